"""CPU oracle for the gradient aggregation rules: test infrastructure only.

Nothing in the product package may import this; see gar_oracle.py.
"""
from .gar_oracle import *  # noqa: F401,F403
