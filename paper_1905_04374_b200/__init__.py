"""B200-native gradient aggregation rules (averaging, median, Krum, multi-Krum,
Bulyan, multi-Bulyan) behind the C ABI of include/gar.h.

`binding` marshals torch tensors into the C calls; `workloads` draws the seeded
synthetic inputs; `build` compiles libgar.so.  All arithmetic runs in the CUDA
kernels of csrc/.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    DISTANCE_MODES, EVEN_MEDIAN, GAR_MAX_N, RULES, GarError, distance_path, gar_selftest_bounded_wait, GarParams, GarSelection, gar_aggregate, gar_aggregate_ex, gar_aggregate_host, gar_aggregate_multi, gar_multi_workspace_bytes, GarTensor, GarMultiParams,
    gar_beta, gar_coordinate_phase, gar_pairwise_distances, gar_pairwise_distances_static, gar_reduce_partials, gar_schedule_from_tables, gar_select, gar_shutdown,
    gar_last_cuda_error, gar_status_string, gar_theta, gar_version, gar_workspace_bytes, lib, new_selection, read_selection,
    write_selection,
)
