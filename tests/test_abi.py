"""CPU-side checks of the C ABI: the library builds, loads and exports every
symbol include/gar.h declares; struct mirrors match; argument and precondition
errors are reported before any CUDA call."""
import ctypes as C
import os
import re
import subprocess

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pkg():
    entry.build()
    import paper_1905_04374_b200 as p
    return p


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "gar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gar_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(pkg):
    names = _declared_functions()
    assert "gar_aggregate" in names and "gar_pairwise_distances" in names and len(names) >= 12
    L = pkg.lib()
    for name in names:
        assert hasattr(L, name), f"{name} declared in gar.h but not exported"


def test_struct_mirrors_match_the_header(pkg, tmp_path):
    src = tmp_path / "sz.cpp"
    src.write_text('#include "gar.h"\n#include <cstdio>\n#include <cstddef>\n'
                   'int main(){printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu %zu\\n", sizeof(gar_selection_t),'
                   'offsetof(gar_selection_t,sets), offsetof(gar_selection_t,nu),'
                   'offsetof(gar_selection_t,add_pos), offsetof(gar_selection_t,scores), sizeof(gar_params_t),'
                   'offsetof(gar_selection_t,even_median), offsetof(gar_selection_t,winners),'
                   'offsetof(gar_params_t,even_median), offsetof(gar_params_t,distance_mode));'
                   'printf("%zu %zu\\n", offsetof(gar_params_t,sgd_params), offsetof(gar_params_t,sgd_lr));'
                   'printf("%zu %zu %zu %zu %zu %zu\\n", sizeof(gar_tensor_t), sizeof(gar_multi_params_t),'
                   'offsetof(gar_multi_params_t,tensors), offsetof(gar_multi_params_t,stream),'
                   'offsetof(gar_tensor_t,sgd_momentum_buf), offsetof(gar_multi_params_t,grads_dtype));}')
    exe = tmp_path / "sz"
    subprocess.check_call(["g++", "-I" + os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    got = [int(v) for v in subprocess.check_output([str(exe)]).split()]
    S = pkg.GarSelection
    P = pkg.GarParams
    assert got == [C.sizeof(S), S.sets.offset, S.nu.offset, S.add_pos.offset, S.scores.offset,
                   C.sizeof(P), S.even_median.offset, S.winners.offset, P.even_median.offset, P.distance_mode.offset,
                   P.sgd_params.offset, P.sgd_lr.offset,
                   C.sizeof(pkg.GarTensor), C.sizeof(pkg.GarMultiParams), pkg.GarMultiParams.tensors.offset,
                   pkg.GarMultiParams.stream.offset, pkg.GarTensor.sgd_momentum_buf.offset,
                   pkg.GarMultiParams.grads_dtype.offset]


def test_version_and_strings(pkg):
    assert pkg.gar_version() == 105
    assert pkg.gar_status_string(0) == "ok"
    assert pkg.gar_last_cuda_error() == (0, "cudaSuccess")      # nothing has failed in this thread yet
    assert "4f+3" in pkg.gar_status_string(2)


def test_theta_beta(pkg):
    # Algorithm 1: theta = n-2f-2, beta = theta-2f; proof of Theorem 2: theta = n-2f
    for n, f in [(11, 2), (23, 5), (39, 9), (51, 12), (15, 3), (20, 3)]:
        assert pkg.gar_theta("multi_bulyan", n, f) == n - 2 * f - 2
        assert pkg.gar_beta("multi_bulyan", n, f) == n - 4 * f - 2
        assert pkg.gar_theta("bulyan", n, f) == n - 2 * f
        assert pkg.gar_beta("bulyan", n, f) == n - 4 * f
        assert pkg.gar_theta("median", n, f) == n and pkg.gar_beta("krum", n, f) == 1
    assert pkg.gar_theta("multi_bulyan", 10, 2) == -1


def test_errors_before_any_launch(pkg):
    L = pkg.lib()
    fake = C.c_void_p(4096)
    # preconditions of Section 2.2 sit exactly at n = 2f+3 / 4f+3
    for f in range(0, 8):
        assert L.gar_aggregate(5, fake, 4 * f + 2, f, 100, fake, None) == 2
        assert L.gar_aggregate(4, fake, 4 * f + 2, f, 100, fake, None) == 2
        assert L.gar_aggregate(3, fake, 2 * f + 2, f, 100, fake, None) == 2
        assert L.gar_aggregate(2, fake, 2 * f + 2, f, 100, fake, None) == 2
    assert L.gar_aggregate(5, fake, 65, 1, 100, fake, None) == 3          # n > 64
    assert L.gar_aggregate(7, fake, 11, 2, 100, fake, None) == 1          # unknown rule
    assert L.gar_aggregate(5, fake, 11, -1, 100, fake, None) == 1
    assert L.gar_aggregate(5, fake, 11, 2, 0, fake, None) == 1
    assert L.gar_aggregate(5, None, 11, 2, 100, fake, None) == 1
    assert L.gar_aggregate(5, fake, 11, 2, 100, None, None) == 1
    assert L.gar_aggregate_ex(None) == 1
    assert pkg.gar_workspace_bytes("multi_bulyan", 11, 2, 1000) > 0
    assert pkg.gar_workspace_bytes("multi_bulyan", 10, 2, 1000) == 0
    p = pkg.GarParams()
    p.rule, p.n, p.f, p.d, p.ld = 5, 11, 2, 100, 50                        # ld < d
    p.grads, p.out = 4096, 1 << 30
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.ld = 100
    p.out = 4096 + 400                                                     # out overlaps grads
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.out = 1 << 30
    p.m = 3                                                                # m only for multi-Krum
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.m, p.theta = 0, 6                                                    # theta > n-2f-2
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.theta = 4                                                            # theta < 2f+1
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.theta, p.even_median = 0, 2                                          # unknown even-median mode
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.even_median, p.distance_mode = 0, 7                                  # unknown distance mode
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.distance_mode, p.grads_dtype = 0, 3                                  # unknown element type
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.grads_dtype = 0
    p.distance_mode = 0
    p.out, p.sgd_params = None, None                                       # neither an output nor a fused step
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.out, p.sgd_momentum_buf = 1 << 30, 1 << 31                            # a momentum buffer without parameters
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    p.sgd_params = (1 << 30) + 40                                          # parameters overlapping the output
    assert L.gar_aggregate_ex(C.byref(p)) == 1
    assert L.gar_pairwise_distances_mode(fake, 11, 100, 100, fake, None, 0, 5, None) == 1
    # the batched call: argument and workspace errors come before any CUDA call
    assert L.gar_aggregate_multi(None) == 1
    assert pkg.gar_multi_workspace_bytes("multi_bulyan", 11, 2, 3) > 0
    assert pkg.gar_multi_workspace_bytes("multi_bulyan", 10, 2, 3) == 0
    assert pkg.gar_multi_workspace_bytes("multi_bulyan", 11, 2, 0) == 0
    tensors = (pkg.GarTensor * 2)()
    tensors[0].grads, tensors[0].out, tensors[0].d, tensors[0].ld = 4096, 1 << 30, 100, 100
    tensors[1].grads, tensors[1].out, tensors[1].d, tensors[1].ld = 1 << 20, 1 << 31, 7, 0
    q = pkg.GarMultiParams()
    q.rule, q.n, q.f, q.count, q.tensors = 5, 11, 2, 2, tensors
    assert L.gar_aggregate_multi(C.byref(q)) == 4                          # no workspace
    q.workspace, q.workspace_bytes = 1 << 32, 1024                         # too small
    assert L.gar_aggregate_multi(C.byref(q)) == 4
    q.n = 10
    assert L.gar_aggregate_multi(C.byref(q)) == 2                          # n < 4f + 3
    q.n, q.count = 11, 0
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    q.count, q.joint = 2, 2
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    q.joint = 0
    tensors[1].ld = 5                                                      # ld < d
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    tensors[1].ld = 0
    tensors[0].out = 4096 + 400                                            # out overlaps its own gradients
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    tensors[0].out = (1 << 20) + 8                                         # ... another tensor's gradients
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    tensors[0].out = (1 << 31) + 4                                         # ... another tensor's output
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    tensors[0].out = 1 << 30
    assert L.gar_aggregate_multi(C.byref(q)) == 4                          # all well again: the workspace is what is missing
    tensors[1].sgd_momentum_buf = 1 << 33                                  # a momentum buffer without parameters
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    tensors[1].sgd_params = (1 << 31) + 8                                  # parameters overlapping the tensor's output
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    tensors[1].sgd_params, tensors[1].out = 1 << 34, None                  # a fused step without the aggregate: fine
    assert L.gar_aggregate_multi(C.byref(q)) == 4
    q.grads_dtype = 3                                                      # unknown element type
    assert L.gar_aggregate_multi(C.byref(q)) == 1
    assert L.gar_reduce_partials(fake, 0, 11, fake, None) == 1 and L.gar_reduce_partials(fake, 2, 65, fake, None) == 3
    assert L.gar_select(5, fake, 11, 2, 0, 0, 0, 3, fake, None) == 1       # unknown even-median mode
    assert L.gar_selftest_bounded_wait(0, fake, None) == 1
    assert L.gar_selftest_bounded_wait(100, None, None) == 1
    assert L.gar_selftest_bounded_wait(1 << 20, fake, None) == 1           # limit above the documented maximum


def test_missing_library_fails_loudly(pkg, monkeypatch):
    from paper_1905_04374_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libgar.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
