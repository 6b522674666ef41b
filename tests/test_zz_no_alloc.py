"""st_sym_moment3_static: the entry point for callers that are not allowed to allocate device
memory (code inside a framework's hot loop, plug-ins that only get input and output buffers,
processes with a fixed device-memory budget).  It must give what st_sym_moment3 gives, call
after call, although every call reuses the same built-in scratch array.

This file is collected last on purpose: a run that stops at the first failure has then
already run every other test."""
import numpy as np
import pytest

import workloads

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle

TOL = 1e-4   # the fp32 tolerance of the parity tests: |a - b| <= TOL * sum |terms|


def _call_static(st, X, out, flags=0):
    """Straight through the C ABI: raw pointers, no workspace argument."""
    N, d = X.shape
    return st.lib().st_sym_moment3_static(X.data_ptr(), N, d, X.stride(0), out.data_ptr(), flags,
                                          torch.cuda.current_stream().cuda_stream)


def test_static_entry_point_matches_the_workspace_one_on_two_calls_in_a_row():
    import paper_2211_10482_b200 as st
    cases = [(workloads.draw((5000, 64), "normal", 901), 0),
             (workloads.draw((777, 40), "uniform", 902), 0),       # smaller second call: stale scratch must not leak
             (workloads.draw((3000, 64), "normal", 903), 0),
             (workloads.draw((300, 16), "normal", 904), st.ST_FLAG_DENSE_CONTROL)]
    for Xh, flags in cases:
        X = torch.from_numpy(Xh).cuda()
        N, d = X.shape
        want = st.st_sym_moment3(X, flags=flags)
        scale = st.st_sym_moment3(X.abs(), flags=flags)            # sum of |terms| of every output
        got = torch.full_like(want, float("nan"))
        before = torch.cuda.memory_allocated()
        assert _call_static(st, X, got, flags) == st.ST_OK
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before             # nothing went through torch's allocator
        assert bool(torch.all(torch.isfinite(got)))
        assert bool(torch.all((got - want).abs() <= TOL * scale)), (N, d)
        # and against the CPU oracle, entry by entry in the packed order i <= j <= k
        ii, jj, kk = (np.array(v) for v in zip(*[(i, j, k) for i in range(d) for j in range(i, d) for k in range(j, d)]))
        T, S = oracle.moment3_at(Xh, ii, jj, kk)
        assert oracle.rel_err(got.cpu().numpy(), T, S) <= TOL, (N, d)
    # the binding of the same name reaches the same entry point
    X = torch.from_numpy(cases[0][0]).cuda()
    out = torch.empty(64 * 65 * 66 // 6, dtype=torch.float32, device="cuda")
    assert torch.equal(st.st_sym_moment3_static(X, out), st.st_sym_moment3(X))


def test_static_entry_point_rejects_bad_requests_without_launching():
    import paper_2211_10482_b200 as st
    X = torch.zeros((64, 64), device="cuda")
    out = torch.zeros(45760, device="cuda")
    L = st.lib()
    s = torch.cuda.current_stream().cuda_stream
    assert L.st_sym_moment3_static(None, 64, 64, 64, out.data_ptr(), 0, s) == st.ST_ERR_NULL
    assert L.st_sym_moment3_static(X.data_ptr(), 64, 72, 72, out.data_ptr(), 0, s) == st.ST_ERR_UNSUPPORTED
    assert L.st_sym_moment3_static(X.data_ptr(), 0, 64, 64, out.data_ptr(), 0, s) == st.ST_ERR_SHAPE
    assert L.st_sym_moment3_static(X.data_ptr(), 64, 64, 64, out.data_ptr(), 8, s) == st.ST_ERR_UNSUPPORTED
    # the size rule: whatever st_workspace_bytes asks for must fit the built-in array
    assert st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, 1 << 20, 64) <= st.ST_STATIC_SCRATCH_BYTES
    assert st.status_string(st.ST_ERR_STATIC_SCRATCH).startswith("request needs more scratch")
