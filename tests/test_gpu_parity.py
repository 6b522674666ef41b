"""GPU parity tests: every C-ABI call against the CPU oracle, element by element, on the same
seeded inputs.  Integer / byte work must be bit-exact; fp32 paths must satisfy
max |gpu - oracle| / sum|terms| <= 1e-4."""
import itertools
import math

import numpy as np
import pytest

import oracle
import workloads

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4


BAND = 4096            # bytes of canary before and after every buffer the binding allocates
CANARY = 0xFF          # all-ones bytes: a NaN in fp32 and bf16, so a read outside a buffer shows up in the result


class GuardAllocator:
    """Allocator handed to the binding: every output and workspace that a test does not pass itself
    sits between two canary bands, which `check` compares on the host."""

    def __init__(self):
        self.live = []

    def __call__(self, numel, dtype, device):
        nbytes = numel * torch.empty(0, dtype=dtype).element_size()
        raw = torch.full((BAND + (nbytes + 255) // 256 * 256 + BAND,), CANARY, dtype=torch.uint8, device=device)
        self.live.append((raw, nbytes))
        return raw[BAND:BAND + nbytes].view(dtype)

    def check(self):
        torch.cuda.synchronize()
        for raw, nbytes in self.live:
            assert bool(torch.all(raw[:BAND] == CANARY)), "a kernel wrote in front of a %d-byte buffer" % nbytes
            assert bool(torch.all(raw[BAND + nbytes:] == CANARY)), "a kernel wrote behind a %d-byte buffer" % nbytes
        self.live.clear()


@pytest.fixture(scope="module")
def st():
    import paper_2211_10482_b200 as m
    m.lib()
    m.set_allocator(GuardAllocator())
    yield m
    m.set_allocator(None)


@pytest.fixture(autouse=True)
def guard_bands_and_device_status(st):
    """After every test: no kernel wrote outside its buffers, and the last compute call left no
    device-side error (a bounded wait that ran out) in its workspace."""
    yield
    import paper_2211_10482_b200 as m
    assert m.st_check_status() == m.ST_OK
    if m._allocator is not None:
        m._allocator.check()


def guarded(st, numel, dtype=None):
    """A buffer with canary bands for the tests that call the C ABI with raw pointers."""
    import paper_2211_10482_b200 as m
    return m._alloc(numel, dtype or torch.float32, torch.device("cuda", torch.cuda.current_device()))


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def okw(layout):
    return dict(kl=layout.kl, ku=layout.ku, nb=layout.nblocks, bs=layout.bs)


# ------------------------------------------------------------------------------ pack / unpack

def layouts(st):
    out = []
    for d in (1, 2, 3, 5, 8, 17, 64, 130):
        out.append(st.Layout(st.ST_TRI_UPPER, d))
    for d in (1, 2, 3, 5, 17, 40):
        out.append(st.Layout(st.ST_TET, d))
    out += [st.Layout(st.ST_BAND, 9, kl=2, ku=3), st.Layout(st.ST_BAND, 4, kl=6, ku=0),
            st.Layout(st.ST_BAND, 33, kl=0, ku=0), st.Layout(st.ST_BAND, 70, kl=1, ku=5)]
    out += [st.Layout(st.ST_BLOCKDIAG, 12, nblocks=3, bs=4), st.Layout(st.ST_BLOCKDIAG, 7, nblocks=7, bs=1),
            st.Layout(st.ST_BLOCKDIAG, 64, nblocks=1, bs=64), st.Layout(st.ST_BLOCKDIAG, 96, nblocks=3, bs=32)]
    # one row / one column of a matrix (the fixed index travels in kl), and the packed 4-simplex
    out += [st.Layout(st.ST_FIXED_ROW, 1, kl=0), st.Layout(st.ST_FIXED_ROW, 9, kl=4), st.Layout(st.ST_FIXED_ROW, 70, kl=69),
            st.Layout(st.ST_FIXED_COL, 1, kl=0), st.Layout(st.ST_FIXED_COL, 9, kl=0), st.Layout(st.ST_FIXED_COL, 70, kl=33)]
    out += [st.Layout(st.ST_SIMPLEX4, d) for d in (1, 2, 3, 5, 9, 17)]
    return out


@pytest.mark.parametrize("inner,dtype", [(1, np.float32), (3, np.float32), (4, np.float32), (36, np.float32),
                                         (1, np.uint16), (5, np.uint16), (8, np.uint16), (1, np.float64),
                                         (3, np.float64), (130, np.float32)])
def test_pack_unpack_bit_exact(st, inner, dtype):
    import dataclasses
    for base in layouts(st):
        lay = dataclasses.replace(base, inner=inner)
        nd = st.st_dense_elems(lay)
        if nd > 3_000_000:
            continue
        rng = np.random.default_rng(nd + inner)
        bits = rng.integers(0, 2 ** 16, size=nd * np.dtype(dtype).itemsize // 2, dtype=np.uint16)
        if dtype == np.float32:      # keep NaN payloads and -0.0 in the mix
            dense = bits.view(np.float32)
        elif dtype == np.float64:
            dense = bits.view(np.float64)
        else:
            dense = bits
        u = {4: np.uint32, 8: np.uint64, 2: np.uint16}[np.dtype(dtype).itemsize]
        tdt = {4: torch.int32, 8: torch.int64, 2: torch.int16}[np.dtype(dtype).itemsize]
        dense_t = torch.from_numpy(dense.view(u).view({4: np.int32, 8: np.int64, 2: np.int16}[dense.itemsize])).cuda()
        want_p = oracle.pack(dense.view(u), lay.kind, lay.d, inner=inner, **okw(lay))
        got_p = st.st_pack(dense_t, lay)
        assert got_p.dtype == tdt
        assert np.array_equal(got_p.cpu().numpy().view(u), want_p), (lay, "pack")
        fills = [st.ST_FILL_ZERO] + ([st.ST_FILL_SYMMETRIC] if lay.kind in (st.ST_TRI_UPPER, st.ST_TET, st.ST_SIMPLEX4) else [])
        for fill in fills:
            want_d = oracle.unpack(want_p, lay.kind, lay.d, inner=inner, fill=fill, **okw(lay)).reshape(-1)
            got_d = st.st_unpack(got_p, lay, fill=fill)
            assert np.array_equal(got_d.cpu().numpy().view(u), want_d), (lay, "unpack", fill)
            # pack(unpack(P)) == P always (band: corner slots are zero both times)
            again = st.st_pack(got_d, lay)
            assert torch.equal(again, got_p), (lay, "round trip")


def test_unpack_of_symmetric_tensor_restores_it(st):
    """Property 5: T = T_C + T_R * T_C for a tensor that has the structure."""
    d = 37
    X = workloads.draw((50, d), "normal", 3)
    T2 = (X.T.astype(np.float64) @ X.astype(np.float64)).astype(np.float32)
    T2 = np.triu(T2) + np.triu(T2, 1).T
    lay = st.Layout(st.ST_TRI_UPPER, d)
    back = st.st_unpack(st.st_pack(dev(T2), lay), lay, fill=st.ST_FILL_SYMMETRIC).cpu().numpy().reshape(d, d)
    assert np.array_equal(back.view(np.uint32), T2.view(np.uint32))


def test_pack_unpack_at_config_sizes(st):
    # tri d=1024 (moment2-large output) and tet d=64 (moment3 output): full comparison
    for lay in (st.Layout(st.ST_TRI_UPPER, 1024), st.Layout(st.ST_TET, 64)):
        n = st.st_packed_elems(lay)
        P = np.random.default_rng(n).integers(0, 2 ** 32, size=n, dtype=np.uint32)
        Pt = torch.from_numpy(P.view(np.int32)).cuda()
        for fill in (st.ST_FILL_ZERO, st.ST_FILL_SYMMETRIC):
            want = oracle.unpack(P, lay.kind, lay.d, fill=fill).reshape(-1)
            got = st.st_unpack(Pt, lay, fill=fill)
            assert np.array_equal(got.cpu().numpy().view(np.uint32), want)
            assert torch.equal(st.st_pack(got, lay), Pt)
    # tri x K with I=512, K=512 (MTTKRP operand): full comparison of pack, unpack on device
    lay = st.Layout(st.ST_TRI_UPPER, 512, inner=512)
    dense = np.random.default_rng(1).integers(0, 2 ** 32, size=512 * 512 * 512, dtype=np.uint32)
    want = oracle.pack(dense, lay.kind, lay.d, inner=512)
    dense_t = torch.from_numpy(dense.view(np.int32)).cuda()
    got = st.st_pack(dense_t, lay)
    assert np.array_equal(got.cpu().numpy().view(np.uint32), want)
    back = st.st_unpack(got, lay).view(512, 512, 512)
    mask = torch.triu(torch.ones(512, 512, dtype=torch.bool, device="cuda"))
    assert torch.equal(back[mask], dense_t.view(512, 512, 512)[mask])
    assert int(torch.count_nonzero(back[~mask])) == 0
    del dense_t, back, got
    # block-diagonal 64 blocks of 64x64 with K=256 (TTM operand): 16 GiB dense, sampled fibres
    lay = st.Layout(st.ST_BLOCKDIAG, 4096, inner=256, nblocks=64, bs=64)
    n = st.st_packed_elems(lay)
    Pt = torch.randint(-2 ** 31, 2 ** 31 - 1, (n,), dtype=torch.int32, device="cuda",
                       generator=torch.Generator(device="cuda").manual_seed(7))
    dense_t = st.st_unpack(Pt, lay).view(4096, 4096, 256)
    rng = np.random.default_rng(11)
    samples = [(0, 0), (63, 63), (63, 64), (64, 63), (4095, 4095), (4095, 4032), (4032, 4031), (100, 70)]
    samples += [tuple(int(v) for v in rng.integers(0, 4096, 2)) for _ in range(24)]
    samples += [(int(b) * 64 + int(a), int(b) * 64 + int(c)) for b, a, c in rng.integers(0, 64, (24, 3))]
    Pv = Pt.view(-1, 256)
    for (i, j) in samples:
        row = oracle.locate(oracle.KIND_BLOCKDIAG, 4096, i, j, nb=64, bs=64)
        if row < 0:
            assert int(torch.count_nonzero(dense_t[i, j])) == 0
        else:
            assert torch.equal(dense_t[i, j], Pv[row])
    assert int(torch.count_nonzero(dense_t)) == int(torch.count_nonzero(Pt))
    assert torch.equal(st.st_pack(dense_t.view(-1), lay), Pt)


def test_pack_unpack_blockdiag_midsize(st):
    # 16 blocks of 64 x 64 fibres of 64 floats: 16.8 MB packed, 268 MB dense (larger than L2); full comparison
    lay = st.Layout(st.ST_BLOCKDIAG, 1024, inner=64, nblocks=16, bs=64)
    n = st.st_packed_elems(lay)
    P = np.random.default_rng(3).integers(0, 2 ** 32, size=n, dtype=np.uint32)
    Pt = torch.from_numpy(P.view(np.int32)).cuda()
    dense = st.st_unpack(Pt, lay)
    want = oracle.unpack(P, oracle.KIND_BLOCKDIAG, 1024, inner=64, nb=16, bs=64).reshape(-1)
    assert np.array_equal(dense.cpu().numpy().view(np.uint32), want)
    assert torch.equal(st.st_pack(dense, lay), Pt)


# ------------------------------------------------------------------------------ moments

def expand2(st, packed, d):
    return oracle.unpack(packed.cpu().numpy(), oracle.KIND_TRI, d, fill=oracle.FILL_SYMMETRIC).astype(np.float64)


def expand3(st, packed, d):
    return oracle.unpack(packed.cpu().numpy(), oracle.KIND_TET, d, fill=oracle.FILL_SYMMETRIC).astype(np.float64)


@pytest.mark.parametrize("d", [1, 2, 3, 5, 8, 17, 64, 100, 130])
@pytest.mark.parametrize("N", [1, 31, 32, 33, 257, 4096])
def test_moment2_f32_small(st, N, d):
    X = workloads.draw((N, d), "uniform", 100 + N + d)
    T, S = oracle.moment2(X)
    for flags in (0, st.ST_FLAG_DENSE_CONTROL):
        got = expand2(st, st.st_sym_moment2(dev(X), flags=flags), d)
        assert oracle.rel_err(got, T, S) <= TOL_F32, (N, d, flags)


@pytest.mark.parametrize("N,d", [(1, 128), (15, 128), (16, 132), (17, 256), (300, 200), (2049, 384), (5000, 516), (40000, 128)])
def test_moment2_f32_many_features(st, N, d):
    # d >= 128 with aligned rows: 128 x 128 tiles, ragged last tiles, sample splits with a ragged tail
    X = workloads.draw((N, d), "normal", 150 + N + d)
    T, S = oracle.moment2(X)
    for flags in (0, st.ST_FLAG_DENSE_CONTROL):
        got = expand2(st, st.st_sym_moment2(dev(X), flags=flags), d)
        assert oracle.rel_err(got, T, S) <= TOL_F32, (N, d, flags)
    assert torch.equal(st.st_sym_moment2(dev(X)), st.st_sym_moment2(dev(X)))
    # the same through a pitch: X as a view of a wider matrix
    if N == 300:
        wide = dev(workloads.draw((N, d + 8), "normal", 151))
        Xv = wide[:, :d]
        out = guarded(st, d * (d + 1) // 2)
        nbytes = st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, N, d, st.ST_F32)
        ws = guarded(st, nbytes, torch.uint8)
        rc = st.lib().st_sym_moment2(Xv.data_ptr(), st.ST_F32, N, d, d + 8, out.data_ptr(), ws.data_ptr(), nbytes, 0,
                                     torch.cuda.current_stream().cuda_stream)
        assert rc == st.ST_OK
        Tw, Sw = oracle.moment2(np.ascontiguousarray(wide.cpu().numpy()[:, :d]))
        assert oracle.rel_err(expand2(st, out, d), Tw, Sw) <= TOL_F32


def test_moment2_f32_strided_rows_and_all_ones(st):
    N, d, ldx = 300, 20, 28
    buf = workloads.draw((N, ldx), "normal", 5)
    Xt = dev(buf)[:, :d]
    T, S = oracle.moment2(np.ascontiguousarray(buf[:, :d]))
    out = guarded(st, d * (d + 1) // 2)
    nbytes = st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, N, d, st.ST_F32)
    ws = guarded(st, nbytes, torch.uint8)
    rc = st.lib().st_sym_moment2(Xt.data_ptr(), st.ST_F32, N, d, ldx, out.data_ptr(), ws.data_ptr(), nbytes, 0,
                                 torch.cuda.current_stream().cuda_stream)
    assert rc == st.ST_OK
    assert oracle.rel_err(expand2(st, out, d), T, S) <= TOL_F32
    ones = torch.ones((777, 64), dtype=torch.float32, device="cuda")
    assert torch.all(st.st_sym_moment2(ones) == 777.0)


def test_moment2_config(st):
    X = workloads.moment_input("moment2")
    assert X.shape == (4096, 64)
    T, S = oracle.moment2(X)
    got = st.st_sym_moment2(dev(X))
    assert got.numel() == 2080
    assert oracle.rel_err(expand2(st, got, 64), T, S) <= TOL_F32
    # two calls give the same bits (fixed-order reduction)
    assert torch.equal(got, st.st_sym_moment2(dev(X)))


def test_moment2_rejects_element_types_it_cannot_compute_on(st):
    # st_pack / st_unpack move any 2-, 4- or 8-byte element as bits; the moments are arithmetic and take
    # float32 or bfloat16 only
    for dt in (torch.float16, torch.int32, torch.float64, torch.int16):
        with pytest.raises(TypeError):
            st.st_sym_moment2(torch.zeros((8, 8), dtype=dt, device="cuda"))


def test_fixed_order_calls_give_the_same_bits_twenty_times(st):
    """The moments, TTM and MTTKRP add their partial sums in a fixed order: repeated calls on the same
    input must agree bit for bit."""
    X2 = dev(workloads.draw((20000, 64), "normal", 31))
    X3 = dev(workloads.draw((9000, 40), "normal", 32))
    Xb = dev(workloads.draw((5000, 512), "normal", 33)).to(torch.bfloat16)
    Bq, U = workloads.ttm_inputs(3, 16, 64, 32)
    Bq, U = dev(Bq), dev(U)
    Bp, C, D = (dev(a) for a in workloads.mttkrp_inputs(96, 64, 32))
    calls = {
        "moment2": lambda: st.st_sym_moment2(X2),
        "moment2_bf16": lambda: st.st_sym_moment2(Xb),
        "moment3": lambda: st.st_sym_moment3(X3),
        "moment3_tf32": lambda: st.st_sym_moment3(X3, flags=st.ST_FLAG_TC_TF32),
        "moment3_bf16": lambda: st.st_sym_moment3(X3, flags=st.ST_FLAG_TC_BF16),
        "moment4": lambda: st.st_sym_moment4(X3[:, :12].contiguous()),
        "ttm": lambda: st.st_ttm_blockdiag(Bq, U, 3, 16),
        "ttm_tf32": lambda: st.st_ttm_blockdiag(Bq, U, 3, 16, flags=st.ST_FLAG_TC_TF32),
        "mttkrp": lambda: st.st_mttkrp_tri(Bp, C, D),
        "mttkrp_tf32": lambda: st.st_mttkrp_tri(Bp, C, D, flags=st.ST_FLAG_TC_TF32),
        "ttm_split": lambda: st.st_ttm_blockdiag(Bq, U, 3, 16, flags=st.ST_FLAG_TC_SPLIT),
        "mttkrp_split": lambda: st.st_mttkrp_tri(Bp, C, D, flags=st.ST_FLAG_TC_SPLIT),
    }
    for name, fn in calls.items():
        first = fn().clone()
        for rep in range(19):
            assert torch.equal(fn(), first), (name, rep)
        st._allocator.check()


@pytest.mark.parametrize("d", [1, 2, 3, 5, 8, 16, 17, 24, 40, 57, 63, 64])
@pytest.mark.parametrize("N", [1, 63, 64, 65, 1000])
def test_moment3_small(st, N, d):
    X = workloads.draw((N, d), "normal", 200 + N + d)
    T, S = oracle.moment3(X)
    got = st.st_sym_moment3(dev(X))
    assert got.numel() == workloads.tet(d)
    assert oracle.rel_err(expand3(st, got, d), T, S) <= TOL_F32, (N, d)


@pytest.mark.parametrize("N,d", [(300, 72), (700, 100), (257, 128), (130, 200), (64, 256)])
def test_moment3_more_than_64_features(st, N, d):
    # the tile table of the call travels through the workspace, stages are shorter, several thread blocks
    # share a sample slice; every unique entry against the oracle
    X = workloads.draw((N, d), "normal", 250 + N + d)
    walk = [(i, j, k) for i in range(d) for j in range(i, d) for k in range(j, d)]
    ii, jj, kk = (np.array(v, dtype=np.int64) for v in zip(*walk))
    T, S = oracle.moment3_at(X, ii, jj, kk)
    ws = guarded(st, st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, N, d), torch.uint8)
    got = st.st_sym_moment3(dev(X), ws=ws)
    assert st.st_check_status(ws) == st.ST_OK
    assert got.numel() == workloads.tet(d) == len(walk)
    assert oracle.rel_err(got.cpu().numpy(), T, S) <= TOL_F32, (N, d)
    assert torch.equal(got, st.st_sym_moment3(dev(X), ws=ws))        # fixed-order sums


def test_moment3_rows_with_a_pitch_that_is_not_aligned(st):
    # X as a view of a wider matrix whose rows are not 16-byte aligned: staged with plain loads
    N, d, ldx = 500, 21, 23
    buf = workloads.draw((N, ldx), "normal", 260)
    Xv = dev(buf)[:, :d]
    got = guarded(st, workloads.tet(d))
    ws = guarded(st, st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, N, d), torch.uint8)
    rc = st.lib().st_sym_moment3(Xv.data_ptr(), N, d, ldx, got.data_ptr(), ws.data_ptr(), ws.numel(), 0,
                                 torch.cuda.current_stream().cuda_stream)
    assert rc == st.ST_OK
    T, S = oracle.moment3(np.ascontiguousarray(buf[:, :d]))
    assert oracle.rel_err(expand3(st, got, d), T, S) <= TOL_F32
    ctl = st.st_sym_moment3(dev(np.ascontiguousarray(buf[:, :d])), flags=st.ST_FLAG_DENSE_CONTROL)
    assert oracle.rel_err(expand3(st, ctl, d), T, S) <= TOL_F32


def test_moment3_dense_control_and_all_ones(st):
    X = workloads.draw((500, 32), "normal", 9)
    T, S = oracle.moment3(X)
    a = st.st_sym_moment3(dev(X))
    b = st.st_sym_moment3(dev(X), flags=st.ST_FLAG_DENSE_CONTROL)
    assert oracle.rel_err(expand3(st, b, 32), T, S) <= TOL_F32
    assert oracle.rel_err(expand3(st, a, 32), T, S) <= TOL_F32
    ones = torch.ones((1234, 64), dtype=torch.float32, device="cuda")
    assert torch.all(st.st_sym_moment3(ones) == 1234.0)


@pytest.fixture(scope="module")
def moment3_config_oracle():
    """The named third-moment configuration and the oracle's value of EVERY unique entry, listed by a
    running walk of i <= j <= k (the packed order)."""
    X = workloads.moment_input("moment3")
    N, d = X.shape
    assert (N, d) == (65536, 64)
    walk = [(i, j, k) for i in range(d) for j in range(i, d) for k in range(j, d)]
    ii, jj, kk = (np.array(v) for v in zip(*walk))
    T, S = oracle.moment3_at(X, ii, jj, kk)
    for p in (0, 1, 63, 64, 2079, 2080, 30000, 45759):
        assert oracle.locate(oracle.KIND_TET, d, *walk[p]) == p
    return X, walk, T, S


def _multiplicity_identity3(X, walk, got, tol):
    # sum over the unique set, weighted by the number of index triples an entry stands for, equals
    # sum_n (sum_i x_i)^3 (holds at any size)
    mult = np.array([{1: 1, 2: 3, 3: 6}[len(set(t))] for t in walk], np.float64)
    Xd = X.astype(np.float64)
    lhs, rhs = float(np.dot(mult, got.astype(np.float64))), float(np.sum(Xd.sum(axis=1) ** 3))
    assert abs(lhs - rhs) <= tol * float(np.sum(np.abs(Xd).sum(axis=1) ** 3))


def test_moment3_config(st, moment3_config_oracle):
    X, walk, T, S = moment3_config_oracle
    got = st.st_sym_moment3(dev(X)).cpu().numpy()
    assert got.size == 45760 == len(walk)
    assert oracle.rel_err(got, T, S) <= TOL_F32          # all 45,760 entries at the full sample count
    _multiplicity_identity3(X, walk, got, TOL_F32)


# tensor-core third moment: pair products made on the fly as the left operand of a tcgen05 GEMM over
# the samples.  TF32: x and x_i*x_j rounded to 10 mantissa bits (three roundings of <= 2^-11 per term).
# bf16: x_k and the fp32 product x_i*x_j rounded to bf16 (two roundings of <= 2^-8 per term, so the
# stated 5e-3 is asserted where rounding errors average out, N >= 1000; 2^-7 holds for any N).
TOL_TC = 5e-3


def _tc_flag(st, kind):
    return st.ST_FLAG_TC_TF32 if kind == "tf32" else st.ST_FLAG_TC_BF16


@pytest.mark.parametrize("d", [1, 2, 5, 8, 16, 17, 33, 40, 63, 64])
@pytest.mark.parametrize("N", [1, 31, 32, 33, 65, 1000])
def test_moment3_tf32_tensor_core_small(st, N, d):
    X = workloads.draw((N, d), "normal", 300 + N + d)
    T, S = oracle.moment3(X)
    got = st.st_sym_moment3(dev(X), flags=st.ST_FLAG_TC_TF32)
    assert st.st_check_status() == st.ST_OK
    assert got.numel() == workloads.tet(d)
    assert oracle.rel_err(expand3(st, got, d), T, S) <= TOL_TC, (N, d)


@pytest.mark.parametrize("N,d", [(1, 5), (63, 64), (64, 16), (129, 40), (1000, 64), (4000, 33), (20000, 64)])
def test_moment3_bf16_tensor_core_small(st, N, d):
    X = workloads.draw((N, d), "normal", 400 + N + d)
    T, S = oracle.moment3(X)
    got = st.st_sym_moment3(dev(X), flags=st.ST_FLAG_TC_BF16)
    assert st.st_check_status() == st.ST_OK
    assert oracle.rel_err(expand3(st, got, d), T, S) <= (TOL_TC if N >= 1000 else 2.0 ** -7), (N, d)


@pytest.mark.parametrize("kind", ["tf32", "bf16"])
def test_moment3_tensor_core_many_slices_of_few_tiles(st, kind):
    # small d (one or two tiles per block) with many sample slices per block: every ring of the kernel
    # wraps many times while few producer warps are at work
    for N, d in ((300000, 8), (200000, 16), (150000, 24)):
        X = workloads.draw((N, d), "uniform", 500 + d)
        got = st.st_sym_moment3(dev(X), flags=_tc_flag(st, kind)).cpu().numpy()
        assert st.st_check_status() == st.ST_OK
        idx = [(i, j, k) for i in range(d) for j in range(i, d) for k in range(j, d)]
        ii, jj, kk = (np.array(v) for v in zip(*idx))
        T, S = oracle.moment3_at(X, ii, jj, kk)
        assert oracle.rel_err(got, T, S) <= TOL_TC, (N, d)


@pytest.mark.parametrize("kind", ["tf32", "bf16"])
def test_moment3_tensor_core_all_ones_strided_rows_and_repeat(st, kind):
    flag = _tc_flag(st, kind)
    ones = torch.ones((1234, 64), dtype=torch.float32, device="cuda")
    assert torch.all(st.st_sym_moment3(ones, flags=flag) == 1234.0)      # 1.0 and small integers are exact
    # rows with a pitch: X is a view of a wider matrix
    wide = dev(workloads.draw((700, 48), "normal", 77))
    Xv = wide[:, :40]
    got = guarded(st, workloads.tet(40))
    ws = guarded(st, st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, 700, 40, 0, 0, flag), torch.uint8)
    rc = st.lib().st_sym_moment3(Xv.data_ptr(), 700, 40, 48, got.data_ptr(), ws.data_ptr(), ws.numel(), flag,
                                 torch.cuda.current_stream().cuda_stream)
    assert rc == st.ST_OK and st.st_check_status(ws) == st.ST_OK
    T, S = oracle.moment3(np.ascontiguousarray(wide.cpu().numpy()[:, :40]))
    assert oracle.rel_err(expand3(st, got, 40), T, S) <= TOL_TC
    # fixed-order reduction: two calls give the same bits
    X = dev(workloads.draw((5000, 64), "normal", 78))
    assert torch.equal(st.st_sym_moment3(X, flags=flag), st.st_sym_moment3(X, flags=flag))
    # the two tensor-core flags exclude each other; the dense control exists for the fp32 kernel only
    both = st.ST_FLAG_TC_TF32 | st.ST_FLAG_TC_BF16
    assert st.lib().st_sym_moment3(X.data_ptr(), 5000, 64, 64, got.data_ptr(), ws.data_ptr(), ws.numel(), both,
                                   torch.cuda.current_stream().cuda_stream) == st.ST_ERR_UNSUPPORTED
    assert st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, 5000, 64, 0, 0, flag | st.ST_FLAG_DENSE_CONTROL) == 0


@pytest.mark.parametrize("kind", ["tf32", "bf16"])
def test_moment3_tensor_core_config(st, kind, moment3_config_oracle):
    X, walk, T, S = moment3_config_oracle
    N, d = X.shape
    ws = guarded(st, st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, N, d, 0, 0, _tc_flag(st, kind)), torch.uint8)
    got = st.st_sym_moment3(dev(X), ws=ws, flags=_tc_flag(st, kind))
    assert st.st_check_status(ws) == st.ST_OK
    got = got.cpu().numpy()
    assert oracle.rel_err(got, T, S) <= TOL_TC           # all 45,760 entries at the full sample count
    _multiplicity_identity3(X, walk, got, TOL_TC)


# fourth moment: packed 4-simplex i<=j<=k<=l in lexicographic order

def simplex4_tuples(d):
    """The unique set in packed order, by a running walk (no closed form)."""
    return [(i, j, k, l) for i in range(d) for j in range(i, d) for k in range(j, d) for l in range(k, d)]


@pytest.mark.parametrize("N,d", [(1, 1), (5, 2), (33, 3), (100, 5), (257, 8), (1000, 11), (64, 12), (500, 16)])
def test_moment4_f32_small(st, N, d):
    X = workloads.draw((N, d), "normal", 600 + N + d)
    T, S = oracle.moment4(X)
    got = st.st_sym_moment4(dev(X)).cpu().numpy()
    tup = simplex4_tuples(d)
    assert got.size == len(tup) == math.comb(d + 3, 4)
    ii, jj, kk, ll = (np.array(v) for v in zip(*tup))
    assert oracle.rel_err(got, T[ii, jj, kk, ll], S[ii, jj, kk, ll]) <= TOL_F32, (N, d)


@pytest.mark.parametrize("flag_name,N,d,tol", [("f32", 3000, 24, TOL_F32), ("f32", 700, 40, TOL_F32),
                                               ("bf16", 1000, 8, 5e-3), ("bf16", 5000, 24, 5e-3),
                                               ("bf16", 2000, 64, 5e-3), ("bf16", 65536, 32, 5e-3)])
def test_moment4_sampled_entries_and_multiplicity_identity(st, flag_name, N, d, tol):
    flags = st.ST_FLAG_TC_BF16 if flag_name == "bf16" else 0
    X = workloads.draw((N, d), "normal", 700 + N + d)
    got = st.st_sym_moment4(dev(X), flags=flags).cpu().numpy()
    assert st.st_check_status() == st.ST_OK
    tup = simplex4_tuples(d)
    assert got.size == len(tup)
    rng = np.random.default_rng(7)
    pick = np.unique(np.concatenate([rng.integers(0, len(tup), 4000), [0, len(tup) - 1]]))
    pick = np.concatenate([pick, [n for n, t in enumerate(tup) if len(set(t)) == 1]])      # all (i,i,i,i)
    ii, jj, kk, ll = (np.array([tup[n][c] for n in pick]) for c in range(4))
    T, S = oracle.moment4_at(X, ii, jj, kk, ll)
    assert oracle.rel_err(got[pick], T, S) <= tol, (N, d)
    # sum over the unique set weighted by the number of index tuples each entry stands for equals
    # sum_n (sum_i x_i)^4 (holds at any size)
    mult = np.array([24 // math.prod(math.factorial(t.count(v)) for v in set(t)) for t in tup], np.float64)
    Xd = X.astype(np.float64)
    lhs, rhs = float(np.dot(mult, got.astype(np.float64))), float(np.sum(Xd.sum(axis=1) ** 4))
    assert abs(lhs - rhs) <= tol * float(np.sum(np.abs(Xd).sum(axis=1) ** 4))


@pytest.mark.parametrize("flag_name,N,d", [("f32", 40, 72), ("bf16", 1200, 72), ("f32", 24, 128)])
def test_moment4_more_than_64_features(st, flag_name, N, d):
    flags = st.ST_FLAG_TC_BF16 if flag_name == "bf16" else 0
    X = workloads.draw((N, d), "normal", 800 + N + d)
    got = st.st_sym_moment4(dev(X), flags=flags).cpu().numpy()
    assert st.st_check_status() == st.ST_OK
    n = math.comb(d + 3, 4)
    assert got.size == n
    # sampled entries, their positions found by the closed form of the running count (checked against the
    # walk for d <= 64 by the host tests) ...
    rng = np.random.default_rng(11)
    tup = np.sort(rng.integers(0, d, (6000, 4)), axis=1)
    tup = np.concatenate([tup, [[0, 0, 0, 0], [d - 1] * 4, [0, 0, 0, d - 1], [0, d - 1, d - 1, d - 1], [63, 64, 64, 65]]])
    def pos(t):     # number of unique 4-tuples that precede t in lexicographic order, by counting
        i, j, k, l = (int(v) for v in t)
        c = sum(math.comb(d - a + 2, 3) for a in range(i))                      # first index smaller
        c += sum(math.comb(d - b + 1, 2) for b in range(i, j))                  # second index smaller
        c += sum(d - e for e in range(j, k))                                    # third index smaller
        return c + (l - k)
    p = np.array([pos(t) for t in tup])
    T, S = oracle.moment4_at(X, tup[:, 0], tup[:, 1], tup[:, 2], tup[:, 3])
    assert oracle.rel_err(got[p], T, S) <= (5e-3 if flags else TOL_F32), (flag_name, N, d)
    # ... and the multiplicity identity over the whole output: sum_n (sum_i x_i)^4
    Xd = X.astype(np.float64)
    idx = np.array(list(itertools.combinations_with_replacement(range(d), 4)), dtype=np.int32) if d <= 72 else None
    if idx is not None:
        assert len(idx) == n
        same = [(idx[:, a] == idx[:, a + 1]) for a in range(3)]
        # multiplicity 24 / prod(run lengths!)
        mult = np.full(n, 24.0)
        run = np.ones(n)
        for a in range(3):
            run = np.where(same[a], run + 1, 1.0)
            mult /= np.where(same[a], run, 1.0)
        lhs, rhs = float(np.dot(mult, got.astype(np.float64))), float(np.sum(Xd.sum(axis=1) ** 4))
        assert abs(lhs - rhs) <= (5e-3 if flags else TOL_F32) * float(np.sum(np.abs(Xd).sum(axis=1) ** 4))


def test_moment4_is_reconstructed_once_at_the_end_of_a_chain(st):
    # fourth moments of two batches are added in packed space (one structure: the sum keeps it) and the dense
    # d^4 tensor is rebuilt once through the redundancy map of the 4-simplex (Section 5.5; Section 6, Property 5)
    d = 9
    Xa, Xb = workloads.draw((400, d), "normal", 1401), workloads.draw((250, d), "normal", 1402)
    m4 = st.st_packed_axpby(1.0, st.st_sym_moment4(dev(Xa)), 1.0, st.st_sym_moment4(dev(Xb)))
    lay = st.Layout(st.ST_SIMPLEX4, d)
    full = st.st_unpack(m4, lay, fill=st.ST_FILL_SYMMETRIC).cpu().numpy().reshape(d, d, d, d)
    T, S = oracle.moment4(np.concatenate([Xa, Xb]))
    assert oracle.rel_err(full, T, S) <= TOL_F32
    for perm in ((1, 0, 2, 3), (3, 2, 1, 0), (0, 2, 3, 1)):
        assert np.array_equal(full, full.transpose(perm))
    assert torch.equal(st.st_pack(dev(full), lay), m4)


def test_moment4_all_ones_pitch_and_errors(st):
    ones = torch.ones((321, 20), dtype=torch.float32, device="cuda")
    assert torch.all(st.st_sym_moment4(ones) == 321.0)
    assert torch.all(st.st_sym_moment4(ones, flags=st.ST_FLAG_TC_BF16) == 321.0)
    wide = dev(workloads.draw((300, 20), "uniform", 5))
    d, N = 9, 300
    out = guarded(st, math.comb(d + 3, 4))
    ws = guarded(st, st.st_workspace_bytes(st.ST_OP_SYM_MOMENT4, N, d), torch.uint8)
    s = torch.cuda.current_stream().cuda_stream
    L = st.lib()
    assert L.st_sym_moment4(wide.data_ptr(), N, d, 20, out.data_ptr(), ws.data_ptr(), ws.numel(), 0, s) == st.ST_OK
    T, S = oracle.moment4(np.ascontiguousarray(wide.cpu().numpy()[:, :d]))
    ii, jj, kk, ll = (np.array(v) for v in zip(*simplex4_tuples(d)))
    assert oracle.rel_err(out.cpu().numpy(), T[ii, jj, kk, ll], S[ii, jj, kk, ll]) <= TOL_F32
    assert L.st_sym_moment4(None, N, d, 20, out.data_ptr(), ws.data_ptr(), ws.numel(), 0, s) == st.ST_ERR_NULL
    assert L.st_sym_moment4(wide.data_ptr(), N, 129, 129, out.data_ptr(), ws.data_ptr(), ws.numel(), 0, s) == st.ST_ERR_UNSUPPORTED
    assert L.st_sym_moment4(wide.data_ptr(), N, d, 20, out.data_ptr(), ws.data_ptr(), 1024, 0, s) == st.ST_ERR_WORKSPACE
    assert L.st_sym_moment4(wide.data_ptr(), N, d, 8, out.data_ptr(), ws.data_ptr(), ws.numel(), 0, s) == st.ST_ERR_SHAPE
    assert L.st_sym_moment4(wide.data_ptr(), N, d, 20, out.data_ptr(), ws.data_ptr(), ws.numel(), 1, s) == st.ST_ERR_UNSUPPORTED


# ------------------------------------------------------------------------------ MTTKRP / TTM

@pytest.mark.parametrize("I,K,R", [(1, 4, 8), (2, 8, 16), (5, 36, 32), (16, 64, 64), (40, 100, 32), (70, 32, 8),
                                   (33, 68, 64),
                                   # fibres far longer than any shared-memory stage; a k tail inside a stage
                                   (12, 2052, 32), (9, 1300, 16),
                                   # every block busy, several units per block, more than one step of 16 units in a block
                                   (150, 20, 64), (200, 16, 8), (390, 16, 64)])
def test_mttkrp_small(st, I, K, R):
    Bp, C, D = workloads.mttkrp_inputs(I, K, R)
    Bd = oracle.unpack(Bp.reshape(-1), oracle.KIND_TRI, I, inner=K)
    A, S = oracle.mttkrp(Bd, C, D)
    got = st.st_mttkrp_tri(dev(Bp), dev(C), dev(D)).cpu().numpy()
    assert oracle.rel_err(got, A, S) <= TOL_F32
    ctl = st.st_mttkrp_tri(dev(Bd), dev(C), dev(D), flags=st.ST_FLAG_DENSE_CONTROL).cpu().numpy()
    assert oracle.rel_err(ctl, A, S) <= TOL_F32


def test_mttkrp_closed_form(st):
    I, K, R = 48, 16, 32
    Bp = torch.ones((I * (I + 1) // 2, K), device="cuda")
    got = st.st_mttkrp_tri(Bp, torch.ones((I, R), device="cuda"), torch.ones((K, R), device="cuda")).cpu().numpy()
    for i in range(I):
        assert np.all(got[i] == (I - i) * K)


@pytest.fixture(scope="module")
def mttkrp_config_oracle():
    """The named MTTKRP configuration and the oracle's A over the full dense iteration space, all 512 rows."""
    Bp, C, D = workloads.mttkrp_inputs()
    assert Bp.shape == (131328, 512) and C.shape == (512, 32) and D.shape == (512, 32)
    Bd = oracle.unpack(Bp.reshape(-1), oracle.KIND_TRI, 512, inner=512)
    A, S = oracle.mttkrp(Bd, C, D)
    return Bp, C, D, A, S


def test_mttkrp_config(st, mttkrp_config_oracle):
    Bp, C, D, A, S = mttkrp_config_oracle
    got = st.st_mttkrp_tri(dev(Bp), dev(C), dev(D)).cpu().numpy()
    assert oracle.rel_err(got, A, S) <= TOL_F32          # every (i, r)


@pytest.mark.parametrize("nb,bs,K,R", [(1, 1, 4, 8), (3, 2, 8, 16), (2, 5, 36, 32), (4, 8, 64, 64), (7, 1, 32, 64),
                                       (2, 17, 100, 8),
                                       # long fibres with a k tail; more than one step of 16 units in a block
                                       (2, 6, 2052, 64), (1, 40, 24, 32), (5, 124, 8, 64)])
def test_ttm_small(st, nb, bs, K, R):
    Bp, U = workloads.ttm_inputs(nb, bs, K, R)
    d = nb * bs
    Bd = oracle.unpack(Bp.reshape(-1), oracle.KIND_BLOCKDIAG, d, inner=K, nb=nb, bs=bs)
    A, S = oracle.ttm(Bd, U)
    got = st.st_ttm_blockdiag(dev(Bp), dev(U), nb, bs).cpu().numpy()
    got_dense = oracle.unpack(got.reshape(-1), oracle.KIND_BLOCKDIAG, d, inner=R, nb=nb, bs=bs)
    assert oracle.rel_err(got_dense, A, S) <= TOL_F32
    ctl = st.st_ttm_blockdiag(dev(Bd), dev(U), nb, bs, flags=st.ST_FLAG_DENSE_CONTROL).cpu().numpy()
    assert oracle.rel_err(ctl.reshape(d, d, R), A, S) <= TOL_F32


def test_ttm_identity_is_bit_exact(st):
    nb, bs, K = 3, 4, 32
    Bp, _ = workloads.ttm_inputs(nb, bs, K, 32)
    got = st.st_ttm_blockdiag(dev(Bp), torch.eye(K, device="cuda"), nb, bs).cpu().numpy()
    assert np.array_equal(got.view(np.uint32), Bp.reshape(-1, K).view(np.uint32))


@pytest.fixture(scope="module")
def ttm_config_oracle():
    """The named TTM configuration and the oracle's result for every one of the 262,144 fibres of the
    diagonal blocks (the fibres of the zero blocks give exact zeros: test_ttm_small checks that on the
    full dense space)."""
    Bp, U = workloads.ttm_inputs()
    assert Bp.shape == (64, 64, 64, 256) and U.shape == (256, 64)
    A, S = oracle.ttm(Bp.reshape(-1, 256), U)
    return Bp, U, A, S


def test_ttm_config(st, ttm_config_oracle):
    Bp, U, A, S = ttm_config_oracle
    got = st.st_ttm_blockdiag(dev(Bp), dev(U), 64, 64).cpu().numpy()
    assert oracle.rel_err(got, A, S) <= TOL_F32          # every fibre, every column
    # the packed row order is the lexicographic walk of the blocks
    for (i, j) in [(0, 0), (63, 63), (64, 64), (130, 190), (4095, 4032)]:
        row = oracle.locate(oracle.KIND_BLOCKDIAG, 4096, i, j, nb=64, bs=64)
        assert row == (i // 64 * 64 + i % 64) * 64 + j % 64


# ------------------------------------------------------------------------------ tensor-core paths

TOL_TC = 5e-3          # stated tolerance of the bf16 / TF32 tensor-core paths


def bf16_dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("d", [64, 128, 192, 256, 320, 520])
@pytest.mark.parametrize("N", [1, 63, 64, 65, 1000, 9000])
def test_moment2_bf16_tensor_core_small(st, N, d):
    X = workloads.draw((N, d), "normal", 300 + N + d)
    bits = workloads.f32_to_bf16_bits(X).reshape(N, d)
    Xb = workloads.bf16_bits_to_f32(bits).reshape(N, d)
    got = expand2(st, st.st_sym_moment2(bf16_dev(bits)), d)
    assert st.st_check_status() == st.ST_OK
    Tb, Sb = oracle.moment2(Xb)         # same rounded inputs: isolates the accumulation error
    assert oracle.rel_err(got, Tb, Sb) <= TOL_F32, (N, d)
    # against the fp32 source of the bf16 copy: every product carries two roundings of relative
    # size <= 2^-8, so 2^-7 bounds any N; the stated 5e-3 is met once rounding errors average out
    T, S = oracle.moment2(X)
    assert oracle.rel_err(got, T, S) <= (TOL_TC if N >= 1000 else 2.0 ** -7 * 1.01), (N, d)
    ctl = expand2(st, st.st_sym_moment2(bf16_dev(bits), flags=st.ST_FLAG_DENSE_CONTROL), d)
    assert oracle.rel_err(ctl, Tb, Sb) <= TOL_F32
    assert st.st_check_status() == st.ST_OK


@pytest.mark.parametrize("N,d", [(1, 4), (31, 8), (100, 36), (33, 128), (1000, 256), (4097, 260), (9000, 520),
                                 (20000, 1024), (3000, 1028)])
def test_moment2_tf32_tensor_core_on_fp32_input(st, N, d):
    """fp32 X read as TF32 by the tensor core (ST_FLAG_TC_TF32): 5e-3 against the oracle on X itself, and 1e-4
    against the oracle on X with the 13 low mantissa bits cleared, which is what the tensor core multiplies."""
    X = workloads.draw((N, d), "normal", 900 + N + d)
    ws = torch.empty(st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, N, d, st.ST_F32, 0, st.ST_FLAG_TC_TF32),
                     dtype=torch.uint8, device="cuda")
    got = expand2(st, st.st_sym_moment2(dev(X), ws=ws, flags=st.ST_FLAG_TC_TF32), d)
    assert st.st_check_status(ws) == st.ST_OK
    T, S = oracle.moment2(X)
    assert oracle.rel_err(got, T, S) <= TOL_TC, (N, d)
    Xt = (X.view(np.uint32) & np.uint32(0xFFFFE000)).view(np.float32)
    Tt, St = oracle.moment2(Xt)
    assert oracle.rel_err(got, Tt, St) <= TOL_F32, (N, d)
    ctl = expand2(st, st.st_sym_moment2(dev(X), ws=ws, flags=st.ST_FLAG_TC_TF32 | st.ST_FLAG_DENSE_CONTROL), d)
    assert oracle.rel_err(ctl, Tt, St) <= TOL_F32
    # a row pitch wider than d
    Xw = torch.zeros((N, d + 12), device="cuda")
    Xw[:, :d] = dev(X)
    out2 = torch.empty(d * (d + 1) // 2, device="cuda")
    assert st.lib().st_sym_moment2(Xw.data_ptr(), st.ST_F32, N, d, d + 12, out2.data_ptr(), ws.data_ptr(), ws.numel(),
                                   st.ST_FLAG_TC_TF32, None) == st.ST_OK
    assert st.st_check_status(ws) == st.ST_OK
    assert np.array_equal(expand2(st, out2, d), got)


@pytest.mark.parametrize("N,d", [(1, 8), (63, 16), (100, 40), (65, 128), (1000, 256), (4097, 264), (9000, 520),
                                 (20000, 1024), (3000, 1032)])
def test_moment2_split_tensor_core_on_fp32_input(st, N, d):
    """fp32 X as hi + lo bf16 parts, three partial products on the tensor cores (ST_FLAG_TC_SPLIT): the fp32 tolerance."""
    X = workloads.draw((N, d), "normal", 950 + N + d)
    ws = torch.empty(st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, N, d, st.ST_F32, 0, st.ST_FLAG_TC_SPLIT),
                     dtype=torch.uint8, device="cuda")
    got = expand2(st, st.st_sym_moment2(dev(X), ws=ws, flags=st.ST_FLAG_TC_SPLIT), d)
    assert st.st_check_status(ws) == st.ST_OK
    T, S = oracle.moment2(X)
    assert oracle.rel_err(got, T, S) <= TOL_F32, (N, d)
    ctl = expand2(st, st.st_sym_moment2(dev(X), ws=ws, flags=st.ST_FLAG_TC_SPLIT | st.ST_FLAG_DENSE_CONTROL), d)
    assert oracle.rel_err(ctl, T, S) <= TOL_F32
    # a row pitch wider than d, and the same result twice
    Xw = torch.zeros((N, d + 12), device="cuda")
    Xw[:, :d] = dev(X)
    out2 = torch.empty(d * (d + 1) // 2, device="cuda")
    assert st.lib().st_sym_moment2(Xw.data_ptr(), st.ST_F32, N, d, d + 12, out2.data_ptr(), ws.data_ptr(), ws.numel(),
                                   st.ST_FLAG_TC_SPLIT, None) == st.ST_OK
    assert st.st_check_status(ws) == st.ST_OK
    assert np.array_equal(expand2(st, out2, d), got)


def test_moment2_split_sums_of_squares_do_not_drift(st):
    """All-positive sums over many samples: the accumulation chain is cut often enough that the diagonal stays
    inside the fp32 tolerance (a tensor-core accumulator rounds towards zero)."""
    N, d = 200000, 64
    X = np.abs(workloads.draw((N, d), "normal", 77)) + 0.5
    got = expand2(st, st.st_sym_moment2(dev(X), flags=st.ST_FLAG_TC_SPLIT), d)
    T, S = oracle.moment2(X)
    assert oracle.rel_err(got, T, S) <= TOL_F32


def test_moment2_tf32_rejects_what_it_cannot_run(st):
    L = st.lib()
    X = torch.zeros((64, 66), device="cuda")
    out = torch.zeros(66 * 67 // 2, device="cuda")
    ws = torch.zeros(1 << 22, dtype=torch.uint8, device="cuda")
    # d not a multiple of 4
    assert L.st_sym_moment2(X.data_ptr(), st.ST_F32, 64, 66, 66, out.data_ptr(), ws.data_ptr(), ws.numel(),
                            st.ST_FLAG_TC_TF32, None) == st.ST_ERR_ALIGN
    # the flag goes with fp32 input only
    Xb = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    assert L.st_sym_moment2(Xb.data_ptr(), st.ST_BF16, 64, 64, 64, out.data_ptr(), ws.data_ptr(), ws.numel(),
                            st.ST_FLAG_TC_TF32, None) == st.ST_ERR_UNSUPPORTED


def test_moment2_bf16_all_ones(st):
    ones = torch.ones((3001, 256), dtype=torch.bfloat16, device="cuda")
    assert torch.all(st.st_sym_moment2(ones) == 3001.0)


def test_moment2_large_config(st):
    cfg = workloads.CONFIGS["moment2_large"]
    N, d = cfg["N"], cfg["d"]
    bits = workloads.draw_rows_bf16(N, d, cfg["dist"], workloads.SEEDS["moment2_large"])
    got = st.st_sym_moment2(bf16_dev(bits)).cpu().numpy()
    assert st.st_check_status() == st.ST_OK
    assert got.size == 524800
    Xb = workloads.bf16_bits_to_f32(bits).reshape(N, d)
    rng = np.random.default_rng(8)
    # sampled entries, each the full sum over 2^20 samples: in every 128 x 128 sub-block of the upper
    # triangle (so of every quadrant of every launched 256 x 256 pair tile) its first and last unique
    # entry and six seeded random ones; all diagonal entries of a stride; seeded random pairs
    pairs = [(i, i) for i in range(0, d, 37)] + [(0, d - 1), (127, 128), (128, 255), (255, 256), (511, 512), (767, 1023)]
    for bi in range(d // 128):
        for bj in range(bi, d // 128):
            sub_pairs = [(bi * 128, bj * 128), (bi * 128 + 127, bj * 128 + 127), (bi * 128, bj * 128 + 127)]
            sub_pairs += [(bi * 128 + int(a), bj * 128 + int(b)) for a, b in rng.integers(0, 128, (6, 2))]
            pairs += [(min(i, j), max(i, j)) for i, j in sub_pairs]
    pairs += [tuple(sorted(int(v) for v in rng.integers(0, d, 2))) for _ in range(200)]
    ii, jj = (np.array(v) for v in zip(*pairs))
    T, S = oracle.moment2_at(Xb, ii, jj)
    pos = ii * (2 * d - ii + 1) // 2 + (jj - ii)
    for (i, j), p in list(zip(pairs, pos))[:40]:
        assert p == oracle.locate(oracle.KIND_TRI, d, i, j)
    assert oracle.rel_err(got[pos], T, S) <= TOL_F32
    # two identities over the WHOLE packed output (they hold at any size):
    # trace: sum_i out[p(i,i)] = ||X||_F^2
    diag = np.array([i * (2 * d - i + 1) // 2 for i in range(d)])
    Xd_sq = 0.0
    row_sum_sq = row_abs_sq = 0.0
    for r0 in range(0, N, 1 << 16):                 # chunks keep the fp64 copies small
        blk = Xb[r0:r0 + (1 << 16)].astype(np.float64)
        Xd_sq += float(np.sum(blk * blk))
        row_sum_sq += float(np.sum(blk.sum(axis=1) ** 2))
        row_abs_sq += float(np.sum(np.abs(blk).sum(axis=1) ** 2))
    g64 = got.astype(np.float64)
    assert abs(float(g64[diag].sum()) - Xd_sq) <= TOL_F32 * Xd_sq
    # every entry: sum_{i,j} T[i,j] = 2 * sum_{i<j} + sum_i = sum_n (sum_i x_i)^2
    weight = np.full(got.size, 2.0)
    weight[diag] = 1.0
    assert abs(float(np.dot(weight, g64)) - row_sum_sq) <= TOL_F32 * row_abs_sq
    del Xb
    # the stated 5e-3 bound of the bf16 path is against the fp32 data that the bf16 copy was rounded from
    X32 = workloads.draw_rows(N, d, cfg["dist"], workloads.SEEDS["moment2_large"])
    assert np.array_equal(workloads.f32_to_bf16_bits(X32[:4096]), bits[:4096])
    T32, S32 = oracle.moment2_at(X32, ii, jj)
    assert oracle.rel_err(got[pos], T32, S32) <= TOL_TC


@pytest.mark.parametrize("nb,bs,K,R", [(1, 1, 4, 16), (3, 2, 8, 16), (2, 5, 36, 32), (4, 8, 64, 64), (7, 3, 32, 48),
                                       (2, 17, 100, 128), (5, 12, 256, 64)])
def test_ttm_tf32_tensor_core_small(st, nb, bs, K, R):
    Bp, U = workloads.ttm_inputs(nb, bs, K, R)
    A, S = oracle.ttm(Bp.reshape(-1, K), U)
    got = st.st_ttm_blockdiag(dev(Bp), dev(U), nb, bs, flags=st.ST_FLAG_TC_TF32).cpu().numpy()
    assert oracle.rel_err(got, A, S) <= TOL_TC
    assert st.st_check_status() == st.ST_OK


def test_ttm_tf32_config(st, ttm_config_oracle):
    Bp, U, A, S = ttm_config_oracle
    got = st.st_ttm_blockdiag(dev(Bp), dev(U), 64, 64, flags=st.ST_FLAG_TC_TF32).cpu().numpy()
    assert oracle.rel_err(got, A, S) <= TOL_TC           # every fibre of all 2,048 tiles, every column
    assert st.st_check_status() == st.ST_OK


def test_ttm_tf32_sixteen_columns_many_tiles(st):
    # R = 16 with more tiles than thread blocks: every block alternates between both accumulator
    # buffers in tensor memory, the second of which starts at column 16
    nb, bs, K, R = 5, 72, 32, 16
    assert nb * bs * bs > 160 * 128
    Bp, U = workloads.ttm_inputs(nb, bs, K, R)
    A, S = oracle.ttm(Bp.reshape(-1, K), U)
    got = st.st_ttm_blockdiag(dev(Bp), dev(U), nb, bs, flags=st.ST_FLAG_TC_TF32).cpu().numpy()
    assert oracle.rel_err(got, A, S) <= TOL_TC
    assert st.st_check_status() == st.ST_OK


# split-bf16 tensor-core path of TTM and MTTKRP: both operands as hi + lo bf16 parts, three partial
# products: held to the fp32 tolerance

@pytest.mark.parametrize("nb,bs,K,R", [(1, 1, 4, 32), (3, 2, 8, 32), (2, 5, 36, 32), (4, 8, 64, 64), (7, 3, 32, 96),
                                       (2, 17, 100, 128), (5, 12, 256, 64), (3, 9, 520, 32), (1, 40, 768, 32)])
def test_ttm_split_tensor_core_small(st, nb, bs, K, R):
    Bp, U = workloads.ttm_inputs(nb, bs, K, R)
    A, S = oracle.ttm(Bp.reshape(-1, K), U)
    got = st.st_ttm_blockdiag(dev(Bp), dev(U), nb, bs, flags=st.ST_FLAG_TC_SPLIT).cpu().numpy()
    assert st.st_check_status() == st.ST_OK
    assert oracle.rel_err(got, A, S) <= TOL_F32


def test_ttm_split_many_tiles_both_accumulators_and_limits(st):
    nb, bs, K, R = 5, 72, 96, 32          # 25,920 fibres = 203 tiles: every block uses both accumulator buffers
    Bp, U = workloads.ttm_inputs(nb, bs, K, R)
    A, S = oracle.ttm(Bp.reshape(-1, K), U)
    got = st.st_ttm_blockdiag(dev(Bp), dev(U), nb, bs, flags=st.ST_FLAG_TC_SPLIT).cpu().numpy()
    assert st.st_check_status() == st.ST_OK
    assert oracle.rel_err(got, A, S) <= TOL_F32
    # all-positive operands: the worst case for a rounding bias of the accumulation
    Bpos, Upos = np.abs(Bp) + 0.5, np.abs(U) + 0.5
    A, S = oracle.ttm(Bpos.reshape(-1, K), Upos)
    got = st.st_ttm_blockdiag(dev(Bpos), dev(Upos), nb, bs, flags=st.ST_FLAG_TC_SPLIT).cpu().numpy()
    assert oracle.rel_err(got, A, S) <= TOL_F32
    # shapes the path does not take, and the two tensor-core flags together
    L, s = st.lib(), torch.cuda.current_stream().cuda_stream
    x = torch.zeros(1 << 20, device="cuda")
    ws = guarded(st, 4096, torch.uint8)
    SP = st.ST_FLAG_TC_SPLIT
    assert L.st_ttm_blockdiag(x.data_ptr(), 2, 2, 8, x.data_ptr(), 48, x.data_ptr(), ws.data_ptr(), 4096, SP, s) == st.ST_ERR_UNSUPPORTED
    assert L.st_ttm_blockdiag(x.data_ptr(), 2, 2, 4096, x.data_ptr(), 32, x.data_ptr(), ws.data_ptr(), 4096, SP, s) == st.ST_ERR_UNSUPPORTED
    assert L.st_ttm_blockdiag(x.data_ptr(), 2, 2, 8, x.data_ptr(), 32, x.data_ptr(), ws.data_ptr(), 4096,
                              SP | st.ST_FLAG_TC_TF32, s) == st.ST_ERR_UNSUPPORTED
    assert st.st_workspace_bytes(st.ST_OP_TTM_BLOCKDIAG, 2, 2, 8, 48, SP) == 0


def test_ttm_split_config(st, ttm_config_oracle):
    Bp, U, A, S = ttm_config_oracle
    got = st.st_ttm_blockdiag(dev(Bp), dev(U), 64, 64, flags=st.ST_FLAG_TC_SPLIT).cpu().numpy()
    assert st.st_check_status() == st.ST_OK
    assert oracle.rel_err(got, A, S) <= TOL_F32          # every fibre, every column, at the fp32 tolerance


@pytest.mark.parametrize("I,K,R", [(1, 4, 32), (5, 36, 32), (16, 64, 64), (40, 100, 32), (70, 32, 96), (33, 68, 64),
                                   (130, 8, 128)])
def test_mttkrp_split_tensor_core_small(st, I, K, R):
    Bp, C, D = workloads.mttkrp_inputs(I, K, R)
    Bd = oracle.unpack(Bp.reshape(-1), oracle.KIND_TRI, I, inner=K)
    A, S = oracle.mttkrp(Bd, C, D)
    got = st.st_mttkrp_tri(dev(Bp), dev(C), dev(D), flags=st.ST_FLAG_TC_SPLIT).cpu().numpy()
    assert st.st_check_status() == st.ST_OK
    assert oracle.rel_err(got, A, S) <= TOL_F32
    ctl = st.st_mttkrp_tri(dev(Bd), dev(C), dev(D), flags=st.ST_FLAG_TC_SPLIT | st.ST_FLAG_DENSE_CONTROL).cpu().numpy()
    assert oracle.rel_err(ctl, A, S) <= TOL_F32


def test_mttkrp_split_config(st, mttkrp_config_oracle):
    Bp, C, D, A, S = mttkrp_config_oracle
    got = st.st_mttkrp_tri(dev(Bp), dev(C), dev(D), flags=st.ST_FLAG_TC_SPLIT)
    assert st.st_check_status() == st.ST_OK
    assert oracle.rel_err(got.cpu().numpy(), A, S) <= TOL_F32      # every (i, r), at the fp32 tolerance
    assert torch.equal(got, st.st_mttkrp_tri(dev(Bp), dev(C), dev(D), flags=st.ST_FLAG_TC_SPLIT))


def test_moment2_bf16_all_tiles_midsize(st):
    """d = 1024 (all 20 launched tiles, both diagonal and off-diagonal kinds) at a sample count
    the oracle can still check on sampled entries quickly; input 256 MiB, larger than L2."""
    N, d = 131072, 1024
    bits = workloads.draw_rows_bf16(N, d, "normal", 4242)
    got = st.st_sym_moment2(bf16_dev(bits)).cpu().numpy()
    Xb = workloads.bf16_bits_to_f32(bits).reshape(N, d)
    rng = np.random.default_rng(9)
    pairs = [(i, i) for i in range(0, d, 61)] + [(r * 128 + a, c * 256 + b) for r in range(8) for c in range(4)
                                                 for a, b in ((0, 0), (127, 255), (5, 200)) if r * 128 + a <= c * 256 + b]
    pairs += [tuple(sorted(int(v) for v in rng.integers(0, d, 2))) for _ in range(200)]
    ii, jj = (np.array(v) for v in zip(*pairs))
    T, S = oracle.moment2_at(Xb, ii, jj)
    pos = ii * (2 * d - ii + 1) // 2 + (jj - ii)
    assert oracle.rel_err(got[pos], T, S) <= TOL_F32


@pytest.mark.parametrize("I,K,R", [(1, 4, 32), (5, 36, 32), (16, 64, 64), (40, 100, 32), (70, 32, 96), (33, 68, 64)])
def test_mttkrp_tf32_tensor_core_small(st, I, K, R):
    Bp, C, D = workloads.mttkrp_inputs(I, K, R)
    Bd = oracle.unpack(Bp.reshape(-1), oracle.KIND_TRI, I, inner=K)
    A, S = oracle.mttkrp(Bd, C, D)
    got = st.st_mttkrp_tri(dev(Bp), dev(C), dev(D), flags=st.ST_FLAG_TC_TF32).cpu().numpy()
    assert st.st_check_status() == st.ST_OK
    assert oracle.rel_err(got, A, S) <= TOL_TC
    ctl = st.st_mttkrp_tri(dev(Bd), dev(C), dev(D), flags=st.ST_FLAG_TC_TF32 | st.ST_FLAG_DENSE_CONTROL).cpu().numpy()
    assert oracle.rel_err(ctl, A, S) <= TOL_TC


def test_mttkrp_tf32_config(st, mttkrp_config_oracle):
    Bp, C, D, A, S = mttkrp_config_oracle
    got = st.st_mttkrp_tri(dev(Bp), dev(C), dev(D), flags=st.ST_FLAG_TC_TF32).cpu().numpy()
    assert oracle.rel_err(got, A, S) <= TOL_TC           # every (i, r)
    assert st.st_check_status() == st.ST_OK


# ------------------------------------------------------------------------------ other structures of Table 1

def _table1_layouts(st, K):
    return [st.Layout(st.ST_TRI_UPPER, 13, inner=K),                      # upper half cube (i <= j)
            st.Layout(st.ST_BLOCKDIAG, 37, inner=K, nblocks=37, bs=1),     # diagonal plane (i = j)
            st.Layout(st.ST_FIXED_ROW, 19, inner=K, kl=7),                 # Table 1 "fixed i"
            st.Layout(st.ST_FIXED_COL, 45, inner=K, kl=44),                # Table 1 "fixed j"
            st.Layout(st.ST_BAND, 21, inner=K, kl=2, ku=1),
            st.Layout(st.ST_BLOCKDIAG, 24, inner=K, nblocks=3, bs=8),
            st.Layout(st.ST_TET, 7, inner=K)]


def _okind(st, lay):
    return {st.ST_TRI_UPPER: oracle.KIND_TRI, st.ST_TET: oracle.KIND_TET, st.ST_BAND: oracle.KIND_BAND,
            st.ST_BLOCKDIAG: oracle.KIND_BLOCKDIAG, st.ST_FIXED_ROW: oracle.KIND_FIXED_ROW,
            st.ST_FIXED_COL: oracle.KIND_FIXED_COL, st.ST_SIMPLEX4: oracle.KIND_SIMPLEX4}[lay.kind]


@pytest.mark.parametrize("flag_name,K,R", [("f32", 36, 32), ("f32", 64, 8), ("tf32", 64, 32), ("tf32", 36, 48),
                                           ("split", 36, 32), ("split", 64, 64)])
def test_ttm_on_every_structure_of_the_first_two_modes(st, flag_name, K, R):
    flags = {"tf32": st.ST_FLAG_TC_TF32, "split": st.ST_FLAG_TC_SPLIT, "f32": 0}[flag_name]
    for n, lay in enumerate(_table1_layouts(st, K)):
        rows = st.st_packed_elems(lay) // K
        Bp = workloads.draw((rows, K), "normal", 800 + n)
        U = workloads.draw((K, R), "normal", 850 + n)
        if lay.kind == st.ST_BAND:      # slots outside the matrix hold zeros in a packed band
            Bp = oracle.pack(oracle.unpack(Bp.reshape(-1), oracle.KIND_BAND, lay.d, inner=K, **okw(lay)),
                             oracle.KIND_BAND, lay.d, inner=K, **okw(lay)).reshape(rows, K)
        # oracle: the dense tensor (zeros outside the structure) times U over the full iteration space,
        # then the structured part of the result
        Bd = oracle.unpack(Bp.reshape(-1), _okind(st, lay), lay.d, inner=K, **okw(lay))
        A, S = oracle.ttm(Bd, U)
        want = oracle.pack(A, _okind(st, lay), lay.d, inner=R, **okw(lay)).reshape(rows, R)
        scale = oracle.pack(S, _okind(st, lay), lay.d, inner=R, **okw(lay)).reshape(rows, R)
        got = st.st_ttm_packed(dev(Bp), dev(U), lay, flags=flags).cpu().numpy()
        assert st.st_check_status() == st.ST_OK
        assert oracle.rel_err(got, want, scale) <= (5e-3 if flag_name == "tf32" else TOL_F32), (flag_name, n)
        # everything outside the structure of the dense result is exactly zero (output keeps B's structure)
        mask = oracle.unpack(np.ones(rows * R, np.float32), _okind(st, lay), lay.d, inner=R, **okw(lay))
        assert np.all(A[mask == 0] == 0)


def test_thp_structured_times_dense(st):
    for n, lay in enumerate(_table1_layouts(st, 12) + [st.Layout(st.ST_TRI_UPPER, 300, inner=5)]):
        K = lay.inner
        elems = st.st_packed_elems(lay)
        Bp = workloads.draw((elems,), "normal", 900 + n)
        Cd = workloads.draw((st.st_dense_elems(lay),), "uniform", 950 + n)
        if lay.kind == st.ST_BAND:
            Bp = oracle.pack(oracle.unpack(Bp, oracle.KIND_BAND, lay.d, inner=K, **okw(lay)), oracle.KIND_BAND, lay.d,
                             inner=K, **okw(lay))
        Bd = oracle.unpack(Bp, _okind(st, lay), lay.d, inner=K, **okw(lay))
        A, _ = oracle.thp(Bd, Cd.reshape(Bd.shape))
        want = oracle.pack(A.astype(np.float32), _okind(st, lay), lay.d, inner=K, **okw(lay))
        got = st.st_thp(dev(Bp), dev(Cd), lay).cpu().numpy()
        # one fp32 multiplication of two fp32 numbers: the correctly rounded product, bit for bit
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), n
        # the dense result is zero wherever B is (the product keeps B's structure)
        mask = oracle.unpack(np.ones(elems, np.float32), _okind(st, lay), lay.d, inner=K, **okw(lay))
        assert np.all(A[mask == 0] == 0)


@pytest.mark.parametrize("flag_name,I,J,K,R", [("f32", 5, 7, 36, 32), ("f32", 300, 40, 64, 8), ("f32", 33, 700, 32, 64),
                                               ("tf32", 5, 7, 36, 32), ("tf32", 300, 260, 64, 64), ("tf32", 1, 1, 4, 32),
                                               ("split", 5, 7, 36, 32), ("split", 300, 260, 64, 64)])
def test_mttkrp_on_slice_structures(st, flag_name, I, J, K, R):
    flags = {"tf32": st.ST_FLAG_TC_TF32, "split": st.ST_FLAG_TC_SPLIT, "f32": 0}[flag_name]
    tol = 5e-3 if flag_name == "tf32" else TOL_F32
    C = workloads.draw((J, R), "uniform", 1100)
    D = workloads.draw((K, R), "uniform", 1101)
    i0, j0 = I // 2, J - 1
    for fi, fj in ((i0, -1), (-1, j0), (i0, j0)):
        rows = (1 if fj >= 0 else J) if fi >= 0 else I
        Bp = workloads.draw((rows, K), "normal", 1102 + rows)
        # oracle: the dense tensor with the slice in place, full iteration space
        Bd = np.zeros((I, J, K), np.float32)
        if fi >= 0 and fj >= 0: Bd[fi, fj, :] = Bp[0]
        elif fi >= 0: Bd[fi, :, :] = Bp
        else: Bd[:, fj, :] = Bp
        A, S = oracle.mttkrp(Bd, C, D)
        got = torch.full((I, R), float("nan"), dtype=torch.float32, device="cuda")
        st.st_mttkrp_slice(dev(Bp), dev(C), dev(D), I, fi, fj, out=got, flags=flags)
        assert st.st_check_status() == st.ST_OK
        assert oracle.rel_err(got.cpu().numpy(), A, S) <= tol, (flag_name, fi, fj)     # rows outside the slice: exactly 0


# ------------------------------------------------------------------------------ chains in compressed space

def test_chain_in_packed_space_with_one_reconstruction_at_the_end(st):
    # covariance blocks of three batches are added up in packed space, scaled, multiplied position by
    # position by a packed upper-triangular mask, and only then reconstructed (Section 5.5)
    d = 24
    batches = [workloads.draw((n, d), "normal", 1200 + n) for n in (700, 1300, 64)]
    acc = None
    for Xb in batches:
        m = st.st_sym_moment2(dev(Xb))
        acc = m if acc is None else st.st_packed_axpby(1.0, acc, 1.0, m, out=acc)
    total = sum(b.shape[0] for b in batches)
    acc = st.st_packed_axpby(1.0 / total, acc, 0.0, acc, out=acc)
    W = workloads.draw((workloads.tri(d),), "uniform", 1299)
    prod = st.st_packed_mul(acc, dev(W))
    full = st.st_unpack(prod, st.Layout(st.ST_TRI_UPPER, d), fill=st.ST_FILL_SYMMETRIC).cpu().numpy().reshape(d, d)
    # oracle: dense second moment of all samples, scaled, times the symmetric expansion of W
    T, S = oracle.moment2(np.concatenate(batches))
    Wd = oracle.unpack(W, oracle.KIND_TRI, d, fill=oracle.FILL_SYMMETRIC).astype(np.float64)
    assert oracle.rel_err(full, T / total * Wd, S / total * np.abs(Wd)) <= 2 * TOL_F32
    # third moments of two batches added in packed space equal the third moment of their union
    Xa, Xb = workloads.draw((900, 16), "normal", 1251), workloads.draw((333, 16), "normal", 1252)
    m3 = st.st_packed_axpby(1.0, st.st_sym_moment3(dev(Xa)), 1.0, st.st_sym_moment3(dev(Xb)))
    T3, S3 = oracle.moment3(np.concatenate([Xa, Xb]))
    assert oracle.rel_err(expand3(st, m3, 16), T3, S3) <= TOL_F32
    # odd sizes and aliasing
    a, b = dev(workloads.draw((1003,), "normal", 1)), dev(workloads.draw((1003,), "normal", 2))
    want = (2.0 * a.double() - 0.5 * b.double()).float()
    assert torch.allclose(st.st_packed_axpby(2.0, a, -0.5, b), want, rtol=1e-6, atol=1e-6)
    assert torch.equal(st.st_packed_mul(a, b, out=a.clone()), a * b)


def test_thp_and_ttm_packed_at_the_benchmark_size(st):
    # the packed upper-half-cube operand of the benchmark (131,328 fibres of 512) times its own dense expansion
    Bp, _, _ = workloads.mttkrp_inputs()
    I, K = 512, 512
    lay = st.Layout(st.ST_TRI_UPPER, I, inner=K)
    Bd = oracle.unpack(Bp.reshape(-1), oracle.KIND_TRI, I, inner=K)
    got = st.st_thp(dev(Bp).view(-1), dev(Bd).view(-1), lay).cpu().numpy()
    assert np.array_equal(got, (Bp.astype(np.float64) ** 2).astype(np.float32).reshape(-1))
    # TTM of the same operand on sampled fibres (first, last, row starts, seeded random)
    U = workloads.draw((K, 64), "normal", 1300)
    A = st.st_ttm_packed(dev(Bp), dev(U), lay, flags=st.ST_FLAG_TC_TF32).cpu().numpy()
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 511, 512, Bp.shape[0] - 1], rng.integers(0, Bp.shape[0], 300)]))
    T, S = oracle.ttm(Bp[rows], U)
    assert oracle.rel_err(A[rows], T, S) <= 5e-3
