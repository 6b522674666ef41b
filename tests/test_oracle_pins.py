"""Pins for the CPU oracle: everything here runs without a GPU and checks the
oracle against things other than itself -- values printed in the paper, closed
forms, brute force in pure Python on tiny inputs, invariants, and textbook
library routines (numpy fp64 matmul / einsum)."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_counts.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = int(v)
    return out


def rnd(shape, seed, dist="normal"):
    return workloads.draw(shape, dist, seed)


# --------------------------------------------------------------------------- moments

def brute_moment(X, order):
    N, d = X.shape
    T = np.zeros((d,) * order)
    S = np.zeros((d,) * order)
    for idx in itertools.product(range(d), repeat=order):
        t = s = 0.0
        for n in range(N):
            term = 1.0
            for a in idx:
                term *= float(X[n, a])
            t += term
            s += abs(term)
        T[idx] = t
        S[idx] = s
    return T, S


@pytest.mark.parametrize("N,d", [(1, 1), (3, 2), (5, 4), (4, 5)])
def test_moments_brute_force(N, d):
    X = rnd((N, d), 7 + N + d)
    for order, fn in ((2, oracle.moment2), (3, oracle.moment3), (4, oracle.moment4)):
        T, S = fn(X)
        Tb, Sb = brute_moment(X, order)
        np.testing.assert_allclose(T, Tb, rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(S, Sb, rtol=1e-13, atol=1e-13)


def test_moments_all_ones_equal_N():
    X = np.ones((37, 6), np.float32)
    for fn in (oracle.moment2, oracle.moment3, oracle.moment4):
        T, S = fn(X)
        assert np.all(T == 37.0) and np.all(S == 37.0)


def test_moment2_is_textbook_gram_matrix():
    X = rnd((257, 19), 3)
    T, S = oracle.moment2(X)
    Xd = X.astype(np.float64)
    np.testing.assert_allclose(T, Xd.T @ Xd, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(S, np.abs(Xd).T @ np.abs(Xd), rtol=1e-12)
    assert abs(np.trace(T) - np.sum(Xd * Xd)) < 1e-9
    assert abs(T.sum() - np.sum(Xd.sum(axis=1) ** 2)) < 1e-8
    assert np.array_equal(T, T.T)


def test_moment2_at_matches_definition_on_samples():
    X = rnd((300, 11), 5)
    Xd = X.astype(np.float64)
    ii = np.array([0, 3, 10, 7, 2])
    jj = np.array([0, 9, 10, 1, 2])
    T, S = oracle.moment2_at(X, ii, jj)
    G = Xd.T @ Xd
    np.testing.assert_allclose(T, G[ii, jj], rtol=1e-12)
    np.testing.assert_allclose(S, (np.abs(Xd).T @ np.abs(Xd))[ii, jj], rtol=1e-12)
    with pytest.raises(IndexError):
        oracle.moment2_at(X, np.array([11]), np.array([0]))


def test_moment3_einsum_permutations_and_multiplicity_identity():
    X = rnd((101, 7), 11)
    Xd = X.astype(np.float64)
    T, S = oracle.moment3(X)
    np.testing.assert_allclose(T, np.einsum("ni,nj,nk->ijk", Xd, Xd, Xd), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(S, np.einsum("ni,nj,nk->ijk", *(np.abs(Xd),) * 3), rtol=1e-11)
    for perm in itertools.permutations(range(3)):
        np.testing.assert_allclose(T, T.transpose(perm), rtol=1e-12, atol=1e-12)
    # sum over the unique set weighted by the orbit size equals sum_n (sum_i x)^3
    d = 7
    acc = 0.0
    for i in range(d):
        for j in range(i, d):
            for k in range(j, d):
                distinct = len({i, j, k})
                mult = {1: 1, 2: 3, 3: 6}[distinct]
                acc += mult * T[i, j, k]
    assert abs(acc - np.sum(Xd.sum(axis=1) ** 3)) < 1e-8
    assert abs(acc - T.sum()) < 1e-8


def test_moment3_at_matches_definition_on_samples():
    X = rnd((90, 6), 17)
    Xd = X.astype(np.float64)
    ii, jj, kk = np.array([0, 1, 5, 2]), np.array([0, 3, 5, 2]), np.array([0, 4, 5, 5])
    T, S = oracle.moment3_at(X, ii, jj, kk)
    full = np.einsum("ni,nj,nk->ijk", Xd, Xd, Xd)
    np.testing.assert_allclose(T, full[ii, jj, kk], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(S, np.einsum("ni,nj,nk->ijk", *(np.abs(Xd),) * 3)[ii, jj, kk], rtol=1e-12)


def test_moment3_d1_is_sum_of_cubes():
    X = rnd((64, 1), 2)
    T, S = oracle.moment3(X)
    assert abs(T[0, 0, 0] - np.sum(X.astype(np.float64) ** 3)) < 1e-12
    assert abs(S[0, 0, 0] - np.sum(np.abs(X.astype(np.float64)) ** 3)) < 1e-12


def test_moment4_at_is_the_dense_sum_at_sampled_entries():
    X = workloads.draw((37, 6), "normal", 21)
    T, S = oracle.moment4(X)
    idx = [(i, j, k, l) for i in range(6) for j in range(6) for k in range(6) for l in range(6)][::7]
    ii, jj, kk, ll = (np.array(v) for v in zip(*idx))
    t, sabs = oracle.moment4_at(X, ii, jj, kk, ll)
    assert np.array_equal(t, T[ii, jj, kk, ll]) and np.array_equal(sabs, S[ii, jj, kk, ll])
    # d = 1 reduces to a plain sum of fourth powers
    x = workloads.draw((50, 1), "uniform", 22)
    t1, _ = oracle.moment4_at(x, [0], [0], [0], [0])
    assert abs(t1[0] - float(np.sum(x.astype(np.float64) ** 4))) <= 1e-12


def test_moment4_einsum():
    X = rnd((33, 5), 13)
    Xd = X.astype(np.float64)
    T, S = oracle.moment4(X)
    np.testing.assert_allclose(T, np.einsum("ni,nj,nk,nl->ijkl", Xd, Xd, Xd, Xd), rtol=1e-11, atol=1e-11)


def test_pr2_covariance_has_65_distinct_elements():
    """Section 2 / Section 3: x = f (+) vec(f (x) f); Sigma = x (x) x is 20 x 20 with
    65 distinct values, and its blocks are the order-2/3/4 moments of f."""
    g = golden()
    n = g["pr2_features"]
    f = np.array([[2.0, 3.0, 5.0, 7.0]], np.float32)  # distinct primes: products collide only by symmetry
    x = np.concatenate([f[0], np.outer(f[0], f[0]).reshape(-1)])[None, :].astype(np.float32)
    assert x.shape[1] == g["pr2_cov_dim"]
    Sigma, _ = oracle.moment2(x)
    assert Sigma.shape == (g["pr2_cov_dim"],) * 2
    assert len(np.unique(Sigma)) == g["pr2_distinct"]
    # the unique-set sizes add up to the same number, counted by walking T_U
    n2 = oracle.packed_rows(oracle.KIND_TRI, n)
    n3 = oracle.packed_rows(oracle.KIND_TET, n)
    n4 = sum(1 for _ in itertools.combinations_with_replacement(range(n), 4))
    assert n2 + n3 + n4 == g["pr2_distinct"]
    # blocks of Sigma are M1, M2, M3 (Section 3): ties moment3 / moment4 to moment2
    M1, _ = oracle.moment2(f)
    M2, _ = oracle.moment3(f)
    M3, _ = oracle.moment4(f)
    assert np.array_equal(Sigma[:n, :n], M1)
    assert np.array_equal(Sigma[:n, n:], M2.reshape(n, n * n))
    assert np.array_equal(Sigma[n:, n:], M3.reshape(n * n, n * n))


def test_redundancy_ratios_stated_in_the_paper():
    g = golden()
    r2 = [d * d / oracle.packed_rows(oracle.KIND_TRI, d) for d in (8, 64, 200)]
    assert all(1.7 < r <= 2.0 for r in r2) and round(r2[-1]) == g["ratio_upper_tri"]
    r3 = {d: d ** 3 / oracle.packed_rows(oracle.KIND_TET, d) for d in (4, 20, 64)}
    assert round(r3[20]) == g["ratio_M2"] and r3[64] < 6.0
    r4 = 100 ** 4 / math.comb(100 + 3, 4)
    assert round(r4) == g["ratio_M3"]


# --------------------------------------------------------------------------- MTTKRP / TTM

def test_mttkrp_brute_force_and_einsum():
    I, J, K, R = 3, 4, 5, 2        # all extents different: a swapped operand cannot pass
    B, C, D = rnd((I, J, K), 1), rnd((J, R), 2), rnd((K, R), 3)
    A, S = oracle.mttkrp(B, C, D)
    Ab = np.zeros((I, R))
    Sb = np.zeros((I, R))
    for i in range(I):
        for r in range(R):
            for j in range(J):
                for k in range(K):
                    t = float(B[i, j, k]) * float(C[j, r]) * float(D[k, r])
                    Ab[i, r] += t
                    Sb[i, r] += abs(t)
    np.testing.assert_allclose(A, Ab, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(S, Sb, rtol=1e-13)
    Bd, Cd, Dd = (a.astype(np.float64) for a in (B, C, D))
    np.testing.assert_allclose(A, np.einsum("ijk,jr,kr->ir", Bd, Cd, Dd), rtol=1e-12, atol=1e-12)
    A1, S1 = oracle.mttkrp(B, C, D, 1, 3)
    assert np.array_equal(A1, A[1:3]) and np.array_equal(S1, S[1:3])


def test_mttkrp_closed_forms():
    I = J = 6
    K, R = 5, 3
    # B = 1 on i<=j, C = D = 1  =>  A[i,r] = (J - i) * K
    B = np.zeros((I, J, K), np.float32)
    for i in range(I):
        B[i, i:, :] = 1.0
    A, S = oracle.mttkrp(B, np.ones((J, R), np.float32), np.ones((K, R), np.float32))
    for i in range(I):
        assert np.all(A[i] == (J - i) * K) and np.all(S[i] == (J - i) * K)
    # B non-zero only at i=j=k (Section 5.4, diagonal tensor): A[i,r] = B[i,i,i] C[i,r] D[i,r]
    n = 5
    Bd = np.zeros((n, n, n), np.float32)
    diag = rnd((n,), 4)
    for i in range(n):
        Bd[i, i, i] = diag[i]
    C, D = rnd((n, R), 5), rnd((n, R), 6)
    A, _ = oracle.mttkrp(Bd, C, D)
    np.testing.assert_allclose(A, diag[:, None].astype(np.float64) * C * D, rtol=1e-13)


def test_ttm_brute_force_einsum_identity():
    I, J, K, R = 3, 4, 5, 6
    B, U = rnd((I, J, K), 8), rnd((K, R), 9)
    A, S = oracle.ttm(B, U)
    Ab = np.zeros((I, J, R))
    for i in range(I):
        for j in range(J):
            for r in range(R):
                for k in range(K):
                    Ab[i, j, r] += float(B[i, j, k]) * float(U[k, r])
    np.testing.assert_allclose(A, Ab, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(A, np.einsum("ijk,kr->ijr", B.astype(np.float64), U.astype(np.float64)),
                               rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(S, np.einsum("ijk,kr->ijr", np.abs(B).astype(np.float64),
                                            np.abs(U).astype(np.float64)), rtol=1e-12)
    Aid, _ = oracle.ttm(B, np.eye(K, dtype=np.float32))
    assert np.array_equal(Aid, B.astype(np.float64))


def test_ttm_keeps_block_diagonal_structure():
    """Unique-set inference for a product + projection (Figure "inference rules for
    unique set"): A_U(i,j,r) = B_U(i,j,.), so off-block outputs are exactly zero."""
    nb, bs, K, R = 3, 2, 4, 3
    Bp, U = workloads.ttm_inputs(nb, bs, K, R)
    d = nb * bs
    Bdense = oracle.unpack(Bp.reshape(-1), oracle.KIND_BLOCKDIAG, d, inner=K, nb=nb, bs=bs)
    A, S = oracle.ttm(Bdense, U)
    for i in range(d):
        for j in range(d):
            if i // bs != j // bs:
                assert np.all(A[i, j] == 0) and np.all(S[i, j] == 0)
            else:
                assert np.any(A[i, j] != 0)
    # bs = 1 is the "diagonal (plane)" row of Table 1
    Bp1, U1 = workloads.ttm_inputs(5, 1, K, R)
    B1 = oracle.unpack(Bp1.reshape(-1), oracle.KIND_BLOCKDIAG, 5, inner=K, nb=5, bs=1)
    A1, _ = oracle.ttm(B1, U1)
    for i in range(5):
        np.testing.assert_allclose(A1[i, i], Bp1[i, 0, 0].astype(np.float64) @ U1.astype(np.float64), rtol=1e-12)
        for j in range(5):
            if i != j:
                assert np.all(A1[i, j] == 0)


def test_thp_brute_force_and_closed_forms():
    """THP of Table 1: A(i,j,k) = B(i,j,k) * C(i,j,k).  Pinned by a pure-Python triple loop on a tensor
    with three different extents, by B = 1 (the product is C itself), and by a B that is non-zero on
    the diagonal plane i = j only (the unique set of a product is the intersection of the operands'
    unique sets, Section 5.1: the result is zero off the plane and b_i * C(i,i,k) on it)."""
    I, J, K = 3, 4, 5
    B, C = rnd((I, J, K), 21), rnd((I, J, K), 22, "uniform")
    A, S = oracle.thp(B, C)
    assert A.dtype == np.float64 and A.shape == (I, J, K)
    for i in range(I):
        for j in range(J):
            for k in range(K):
                want = float(B[i, j, k]) * float(C[i, j, k])      # exact in fp64: two 24-bit significands
                assert A[i, j, k] == want and S[i, j, k] == abs(want)
    # the operands are not interchangeable with their transposes: a reshaped or transposed C fails this
    assert not np.array_equal(A, oracle.thp(B, np.ascontiguousarray(C.transpose(0, 2, 1)).reshape(I, J, K))[0])
    A1, _ = oracle.thp(np.ones((I, J, K), np.float32), C)
    assert np.array_equal(A1, C.astype(np.float64))
    d = 4
    b = rnd((d,), 23)
    Bd = np.zeros((d, d, K), np.float32)
    for i in range(d):
        Bd[i, i, :] = b[i]
    Cd = rnd((d, d, K), 24)
    Ad, Sd = oracle.thp(Bd, Cd)
    for i in range(d):
        for j in range(d):
            if i == j:
                assert np.array_equal(Ad[i, i], np.float64(b[i]) * Cd[i, i].astype(np.float64))
            else:
                assert np.all(Ad[i, j] == 0) and np.all(Sd[i, j] == 0)
    # widening happens before the product: the fp64 product of two fp32 numbers is not the fp32 one
    x = np.array([[[1.0 + 2.0 ** -23]]], np.float32)
    assert oracle.thp(x, x)[0][0, 0, 0] == (1.0 + 2.0 ** -23) ** 2 != float(np.float32(x[0, 0, 0] * x[0, 0, 0]))
    with pytest.raises(AssertionError):
        oracle.thp(B, C[:, :, :4])


# --------------------------------------------------------------------------- layouts

def test_unique_set_counts_closed_forms():
    for d in range(1, 40):
        assert oracle.packed_rows(oracle.KIND_TRI, d) == math.comb(d + 1, 2) == workloads.tri(d)
        assert oracle.packed_rows(oracle.KIND_TET, d) == math.comb(d + 2, 3) == workloads.tet(d)
    assert oracle.packed_rows(oracle.KIND_TRI, 64) == 2080
    assert oracle.packed_rows(oracle.KIND_TET, 64) == 45760
    assert oracle.packed_rows(oracle.KIND_TRI, 1024) == 524800
    assert oracle.packed_rows(oracle.KIND_BAND, 9, kl=2, ku=3) == 9 * 6
    assert oracle.packed_rows(oracle.KIND_BLOCKDIAG, 12, nb=3, bs=4) == 48
    assert oracle.packed_rows(oracle.KIND_BLOCKDIAG, 13, nb=3, bs=4) == -1


def in_unique(kind, idx, d, kl=0, ku=0, bs=1):
    if kind == oracle.KIND_TRI:
        return idx[0] <= idx[1]
    if kind == oracle.KIND_TET:
        return idx[0] <= idx[1] <= idx[2]
    if kind == oracle.KIND_SIMPLEX4:
        return idx[0] <= idx[1] <= idx[2] <= idx[3]
    if kind == oracle.KIND_BAND:
        return idx[0] - kl <= idx[1] <= idx[0] + ku
    if kind == oracle.KIND_FIXED_ROW:       # R_r of Figure "matrix structures": the fixed index travels in kl
        return idx[0] == kl
    if kind == oracle.KIND_FIXED_COL:       # C_c
        return idx[1] == kl
    return idx[0] // bs == idx[1] // bs


def order_of(kind):
    return {oracle.KIND_TET: 3, oracle.KIND_SIMPLEX4: 4}.get(kind, 2)


LAYOUTS = [
    (oracle.KIND_TRI, 7, {}), (oracle.KIND_TET, 5, {}),
    (oracle.KIND_BAND, 8, dict(kl=2, ku=1)), (oracle.KIND_BAND, 4, dict(kl=5, ku=0)),
    (oracle.KIND_BLOCKDIAG, 6, dict(nb=3, bs=2)),
    (oracle.KIND_FIXED_ROW, 5, dict(kl=3)), (oracle.KIND_FIXED_COL, 6, dict(kl=0)), (oracle.KIND_FIXED_COL, 4, dict(kl=3)),
    (oracle.KIND_SIMPLEX4, 4, {}),
]


@pytest.mark.parametrize("kind,d,kw", LAYOUTS)
@pytest.mark.parametrize("inner", [1, 3])
def test_pack_is_lexicographic_walk_of_unique_set(kind, d, kw, inner):
    order = order_of(kind)
    shape = (d,) * order + (inner,)
    dense = np.arange(np.prod(shape), dtype=np.int32).reshape(shape) + 1
    packed = oracle.pack(dense, kind, d, inner=inner, **kw).reshape(-1, inner)
    expect = []
    if kind == oracle.KIND_BAND:
        for i in range(d):
            for j in range(i - kw["kl"], i + kw["ku"] + 1):
                expect.append(dense[i, j] if 0 <= j < d else np.zeros(inner, np.int32))
    else:
        for idx in itertools.product(range(d), repeat=order):
            if in_unique(kind, idx, d, kl=kw.get("kl", 0), bs=kw.get("bs", 1)):
                expect.append(dense[idx])
    assert np.array_equal(packed, np.array(expect))
    # locate() agrees with the position found above
    pos = 0
    if kind != oracle.KIND_BAND:
        for idx in itertools.product(range(d), repeat=order):
            a = tuple(idx) + (0,) * (4 - order)
            if in_unique(kind, idx, d, kl=kw.get("kl", 0), bs=kw.get("bs", 1)):
                assert oracle.locate(kind, d, *a, **kw) == pos
                pos += 1
            else:
                assert oracle.locate(kind, d, *a, **kw) == -1


@pytest.mark.parametrize("kind,d,kw", LAYOUTS)
def test_round_trips_and_properties(kind, d, kw):
    order = order_of(kind)
    inner = 2
    rows = oracle.packed_rows(kind, d, **kw)
    P = workloads.draw((rows, inner), "normal", 99)
    dense = oracle.unpack(P, kind, d, inner=inner, **kw)
    # pack(unpack(P)) == P bit for bit, apart from the band's out-of-matrix slots
    P2 = oracle.pack(dense, kind, d, inner=inner, **kw).reshape(rows, inner)
    if kind == oracle.KIND_BAND:
        slot = 0
        for i in range(d):
            for j in range(i - kw["kl"], i + kw["ku"] + 1):
                if 0 <= j < d:
                    assert np.array_equal(P2[slot].view(np.uint32), P[slot].view(np.uint32))
                else:
                    assert np.all(P2[slot].view(np.uint32) == 0)
                slot += 1
    else:
        assert np.array_equal(P2.view(np.uint32), P.view(np.uint32))
    # T * T_U: positions outside the unique set are +0.0 (Property 2, T_C = T_U * T)
    for idx in itertools.product(range(d), repeat=order):
        if not in_unique(kind, idx, d, kw.get("kl", 0), kw.get("ku", 0), kw.get("bs", 1)):
            assert np.all(dense[idx].view(np.uint32) == 0)


def test_symmetric_reconstruction_property5():
    """T = T_C + T_R * T_C for the symmetric structure, and its order-3 extension."""
    d = 6
    X = rnd((9, d), 21)
    T2, _ = oracle.moment2(X)
    P = oracle.pack(T2, oracle.KIND_TRI, d)
    assert np.array_equal(oracle.unpack(P, oracle.KIND_TRI, d, fill=oracle.FILL_SYMMETRIC), T2)
    upper = oracle.unpack(P, oracle.KIND_TRI, d)
    assert np.array_equal(upper, np.triu(T2))
    # a non-symmetric source: pack reads only T_U, so the lower triangle is ignored
    M = rnd((d, d), 22)
    R = oracle.unpack(oracle.pack(M, oracle.KIND_TRI, d), oracle.KIND_TRI, d, fill=oracle.FILL_SYMMETRIC)
    assert np.array_equal(np.triu(R), np.triu(M)) and np.array_equal(R, R.T)
    T3, _ = oracle.moment3(X)
    # make it exactly permutation invariant first (fp64 sums differ in the last bit by order of factors)
    P3 = oracle.pack(T3, oracle.KIND_TET, d)
    R3 = oracle.unpack(P3, oracle.KIND_TET, d, fill=oracle.FILL_SYMMETRIC)
    for perm in itertools.permutations(range(3)):
        assert np.array_equal(R3, R3.transpose(perm))
    np.testing.assert_allclose(R3, T3, rtol=1e-13, atol=1e-13)
    for i in range(d):
        for j in range(i, d):
            for k in range(j, d):
                assert R3[i, j, k] == T3[i, j, k]
    with pytest.raises(ValueError):
        oracle.unpack(np.zeros(12, np.float32), oracle.KIND_BLOCKDIAG, 6, nb=3, bs=2, fill=oracle.FILL_SYMMETRIC)


def test_four_simplex_counts_redundancy_map_and_slice_structures():
    """The unique 4-tuples of M3 (Section 3): 35 of them at 4 features (Section 2: 65 = 10 + 20 + 35), about
    23x fewer than d^4; the redundancy map sends every index tuple to its sorted representative; the
    one-row / one-column structures hold d positions."""
    g = golden()
    n4 = g["pr2_distinct"] - oracle.packed_rows(oracle.KIND_TRI, 4) - oracle.packed_rows(oracle.KIND_TET, 4)
    assert oracle.packed_rows(oracle.KIND_SIMPLEX4, 4) == n4 == 35
    for d in range(1, 9):
        assert oracle.packed_rows(oracle.KIND_SIMPLEX4, d) == math.comb(d + 3, 4)
    assert 20 < 64 ** 4 / oracle.packed_rows(oracle.KIND_SIMPLEX4, 64) < 24
    d = 4
    rows = oracle.packed_rows(oracle.KIND_SIMPLEX4, d)
    ids = np.arange(1, rows + 1, dtype=np.int32)
    dense = oracle.unpack(ids, oracle.KIND_SIMPLEX4, d, fill=oracle.FILL_SYMMETRIC)
    assert dense.shape == (d, d, d, d)
    covered = 0
    for idx in itertools.product(range(d), repeat=4):
        rep = tuple(sorted(idx))
        assert dense[idx] == ids[oracle.locate(oracle.KIND_SIMPLEX4, d, *rep)]
        covered += 1
    assert covered == d ** 4
    # Property 5 on a real fourth moment: the symmetric fill restores the dense tensor
    X = rnd((7, d), 31)
    T4, _ = oracle.moment4(X)
    P4 = oracle.pack(T4, oracle.KIND_SIMPLEX4, d)
    R4 = oracle.unpack(P4, oracle.KIND_SIMPLEX4, d, fill=oracle.FILL_SYMMETRIC)
    np.testing.assert_allclose(R4, T4, rtol=1e-13, atol=1e-13)
    for perm in itertools.permutations(range(4)):
        assert np.array_equal(R4, R4.transpose(perm))
    # one row / one column of a matrix
    for kind, fixed in ((oracle.KIND_FIXED_ROW, 2), (oracle.KIND_FIXED_COL, 4)):
        assert oracle.packed_rows(kind, 6, kl=fixed) == 6
        assert oracle.packed_rows(kind, 6, kl=6) == -1
        M = rnd((6, 6), 32)
        P = oracle.pack(M, kind, 6, kl=fixed)
        assert np.array_equal(P, M[fixed, :] if kind == oracle.KIND_FIXED_ROW else M[:, fixed])
        back = oracle.unpack(P, kind, 6, kl=fixed)
        keep = np.zeros((6, 6), bool)
        if kind == oracle.KIND_FIXED_ROW:
            keep[fixed, :] = True
        else:
            keep[:, fixed] = True
        assert np.array_equal(back, np.where(keep, M, 0.0))


def test_unique_and_redundant_sets_partition_the_index_space():
    """Property 1 (T_U * T_R is empty) and |orbits| sum to d^k for the symmetric structures."""
    d = 5
    total2 = sum(1 if i == j else 2 for i in range(d) for j in range(i, d))
    assert total2 == d * d
    total3 = 0
    for i in range(d):
        for j in range(i, d):
            for k in range(j, d):
                total3 += {1: 1, 2: 3, 3: 6}[len({i, j, k})]
    assert total3 == d ** 3
    # unpack with symmetric fill writes every dense position from exactly one packed position
    rows = oracle.packed_rows(oracle.KIND_TET, d)
    ids = np.arange(1, rows + 1, dtype=np.int32)
    dense = oracle.unpack(ids, oracle.KIND_TET, d, fill=oracle.FILL_SYMMETRIC)
    for i, j, k in itertools.product(range(d), repeat=3):
        a, b, c = sorted((i, j, k))
        assert dense[i, j, k] == ids[oracle.locate(oracle.KIND_TET, d, a, b, c)]


def test_mttkrp_on_upper_half_cube_uses_only_unique_set():
    """Expanding a packed (i<=j, k) tensor and running the dense definition equals the sum
    restricted to j >= i (Table 1, "upper half cube")."""
    I, K, R = 5, 3, 2
    Bp, C, D = workloads.mttkrp_inputs(I, K, R)
    Bd = oracle.unpack(Bp.reshape(-1), oracle.KIND_TRI, I, inner=K)
    A, S = oracle.mttkrp(Bd, C, D)
    ref = np.zeros((I, R))
    p = 0
    for i in range(I):
        for j in range(i, I):
            for k in range(K):
                ref[i] += float(Bp[p, k]) * C[j].astype(np.float64) * D[k].astype(np.float64)
            p += 1
    np.testing.assert_allclose(A, ref, rtol=1e-12, atol=1e-12)


# --------------------------------------------------------------------------- metric, inputs

def test_rel_err_metric_separates_ulp_noise_from_real_errors():
    X = rnd((200, 8), 31)
    T, S = oracle.moment2(X)
    ok = T.astype(np.float32).astype(np.float64)
    assert oracle.rel_err(ok, T, S) < 1e-6
    bad = T.copy()
    bad[2, 3] += 1e-3 * S[2, 3]
    assert oracle.rel_err(bad, T, S) > 5e-4
    z = np.zeros_like(T)
    assert oracle.rel_err(z + 1e-30, z, z) == float("inf")
    assert oracle.rel_err(z, z, z) == 0.0


def test_workload_generators_are_seeded_and_prefix_stable():
    a = workloads.moment_input("moment3", N=70000, d=8)
    b = workloads.moment_input("moment3", N=65536, d=8)
    assert np.array_equal(a[:65536], b)
    assert a.dtype == np.float32
    u = workloads.moment_input("moment2", N=1000, d=4)
    assert u.min() >= -1.0 and u.max() < 1.0 and abs(u.mean()) < 0.05
    bits = workloads.f32_to_bf16_bits(np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0], np.float32))
    back = workloads.bf16_bits_to_f32(bits)
    assert back[0] == 1.0 and back[3] == -2.5 and back[4] == 0.0
    assert back[1] == 1.0            # 1 + 2^-8 is a tie: rounds to even (1.0)
    assert back[2] == 1.015625       # 1 + 3*2^-8 is a tie: rounds to even (1 + 2^-6)
