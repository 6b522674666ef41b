// Closed-form index arithmetic of the packed layouts (host + device).
//
// The packed order is the lexicographic order of the unique set T_U (Section 4,
// "Compressed Tensor"; Section 5.5: loop nests follow the syntactic order of the index
// variables).  The paper itself keeps compressed tensors in full n-d arrays and names
// better layouts as future work (Section 8); the closed forms below are this library's.
#pragma once
#include <cstdint>
#include <cmath>

#if defined(__CUDACC__)
#define ST_HD __host__ __device__ __forceinline__
#else
#define ST_HD inline
#endif

namespace st {

ST_HD int64_t tri_rows(int64_t d) { return d * (d + 1) / 2; }
ST_HD int64_t tet_rows(int64_t d) { return (d * (d + 1) / 2) * (d + 2) / 3; }  // exact: one of the factors is divisible by 3

// First packed row of matrix row i in an upper triangle of side d.
ST_HD int64_t tri_row_start(int64_t d, int64_t i) { return i * (2 * d - i + 1) / 2; }
ST_HD int64_t tri_encode(int64_t d, int64_t i, int64_t j) { return tri_row_start(d, i) + (j - i); }

// Inverse of tri_encode: the largest i with tri_row_start(d,i) <= p.  The discriminant is an exact
// integer; only its square root is taken in floating point -- single precision, which the GPU
// evaluates at full rate -- and the estimate is corrected with integer comparisons, so the result is
// exact for every p.
ST_HD void tri_decode(int64_t d, int64_t p, int64_t &i, int64_t &j)
{
    const int64_t b = 2 * d + 1;
    int64_t disc = b * b - 8 * p;
    if (disc < 0) disc = 0;
    int64_t ii = (b - (int64_t)sqrtf((float)disc)) >> 1;
    if (ii < 0) ii = 0;
    if (ii > d - 1) ii = d - 1;
    while (ii > 0 && tri_row_start(d, ii) > p) --ii;
    while (ii + 1 < d && tri_row_start(d, ii + 1) <= p) ++ii;
    i = ii;
    j = ii + (p - tri_row_start(d, ii));
}

// Number of packed rows of the slabs 0..i-1 of a tetrahedron of side d.
ST_HD int64_t tet_slab_start(int64_t d, int64_t i) { return tet_rows(d) - tet_rows(d - i); }
ST_HD int64_t tet_encode(int64_t d, int64_t i, int64_t j, int64_t k)
{
    return tet_slab_start(d, i) + tri_encode(d - i, j - i, k - i);
}

// Inverse of tet_encode: cube-root estimate of the slab, integer fix-up, then a
// triangle decode of side d-i.
ST_HD void tet_decode(int64_t d, int64_t q, int64_t &i, int64_t &j, int64_t &k)
{
    const int64_t r = tet_rows(d) - q;          // positions left, 1 <= r <= tet(d)
    int64_t m = (int64_t)cbrtf(6.0f * (float)r); // slab i has side m = d-i: tet(m-1) < r <= tet(m)
    if (m < 1) m = 1;
    if (m > d) m = d;
    while (m > 1 && tet_rows(m - 1) >= r) --m;
    while (m < d && tet_rows(m) < r) ++m;
    i = d - m;
    int64_t jj, kk;
    tri_decode(m, q - tet_slab_start(d, i), jj, kk);
    j = i + jj;
    k = i + kk;
}

// Packed 4-simplex 0<=i<=j<=k<=l<d in lexicographic order: slabs i, each a tetrahedron of side d-i.
ST_HD int64_t simp4_rows(int64_t d) { return tet_rows(d) * (d + 3) / 4; }   // C(d+3, 4), exact
ST_HD int64_t simp4_slab_start(int64_t d, int64_t i) { return simp4_rows(d) - simp4_rows(d - i); }
ST_HD int64_t simp4_encode(int64_t d, int64_t i, int64_t j, int64_t k, int64_t l)
{
    return simp4_slab_start(d, i) + tet_encode(d - i, j - i, k - i, l - i);
}

}  // namespace st
