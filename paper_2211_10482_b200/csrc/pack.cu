// st_pack / st_unpack: gather the unique set T_U of a dense tensor into the packed layout
// (T_C = T * T_U, Section 4) and reconstruct the dense tensor from it
// (T = T_C + T_R * T_C, Section 6, Property 5).  HBM-bound index-decode copies.
//
// Two kernels.
//   slice_copy_kernel (st_pack, st_unpack with zero fill): the dense array is cut into slices
//   along its last structured index (matrix row i; pair (i,j) of an order-3 tensor).  In every
//   supported structure the unique positions of a slice are ONE contiguous run of columns
//   [lo,hi) that is also contiguous in the packed array, so a slice is "zeros, one flat copy,
//   zeros" and needs no per-element index arithmetic at all: the run and its packed offset come
//   from the closed forms of st_index.cuh once per slice.  Copies run in units of U bytes (16
//   where the row width allows); long slices are split into parts over several thread groups.
//   structured_copy_kernel (st_unpack with symmetric fill): one lane group per dense row
//   decodes its index tuple, maps it through the redundancy map and copies the row.
#include "st_common.cuh"
#include "st_index.cuh"

namespace st {

struct LayoutArgs {
    int kind;
    int fill;
    int64_t d, kl, ku, nb, bs;
    int64_t width;       // band: kl+ku+1
    int64_t packed_rows;
    int64_t dense_rows;
    int64_t chunks;      // units of U bytes per row
};

// Dense row index of packed row p, or -1 for a band slot outside the matrix.
template <int KIND>
__device__ __forceinline__ int64_t dense_row_of_packed(const LayoutArgs &a, int64_t p)
{
    if (KIND == ST_TRI_UPPER) {
        int64_t i, j;
        tri_decode(a.d, p, i, j);
        return i * a.d + j;
    } else if (KIND == ST_TET) {
        int64_t i, j, k;
        tet_decode(a.d, p, i, j, k);
        return (i * a.d + j) * a.d + k;
    } else if (KIND == ST_BAND) {
        const int64_t i = p / a.width;
        const int64_t j = i + (p - i * a.width) - a.kl;
        return (j >= 0 && j < a.d) ? i * a.d + j : -1;
    } else if (KIND == ST_FIXED_ROW) {
        return a.kl * a.d + p;
    } else if (KIND == ST_FIXED_COL) {
        return p * a.d + a.kl;
    } else if (KIND == ST_SIMPLEX4) {
        int64_t i = 0;                                   // slab i: the largest i with simp4_slab_start(d, i) <= p
        while (i + 1 < a.d && simp4_slab_start(a.d, i + 1) <= p) ++i;
        int64_t j, k, l;
        tet_decode(a.d - i, p - simp4_slab_start(a.d, i), j, k, l);
        return (((i * a.d) + (i + j)) * a.d + (i + k)) * a.d + (i + l);
    } else {
        const int64_t bb = a.bs * a.bs;
        const int64_t b = p / bb;
        const int64_t rem = p - b * bb;
        const int64_t ii = rem / a.bs;
        const int64_t jj = rem - ii * a.bs;
        return (b * a.bs + ii) * a.d + b * a.bs + jj;
    }
}

// Packed row that dense row r is read from, or -1 when the position is a structural zero.
template <int KIND>
__device__ __forceinline__ int64_t packed_row_of_dense(const LayoutArgs &a, int64_t r)
{
    if (KIND == ST_TRI_UPPER) {
        int64_t i = r / a.d, j = r - i * a.d;
        if (i > j) {
            if (a.fill != ST_FILL_SYMMETRIC) return -1;
            int64_t t = i; i = j; j = t;     // T_R(i,j,i',j') = (j<i)*(i'=j)*(j'=i)
        }
        return tri_encode(a.d, i, j);
    } else if (KIND == ST_TET) {
        const int64_t ij = r / a.d;
        int64_t k = r - ij * a.d;
        int64_t i = ij / a.d, j = ij - i * a.d;
        if (!(i <= j && j <= k)) {
            if (a.fill != ST_FILL_SYMMETRIC) return -1;
            int64_t t;                        // representative = sorted index triple
            if (i > j) { t = i; i = j; j = t; }
            if (j > k) { t = j; j = k; k = t; }
            if (i > j) { t = i; i = j; j = t; }
        }
        return tet_encode(a.d, i, j, k);
    } else if (KIND == ST_BAND) {
        const int64_t i = r / a.d, j = r - i * a.d;
        const int64_t s = j - i + a.kl;
        return (s >= 0 && s < a.width) ? i * a.width + s : -1;
    } else if (KIND == ST_FIXED_ROW) {
        const int64_t i = r / a.d;
        return i == a.kl ? r - i * a.d : -1;
    } else if (KIND == ST_FIXED_COL) {
        const int64_t i = r / a.d;
        return r - i * a.d == a.kl ? i : -1;
    } else if (KIND == ST_SIMPLEX4) {
        int64_t v[4];
        int64_t q = r;
        v[3] = q % a.d; q /= a.d;
        v[2] = q % a.d; q /= a.d;
        v[1] = q % a.d; v[0] = q / a.d;
        if (!(v[0] <= v[1] && v[1] <= v[2] && v[2] <= v[3])) {
            if (a.fill != ST_FILL_SYMMETRIC) return -1;
            // representative = sorted index tuple (sorting network for four keys)
#define ST_CSWAP(x, y) { if (v[x] > v[y]) { const int64_t t = v[x]; v[x] = v[y]; v[y] = t; } }
            ST_CSWAP(0, 1) ST_CSWAP(2, 3) ST_CSWAP(0, 2) ST_CSWAP(1, 3) ST_CSWAP(1, 2)
#undef ST_CSWAP
        }
        return simp4_encode(a.d, v[0], v[1], v[2], v[3]);
    } else {
        const int64_t i = r / a.d, j = r - i * a.d;
        const int64_t b = i / a.bs;
        if (j / a.bs != b) return -1;
        return (i * a.bs) + (j - b * a.bs);   // ((b*bs + i')*bs + j') with b*bs+i' = i
    }
}

template <typename U>
__device__ __forceinline__ U zero_unit();
template <> __device__ __forceinline__ uint4 zero_unit<uint4>() { return make_uint4(0, 0, 0, 0); }
template <> __device__ __forceinline__ uint2 zero_unit<uint2>() { return make_uint2(0, 0); }
template <> __device__ __forceinline__ uint32_t zero_unit<uint32_t>() { return 0u; }
template <> __device__ __forceinline__ uint16_t zero_unit<uint16_t>() { return 0; }

// Element-wise product of two units of fp32 values (the Hadamard variant of st_pack).
__device__ __forceinline__ uint4 mul_unit(uint4 a, uint4 b)
{
    return make_uint4(__float_as_uint(__uint_as_float(a.x) * __uint_as_float(b.x)),
                      __float_as_uint(__uint_as_float(a.y) * __uint_as_float(b.y)),
                      __float_as_uint(__uint_as_float(a.z) * __uint_as_float(b.z)),
                      __float_as_uint(__uint_as_float(a.w) * __uint_as_float(b.w)));
}
__device__ __forceinline__ uint2 mul_unit(uint2 a, uint2 b)
{
    return make_uint2(__float_as_uint(__uint_as_float(a.x) * __uint_as_float(b.x)),
                      __float_as_uint(__uint_as_float(a.y) * __uint_as_float(b.y)));
}
__device__ __forceinline__ uint32_t mul_unit(uint32_t a, uint32_t b)
{
    return __float_as_uint(__uint_as_float(a) * __uint_as_float(b));
}
__device__ __forceinline__ uint16_t mul_unit(uint16_t a, uint16_t) { return a; }   // not reached: fp32 rows are whole words

// PACK = true : rows of `dst` are packed rows, source rows are dense rows.
// PACK = false: rows of `dst` are dense rows, source rows are packed rows.
template <int KIND, typename U, bool PACK>
__global__ void __launch_bounds__(256)
structured_copy_kernel(const U *__restrict__ src, U *__restrict__ dst, LayoutArgs a, int group_shift)
{
    const int64_t rows = PACK ? a.packed_rows : a.dense_rows;
    const int g = 1 << group_shift;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t groups = ((int64_t)gridDim.x * blockDim.x) >> group_shift;
    const int lane = (int)(tid & (g - 1));
    for (int64_t row = tid >> group_shift; row < rows; row += groups) {
        const int64_t srow = PACK ? dense_row_of_packed<KIND>(a, row) : packed_row_of_dense<KIND>(a, row);
        U *out = dst + row * a.chunks;
        if (srow >= 0 && !ST_BOUNDS_OK(srow, PACK ? a.dense_rows : a.packed_rows, 1)) continue;
        if (srow >= 0) {
            const U *in = src + srow * a.chunks;
            for (int64_t c = lane; c < a.chunks; c += g) out[c] = in[c];
        } else {
            for (int64_t c = lane; c < a.chunks; c += g) out[c] = zero_unit<U>();
        }
    }
}

// Symmetric fill of a plain matrix / order-3 tensor of 4-byte elements (the reconstruction of a moment
// output): one thread per dense element, indices from the thread coordinates, 32-bit arithmetic only.
template <int KIND>
__global__ void __launch_bounds__(256)
sym_unpack32_kernel(const uint32_t *__restrict__ packed, uint32_t *__restrict__ dense, unsigned d)
{
    const unsigned x = blockIdx.x * blockDim.x + threadIdx.x, y = blockIdx.y * blockDim.y + threadIdx.y;
    if (x >= d || y >= d) return;
    if (KIND == ST_TRI_UPPER) {
        const unsigned i = y < x ? y : x, j = y < x ? x : y;             // representative (min, max): T_R of the symmetric structure
        dense[y * d + x] = packed[i * (2 * d - i + 1) / 2 + (j - i)];
    } else {
        unsigned a = blockIdx.z, b = y, c = x, t;                        // dense (i, j, k) = (z, y, x); sort to a <= b <= c
        if (a > b) { t = a; a = b; b = t; }
        if (b > c) { t = b; b = c; c = t; }
        if (a > b) { t = a; a = b; b = t; }
        const unsigned m = d - a, jj = b - a, kk = c - a;
        const unsigned slab = d * (d + 1) / 2 * (d + 2) / 3 - m * (m + 1) / 2 * (m + 2) / 3;
        dense[(blockIdx.z * d + y) * d + x] = packed[slab + jj * (2 * m - jj + 1) / 2 + (kk - jj)];
    }
}

// Run of unique columns of slice s, in rows of `chunks` units: dense columns [lo,hi) of the
// slice map to packed rows prow.. (contiguous).  For ST_BAND also the extent of the fixed-width
// packed row [band0, band1) whose slots outside the run are zero-filled by pack.
template <int KIND>
__device__ __forceinline__ void slice_run(const LayoutArgs &a, int64_t s, int64_t &lo, int64_t &hi, int64_t &prow)
{
    if (KIND == ST_TRI_UPPER) {
        lo = s; hi = a.d; prow = tri_row_start(a.d, s);
    } else if (KIND == ST_TET) {
        const int64_t i = s / a.d, j = s - i * a.d;
        if (j < i) { lo = hi = 0; prow = 0; }
        else { lo = j; hi = a.d; prow = tet_encode(a.d, i, j, j); }
    } else if (KIND == ST_BAND) {
        lo = s - a.kl; if (lo < 0) lo = 0;
        hi = s + a.ku + 1; if (hi > a.d) hi = a.d;
        if (hi < lo) hi = lo;
        prow = s * a.width + (lo - (s - a.kl));
    } else if (KIND == ST_FIXED_ROW) {
        if (s == a.kl) { lo = 0; hi = a.d; } else { lo = hi = 0; }
        prow = 0;
    } else if (KIND == ST_FIXED_COL) {
        lo = a.kl; hi = a.kl + 1; prow = s;
    } else if (KIND == ST_SIMPLEX4) {
        // slice s = (i, j, k): its unique entries are l = k .. d-1 when i <= j <= k
        const int64_t ij = s / a.d, k = s - ij * a.d;
        const int64_t i = ij / a.d, j = ij - i * a.d;
        if (i <= j && j <= k) { lo = k; hi = a.d; prow = simp4_encode(a.d, i, j, k, k); }
        else { lo = hi = 0; prow = 0; }
    } else {
        const int64_t b = s / a.bs;
        lo = b * a.bs; hi = lo + a.bs; prow = s * a.bs;
    }
}

template <int KIND, typename U, bool PACK>
__global__ void __launch_bounds__(256)
slice_copy_kernel(const U *__restrict__ src, U *__restrict__ dst, LayoutArgs a, int group_shift, int parts,
                  int64_t part_units, const U *__restrict__ mul)
{
    // mul (pack only, fp32 elements): a second packed operand; the gathered values are multiplied by it
    const int g = 1 << group_shift;
    const int lane = (int)(threadIdx.x & (g - 1));
    const int64_t gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> group_shift;
    const int64_t ngroups = ((int64_t)gridDim.x * blockDim.x) >> group_shift;
    const int64_t nslices = (KIND == ST_TET) ? a.d * a.d : (KIND == ST_SIMPLEX4) ? a.d * a.d * a.d : a.d;
    const int64_t su = a.d * a.chunks;                        // units per dense slice
    for (int64_t item = gid; item < nslices * parts; item += ngroups) {
        const int64_t s = item / parts;
        const int64_t part = item - s * parts;
        int64_t lo, hi, prow;
        slice_run<KIND>(a, s, lo, hi, prow);
        // a non-empty run lies inside the slice and inside the packed array
        if (hi > lo && !(ST_BOUNDS_OK(lo, a.d, 1) && ST_BOUNDS_OK(hi - 1, a.d, 1) && ST_BOUNDS_OK(prow, a.packed_rows, 1) &&
                         ST_BOUNDS_OK(prow + (hi - lo) - 1, a.packed_rows, 1)))
            continue;
        const int64_t c0 = lo * a.chunks, c1 = hi * a.chunks;  // units of the run inside the slice
        // pack splits the run itself into parts, unpack the whole dense slice (it writes all of it)
        const int64_t r0 = PACK ? c0 : 0, r1 = PACK ? c1 : su;
        int64_t u0 = r0 + part * part_units;                  // this part covers dense units [u0, u1) of the slice
        int64_t u1 = u0 + part_units;
        if (u0 > r1) u0 = r1;
        if (u1 > r1) u1 = r1;
        const int64_t x0 = u0 > c0 ? u0 : c0, x1 = u1 < c1 ? u1 : c1;   // run clipped to this part
        if (PACK) {
            const U *in = src + s * su;
            U *out = dst + prow * a.chunks - c0;                // out[u] for dense unit u of the run
            if (mul) {
                const U *m = mul + prow * a.chunks - c0;
                for (int64_t u = x0 + lane; u < x1; u += g) out[u] = mul_unit(in[u], m[u]);
            } else {
                for (int64_t u = x0 + lane; u < x1; u += g) out[u] = in[u];
            }
            if (KIND == ST_BAND && part == 0) {
                // slots of the fixed-width packed row that fall outside the matrix
                U *row = dst + s * a.width * a.chunks;
                const int64_t first = (prow - s * a.width) * a.chunks, last = first + (c1 - c0);
                const int64_t wu = a.width * a.chunks;
                for (int64_t u = lane; u < first; u += g) row[u] = zero_unit<U>();
                for (int64_t u = last + lane; u < wu; u += g) row[u] = zero_unit<U>();
            }
        } else {
            U *out = dst + s * su;
            const U *in = src + prow * a.chunks - c0;
            const int64_t z1 = u1 < c0 ? u1 : c0;               // zeros before the run
            for (int64_t u = u0 + lane; u < z1; u += g) out[u] = zero_unit<U>();
            for (int64_t u = x0 + lane; u < x1; u += g) out[u] = in[u];
            const int64_t z2 = u0 > c1 ? u0 : c1;               // zeros after the run
            for (int64_t u = z2 + lane; u < u1; u += g) out[u] = zero_unit<U>();
        }
    }
}

// out = alpha * a + beta * b (OP 0) or out = a * b (OP 1) over packed arrays of the same layout.
// `out` may be `a` or `b` (a thread reads the elements it later writes, and nobody else's), so none of
// the pointers is declared restrict.
template <int OP>
__global__ void __launch_bounds__(256)
packed_binary_kernel(const float *a, const float *b, float *out, int64_t n, float alpha, float beta)
{
    const int64_t n4 = n >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += stride) {
        const float4 x = reinterpret_cast<const float4 *>(a)[e];
        const float4 y = reinterpret_cast<const float4 *>(b)[e];
        float4 r;
        if (OP == 0) r = make_float4(alpha * x.x + beta * y.x, alpha * x.y + beta * y.y, alpha * x.z + beta * y.z, alpha * x.w + beta * y.w);
        else r = make_float4(x.x * y.x, x.y * y.y, x.z * y.z, x.w * y.w);
        reinterpret_cast<float4 *>(out)[e] = r;
    }
    for (int64_t e = 4 * n4 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += stride)
        out[e] = OP == 0 ? alpha * a[e] + beta * b[e] : a[e] * b[e];
}

static bool layout_ok(const st_layout *L)
{
    if (!L) return false;
    if (L->reserved != 0) return false;
    if (L->d <= 0 || L->inner <= 0) return false;
    if (L->d > (int64_t(1) << 31)) return false;
    switch (L->kind) {
    case ST_TRI_UPPER: return true;
    case ST_TET: return L->d <= (int64_t(1) << 20);
    case ST_SIMPLEX4: return L->d <= 32768;
    case ST_FIXED_ROW:
    case ST_FIXED_COL: return L->kl >= 0 && L->kl < L->d;
    case ST_BAND: return L->kl >= 0 && L->ku >= 0 && L->kl < (int64_t(1) << 31) && L->ku < (int64_t(1) << 31);
    case ST_BLOCKDIAG: return L->nblocks > 0 && L->bs > 0 && L->nblocks * L->bs == L->d;
    default: return false;
    }
}

static int64_t packed_rows_of(const st_layout *L)
{
    switch (L->kind) {
    case ST_TRI_UPPER: return tri_rows(L->d);
    case ST_TET: return tet_rows(L->d);
    case ST_SIMPLEX4: return simp4_rows(L->d);
    case ST_FIXED_ROW:
    case ST_FIXED_COL: return L->d;
    case ST_BAND: return L->d * (L->kl + L->ku + 1);
    default: return L->nblocks * L->bs * L->bs;
    }
}

static int64_t dense_rows_of(const st_layout *L)
{
    if (L->kind == ST_SIMPLEX4) return L->d * L->d * L->d * L->d;
    return L->kind == ST_TET ? L->d * L->d * L->d : L->d * L->d;
}

static int dtype_bytes(st_dtype t)
{
    switch (t) {
    case ST_F32: return 4;
    case ST_BF16: return 2;
    case ST_F64: return 8;
    default: return 0;
    }
}

template <int KIND, typename U, bool PACK>
static st_status launch_copy(const void *src, void *dst, const LayoutArgs &a, cudaStream_t s, const void *mul)
{
    const int64_t cap = (int64_t)sm_count_or_default() * 16;
    if (!PACK && a.fill == ST_FILL_SYMMETRIC && sizeof(U) == 4 && a.chunks == 1 &&
        ((KIND == ST_TRI_UPPER && a.d <= 32768) || (KIND == ST_TET && a.d <= 1024))) {
        const dim3 block(32, 8), grid((unsigned)((a.d + 31) / 32), (unsigned)((a.d + 7) / 8), KIND == ST_TET ? (unsigned)a.d : 1u);
        sym_unpack32_kernel<(KIND == ST_TET ? ST_TET : ST_TRI_UPPER)><<<grid, block, 0, s>>>((const uint32_t *)src, (uint32_t *)dst, (unsigned)a.d);
        return launch_status();
    }
    if (!PACK && a.fill == ST_FILL_SYMMETRIC) {
        // redundancy map: one lane group per dense row
        int shift = 0;
        while ((1 << shift) < 32 && (int64_t(1) << shift) < a.chunks) ++shift;
        const int64_t threads = a.dense_rows << shift;
        const int64_t want = (threads + 255) / 256;
        const int grid = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
        structured_copy_kernel<KIND, U, PACK><<<grid, 256, 0, s>>>((const U *)src, (U *)dst, a, shift);
        return launch_status();
    }
    // slices: about 8 units per thread, at most 8192 units per (slice, part).  Pack splits the
    // longest run of unique columns, unpack the whole dense slice.
    int64_t run_rows = a.d;
    if (KIND == ST_BAND) run_rows = a.width < a.d ? a.width : a.d;
    if (KIND == ST_BLOCKDIAG) run_rows = a.bs;
    if (KIND == ST_FIXED_COL) run_rows = 1;
    const int64_t su = (PACK ? run_rows : a.d) * a.chunks;
    int parts = (int)((su + 8191) / 8192);
    if (parts < 1) parts = 1;
    const int64_t pu = (su + parts - 1) / parts;
    int shift = 0;
    while ((1 << shift) < 256 && (int64_t(8) << shift) < pu) ++shift;
    const int64_t nslices = (KIND == ST_TET) ? a.d * a.d : (KIND == ST_SIMPLEX4) ? a.d * a.d * a.d : a.d;
    const int64_t threads = (nslices * parts) << shift;
    const int64_t want = (threads + 255) / 256;
    const int grid = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
    slice_copy_kernel<KIND, U, PACK><<<grid, 256, 0, s>>>((const U *)src, (U *)dst, a, shift, parts, pu, (const U *)mul);
    return launch_status();
}

template <typename U, bool PACK>
static st_status dispatch_kind(const void *src, void *dst, const LayoutArgs &a, cudaStream_t s, const void *mul)
{
    switch (a.kind) {
    case ST_TRI_UPPER: return launch_copy<ST_TRI_UPPER, U, PACK>(src, dst, a, s, mul);
    case ST_TET: return launch_copy<ST_TET, U, PACK>(src, dst, a, s, mul);
    case ST_BAND: return launch_copy<ST_BAND, U, PACK>(src, dst, a, s, mul);
    case ST_FIXED_ROW: return launch_copy<ST_FIXED_ROW, U, PACK>(src, dst, a, s, mul);
    case ST_FIXED_COL: return launch_copy<ST_FIXED_COL, U, PACK>(src, dst, a, s, mul);
    case ST_SIMPLEX4: return launch_copy<ST_SIMPLEX4, U, PACK>(src, dst, a, s, mul);
    default: return launch_copy<ST_BLOCKDIAG, U, PACK>(src, dst, a, s, mul);
    }
}

template <bool PACK>
static st_status copy_entry(const st_layout *L, st_dtype dtype, const void *src, void *dst, int fill,
                            void *stream, const void *mul = nullptr)
{
    if (!L || !src || !dst) return ST_ERR_NULL;
    if (!layout_ok(L)) return ST_ERR_SHAPE;
    const int es = dtype_bytes(dtype);
    if (es == 0) return ST_ERR_DTYPE;
    if (fill != ST_FILL_ZERO && fill != ST_FILL_SYMMETRIC) return ST_ERR_UNSUPPORTED;
    if (fill == ST_FILL_SYMMETRIC && L->kind != ST_TRI_UPPER && L->kind != ST_TET && L->kind != ST_SIMPLEX4)
        return ST_ERR_UNSUPPORTED;
    if (!aligned16(src) || !aligned16(dst)) return ST_ERR_ALIGN;
    LayoutArgs a;
    a.kind = L->kind;
    a.fill = fill;
    a.d = L->d; a.kl = L->kl; a.ku = L->ku; a.nb = L->nblocks; a.bs = L->bs;
    a.width = L->kl + L->ku + 1;
    a.packed_rows = packed_rows_of(L);
    a.dense_rows = dense_rows_of(L);
    const int64_t w = L->inner * es;   // bytes per row
    cudaStream_t s = (cudaStream_t)stream;
    if (w % 16 == 0) { a.chunks = w / 16; return dispatch_kind<uint4, PACK>(src, dst, a, s, mul); }
    if (w % 8 == 0)  { a.chunks = w / 8;  return dispatch_kind<uint2, PACK>(src, dst, a, s, mul); }
    if (w % 4 == 0)  { a.chunks = w / 4;  return dispatch_kind<uint32_t, PACK>(src, dst, a, s, mul); }
    a.chunks = w / 2;
    return dispatch_kind<uint16_t, PACK>(src, dst, a, s, mul);
}

}  // namespace st

extern "C" {

int64_t st_packed_elems(const st_layout *layout)
{
    if (!st::layout_ok(layout)) return -1;
    return st::packed_rows_of(layout) * layout->inner;
}

int64_t st_dense_elems(const st_layout *layout)
{
    if (!st::layout_ok(layout)) return -1;
    return st::dense_rows_of(layout) * layout->inner;
}

st_status st_pack(const st_layout *layout, st_dtype dtype, const void *dense, void *packed, void *stream)
{
    return st::copy_entry<true>(layout, dtype, dense, packed, ST_FILL_ZERO, stream);
}

static st_status packed_binary(int op, int64_t n, const float *a, const float *b, float *out, float alpha, float beta,
                               void *stream)
{
    if (!a || !b || !out) return ST_ERR_NULL;
    if (n <= 0) return ST_ERR_SHAPE;
    if (!st::aligned16(a) || !st::aligned16(b) || !st::aligned16(out)) return ST_ERR_ALIGN;
    const int64_t want = (n / 4 + 255) / 256, cap = (int64_t)st::sm_count_or_default() * 16;
    const unsigned grid = (unsigned)(want < 1 ? 1 : (want < cap ? want : cap));
    if (op == 0) st::packed_binary_kernel<0><<<grid, 256, 0, (cudaStream_t)stream>>>(a, b, out, n, alpha, beta);
    else st::packed_binary_kernel<1><<<grid, 256, 0, (cudaStream_t)stream>>>(a, b, out, n, alpha, beta);
    return st::launch_status();
}

st_status st_packed_axpby(int64_t n, float alpha, const float *a, float beta, const float *b, float *out, void *stream)
{
    return packed_binary(0, n, a, b, out, alpha, beta, stream);
}

st_status st_packed_mul(int64_t n, const float *a, const float *b, float *out, void *stream)
{
    return packed_binary(1, n, a, b, out, 0.f, 0.f, stream);
}

st_status st_thp(const st_layout *layout, const float *Bp, const float *C_dense, float *Ap, void *stream)
{
    if (!Bp) return ST_ERR_NULL;
    if (!st::aligned16(Bp)) return ST_ERR_ALIGN;
    // the pack of C with every gathered value multiplied by the packed operand at the same position
    return st::copy_entry<true>(layout, ST_F32, C_dense, Ap, ST_FILL_ZERO, stream, Bp);
}

st_status st_unpack(const st_layout *layout, st_dtype dtype, const void *packed, void *dense, st_fill fill,
                    void *stream)
{
    return st::copy_entry<false>(layout, dtype, packed, dense, (int)fill, stream);
}

}  // extern "C"
