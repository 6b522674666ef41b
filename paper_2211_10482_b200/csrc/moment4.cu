// st_sym_moment4: out[s(i,j,k,l)] = sum_n X[n,i] X[n,j] X[n,k] X[n,l] over the unique set
// 0<=i<=j<=k<=l<d (Section 3, M3 = vec(f (x) f) (x) vec(f (x) f) summed over samples; its unique
// elements are the 4-tuples with repetition, about 23x fewer than d^4).
//
// M3 is the second moment of the pair features: with P[n,(i,j)] = X[n,i] X[n,j] over the unique
// pairs i<=j (the rows of vec(f (x) f) that are not redundant),
//     out[s(i,j,k,l)] = sum_n P[n,(i,j)] P[n,(k,l)],
// and (i,j,k,l) is a unique 4-tuple exactly when j <= k.  Three steps, all on the GPU:
//   1. pair_expand_kernel    P [N, dP], dP = d(d+1)/2 rounded up to 64 (zero columns), fp32 or bf16
//   2. st_sym_moment2 on P   the packed upper triangle of P^T P: the tensor-core triangular tile GEMM, on P rounded
//                            to bf16 (ST_FLAG_TC_BF16, 5e-3) or, for the fp32 tolerance, on P written as hi + lo
//                            bf16 parts and multiplied in three partial products (d <= 89: the pair features
//                            fit the kernel's 4096 columns); beyond that the fp32 FMA kernel on an fp32 P
//   3. simplex_gather_kernel all entries (i,j,*,*) of the 4-simplex are one run of row (i,j) of that triangle,
//                            from column (j,j) on: contiguous on both sides
// Step 2 works on the symmetric pair-by-pair matrix, whose unique set (pairs p <= q) is about
// three times larger than the set of unique 4-tuples: the entries with j > k are computed and
// not gathered.
#include "st_common.cuh"
#include "st_index.cuh"
#include <cuda_bf16.h>
#include <type_traits>

namespace st {

size_t moment2_workspace(int64_t N, int64_t d, int xdt, unsigned flags);
int64_t moment2_split_part_rows(int64_t N);
size_t moment2_split_parts_workspace(int64_t N, int64_t d);
st_status moment2_split_tc_parts(const void *Z, int64_t N, int64_t d, float *out, void *ws, size_t ws_bytes, cudaStream_t stream);

namespace m4 {

constexpr int MAX_D = 128;          // fp32 path; the bf16 path ends where the pair features exceed the tensor-core kernel's 4096 columns (d <= 89)
constexpr int EXP_ROWS = 32;        // sample rows per pass of a block
constexpr int EXP_THREADS = 192;

struct Plan {
    int64_t dP, p_bytes, m2_elems, m2_ws, Np;
    size_t off_p, off_m2, off_ws, total;
    bool bf16, split, ok;
};

static Plan plan(int64_t N, int64_t d, unsigned flags)
{
    Plan p{};
    p.ok = false;
    if (N <= 0 || d < 1 || d > MAX_D) return p;
    p.bf16 = (flags & ST_FLAG_TC_BF16) != 0;
    p.dP = (tri_rows(d) + 63) / 64 * 64;
    p.m2_elems = tri_rows(p.dP);
    // fp32 result: the pair features are written as hi + lo bf16 parts and multiplied on the tensor cores in three
    // partial products (the fp32 tolerance) wherever that kernel reaches; else fp32 features and the fp32 FMA kernel
    p.Np = moment2_split_part_rows(N);
    p.m2_ws = p.bf16 ? 0 : (int64_t)moment2_split_parts_workspace(N, p.dP);
    p.split = !p.bf16 && p.m2_ws != 0;
    if (p.split) {
        p.p_bytes = 2 * p.Np * p.dP * 2;
    } else {
        p.p_bytes = N * p.dP * (p.bf16 ? 2 : 4);
        p.m2_ws = (int64_t)moment2_workspace(N, p.dP, p.bf16 ? ST_BF16 : ST_F32, 0);
    }
    if (p.m2_ws == 0) return p;
    p.off_p = kWsHeaderBytes;
    p.off_m2 = round_up(p.off_p + (size_t)p.p_bytes, 256);
    p.off_ws = round_up(p.off_m2 + (size_t)p.m2_elems * 4, 256);
    p.total = p.off_ws + (size_t)p.m2_ws;
    p.ok = true;
    return p;
}

__device__ __forceinline__ void store4(float *dst, float a, float b, float c, float e)
{
    *reinterpret_cast<float4 *>(dst) = make_float4(a, b, c, e);
}
__device__ __forceinline__ void store4(__nv_bfloat16 *dst, float a, float b, float c, float e)
{
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, e);
    *reinterpret_cast<uint2 *>(dst) = make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
}

// P[n, p(i,j)] = X[n,i] X[n,j] for the unique pairs in packed order, zeros in the padding
// columns.  A block stages EXP_ROWS rows of X per pass (one extra column holds zero); a thread owns
// four adjacent columns of P, decodes their index pairs once and writes them for every staged
// row with one 8- or 16-byte store.  HBM bound: the write of P.
// SPLIT: every product p is written twice, hi = bf16(p) in row n and lo = bf16(p - hi) in row Np + n; the rows
// N .. Np-1 of either part are zero.
// COLS: columns of a staged row per lane, (d + 1 + 31) / 32 rounded up to an instance (2, 3 or 5).
template <typename OutT, bool SPLIT, int COLS>
__global__ void __launch_bounds__(EXP_THREADS)
pair_expand_kernel(const float *__restrict__ X, int64_t N, int d, int64_t ldx, OutT *__restrict__ P, int dP, int npairs,
                   int64_t Np)
{
    extern __shared__ __align__(16) float xs[];                       // 2 x [EXP_ROWS][d + 1], column d is zero
    const int pitch = d + 1;
    // gridDim.x = column groups, gridDim.y = row groups
    const int p = (blockIdx.x * EXP_THREADS + threadIdx.x) * 4;       // this thread's columns p .. p+3
    int ci[4], cj[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        ci[u] = cj[u] = d;                                            // padding column: 0 * 0
        if (p + u < npairs) {
            int64_t a, b;
            tri_decode(d, p + u, a, b);
            ci[u] = (int)a;
            cj[u] = (int)b;
        }
    }
    const bool inside = p < dP;
    const int64_t rows_total = SPLIT ? Np : N;
    // Two stage buffers: the rows of the next pass travel from global memory into registers while the current ones are
    // multiplied, and one block barrier per pass is enough (a buffer is rewritten two passes later, after every
    // thread has gone through the barrier of the pass in between).
    constexpr int NW = EXP_THREADS / 32, RPW = (EXP_ROWS + NW - 1) / NW;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float reg[RPW][COLS];
    auto gload = [&](int64_t row0) {
#pragma unroll
        for (int q = 0; q < RPW; ++q) {
            const int64_t n = row0 + warp + q * NW;
            const bool row_in = warp + q * NW < EXP_ROWS && n < N;
#pragma unroll
            for (int c = 0; c < COLS; ++c) {
                const int col = lane + 32 * c;
                reg[q][c] = (row_in && col < d) ? X[n * ldx + col] : 0.f;
            }
        }
    };
    auto sstore = [&](float *buf) {
#pragma unroll
        for (int q = 0; q < RPW; ++q) {
            const int r = warp + q * NW;
#pragma unroll
            for (int c = 0; c < COLS; ++c) {
                const int col = lane + 32 * c;
                if (r < EXP_ROWS && col < pitch) buf[r * pitch + col] = reg[q][c];
            }
        }
    };
    const int64_t step = (int64_t)gridDim.y * EXP_ROWS;
    int64_t row0 = (int64_t)blockIdx.y * EXP_ROWS;
    if (row0 < rows_total) gload(row0);
    int buf = 0;
    for (; row0 < rows_total; row0 += step, buf ^= 1) {
        const int nrows = rows_total - row0 < EXP_ROWS ? (int)(rows_total - row0) : EXP_ROWS;
        float *xb = xs + buf * (EXP_ROWS * pitch);
        sstore(xb);
        __syncthreads();
        if (row0 + step < rows_total) gload(row0 + step);
        if (!inside) continue;
        OutT *dst = P + row0 * dP + p;
        const float *x = xb;
#pragma unroll 4
        for (int r = 0; r < nrows; ++r, dst += dP, x += pitch) {
            const float v0 = x[ci[0]] * x[cj[0]], v1 = x[ci[1]] * x[cj[1]], v2 = x[ci[2]] * x[cj[2]], v3 = x[ci[3]] * x[cj[3]];
            store4(dst, v0, v1, v2, v3);
            if (SPLIT) {
                const float h0 = __bfloat162float(__float2bfloat16_rn(v0)), h1 = __bfloat162float(__float2bfloat16_rn(v1)),
                            h2 = __bfloat162float(__float2bfloat16_rn(v2)), h3 = __bfloat162float(__float2bfloat16_rn(v3));
                store4(dst + Np * dP, v0 - h0, v1 - h1, v2 - h2, v3 - h3);
            }
        }
    }
}

// One block per unique pair (i,j): the entries (i,j,k,l), j <= k <= l, follow each other in the 4-simplex in the
// order of the pairs (k,l), and in row (i,j) of the packed pair-by-pair triangle they are the columns from pair
// (j,j) to the last one: one contiguous run on both sides, of d-j + ... + 1 elements.
__global__ void __launch_bounds__(128)
simplex_gather_kernel(const float *__restrict__ M2, float *__restrict__ out, int d, int64_t dP, unsigned *status,
                      const unsigned *inner_status)
{
    // the second-moment step ran on its own part of the workspace: its status becomes the call's
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        status[kWsStatusWord] = inner_status[kWsStatusWord];
        status[kWsDetailWord] = inner_status[kWsDetailWord];
    }
    const int64_t p = blockIdx.x;
    int64_t i, j;
    tri_decode(d, p, i, j);
    const int64_t q0 = tri_encode(d, j, j);                               // p <= q0 because i <= j
    const int len = (int)(tri_rows(d) - q0);
    const float *src = M2 + tri_encode(dP, p, q0);
    float *dst = out + simp4_encode(d, i, j, j, j);
    if (!(ST_BOUNDS_OK(tri_encode(dP, p, q0) + len - 1, tri_rows(dP), 7) &&
          ST_BOUNDS_OK(simp4_encode(d, i, j, j, j) + len - 1, simp4_rows(d), 7)))
        return;
    for (int o = threadIdx.x; o < len; o += 128) dst[o] = src[o];
}

}  // namespace m4

size_t moment4_workspace(int64_t N, int64_t d, unsigned flags)
{
    const m4::Plan p = m4::plan(N, d, flags);
    return p.ok ? p.total : 0;
}

}  // namespace st

extern "C" st_status st_sym_moment4(const float *X, int64_t N, int64_t d, int64_t ldx, float *out_packed, void *ws,
                                    size_t ws_bytes, unsigned flags, void *stream_)
{
    using namespace st;
    using namespace st::m4;
    if (!X || !out_packed) return ST_ERR_NULL;
    if (N <= 0 || d <= 0 || ldx < d) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_TC_BF16)) return ST_ERR_UNSUPPORTED;
    if (d > MAX_D) return ST_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(out_packed)) return ST_ERR_ALIGN;
    const Plan p = plan(N, d, flags);
    if (!p.ok) return ST_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < p.total) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    cudaStream_t stream = (cudaStream_t)stream_;
    unsigned char *w = (unsigned char *)ws;
    float *M2 = (float *)(w + p.off_m2);
    const int npairs = (int)tri_rows(d);
    const size_t smem = (size_t)2 * EXP_ROWS * (d + 1) * sizeof(float);
    const unsigned col_groups = (unsigned)((p.dP + 4 * EXP_THREADS - 1) / (4 * EXP_THREADS));
    const int64_t passes = ((p.split ? p.Np : N) + EXP_ROWS - 1) / EXP_ROWS;
    const int64_t cap = ((int64_t)sm_count_or_default() * 8 + col_groups - 1) / col_groups;
    const dim3 grid(col_groups, (unsigned)(passes < cap ? passes : cap));
    auto expand = [&](auto tag, auto split_tag) {
        using T = decltype(tag);
        constexpr bool SP = decltype(split_tag)::value;
        T *dst = (T *)(w + p.off_p);
        if (d + 1 <= 64)
            pair_expand_kernel<T, SP, 2><<<grid, EXP_THREADS, smem, stream>>>(X, N, (int)d, ldx, dst, (int)p.dP, npairs, p.Np);
        else if (d + 1 <= 96)
            pair_expand_kernel<T, SP, 3><<<grid, EXP_THREADS, smem, stream>>>(X, N, (int)d, ldx, dst, (int)p.dP, npairs, p.Np);
        else
            pair_expand_kernel<T, SP, 5><<<grid, EXP_THREADS, smem, stream>>>(X, N, (int)d, ldx, dst, (int)p.dP, npairs, p.Np);
    };
    if (p.split) expand(__nv_bfloat16(), std::true_type());
    else if (p.bf16) expand(__nv_bfloat16(), std::false_type());
    else expand(float(), std::false_type());
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    const st_status rc = p.split ? moment2_split_tc_parts(w + p.off_p, N, p.dP, M2, w + p.off_ws, (size_t)p.m2_ws, stream)
                                 : st_sym_moment2(w + p.off_p, p.bf16 ? ST_BF16 : ST_F32, N, p.dP, p.dP, M2, w + p.off_ws,
                                                  (size_t)p.m2_ws, 0, stream_);
    if (rc != ST_OK) return rc;
    simplex_gather_kernel<<<(unsigned)npairs, 128, 0, stream>>>(M2, out_packed, (int)d, p.dP, (unsigned *)w,
                                                                (const unsigned *)(w + p.off_ws));
    return launch_status();
}
