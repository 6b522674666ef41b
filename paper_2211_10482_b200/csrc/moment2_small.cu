// st_sym_moment2, fp32 path for few features (d % 8 == 0, d <= 64) and many samples -- the regime
// of the paper's covariance workloads (Section 7.2; its real datasets have 6 and 13 features).
//
// out[p(i,j)] = sum_n X[n,i] X[n,j], 0 <= i <= j < d  (Section 3, M1; Section 5.5, y_U = i <= j).
//
// The upper triangle is cut into 8x8 register tiles (ib <= jb): 36 of the 64 tiles for d = 64; tiles
// below the diagonal do not exist here.  The rows of a shared-memory stage are dealt to RG "row
// groups"; one thread owns (tile, row group) and keeps the 64 sums of its tile over its rows in
// registers, so a block of tiles*RG threads needs 4 shared-memory loads per 64 FMAs.  Blocks own
// slices of the samples (one block per SM), stream them through a 3-buffer cp.async pipeline in
// the same bank-conflict-free "split halves" row layout as the third-moment kernel, add their row
// groups in shared memory and write one partial per block; a second kernel adds the partials in
// fixed order.  Diagonal tiles compute all 64 products (the 28 below the diagonal are dropped):
// 36*64 = 2304 FMAs issued per sample for 2080 useful.
#include "st_common.cuh"
#include "st_index.cuh"

namespace st {

constexpr int M2S_MAX_THREADS = 512;
constexpr int M2S_ROWS_PER_GROUP = 8;      // rows of a stage handled by one row group
constexpr int M2S_BUFFERS = 3;
constexpr int M2S_RED_STRIDE = 65;         // floats per tile in the block-level sum array

__device__ __forceinline__ void m2s_cp_async16(void *smem, const void *gmem, bool valid)
{
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    const int sz = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(sz));
}

struct M2SmallArgs {
    const float *X;
    float *partials;      // [slices][ntiles*64]
    int64_t N, ldx, rows_per_slice;
    int d, nbk, ntiles, rg, dense;
};

__global__ void __launch_bounds__(M2S_MAX_THREADS, 1) moment2_small_kernel(const M2SmallArgs a)
{
    extern __shared__ __align__(16) float smem[];
    const int stage_rows = a.rg * M2S_ROWS_PER_GROUP;
    const int stage_floats = stage_rows * a.d;
    float *red = smem + M2S_BUFFERS * stage_floats;          // [ntiles][M2S_RED_STRIDE] block-level sums
    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int item_rg = tid / a.ntiles, tile = tid - item_rg * a.ntiles;
    const bool active = item_rg < a.rg;
    int ib, jb;
    if (a.dense) {
        ib = tile / a.nbk;
        jb = tile - ib * a.nbk;
    } else {
        int64_t x, y;
        tri_decode(a.nbk, tile, x, y);
        ib = (int)x;
        jb = (int)y;
    }
    const int half = 4 * a.nbk;
    const int oi = 4 * ib, oj = 4 * jb;

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    const int64_t n_begin = (int64_t)blockIdx.x * a.rows_per_slice;
    int64_t n_end = n_begin + a.rows_per_slice;
    if (n_end > a.N) n_end = a.N;
    const int chunks_per_row = a.d / 4;
    const int stage_chunks = stage_rows * chunks_per_row;

    auto load_stage = [&](int buf, int64_t n0) {
        float *dst = smem + buf * stage_floats;
        for (int c = tid; c < stage_chunks; c += nthreads) {
            const int r = c / chunks_per_row, g = c - r * chunks_per_row;
            const int64_t n = n0 + r;
            const int sc = (g & 1) ? a.nbk + (g >> 1) : (g >> 1);    // split-half position of chunk g
            const bool ok = n < n_end;
            m2s_cp_async16(dst + r * a.d + 4 * sc, a.X + (ok ? n : n_begin) * a.ldx + 4 * g, ok);
        }
        asm volatile("cp.async.commit_group;\n" ::);
    };

    const int64_t nstages = (n_end > n_begin) ? (n_end - n_begin + stage_rows - 1) / stage_rows : 0;
    for (int s = 0; s < M2S_BUFFERS - 1; ++s) {
        if (s < nstages) load_stage(s, n_begin + (int64_t)s * stage_rows);
        else asm volatile("cp.async.commit_group;\n" ::);
    }
    for (int64_t s = 0; s < nstages; ++s) {
        asm volatile("cp.async.wait_group %0;\n" ::"n"(M2S_BUFFERS - 2));
        __syncthreads();
        if (s + M2S_BUFFERS - 1 < nstages)
            load_stage((int)((s + M2S_BUFFERS - 1) % M2S_BUFFERS), n_begin + (s + M2S_BUFFERS - 1) * stage_rows);
        else
            asm volatile("cp.async.commit_group;\n" ::);
        if (active) {
            const float *xs = smem + (int)(s % M2S_BUFFERS) * stage_floats + item_rg * a.d;
            const int step = a.rg * a.d;
#pragma unroll 2
            for (int q = 0; q < M2S_ROWS_PER_GROUP; ++q) {
                const float *row = xs + q * step;
                const float4 i0 = *reinterpret_cast<const float4 *>(row + oi);
                const float4 i1 = *reinterpret_cast<const float4 *>(row + oi + half);
                const float4 j0 = *reinterpret_cast<const float4 *>(row + oj);
                const float4 j1 = *reinterpret_cast<const float4 *>(row + oj + half);
                const float xi[8] = {i0.x, i0.y, i0.z, i0.w, i1.x, i1.y, i1.z, i1.w};
                const float xj[8] = {j0.x, j0.y, j0.z, j0.w, j1.x, j1.y, j1.z, j1.w};
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(xi[i], xj[j], acc[i][j]);
            }
        }
    }
    asm volatile("cp.async.wait_group 0;\n" ::);

    // add the row groups of the block one after the other (fixed order: the result is reproducible)
    for (int g = 0; g < a.rg; ++g) {
        if (active && item_rg == g) {
            float *t = red + tile * M2S_RED_STRIDE;      // odd stride: lanes (tiles) hit different banks
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) t[i * 8 + j] = (g == 0 ? 0.f : t[i * 8 + j]) + acc[i][j];
        }
        __syncthreads();
    }
    float *mine = a.partials + (size_t)blockIdx.x * a.ntiles * 64;
    for (int e = tid; e < a.ntiles * 64; e += nthreads) mine[e] = red[(e >> 6) * M2S_RED_STRIDE + (e & 63)];
}

// out[p(i,j)] = sum over the slices, in slice order, i <= j only.
__global__ void __launch_bounds__(256)
moment2_small_reduce_kernel(const float *__restrict__ partials, float *__restrict__ out, int d, int nbk, int ntiles,
                            int slices, int dense)
{
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e >= ntiles * 64) return;
    const int tile = e >> 6, i8 = (e >> 3) & 7, j8 = e & 7;
    int ib, jb;
    if (dense) {
        ib = tile / nbk;
        jb = tile - ib * nbk;
    } else {
        int64_t x, y;
        tri_decode(nbk, tile, x, y);
        ib = (int)x;
        jb = (int)y;
    }
    const int gi = 8 * ib + i8, gj = 8 * jb + j8;
    if (gi > gj) return;
    float s = 0.f;
    const size_t stride = (size_t)ntiles * 64;
    for (int k0 = 0; k0 < slices; k0 += 32) {
        float v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) v[u] = (k0 + u < slices) ? __ldcg(partials + (size_t)(k0 + u) * stride + e) : 0.f;
#pragma unroll
        for (int u = 0; u < 32; ++u) s += v[u];
    }
    out[tri_encode(d, gi, gj)] = s;
}

struct M2SmallPlan {
    int nbk, ntiles, rg, threads, slices;
    int64_t rows_per_slice;
    size_t smem, partial_bytes;
};

bool moment2_small_applies(int64_t N, int64_t d)
{
    return d % 8 == 0 && d >= 8 && d <= 64 && N >= 1;
}

static M2SmallPlan moment2_small_plan(int64_t N, int64_t d, unsigned flags)
{
    M2SmallPlan p;
    p.nbk = (int)d / 8;
    p.ntiles = (flags & ST_FLAG_DENSE_CONTROL) ? p.nbk * p.nbk : p.nbk * (p.nbk + 1) / 2;
    p.rg = M2S_MAX_THREADS / p.ntiles;
    if (p.rg > 16) p.rg = 16;
    if (p.rg < 1) p.rg = 1;
    p.threads = (p.ntiles * p.rg + 31) / 32 * 32;
    const int stage_rows = p.rg * M2S_ROWS_PER_GROUP;
    int64_t slices = sm_count_or_default();
    const int64_t max_slices = (N + stage_rows - 1) / stage_rows;
    if (slices > max_slices) slices = max_slices;
    p.rows_per_slice = (N + slices - 1) / slices;
    p.slices = (int)((N + p.rows_per_slice - 1) / p.rows_per_slice);
    p.smem = ((size_t)M2S_BUFFERS * stage_rows * d + (size_t)p.ntiles * M2S_RED_STRIDE) * sizeof(float);
    p.partial_bytes = (size_t)p.slices * p.ntiles * 64 * sizeof(float);
    return p;
}

size_t moment2_small_workspace(int64_t N, int64_t d, unsigned flags)
{
    return kWsHeaderBytes + moment2_small_plan(N, d, flags).partial_bytes;
}

st_status moment2_small(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                        unsigned flags, cudaStream_t stream)
{
    const M2SmallPlan p = moment2_small_plan(N, d, flags);
    if (!ws || ws_bytes < kWsHeaderBytes + p.partial_bytes) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    M2SmallArgs a;
    a.X = X;
    a.partials = (float *)((unsigned char *)ws + kWsHeaderBytes);
    a.N = N; a.ldx = ldx; a.rows_per_slice = p.rows_per_slice;
    a.d = (int)d; a.nbk = p.nbk; a.ntiles = p.ntiles; a.rg = p.rg;
    a.dense = (flags & ST_FLAG_DENSE_CONTROL) ? 1 : 0;
    if (!ensure_dynamic_smem(moment2_small_kernel, p.smem)) return ST_ERR_CUDA;
    moment2_small_kernel<<<p.slices, p.threads, p.smem, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    const int n = p.ntiles * 64;
    moment2_small_reduce_kernel<<<(n + 255) / 256, 256, 0, stream>>>(a.partials, out, (int)d, p.nbk, p.ntiles, p.slices,
                                                                     a.dense);
    return launch_status();
}

}  // namespace st
