// st_sym_moment2, fp32 path for few features (d % 8 == 0, d <= 64) and many samples -- the regime
// of the paper's covariance workloads (Section 7.2; its real datasets have 6 and 13 features).
//
// out[p(i,j)] = sum_n X[n,i] X[n,j], 0 <= i <= j < d  (Section 3, M1; Section 5.5, y_U = i <= j).
//
// The d columns are dealt to d/8 "column blocks"; block b owns columns 4b..4b+3 of the first half
// of a row and the same four of the second half (two 16-byte chunks, so that the threads of a warp
// read one contiguous 128-byte segment per load and a row can stay in its natural layout).  Every
// unordered pair of columns lies in exactly one unordered pair of blocks, so the 8x8 register tiles
// (ib <= jb) cover the unique set once: 36 tiles for d = 64, not 64.  The rows of a shared-memory
// stage are dealt to RG "row groups"; one thread owns (tile, row group) and keeps the 64 sums of
// its tile over its rows in registers: 4 shared-memory loads per 64 FMAs.  Blocks own slices of the
// samples (one block per SM), stream them through a 3-buffer cp.async pipeline, add their row
// groups in shared memory in a fixed order and write one partial per block; a second kernel adds
// the partials in slice order.  Diagonal tiles compute all 64 products (the 28 below the diagonal
// are dropped): 36*64 = 2304 FMAs issued per sample for 2080 useful.
#include "st_common.cuh"
#include "st_index.cuh"
#include "tc_common.cuh"

namespace st {

constexpr int M2S_MAX_THREADS = 512;
constexpr int M2S_BUFFERS = 3;
constexpr int M2S_STAGE_BYTES = 57344;     // upper bound of one stage (3 stages + slack fit in 227 KB)

// bulk copy global -> shared of `bytes` (a multiple of 16, both addresses 16-byte aligned),
// completion counted in bytes on `bar`
__device__ __forceinline__ void m2s_bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     tc::smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(tc::smem_u32(bar))
                 : "memory");
}

struct M2SmallArgs {
    const float *X;
    float *partials;      // [slices][64][ntiles]
    unsigned *status;     // workspace header (status and detail words)
    int64_t N, ldx, rows_per_slice;
    int d, nbk, ntiles, rg, rpg, dense, bar_floats;
};

// column of element e (0..7) of column block b
__device__ __forceinline__ int m2s_column(int b, int e, int half) { return (e < 4) ? 4 * b + e : half + 4 * b + (e - 4); }

__device__ __forceinline__ void m2s_tile(int tile, int nbk, int dense, int &ib, int &jb)
{
    if (dense) {
        ib = tile / nbk;
        jb = tile - ib * nbk;
    } else {
        int64_t x, y;
        tri_decode(nbk, tile, x, y);
        ib = (int)x;
        jb = (int)y;
    }
}

__global__ void __launch_bounds__(M2S_MAX_THREADS, 1) moment2_small_kernel(const M2SmallArgs a)
{
    extern __shared__ __align__(16) float smem[];
    const int stage_rows = a.rg * a.rpg;
    const int stage_floats = stage_rows * a.d;
    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int item_rg = tid / a.ntiles, tile = tid - item_rg * a.ntiles;
    const bool active = item_rg < a.rg;
    int ib, jb;
    m2s_tile(tile, a.nbk, a.dense, ib, jb);
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

    uint64_t *full = reinterpret_cast<uint64_t *>(smem + a.bar_floats);      // one barrier per buffer
    volatile int *abort_flag = reinterpret_cast<volatile int *>(full + M2S_BUFFERS);
    if (tid == 0) {
        for (int b = 0; b < M2S_BUFFERS; ++b) tc::mbar_init(&full[b], 1);
        *abort_flag = 0;
        if (blockIdx.x == 0) {      // a time-out report can only be written 2^24 failed polls later
            a.status[kWsStatusWord] = 0;
            a.status[kWsDetailWord] = 0;
        }
        tc::fence_barrier_init();
    }
    __syncthreads();

    const int nstages = (n_end > n_begin) ? (int)((n_end - n_begin + stage_rows - 1) / stage_rows) : 0;
    const bool contiguous = (a.ldx == a.d);
    // the rows of a stage arrive by bulk copies issued from warp 0: one copy when the rows are
    // contiguous in memory, one per row otherwise; rows past the end of the slice are not copied
    // and not read
    auto issue_stage = [&](int buf, int s) {
        if (tid >= 32) return;
        const int64_t n0 = n_begin + (int64_t)s * stage_rows;
        const int rows = (n_end - n0 < stage_rows) ? (int)(n_end - n0) : stage_rows;
        float *dst = smem + buf * stage_floats;
        const uint32_t row_bytes = (uint32_t)a.d * 4u;
        if (tid == 0) tc::mbar_expect_tx(&full[buf], (uint32_t)rows * row_bytes);
        __syncwarp();
        if (contiguous) {
            if (tid == 0) m2s_bulk_load(dst, a.X + n0 * a.ldx, (uint32_t)rows * row_bytes, &full[buf]);
        } else {
            for (int r = tid; r < rows; r += 32) m2s_bulk_load(dst + r * a.d, a.X + (n0 + r) * a.ldx, row_bytes, &full[buf]);
        }
    };

    for (int s = 0; s < M2S_BUFFERS - 1 && s < nstages; ++s) issue_stage(s, s);
    const int step = a.rg * a.d;
    int buf = 0;
    uint32_t parity = 0;
    for (int s = 0; s < nstages; ++s) {
        // a wait that gives up raises the abort flag; every thread still walks all stages so that
        // the block-wide barriers stay matched, and the host reads the status word afterwards
        (void)tc::mbar_wait(&full[buf], parity, abort_flag, a.status, 1);
        __syncthreads();                                // stage s-1 is consumed: its buffer may be refilled
        if (s + M2S_BUFFERS - 1 < nstages) issue_stage(buf == 0 ? M2S_BUFFERS - 1 : buf - 1, s + M2S_BUFFERS - 1);
        int qn = a.rpg;
        if (s == nstages - 1) {                         // last stage of the slice: only the rows that exist
            const int rows = (int)(n_end - n_begin - (int64_t)s * stage_rows);
            qn = (rows - item_rg + a.rg - 1) / a.rg;
            if (qn > a.rpg) qn = a.rpg;
        }
        if (active) {
            const float *row = smem + buf * stage_floats + item_rg * a.d;
#pragma unroll 2
            for (int q = 0; q < qn; ++q, row += step) {
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
        if (++buf == M2S_BUFFERS) {
            buf = 0;
            parity ^= 1u;
        }
    }
    if (*abort_flag && tid == 0) {
        // after a time-out: give the copies still in flight a bounded time to land before the
        // shared memory is reused or released
        for (int s = (nstages > M2S_BUFFERS ? nstages - M2S_BUFFERS : 0); s < nstages; ++s)
            for (uint32_t it = 0; it < tc::kSpinLimit; ++it)
                if (tc::mbar_try_wait(&full[s % M2S_BUFFERS], (uint32_t)((s / M2S_BUFFERS) & 1))) break;
    }
    __syncthreads();                                   // every thread is done with the stage buffers

    // block-level sum over the row groups, in group order (reproducible): the sums go to shared
    // memory as red[k][group][tile] (consecutive threads, consecutive words), output (k, tile) is
    // then summed over the groups by `parts` threads, each over a fixed range, and by one thread
    // over the parts.
    float *red = smem;
    const int items = a.rg * a.ntiles;
    if (active) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) red[(i * 8 + j) * items + tid] = acc[i][j];
    }
    __syncthreads();
    const int nout = 64 * a.ntiles;
    int parts = nthreads / nout;
    if (parts < 1) parts = 1;
    if (parts > a.rg) parts = a.rg;
    float *mine = a.partials + (size_t)blockIdx.x * nout;
    if (parts == 1) {
        for (int o = tid; o < nout; o += nthreads) {
            const int k = o / a.ntiles, t = o - k * a.ntiles;
            const float *p = red + k * items + t;
            float sum = 0.f;
            for (int g = 0; g < a.rg; ++g) sum += p[g * a.ntiles];
            mine[o] = sum;
        }
    } else {
        float *scratch = red + 64 * items;             // [parts][nout]
        const int per = (a.rg + parts - 1) / parts;
        if (tid < parts * nout) {
            const int part = tid / nout, o = tid - part * nout;
            const int k = o / a.ntiles, t = o - k * a.ntiles;
            const float *p = red + k * items + t;
            int g_end = (part + 1) * per;
            if (g_end > a.rg) g_end = a.rg;
            float sum = 0.f;
            for (int g = part * per; g < g_end; ++g) sum += p[g * a.ntiles];
            scratch[part * nout + o] = sum;
        }
        __syncthreads();
        if (tid < nout) {
            float sum = 0.f;
            for (int part = 0; part < parts; ++part) sum += scratch[part * nout + tid];
            mine[tid] = sum;
        }
    }
}

// out[p(ci,cj)] = sum over the slices, in slice order, of element (k, tile) of the partials.
__global__ void __launch_bounds__(256)
moment2_small_reduce_kernel(const float *__restrict__ partials, float *__restrict__ out, int d, int nbk, int ntiles,
                            int slices, int dense)
{
    const int o = blockIdx.x * 256 + threadIdx.x;
    if (o >= ntiles * 64) return;
    const int k = o / ntiles, tile = o - k * ntiles;
    const int i8 = k >> 3, j8 = k & 7;
    int ib, jb;
    m2s_tile(tile, nbk, dense, ib, jb);
    if (ib > jb || (ib == jb && i8 > j8)) return;      // dense control: the other half is discarded
    const int ci = m2s_column(ib, i8, 4 * nbk), cj = m2s_column(jb, j8, 4 * nbk);
    float s = 0.f;
    const size_t stride = (size_t)ntiles * 64;
    for (int k0 = 0; k0 < slices; k0 += 32) {
        float v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) v[u] = (k0 + u < slices) ? __ldcg(partials + (size_t)(k0 + u) * stride + o) : 0.f;
#pragma unroll
        for (int u = 0; u < 32; ++u) s += v[u];
    }
    out[tri_encode(d, ci < cj ? ci : cj, ci < cj ? cj : ci)] = s;
}

struct M2SmallPlan {
    int nbk, ntiles, rg, rpg, threads, slices;
    int64_t rows_per_slice;
    size_t smem, data_bytes, partial_bytes;
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
    const int max_stage_rows = M2S_STAGE_BYTES / (4 * (int)d);
    p.rg = M2S_MAX_THREADS / p.ntiles;
    if (p.rg > max_stage_rows / 8) p.rg = max_stage_rows / 8;
    if (p.rg < 1) p.rg = 1;
    p.threads = (p.ntiles * p.rg + 31) / 32 * 32;
    p.rpg = 8;
    int64_t slices = sm_count_or_default();
    const int64_t max_slices = (N + p.rg * 8 - 1) / (p.rg * 8);
    if (slices > max_slices) slices = max_slices;
    p.rows_per_slice = (N + slices - 1) / slices;
    p.slices = (int)((N + p.rows_per_slice - 1) / p.rows_per_slice);
    // long slices: 16 rows per thread and stage halve the number of block-wide barriers
    if (p.rg * 16 <= max_stage_rows && p.rows_per_slice >= 4 * p.rg * 16) p.rpg = 16;
    const size_t items = (size_t)p.rg * p.ntiles;
    const size_t main_bytes = (size_t)M2S_BUFFERS * p.rg * p.rpg * d * sizeof(float);
    const size_t sum_bytes = (64 * items + (size_t)M2S_MAX_THREADS) * sizeof(float);
    p.data_bytes = round_up(main_bytes > sum_bytes ? main_bytes : sum_bytes, 16);
    p.smem = p.data_bytes + 64;                        // barriers and the abort flag behind the data
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
    a.d = (int)d; a.nbk = p.nbk; a.ntiles = p.ntiles; a.rg = p.rg; a.rpg = p.rpg;
    a.status = (unsigned *)ws;
    a.bar_floats = (int)(p.data_bytes / sizeof(float));
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
