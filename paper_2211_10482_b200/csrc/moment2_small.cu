// st_sym_moment2, fp32 path for few features (d % 8 == 0, d <= 64) and many samples -- the regime
// of the paper's covariance workloads (Section 7.2; its real datasets have 6 and 13 features).
//
// out[p(i,j)] = sum_n X[n,i] X[n,j], 0 <= i <= j < d  (Section 3, M1; Section 5.5, y_U = i <= j).
//
// The d columns are dealt to d/8 "column blocks"; block b owns columns 4b..4b+3 of the first half
// of a row and the same four of the second half (two 16-byte chunks, so that the threads of a warp
// read one contiguous 128-byte segment per load and a row can stay in its natural layout).  Every
// unordered pair of columns lies in exactly one unordered pair of blocks, so the 8x8 tiles {x,y}
// (x <= y) cover the unique set once: 36 tiles for d = 64, not 64.
//
// Shared memory returns 32 words per cycle to the registers of an SM, against 128 FMA lanes: an
// 8x8 register tile (16 operand words per 64 FMAs) saturates both at once.  A work item is
// therefore two tiles with one block in common, {s,p} and {s,q}: 24 operand words per 128 FMAs.
// The host pairs the tiles up (an odd one out computes its tile twice and drops one copy).  The
// rows of a shared-memory stage are dealt to RG "row groups"; one thread owns (item, row group)
// and keeps the 128 sums of its item over its rows in registers.  Blocks own slices of the samples
// (one block per SM), receive them in a 3-buffer pipeline of bulk copies, add their row groups in
// shared memory in a fixed order and write one partial per block; a second kernel adds the
// partials in slice order.  Diagonal tiles compute all 64 products (the 28 below the diagonal are
// dropped): 36*64 = 2304 FMAs issued per sample for 2080 useful.
#include "st_common.cuh"
#include "st_index.cuh"
#include "tc_common.cuh"

namespace st {

constexpr int M2S_MAX_THREADS = 256;
constexpr int M2S_MAX_ITEMS = 32;
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

// work items: tiles {s,p} and {s,q} of column blocks; q == 255 marks an item with one tile only
struct M2SmallItems {
    int n;
    unsigned char s[M2S_MAX_ITEMS], p[M2S_MAX_ITEMS], q[M2S_MAX_ITEMS];
};

struct M2SmallArgs {
    const float *X;
    float *partials;      // [slices][128][nitems]
    unsigned *status;     // workspace header (status and detail words)
    int64_t N, ldx, rows_per_slice;
    int d, nbk, rg, rpg, dense, bar_floats;
    M2SmallItems items;
};

// column of element e (0..7) of column block b
__device__ __forceinline__ int m2s_column(int b, int e, int half) { return (e < 4) ? 4 * b + e : half + 4 * b + (e - 4); }

__global__ void __launch_bounds__(M2S_MAX_THREADS, 1) moment2_small_kernel(const M2SmallArgs a)
{
    extern __shared__ __align__(16) float smem[];
    const int stage_rows = a.rg * a.rpg;
    const int stage_floats = stage_rows * a.d;
    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int nitems = a.items.n;
    const int item_rg = tid / nitems, item = tid - item_rg * nitems;
    const bool active = item_rg < a.rg;
    const int half = 4 * a.nbk;
    const int bs = a.items.s[item], bp = a.items.p[item];
    const int bq = a.items.q[item] == 255 ? bp : a.items.q[item];
    const int os = 4 * bs, op = 4 * bp, oq = 4 * bq;

    float accp[8][8], accq[8][8];                      // tiles {s,p} and {s,q}
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) accp[i][j] = accq[i][j] = 0.f;

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
                const float4 s0 = *reinterpret_cast<const float4 *>(row + os);
                const float4 s1 = *reinterpret_cast<const float4 *>(row + os + half);
                const float4 p0 = *reinterpret_cast<const float4 *>(row + op);
                const float4 p1 = *reinterpret_cast<const float4 *>(row + op + half);
                const float4 q0 = *reinterpret_cast<const float4 *>(row + oq);
                const float4 q1 = *reinterpret_cast<const float4 *>(row + oq + half);
                const float xs[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
                const float xp[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
                const float xq[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        accp[i][j] = fmaf(xs[i], xp[j], accp[i][j]);
                        accq[i][j] = fmaf(xs[i], xq[j], accq[i][j]);
                    }
            }
        }
        if (++buf == M2S_BUFFERS) {
            buf = 0;
            parity ^= 1u;
        }
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the sum over the slices may be launched; it waits for this grid to end
    if (*abort_flag && tid == 0) {
        // after a time-out: give the copies still in flight a bounded time to land before the
        // shared memory is reused or released
        for (int s = (nstages > M2S_BUFFERS ? nstages - M2S_BUFFERS : 0); s < nstages; ++s)
            for (uint32_t it = 0; it < tc::kSpinLimit; ++it)
                if (tc::mbar_try_wait(&full[s % M2S_BUFFERS], (uint32_t)((s / M2S_BUFFERS) & 1))) break;
    }
    __syncthreads();                                   // every thread is done with the stage buffers

    // block-level sum over the row groups, in group order (reproducible): the sums go to shared
    // memory as red[k][group][item] (consecutive threads, consecutive words; k < 64 is tile {s,p},
    // k >= 64 tile {s,q}), output (k, item) is then summed over the groups by `parts` threads, each
    // over a fixed range, and by one thread over the parts.
    float *red = smem;
    const int cells = a.rg * nitems;
    if (active) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                red[(i * 8 + j) * cells + tid] = accp[i][j];
                red[(64 + i * 8 + j) * cells + tid] = accq[i][j];
            }
    }
    __syncthreads();
    const int nout = 128 * nitems;
    int parts = nthreads / nout;
    if (parts < 1) parts = 1;
    if (parts > a.rg) parts = a.rg;
    float *mine = a.partials + (size_t)blockIdx.x * nout;
    if (parts == 1) {
        for (int o = tid; o < nout; o += nthreads) {
            const int k = o / nitems, t = o - k * nitems;
            const float *p = red + k * cells + t;
            float sum = 0.f;
            for (int g = 0; g < a.rg; ++g) sum += p[g * nitems];
            mine[o] = sum;
        }
    } else {
        float *scratch = red + 128 * cells;            // [parts][nout]
        const int per = (a.rg + parts - 1) / parts;
        if (tid < parts * nout) {
            const int part = tid / nout, o = tid - part * nout;
            const int k = o / nitems, t = o - k * nitems;
            const float *p = red + k * cells + t;
            int g_end = (part + 1) * per;
            if (g_end > a.rg) g_end = a.rg;
            float sum = 0.f;
            for (int g = part * per; g < g_end; ++g) sum += p[g * nitems];
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

// out[p(ci,cj)] = sum over the slices, in slice order, of element (k, item) of the partials.
__global__ void __launch_bounds__(256)
moment2_small_reduce_kernel(const float *__restrict__ partials, float *__restrict__ out, int d, int nbk, int slices,
                            int dense, const M2SmallItems items)
{
    // launched as a programmatic dependent of the kernel that writes the partial sums: the launch overlaps
    // that kernel's tail, and nothing is read before it has completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int o = blockIdx.x * 256 + threadIdx.x;
    const int nitems = items.n;
    if (o >= nitems * 128) return;
    const int k = o / nitems, item = o - k * nitems;
    const int i8 = (k >> 3) & 7, j8 = k & 7;
    const int x = items.s[item];
    const int y = (k < 64) ? items.p[item] : items.q[item];
    if (y == 255) return;                              // odd item out: no second tile
    // a diagonal tile keeps its upper half; the dense control also computes the tiles below the
    // diagonal and discards them here
    if ((x == y && i8 > j8) || (dense && x > y)) return;
    const int ci = m2s_column(x, i8, 4 * nbk), cj = m2s_column(y, j8, 4 * nbk);
    float s = 0.f;
    const size_t stride = (size_t)nitems * 128;
    for (int k0 = 0; k0 < slices; k0 += 32) {
        float v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) v[u] = (k0 + u < slices) ? __ldcg(partials + (size_t)(k0 + u) * stride + o) : 0.f;
#pragma unroll
        for (int u = 0; u < 32; ++u) s += v[u];
    }
    const int64_t at = tri_encode(d, ci < cj ? ci : cj, ci < cj ? cj : ci);
    if (ST_BOUNDS_OK(at, tri_rows(d), 2)) out[at] = s;
}

struct M2SmallPlan {
    int nbk, rg, rpg, threads, slices;
    int64_t rows_per_slice;
    size_t smem, data_bytes, partial_bytes;
    M2SmallItems items;
};

bool moment2_small_applies(int64_t N, int64_t d)
{
    return d % 8 == 0 && d >= 8 && d <= 64 && N >= 1;
}

// Pairs the tiles up into items with a common block.  Structured: for every block y the tiles
// {x,y}, x <= y, are paired along x with y as the common block; when their number is odd, tile
// {0,y} is held back, and the held-back tiles are paired with block 0 in common.  Dense control:
// all ordered tiles (x,y), paired along y with x in common.
static M2SmallItems moment2_small_items(int nbk, bool dense)
{
    M2SmallItems t;
    t.n = 0;
    auto add = [&](int s, int p, int q) {
        t.s[t.n] = (unsigned char)s;
        t.p[t.n] = (unsigned char)p;
        t.q[t.n] = (unsigned char)q;
        ++t.n;
    };
    if (dense) {
        for (int x = 0; x < nbk; ++x)
            for (int y = 0; y < nbk; y += 2) add(x, y, y + 1 < nbk ? y + 1 : 255);
    } else {
        int held[8], nheld = 0;
        for (int y = 0; y < nbk; ++y) {
            int x = 0;
            if ((y + 1) % 2 == 1) {
                held[nheld++] = y;
                x = 1;
            }
            for (; x + 1 <= y; x += 2) add(y, x, x + 1);
        }
        for (int h = 0; h < nheld; h += 2) add(0, held[h], h + 1 < nheld ? held[h + 1] : 255);
    }
    for (int i = t.n; i < M2S_MAX_ITEMS; ++i) t.s[i] = t.p[i] = t.q[i] = 0;
    return t;
}

static M2SmallPlan moment2_small_plan(int64_t N, int64_t d, unsigned flags)
{
    M2SmallPlan p;
    p.nbk = (int)d / 8;
    p.items = moment2_small_items(p.nbk, (flags & ST_FLAG_DENSE_CONTROL) != 0);
    const int nitems = p.items.n;
    const int max_stage_rows = M2S_STAGE_BYTES / (4 * (int)d);
    p.rg = M2S_MAX_THREADS / nitems;
    if (p.rg > max_stage_rows / 8) p.rg = max_stage_rows / 8;
    if (p.rg < 1) p.rg = 1;
    p.threads = (nitems * p.rg + 31) / 32 * 32;
    p.rpg = 8;
    int64_t slices = sm_count_or_default();
    const int64_t max_slices = (N + p.rg * 8 - 1) / (p.rg * 8);
    if (slices > max_slices) slices = max_slices;
    p.rows_per_slice = (N + slices - 1) / slices;
    p.slices = (int)((N + p.rows_per_slice - 1) / p.rows_per_slice);
    // long slices: 16 rows per thread and stage halve the number of block-wide barriers
    if (p.rg * 16 <= max_stage_rows && p.rows_per_slice >= 4 * p.rg * 16) p.rpg = 16;
    const size_t cells = (size_t)p.rg * nitems;
    const size_t main_bytes = (size_t)M2S_BUFFERS * p.rg * p.rpg * d * sizeof(float);
    const size_t sum_bytes = (128 * cells + (size_t)M2S_MAX_THREADS) * sizeof(float);
    p.data_bytes = round_up(main_bytes > sum_bytes ? main_bytes : sum_bytes, 16);
    p.smem = p.data_bytes + 64;                        // barriers and the abort flag behind the data
    p.partial_bytes = (size_t)p.slices * nitems * 128 * sizeof(float);
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
    a.d = (int)d; a.nbk = p.nbk; a.rg = p.rg; a.rpg = p.rpg;
    a.items = p.items;
    a.status = (unsigned *)ws;
    a.bar_floats = (int)(p.data_bytes / sizeof(float));
    a.dense = (flags & ST_FLAG_DENSE_CONTROL) ? 1 : 0;
    if (!ensure_dynamic_smem(moment2_small_kernel, p.smem)) return ST_ERR_CUDA;
    moment2_small_kernel<<<p.slices, p.threads, p.smem, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    const int n = p.items.n * 128;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((n + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float *partials = a.partials;
    const int di = (int)d, dense = a.dense;
    if (cudaLaunchKernelEx(&cfg, moment2_small_reduce_kernel, partials, out, di, p.nbk, p.slices, dense, p.items) != cudaSuccess) {
        (void)cudaGetLastError();
        return ST_ERR_CUDA;
    }
    return ST_OK;
}

}  // namespace st
