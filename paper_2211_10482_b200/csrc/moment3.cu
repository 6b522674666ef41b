// st_sym_moment3: out[q(i,j,k)] = sum_n X[n,i] X[n,j] X[n,k] over the unique set
// 0<=i<=j<=k<d (Section 3, M2; Section 2, "Tensor Structures").  fp32 FMA bound.
//
// Work decomposition.  The unique set is cut into register tiles (i; 8 values of j; 8 values
// of k) aligned to blocks of 8: tile (i, jb, kb) with block(i) <= jb <= kb.  One thread owns
// one tile for a slice of the samples and keeps its <= 64 sums in registers; per sample it
// reads x_i, the 8 x_j and the 8 x_k of the row from shared memory, forms the pair product
// p = x_i * x_j once per j (loop-invariant code motion of Section 5.5 applied to the k loop)
// and issues one FMA per unique triple (two per packed f32x2 instruction; on a triangular
// tile a pair that straddles k = j carries one unused lane) -- no other work outside i<=j<=k:
//     variant 0        full 8x8 tile            (jb > block(i) or i at a block start, kb > jb)
//     variant 1        triangular, k >= j       (kb == jb; rows j < i are not stored)
//     variant 1+s      rows j >= i only, s=i%8  (jb == block(i), kb > jb), s = 1..7
// Threads are grouped into warps of one variant so no lane diverges; warps are dealt to
// G thread blocks x 4 schedulers so that every scheduler gets the same FMA count.  The
// tile table is built on the host for the given d and travels as a kernel parameter.
//
// The sample range is split over gridDim.y slices; every slice writes its partial sums to
// the workspace and a second kernel adds the slices in a fixed order.
//
// Any 1 <= d <= 256.  A stage holds whole rows, padded with zero columns to a multiple of 8 (tiles
// that reach into the padding compute zeros that are never stored).  Up to d = 64 the tile table
// travels as a kernel parameter; beyond that it is copied into the workspace before the launch,
// stages get shorter (three of them must fit in shared memory) and more thread blocks share a
// sample slice.  Rows that are not 16-byte aligned (d or ldx not a multiple of 4) are staged with
// plain 4-byte loads instead of asynchronous 16-byte copies.
#include "st_common.cuh"
#include "st_index.cuh"
#include <algorithm>
#include <mutex>
#include <vector>

namespace st {

constexpr int M3_THREADS = 512;            // 16 warps per block
constexpr int M3_WPB = M3_THREADS / 32;
constexpr int M3_STAGE_ROWS = 128;         // most sample rows per shared-memory stage
constexpr int M3_PARAM_D = 64;             // largest d whose tile table travels as a kernel parameter
constexpr int M3_MAX_D = 256;
constexpr int M3_BUFFERS = 3;               // shared-memory stages in flight
constexpr size_t M3_SMEM_BUDGET = 220 * 1024;

// tile word: i | jb << 9 | kb << 15 | valid << 31
__host__ __device__ inline unsigned m3_tile_word(int i, int jb, int kb) { return (unsigned)i | ((unsigned)jb << 9) | ((unsigned)kb << 15) | (1u << 31); }

// The table as a kernel parameter (d <= 64): tile words packed into 16 bits, i | jb << 6 | kb << 9 | valid << 15,
// so that the parameters of the common launch stay below 4 KB.
template <int WARPS>
struct M3Table {
    unsigned char variant[WARPS];          // per warp slot (group-major): variant id, 255 = idle
    unsigned short tile[WARPS * 32];       // per thread slot
};
__host__ __device__ inline unsigned short m3_pack16(unsigned t)
{
    return (unsigned short)((t & 63u) | (((t >> 9) & 7u) << 6) | (((t >> 15) & 7u) << 9) | ((t >> 31) << 15));
}
__host__ __device__ inline unsigned m3_unpack16(unsigned short h)
{
    return (h & 63u) | (((h >> 6) & 7u) << 9) | (((h >> 9) & 7u) << 15) | ((unsigned)(h >> 15) << 31);
}

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem, bool valid)
{
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    const int sz = valid ? 16 : 0;         // src-size 0: the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

// One stage of rows for one tile.  Row layout in shared memory ("split halves"): columns
// 8b..8b+3 of block b sit at floats 4b.., columns 8b+4..8b+7 at floats 4*nbk+4b.., so that a
// 128-bit load of "the first (second) half of block b" by lanes with arbitrary b touches
// each bank once.
// Packed fp32 pairs: sm_100 executes fma.rn.f32x2 on a 64-bit register pair, which halves the
// issue slots per FMA and leaves room for the shared-memory loads and the pair products.
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// One stage of rows for one tile.  acc[a][c] holds the sums for j = a, k = 2c and 2c+1.
// DC > 0: the row length is the compile-time constant DC, so that every shared-memory address of
// the loop is "row base + immediate" (integer multiply-adds share the FMA pipe: with run-time strides
// the kernel was 9 % slower at d = 64).
template <int J0, bool DIAG, int DC>
__device__ __forceinline__ void m3_stage(const float *__restrict__ xs, int rows_, int d_, int pi, int oj, int ok, int half_,
                                         uint64_t (&acc)[8][4])
{
    const int d = DC > 0 ? DC : d_, half = DC > 0 ? DC / 2 : half_;
    const int rows = DC > 0 ? M3_STAGE_ROWS : rows_;      // the instance with compile-time strides has full stages
#pragma unroll 2
    for (int r = 0; r < rows; ++r) {
        const float *row = xs + r * d;
        const float xi = row[pi];
        const float4 ja = *reinterpret_cast<const float4 *>(row + oj);
        const float4 jb = *reinterpret_cast<const float4 *>(row + oj + half);
        float4 ka, kb;
        if (DIAG) {
            ka = ja;
            kb = jb;
        } else {
            ka = *reinterpret_cast<const float4 *>(row + ok);
            kb = *reinterpret_cast<const float4 *>(row + ok + half);
        }
        const float xj[8] = {ja.x, ja.y, ja.z, ja.w, jb.x, jb.y, jb.z, jb.w};
        const uint64_t xk[4] = {pack2(ka.x, ka.y), pack2(ka.z, ka.w), pack2(kb.x, kb.y), pack2(kb.z, kb.w)};
#pragma unroll
        for (int a = J0; a < 8; ++a) {
            const float p = xi * xj[a];
            const uint64_t pp = pack2(p, p);
#pragma unroll
            for (int c = (DIAG ? a / 2 : 0); c < 4; ++c) acc[a][c] = ffma2(pp, xk[c], acc[a][c]);
        }
    }
}

// d: columns of X; dp: d rounded up to a multiple of 8 (row length of a stage); rows: sample rows per stage
// (a multiple of 8, at most M3_STAGE_ROWS).  The tile table comes from `tab` when gtile is NULL.
struct M3Args {
    const float *X;
    float *partials;
    unsigned *status;
    const unsigned char *gvariant;         // tile table in global memory (d > M3_PARAM_D), else NULL
    const unsigned *gtile;
    int64_t N, ldx, rows_per_slice;
    int d, dp, rows, out_elems;
};

// ALIGNED: rows are staged by asynchronous 16-byte copies; otherwise by plain 4-byte loads (an instance of
// its own: with both loaders in one kernel the common one ran 7 % slower).
template <int WARPS, int DC, bool ALIGNED>
__global__ void __launch_bounds__(M3_THREADS, 1)
moment3_kernel(const M3Args a, const __grid_constant__ M3Table<WARPS> tab)
{
    const float *__restrict__ X = a.X;
    const int64_t N = a.N, ldx = a.ldx, rows_per_slice = a.rows_per_slice;
    const int d = a.d, dp = DC > 0 ? DC : a.dp, out_elems = a.out_elems;
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {   // this kernel has no bounded waits: the status is "ok"
        a.status[kWsStatusWord] = 0;
        a.status[kWsDetailWord] = 0;
    }
    extern __shared__ __align__(16) float smem[];   // M3_BUFFERS stages of a.rows x dp floats
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = blockIdx.x;
    const int slot = group * M3_WPB + warp;
    const int variant = a.gtile ? a.gvariant[slot] : tab.variant[slot];
    const unsigned t = a.gtile ? a.gtile[slot * 32 + lane] : m3_unpack16(tab.tile[slot * 32 + lane]);
    const bool valid = (t >> 31) != 0u;
    const int ti = t & 511, tjb = (t >> 9) & 63, tkb = (t >> 15) & 63;
    const int nbk = dp / 8;
    const int half = 4 * nbk;
    // shared-memory float offset of column c: block c/8, half (c%8)/4
    const int pi = ((ti & 7) < 4) ? 4 * (ti >> 3) + (ti & 3) : half + 4 * (ti >> 3) + (ti & 3);
    const int oj = 4 * tjb, ok = 4 * tkb;

    uint64_t acc[8][4];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = 0ull;

    const int64_t n_begin = (int64_t)blockIdx.y * rows_per_slice;
    int64_t n_end = n_begin + rows_per_slice;
    if (n_end > N) n_end = N;
    const int stage_rows = DC > 0 ? M3_STAGE_ROWS : a.rows;
    const int stage_floats = stage_rows * dp;
    const int chunks_per_row = dp / 4;
    const int stage_chunks = stage_rows * chunks_per_row;

    auto load_stage = [&](int buf, int64_t n0) {
        float *dst = smem + buf * stage_floats;
        if (ALIGNED) {
            for (int c = tid; c < stage_chunks; c += M3_THREADS) {
                const int r = c / chunks_per_row, g = c - r * chunks_per_row;
                const int64_t n = n0 + r;
                const int sc = (g & 1) ? nbk + (g >> 1) : (g >> 1);   // split-half position of chunk g
                const bool in = n < n_end && 4 * g < d;                // padding columns and rows past the end: zeros
                cp_async16(dst + r * dp + 4 * sc, X + (in ? n * ldx + 4 * g : 0), in);
            }
        } else {
            // rows that are not 16-byte aligned: one float at a time (the barrier of the stage orders the stores)
            for (int e = tid; e < stage_rows * dp; e += M3_THREADS) {
                const int r = e / dp, c = e - r * dp;
                const int64_t n = n0 + r;
                const int g = c >> 2, sc = (g & 1) ? nbk + (g >> 1) : (g >> 1);
                dst[r * dp + 4 * sc + (c & 3)] = (n < n_end && c < d) ? X[n * ldx + c] : 0.f;
            }
        }
        cp_async_commit();
    };

    const int64_t nstages = (n_end > n_begin) ? (n_end - n_begin + stage_rows - 1) / stage_rows : 0;
    // three buffers, one barrier per stage: stage s+2 is issued after the barrier of stage s, which
    // every warp passes only after it has finished stage s-1 (the previous user of that buffer)
    for (int s = 0; s < M3_BUFFERS - 1; ++s) {
        if (s < nstages) load_stage(s, n_begin + (int64_t)s * stage_rows);
        else cp_async_commit();
    }
    for (int64_t s = 0; s < nstages; ++s) {
        cp_async_wait<M3_BUFFERS - 2>();
        __syncthreads();
        if (s + M3_BUFFERS - 1 < nstages)
            load_stage((int)((s + M3_BUFFERS - 1) % M3_BUFFERS), n_begin + (s + M3_BUFFERS - 1) * stage_rows);
        else
            cp_async_commit();
        const float *xs = smem + (int)(s % M3_BUFFERS) * stage_floats;
        switch (variant) {
        case 0: m3_stage<0, false, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        case 1: m3_stage<0, true, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        case 2: m3_stage<1, false, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        case 3: m3_stage<2, false, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        case 4: m3_stage<3, false, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        case 5: m3_stage<4, false, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        case 6: m3_stage<5, false, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        case 7: m3_stage<6, false, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        case 8: m3_stage<7, false, DC>(xs, stage_rows, dp, pi, oj, ok, half, acc); break;
        default: break;
        }
    }
    cp_async_wait<0>();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the slice sums may be launched; they wait for this grid to end

    if (!valid || variant == 255) return;
    float *mine = a.partials + (size_t)blockIdx.y * out_elems;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const int j = 8 * tjb + r;
        if (j < ti || j >= d) continue;                  // j >= d: padding columns
        const int base = (int)tet_encode(d, ti, j, j);   // row (i,j,*) is contiguous in k
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float lo, hi;
            unpack2(acc[r][c], lo, hi);
            const int k = 8 * tkb + 2 * c;
            if (k >= j && k < d && ST_BOUNDS_OK(base + (k - j), out_elems, 3)) mine[base + (k - j)] = lo;
            if (k + 1 >= j && k + 1 < d && ST_BOUNDS_OK(base + (k + 1 - j), out_elems, 3)) mine[base + (k + 1 - j)] = hi;
        }
    }
}

// out[e] = sum over slices of partials[slice][e], in a fixed order.  A block covers 32 consecutive
// elements; warp w adds the slices w, w+8, w+16, ... (all loads of a batch in flight before the first
// add), then the eight partial sums are added through shared memory.
constexpr int SUM_GROUPS = 8;
__global__ void __launch_bounds__(32 * SUM_GROUPS)
sum_slices_kernel(const float *__restrict__ partials, float *__restrict__ out, int64_t elems, int slices)
{
    __shared__ float part[SUM_GROUPS][32];
    // launched as a programmatic dependent of the kernel that writes the partial sums: the launch itself
    // overlaps that kernel's tail, and nothing is read before that kernel has completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
    const int64_t e = (int64_t)blockIdx.x * 32 + lane;
    float s = 0.f;
    if (e < elems) {
        constexpr int BATCH = 12;
        for (int k0 = g; k0 < slices; k0 += BATCH * SUM_GROUPS) {
            float v[BATCH];
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int k = k0 + u * SUM_GROUPS;
                v[u] = k < slices ? __ldcg(&partials[(size_t)k * elems + e]) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < BATCH; ++u) s += v[u];
        }
    }
    part[g][lane] = s;
    __syncthreads();
    if (g == 0 && e < elems) {
        float t = part[0][lane];
#pragma unroll
        for (int w = 1; w < SUM_GROUPS; ++w) t += part[w][lane];
        out[e] = t;
    }
}

st_status sum_slices_launch(const float *partials, float *out, int64_t elems, int slices, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((elems + 31) / 32));
    cfg.blockDim = dim3(32 * SUM_GROUPS);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, sum_slices_kernel, partials, out, elems, slices) != cudaSuccess) {
        (void)cudaGetLastError();
        return ST_ERR_CUDA;
    }
    return ST_OK;
}

// ---- host side: tile table ------------------------------------------------------------

struct WarpDesc {
    int variant;
    int cost;
    std::vector<unsigned> tiles;
};

static int variant_cost(int v)
{
    // fp32-pipe cycles per sample row: two per packed FMA, one per pair product, one per pair move
    if (v == 0) return 64 + 16;
    if (v == 1) return 40 + 16;
    const int rows = 8 - (v - 1);
    return rows * 8 + 2 * rows;
}

// The per-thread tile table of side d (dp = d rounded up to a multiple of 8): variant per warp slot
// and tile word per thread slot, group-major.
struct M3HostTable {
    int groups = 0;
    std::vector<unsigned char> variant;    // groups * M3_WPB
    std::vector<unsigned> tile;            // groups * M3_WPB * 32
};

static void build_table(int d, bool dense, M3HostTable &tab)
{
    const int nbk = (d + 7) / 8;
    std::vector<std::vector<unsigned>> lists(9);
    for (int i = 0; i < d; ++i) {
        const int ib = i / 8, s = i % 8;
        for (int jb = dense ? 0 : ib; jb < nbk; ++jb)
            for (int kb = dense ? 0 : jb; kb < nbk; ++kb) {
                int v;
                if (dense) v = 0;
                else if (kb == jb) v = 1;
                else if (jb == ib && s != 0) v = 1 + s;
                else v = 0;
                lists[v].push_back(m3_tile_word(i, jb, kb));
            }
    }
    std::vector<WarpDesc> warps;
    for (int v = 0; v < 9; ++v)
        for (size_t o = 0; o < lists[v].size(); o += 32) {
            WarpDesc w;
            w.variant = v;
            w.cost = variant_cost(v);
            w.tiles.assign(lists[v].begin() + o, lists[v].begin() + std::min(lists[v].size(), o + 32));
            warps.push_back(w);
        }
    const int nw = (int)warps.size();
    const int groups = (nw + M3_WPB - 1) / M3_WPB;
    // deal warps, most expensive first, to the scheduler bin (group, warp%4) with the least load,
    // then swap warps between the fullest bin and the others while that lowers the maximum
    std::stable_sort(warps.begin(), warps.end(), [](const WarpDesc &a, const WarpDesc &b) { return a.cost > b.cost; });
    const int bins = groups * 4;
    const int cap = M3_WPB / 4;
    std::vector<int> load(bins, 0);
    std::vector<std::vector<int>> members(bins);
    int next_bin = 0;
    for (int w = 0; w < nw; ++w) {
        int best = -1;
        if (bins <= 64) {
            for (int b = 0; b < bins; ++b)
                if ((int)members[b].size() < cap && (best < 0 || load[b] < load[best])) best = b;
        } else {
            // many bins: round robin over the bins in order of decreasing cost is as even and linear in time
            while ((int)members[next_bin].size() >= cap) next_bin = (next_bin + 1) % bins;
            best = next_bin;
            next_bin = (next_bin + 1) % bins;
        }
        members[best].push_back(w);
        load[best] += warps[w].cost;
    }
    for (int iter = 0; iter < 200 && bins <= 64; ++iter) {
        int hi = 0;
        for (int b = 1; b < bins; ++b)
            if (load[b] > load[hi]) hi = b;
        bool improved = false;
        for (int b = 0; b < bins && !improved; ++b) {
            if (b == hi) continue;
            for (size_t x = 0; x < members[hi].size() && !improved; ++x) {
                const int cx = warps[members[hi][x]].cost;
                // move x to b
                if ((int)members[b].size() < cap && load[b] + cx < load[hi]) {
                    load[b] += cx; load[hi] -= cx;
                    members[b].push_back(members[hi][x]);
                    members[hi].erase(members[hi].begin() + x);
                    improved = true;
                    break;
                }
                for (size_t y = 0; y < members[b].size(); ++y) {
                    const int cy = warps[members[b][y]].cost;
                    if (cy < cx && load[b] - cy + cx < load[hi]) {
                        load[b] += cx - cy; load[hi] -= cx - cy;
                        std::swap(members[hi][x], members[b][y]);
                        improved = true;
                        break;
                    }
                }
            }
        }
        if (!improved) break;
    }
    tab.groups = groups;
    tab.variant.assign((size_t)groups * M3_WPB, 255);
    tab.tile.assign((size_t)groups * M3_WPB * 32, 0u);
    for (int b = 0; b < bins; ++b) {
        const int g = b / 4, sched = b % 4;
        for (size_t k = 0; k < members[b].size(); ++k) {
            const WarpDesc &w = warps[members[b][k]];
            const int slot = g * M3_WPB + sched + 4 * (int)k;   // warp index % 4 = scheduler
            tab.variant[slot] = (unsigned char)w.variant;
            for (size_t l = 0; l < w.tiles.size(); ++l) tab.tile[(size_t)slot * 32 + l] = w.tiles[l];
        }
    }
}

// The table depends on (d, dense) only; building it costs tens of microseconds of host time (milliseconds
// for the largest d) during which the GPU would sit idle, so it is built once and kept.
static const M3HostTable &cached_table(int d, bool dense)
{
    static M3HostTable cache[2][M3_MAX_D + 1];
    static bool cached[2][M3_MAX_D + 1] = {{false}};
    static std::mutex lock;
    std::lock_guard<std::mutex> guard(lock);
    M3HostTable &t = cache[dense ? 1 : 0][d];
    if (!cached[dense ? 1 : 0][d]) {
        build_table(d, dense, t);
        cached[dense ? 1 : 0][d] = true;
    }
    return t;
}

struct M3Plan {
    int groups, slices, dp, rows;
    int64_t rows_per_slice;
    int64_t out_elems;
    size_t table_bytes;                    // tile table in the workspace (0 when it travels as a parameter)
    size_t smem;
};

// Block groups per sample slice; slices fill the SMs once.
static M3Plan moment3_plan(int64_t N, int64_t d, int groups)
{
    M3Plan p;
    p.groups = groups;
    p.dp = (int)((d + 7) / 8 * 8);
    p.out_elems = tet_rows(d);
    int rows = (int)(M3_SMEM_BUDGET / ((size_t)M3_BUFFERS * p.dp * sizeof(float))) / 8 * 8;
    p.rows = rows > M3_STAGE_ROWS ? M3_STAGE_ROWS : rows;
    p.smem = (size_t)M3_BUFFERS * p.rows * p.dp * sizeof(float);
    const int sms = sm_count_or_default();
    int64_t slices = sms / groups;
    if (slices < 1) slices = 1;
    const int64_t max_slices = (N + p.rows - 1) / p.rows;
    if (slices > max_slices) slices = max_slices;
    p.rows_per_slice = (N + slices - 1) / slices;
    p.slices = (int)((N + p.rows_per_slice - 1) / p.rows_per_slice);
    p.table_bytes = d > M3_PARAM_D ? round_up((size_t)groups * M3_WPB * (1 + 32 * sizeof(unsigned)), 256) : 0;
    return p;
}

template <int WARPS>
static st_status moment3_launch(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws,
                                size_t ws_bytes, unsigned flags, cudaStream_t stream)
{
    const bool dense = (flags & ST_FLAG_DENSE_CONTROL) != 0;
    const M3HostTable &tab = cached_table((int)d, dense);
    const M3Plan p = moment3_plan(N, d, tab.groups);
    const size_t need = kWsHeaderBytes + p.table_bytes + (size_t)p.slices * p.out_elems * sizeof(float);
    if (!ws || ws_bytes < need) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    const DeviceInfo di = device_info();
    if (!di.ok) return ST_ERR_CUDA;
    if (p.smem > (size_t)di.max_smem_optin) return ST_ERR_UNSUPPORTED;
    unsigned char *w = (unsigned char *)ws;
    M3Args a;
    a.X = X; a.partials = (float *)(w + kWsHeaderBytes + p.table_bytes); a.status = (unsigned *)ws;
    a.gvariant = nullptr; a.gtile = nullptr;
    a.N = N; a.ldx = ldx; a.rows_per_slice = p.rows_per_slice;
    a.d = (int)d; a.dp = p.dp; a.rows = p.rows; a.out_elems = (int)p.out_elems;
    const bool aligned = d % 4 == 0 && ldx % 4 == 0;
    static M3Table<WARPS> empty_table;      // the parameter slot of launches that read the table from memory
    M3Table<WARPS> local;
    const M3Table<WARPS> *param = &empty_table;
    if (p.table_bytes == 0) {
        if ((size_t)tab.groups * M3_WPB > (size_t)WARPS) return ST_ERR_UNSUPPORTED;
        for (int i = 0; i < WARPS; ++i) local.variant[i] = i < (int)tab.variant.size() ? tab.variant[i] : 255;
        for (int i = 0; i < WARPS * 32; ++i) local.tile[i] = i < (int)tab.tile.size() ? m3_pack16(tab.tile[i]) : (unsigned short)0;
        param = &local;
    } else {
        // the table goes to the workspace: tile words first (4-byte aligned), variants behind them
        unsigned *gt = (unsigned *)(w + kWsHeaderBytes);
        unsigned char *gv = (unsigned char *)(gt + tab.tile.size());
        if (cudaMemcpyAsync(gt, tab.tile.data(), tab.tile.size() * sizeof(unsigned), cudaMemcpyHostToDevice, stream) != cudaSuccess ||
            cudaMemcpyAsync(gv, tab.variant.data(), tab.variant.size(), cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return ST_ERR_CUDA;
        a.gtile = gt;
        a.gvariant = gv;
    }
    dim3 grid(p.groups, p.slices);
    if (!aligned) {
        if (!ensure_dynamic_smem(moment3_kernel<WARPS, 0, false>, p.smem)) return ST_ERR_CUDA;
        moment3_kernel<WARPS, 0, false><<<grid, M3_THREADS, p.smem, stream>>>(a, *param);
    } else if (p.dp == M3_PARAM_D && p.rows == M3_STAGE_ROWS) {   // d = 60, 64 has its own instance with compile-time strides
        if (!ensure_dynamic_smem(moment3_kernel<WARPS, M3_PARAM_D, true>, p.smem)) return ST_ERR_CUDA;
        moment3_kernel<WARPS, M3_PARAM_D, true><<<grid, M3_THREADS, p.smem, stream>>>(a, *param);
    } else {
        if (!ensure_dynamic_smem(moment3_kernel<WARPS, 0, true>, p.smem)) return ST_ERR_CUDA;
        moment3_kernel<WARPS, 0, true><<<grid, M3_THREADS, p.smem, stream>>>(a, *param);
    }
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    return sum_slices_launch(a.partials, out, p.out_elems, p.slices, stream);
}

size_t moment3_tc_workspace(int64_t N, int64_t d, bool bf16);
st_status moment3_tc(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                     bool bf16, cudaStream_t stream);

size_t moment3_workspace(int64_t N, int64_t d, unsigned flags)
{
    if (flags & (ST_FLAG_TC_TF32 | ST_FLAG_TC_BF16))
        return (flags & ST_FLAG_DENSE_CONTROL) ? 0 : moment3_tc_workspace(N, d, (flags & ST_FLAG_TC_BF16) != 0);
    if (N <= 0 || d < 1 || d > M3_MAX_D) return 0;
    const M3HostTable &tab = cached_table((int)d, (flags & ST_FLAG_DENSE_CONTROL) != 0);
    const M3Plan p = moment3_plan(N, d, tab.groups);
    return kWsHeaderBytes + p.table_bytes + (size_t)p.slices * p.out_elems * sizeof(float);
}

}  // namespace st

extern "C" st_status st_sym_moment3(const float *X, int64_t N, int64_t d, int64_t ldx, float *out_packed,
                                    void *ws, size_t ws_bytes, unsigned flags, void *stream)
{
    if (!X || !out_packed) return ST_ERR_NULL;
    if (N <= 0 || d <= 0 || ldx < d) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_DENSE_CONTROL | ST_FLAG_TC_TF32 | ST_FLAG_TC_BF16)) return ST_ERR_UNSUPPORTED;
    if (flags & (ST_FLAG_TC_TF32 | ST_FLAG_TC_BF16)) {
        if ((flags & ST_FLAG_DENSE_CONTROL) || d > st::M3_PARAM_D) return ST_ERR_UNSUPPORTED;
        if ((flags & ST_FLAG_TC_TF32) && (flags & ST_FLAG_TC_BF16)) return ST_ERR_UNSUPPORTED;
        if (!st::aligned16(X) || !st::aligned16(out_packed)) return ST_ERR_ALIGN;
        return st::moment3_tc(X, N, d, ldx, out_packed, ws, ws_bytes, (flags & ST_FLAG_TC_BF16) != 0,
                              (cudaStream_t)stream);
    }
    if (d > st::M3_MAX_D) return ST_ERR_UNSUPPORTED;
    if (!st::aligned16(X) || !st::aligned16(out_packed)) return ST_ERR_ALIGN;
    if ((flags & ST_FLAG_DENSE_CONTROL) && d <= st::M3_PARAM_D)
        return st::moment3_launch<128>(X, N, d, ldx, out_packed, ws, ws_bytes, flags, (cudaStream_t)stream);
    return st::moment3_launch<32>(X, N, d, ldx, out_packed, ws, ws_bytes, flags, (cudaStream_t)stream);
}

// ---- st_sym_moment3_static: the same kernels with built-in scratch ---------------------
//
// The per-slice partial sums normally live in a workspace the caller allocates.  Some callers
// cannot allocate device memory at the point where they need the result: code running inside a
// framework that owns the allocator and forbids cudaMalloc in its hot loop, plug-ins that are
// handed only input and output buffers, or a process whose memory budget was fixed at start-up.
// For them the partial sums go to an array that is part of the library image.  It is reserved
// on every GPU that loads the library, for the lifetime of the process.
namespace st {

constexpr size_t kStaticScratchBytes = ST_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_moment3_scratch[kStaticScratchBytes];

// In host code `g_moment3_scratch` only names the symbol; the device address has to be asked
// for, once per device and with that device current.
static st_status moment3_static_scratch(void **ptr)
{
    static void *addr[64] = {nullptr};
    static std::mutex lock;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ST_ERR_CUDA;
    std::lock_guard<std::mutex> guard(lock);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_moment3_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return ST_ERR_CUDA;
        }
        addr[dev] = p;
    }
    *ptr = addr[dev];
    return ST_OK;
}

}  // namespace st

extern "C" st_status st_sym_moment3_static(const float *X, int64_t N, int64_t d, int64_t ldx, float *out_packed,
                                           unsigned flags, void *stream)
{
    if (!X || !out_packed) return ST_ERR_NULL;
    if (N <= 0 || d <= 0 || ldx < d) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_DENSE_CONTROL)) return ST_ERR_UNSUPPORTED;
    if (d < 8 || d > st::M3_PARAM_D || d % 8) return ST_ERR_UNSUPPORTED;
    if (!st::aligned16(X) || !st::aligned16(out_packed) || ldx % 4) return ST_ERR_ALIGN;
    // the request must fit the built-in array; nothing is launched otherwise
    const size_t need = st::moment3_workspace(N, d, flags);
    if (need == 0) return ST_ERR_UNSUPPORTED;
    if (need > st::kStaticScratchBytes) return ST_ERR_STATIC_SCRATCH;
    void *scratch = nullptr;
    const st_status rc = st::moment3_static_scratch(&scratch);
    if (rc != ST_OK) return rc;
    // every partial sum that the second kernel reads is written by the first one in the same
    // call, so nothing in the array has to start at zero
    if (flags & ST_FLAG_DENSE_CONTROL)
        return st::moment3_launch<128>(X, N, d, ldx, out_packed, scratch, st::kStaticScratchBytes, flags,
                                       (cudaStream_t)stream);
    return st::moment3_launch<32>(X, N, d, ldx, out_packed, scratch, st::kStaticScratchBytes, flags,
                                  (cudaStream_t)stream);
}
