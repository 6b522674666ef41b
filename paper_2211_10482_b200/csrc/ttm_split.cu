// st_ttm_blockdiag / st_ttm_packed / st_mttkrp_tri / st_mttkrp_slice, tensor-core path with fp32-class
// accuracy (ST_FLAG_TC_SPLIT):  Y[m, r] = sum_k Bp[m, k] W[k, r] over the packed fibres m only
// (Table 1, TTM and the inner contraction of MTTKRP), read once from HBM.
//
// Both operands are split into two bf16 parts, x = hi + lo + O(2^-18 x) with hi = bf16(x) and
// lo = bf16(x - hi), and three of the four partial products are kept:
//     Y = Bh Wh + Bh Wl + Bl Wh          (Bl Wl is of relative size 2^-18 and dropped).
// Per term the result differs from the exact product by at most about 3 * 2^-18 = 1.2e-5, and the fp32
// accumulation of at most 3 K / 16 tensor-core instructions adds less than that for the K this path
// accepts: it is held to the 1e-4 tolerance of the fp32 kernels.  HBM bound (the fp32 FMA kernel of
// the same contraction is bound by arithmetic at more than twice the time).
//
// Persistent blocks walk tiles of 128 fibres.  Sixteen converter warps copy slices of 64 k-values
// asynchronously into a landing ring (16-byte copies, every thread later reads back the chunks it
// copied itself: no barrier), split them and store hi and lo as two K-major, 128-byte-swizzled bf16
// operands.  (Asking for whole tiles to be brought into L2 ahead of the copies, so that DRAM would see
// long sequential reads, was measured and made the kernel 12-20 % slower.)  W is split once per block into [Wh; Wl] stacked along N.  Per 16
// k-values the issuing thread runs
//     D[128 x 2R] += Bh x [Wh; Wl]^T     (N = 2R)
//     D[128 x  R] += Bl x  Wh^T          (N = R, the first R columns of the same accumulator)
// so the two products with Bh cost one instruction (an MMA of M = 128 takes the same time for any
// N <= 128).  The epilogue adds the two halves of the accumulator, D[:, r] + D[:, R + r]; it is
// double buffered in tensor memory.  Warps 0-3 epilogue (and the split of W), warp 4 MMA issue and
// tensor-memory owner, warps 5-20 converters (what bounds them is the latency of the chain copy ->
// convert -> store -> proxy fence -> barrier, so there are four of them per scheduler).
#include "tc_common.cuh"
#include "st_index.cuh"
#include "mttkrp_common.cuh"
#include <cuda_bf16.h>

namespace st {

namespace split {
constexpr int BM = 128;                    // fibres per tile
constexpr int KC = 64;                     // k-values per operand stage (128 bytes of bf16 per fibre)
constexpr int OP_BYTES = BM * 128;         // one operand (hi or lo) of a stage: 16 KiB
constexpr int STAGE_BYTES = 2 * OP_BYTES;  // hi + lo
constexpr int MAX_STAGES = 4;
constexpr int EPI_WARPS = 4, MMA_WARP = 4, CONV_WARP0 = 5, CONV_WARPS = 16;
constexpr int CONV_THREADS = 32 * CONV_WARPS;
constexpr int THREADS = 32 * (CONV_WARP0 + CONV_WARPS);
constexpr int LOADS = BM * (KC / 4) / CONV_THREADS;   // 16-byte copies per converter thread and stage: 4
constexpr int ROW_STEP = CONV_THREADS / 16;           // fibres between two copies of a thread: 32
constexpr int LAND_BYTES = BM * KC * 4;     // one stage of the landing ring of the fp32 data: 32 KiB
constexpr int MAX_K = 2048;                // longest accumulation chain: 3 * 2048 / 16 = 384 instructions
}  // namespace split

enum { SP_TTM = 0, SP_MTTKRP_PACKED = 1, SP_MTTKRP_DENSE = 2 };

struct SplitArgs {
    const float *B;      // [rows, K]
    const float *W;      // [K, R]
    const float *C;      // MTTKRP: [., R]
    int I, mode;
    int64_t div;
    float *out;          // TTM: [rows, R];  MTTKRP: partial slots
    unsigned *status;
    int64_t rows;
    int K, R, kchunks, ntiles, stages;
    uint32_t tmem_cols;
};
struct SplitPlan {
    int kchunks, stages, land;
    uint32_t tmem_cols;
    size_t smem;
    bool ok;
};

// two floats -> two bf16 in one word (first argument in the low half)
__device__ __forceinline__ uint32_t bf16x2(float lo, float hi)
{
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&p);
}

// (hi, lo) words of the split of two floats: hi = bf16(x), lo = bf16(x - hi)
__device__ __forceinline__ void split2(float x0, float x1, uint32_t &hi, uint32_t &lo)
{
    hi = bf16x2(x0, x1);
    const float h0 = __uint_as_float(hi << 16), h1 = __uint_as_float(hi & 0xffff0000u);
    lo = bf16x2(x0 - h0, x1 - h1);
}

// LAND: stages of the landing ring (3 when shared memory has room beside W, else 2)
template <int LAND>
__global__ void __launch_bounds__(split::THREADS, 1) ttm_split_kernel(const SplitArgs a)
{
    using namespace split;
    using namespace tc;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int w_region = 2 * a.R * 128;                               // [Wh; Wl] of one chunk of 64 k-values
    unsigned char *w_smem = smem;
    unsigned char *stage0 = smem + (size_t)a.kchunks * w_region;
    uint64_t *bars = (uint64_t *)(stage0 + (size_t)a.stages * STAGE_BYTES);
    uint64_t *op_full = bars, *op_empty = bars + MAX_STAGES, *acc_full = bars + 2 * MAX_STAGES,
             *acc_empty = bars + 2 * MAX_STAGES + 2;
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * MAX_STAGES + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) {
            mbar_init(&op_full[s], CONV_WARPS);   // one arrival per converter warp
            mbar_init(&op_empty[s], 1);           // tcgen05.commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], EPI_WARPS);
        }
        *abort_flag = 0;
        if (blockIdx.x == 0) {      // a time-out report can only be written 2^24 failed polls later
            a.status[kWsStatusWord] = 0;
            a.status[kWsDetailWord] = 0;
        }
        fence_barrier_init();
    }
    if (warp == MMA_WARP) {
        tmem_alloc(tmem_slot, a.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int my_tiles = (a.ntiles > (int)blockIdx.x) ? (a.ntiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int R = a.R;

    // ---- converter set-up (used again in the converter branch below).  Copy u of a thread covers fibre
    // (ct / 16 + 32 u) of the tile and the four k-values 4 * (ct % 16) of the chunk: the 16 lanes of a
    // half-warp copy one fibre's 256 contiguous bytes and later write its 128-byte row of each operand.
    // The fp32 data travel global -> shared by asynchronous 16-byte copies into a landing ring of LAND
    // stages; every thread reads back exactly the chunks it copied itself, so the ring needs no barrier,
    // only the thread's own wait on its copy groups.  LAND - 1 stages are in flight per block while one
    // is converted.
    const int ct = threadIdx.x - 32 * CONV_WARP0;
    const int g = ct & 15, r_base = ct >> 4;                          // rows r_base + 32 u
    const int total = my_tiles * a.kchunks;                           // stages of this block (< 2^31: see the launch)
    const uint32_t land0 = smem_u32(stage0 + (size_t)a.stages * STAGE_BYTES + 256) + (uint32_t)ct * 16u;
    // State of the copy stream, advanced by one stage per call: all of it in 32-bit counters and one pointer
    // (the sixteen converter warps all run this code: divisions and 64-bit products here would cost more
    // issue slots than the conversion itself).
    int ld_it = 0, ld_kc = 0, ld_slot = 0;
    const int64_t first_row = (int64_t)blockIdx.x * BM + r_base;
    int64_t ld_rows_left = a.rows - first_row;                        // fibres from this thread's first row of the tile to the end
    const float *ld_src = a.B + first_row * (int64_t)a.K + g * 4;       // that row, this thread's k-offset, chunk 0
    const int64_t tile_step = (int64_t)gridDim.x * BM;                // fibres between two tiles of this block
    auto load = [&]() {
        if (ld_it < total) {
            const bool k_in = ld_kc * KC + g * 4 < a.K;
            const uint32_t dst = land0 + (uint32_t)ld_slot * (uint32_t)LAND_BYTES;
            const float *src = ld_src + ld_kc * KC;
#pragma unroll
            for (int u = 0; u < LOADS; ++u) {
                const bool in = k_in && ROW_STEP * u < ld_rows_left;
                const int sz = in ? 16 : 0;                          // src-size 0: the 16 bytes are zero-filled
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + (uint32_t)u * (CONV_THREADS * 16u)),
                             "l"(in ? src + (int64_t)(ROW_STEP * u) * a.K : a.B), "r"(sz)
                             : "memory");
            }
            ++ld_it;
            if (++ld_slot == LAND) ld_slot = 0;
            if (++ld_kc == a.kchunks) {
                ld_kc = 0;
                ld_rows_left -= tile_step;
                ld_src += tile_step * a.K;
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");           // one group per stage, empty past the end
    };
    // the first slices are requested before anything else, so that they travel while W is split
    if (warp >= CONV_WARP0)
        for (int p = 0; p < LAND; ++p) load();

    if (warp != MMA_WARP) {
        // ---- split W (all warps but the issuer: one cold round trip to memory each): chunk kc of 64 k-values
        // becomes 2R rows of 128 bytes, row r = Wh[., r], row R + r = Wl[., r], K-major with the 128-byte
        // swizzle (16-byte unit u of row n sits at unit u ^ (n & 7)).  A warp takes (chunk, 16 columns r):
        // lane = (4 columns rg, unit q of 8 k-values); it loads the float4 W[8q + e, 4rg ..] for e = 0..7
        // (64 contiguous bytes per k across the 4 rg lanes) and stores one 16-byte unit per column and part
        // (the 8 lanes q of a column fill one 128-byte row).
        const int items = a.kchunks * (R / 16);
        const int wi = warp < MMA_WARP ? warp : warp - 1;
        for (int it = wi; it < items; it += EPI_WARPS + CONV_WARPS) {
            const int kc = it / (R / 16), r0 = (it - kc * (R / 16)) * 16 + (lane >> 3) * 4;
            const int q = lane & 7, k0 = kc * KC + q * 8;
            float4 v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
                v[e] = (k0 + e < a.K) ? __ldg(reinterpret_cast<const float4 *>(a.W + (size_t)(k0 + e) * R + r0))
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
            unsigned char *reg = w_smem + (size_t)kc * w_region;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float x[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] = j == 0 ? v[e].x : j == 1 ? v[e].y : j == 2 ? v[e].z : v[e].w;
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) split2(x[2 * e], x[2 * e + 1], hi[e], lo[e]);
                const int r = r0 + j;
                const uint32_t off = (uint32_t)r * 128u + (uint32_t)((q ^ (r & 7)) << 4);
                *reinterpret_cast<uint4 *>(reg + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4 *>(reg + (size_t)R * 128 + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
        }
        fence_proxy_async();      // make the generic-proxy writes of W visible to the tensor core
    }
    __syncthreads();              // W is in place

    if (warp < EPI_WARPS) {
        // ---- epilogue
        const int q = warp;       // TMEM lanes 32q .. 32q + 31
        for (int t = 0; t < my_tiles; ++t) {
            const int buf = t & 1;
            const int64_t tile = blockIdx.x + (int64_t)t * gridDim.x;
            const int64_t row = tile * BM + q * 32 + lane;
            const bool valid = row < a.rows;
            // MTTKRP: the fibre's (i, j) and, for R = 32, its row of C are fetched before the accumulator is
            // waited for -- with the memory system saturated by the fibre stream a dependent load costs
            // microseconds, which would otherwise stall the tile after next
            int64_t gi = -1, gj = 0;
            WarpRuns runs{0u, 0u};
            float4 cpre[8];
            const bool pre = a.mode != SP_TTM && R == 32;
            if (a.mode != SP_TTM) {
                if (valid) {
                    if (a.mode == SP_MTTKRP_PACKED) tri_decode(a.I, row, gi, gj);
                    else { gi = row / a.div; gj = row - gi * a.div; }
                }
                runs = warp_runs(valid, (int)gi, lane);
                if (pre) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        cpre[e] = valid ? __ldg(reinterpret_cast<const float4 *>(a.C + gj * R) + e) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            if (!mbar_wait(&acc_full[buf], (uint32_t)((t >> 1) & 1), abort_flag, a.status, 4)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 2 * R);
            // 16 columns at a time keeps the register count low; cv = the fibre's four float4 of C for them
            auto chunk = [&](int c0, const float4 &cv0, const float4 &cv1, const float4 &cv2, const float4 &cv3) {
                float v[16];
                {
                    uint32_t r1[16], r2[16];
                    tmem_ld_32x16(taddr + (uint32_t)c0, r1);
                    tmem_ld_32x16(taddr + (uint32_t)(R + c0), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = __uint_as_float(r1[e]) + __uint_as_float(r2[e]);
                }
                if (a.mode == SP_TTM) {
                    if (valid) {
                        float4 *dst = reinterpret_cast<float4 *>(a.out + row * R + c0);
#pragma unroll
                        for (int e = 0; e < 4; ++e) dst[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                    }
                } else {
                    const float4 cv[4] = {cv0, cv1, cv2, cv3};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {            // lanes without a fibre hold zeros in cv
                        v[4 * e + 0] *= cv[e].x;
                        v[4 * e + 1] *= cv[e].y;
                        v[4 * e + 2] *= cv[e].z;
                        v[4 * e + 3] *= cv[e].w;
                    }
                    warp_store_runs16(v, runs, valid, (int)gi, tile * (BM / 32) + q, lane, a.out, R, c0,
                                      mttkrp_slots(a.rows, 32, a.I, 1));
                }
            };
            if (pre) {
                chunk(0, cpre[0], cpre[1], cpre[2], cpre[3]);
                chunk(16, cpre[4], cpre[5], cpre[6], cpre[7]);
            } else {
                const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int c0 = 0; c0 < R; c0 += 16) {
                    float4 cv[4] = {z, z, z, z};
                    if (a.mode != SP_TTM && valid) {
                        const float4 *crow = reinterpret_cast<const float4 *>(a.C + gj * R + c0);
#pragma unroll
                        for (int e = 0; e < 4; ++e) cv[e] = __ldg(crow + e);
                    }
                    chunk(c0, cv[0], cv[1], cv[2], cv[3]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    } else if (warp == MMA_WARP) {
        if (elect_one()) {
            const uint32_t idesc2 = make_idesc(1, 0, 0, BM, (uint32_t)(2 * R));    // bf16 x bf16, both K-major
            const uint32_t idesc1 = make_idesc(1, 0, 0, BM, (uint32_t)R);
            int s = 0;
            uint32_t full_parity = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int buf = t & 1, use = t >> 1;
                if (use > 0 && !mbar_wait(&acc_empty[buf], (uint32_t)((use - 1) & 1), abort_flag, a.status, 2)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 2 * R);
                for (int kc = 0; kc < a.kchunks; ++kc) {
                    if (!mbar_wait(&op_full[s], full_parity, abort_flag, a.status, 3)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sh = smem_u32(stage0 + (size_t)s * STAGE_BYTES), sl = sh + OP_BYTES;
                    const uint32_t sw = smem_u32(w_smem + (size_t)kc * w_region);
                    const int kleft = a.K - kc * KC;                  // slices of 16 beyond K hold zeros: not issued
#pragma unroll
                    for (int kk = 0; kk < KC / 16; ++kk) {
                        if (kk * 16 < kleft) {
                            const uint64_t wdesc = make_smem_desc(sw + kk * 32, 16, 1024);
                            mma_bf16(d_tmem, make_smem_desc(sh + kk * 32, 16, 1024), wdesc, idesc2, (kc > 0 || kk > 0) ? 1u : 0u);
                            mma_bf16(d_tmem, make_smem_desc(sl + kk * 32, 16, 1024), wdesc, idesc1, 1u);
                        }
                    }
                    tc_commit(&op_empty[s]);
                    if (++s == a.stages) {
                        s = 0;
                        full_parity ^= 1u;
                    }
                }
                tc_commit(&acc_full[buf]);
            }
        }
    } else {
        // ---- converters
        const uint32_t op0 = smem_u32(stage0);
        // byte offset of this thread's 8 bytes inside an operand, for its first row; row r_base + 32 u has the
        // same swizzle phase (32 u is a multiple of 8), so the others follow at 32 * 128 bytes each
        const uint32_t op_off = (uint32_t)r_base * 128u + (uint32_t)(((g >> 1) ^ (r_base & 7)) << 4) + (uint32_t)((g & 1) << 3);
        int slot = 0, s = 0;
        uint32_t empty_parity = 0;                                    // (first pass over the operand ring: nothing to wait for)
        bool first_pass = true;
        for (int it = 0; it < total; ++it) {
            asm volatile("cp.async.wait_group %0;" ::"n"(LAND - 1) : "memory");   // stage `it` has landed
            const uint32_t land = land0 + (uint32_t)slot * (uint32_t)LAND_BYTES;
            if (++slot == LAND) slot = 0;
            float4 x[LOADS];
#pragma unroll
            for (int u = 0; u < LOADS; ++u)
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(x[u].x), "=f"(x[u].y), "=f"(x[u].z), "=f"(x[u].w)
                             : "r"(land + (uint32_t)u * (CONV_THREADS * 16u)));
            uint32_t h[LOADS][2], l[LOADS][2];
#pragma unroll
            for (int u = 0; u < LOADS; ++u) {
                split2(x[u].x, x[u].y, h[u][0], l[u][0]);
                split2(x[u].z, x[u].w, h[u][1], l[u][1]);
            }
            // the thread's chunks of this landing slot are in registers: the slot takes stage it + LAND at once,
            // so that LAND stages are in flight whatever the tensor core is doing
            load();
            if (!first_pass && !mbar_wait(&op_empty[s], empty_parity, abort_flag, a.status, 1)) break;
            const uint32_t op = op0 + (uint32_t)s * (uint32_t)STAGE_BYTES + op_off;
#pragma unroll
            for (int u = 0; u < LOADS; ++u) {
                const uint32_t o = op + (uint32_t)u * (ROW_STEP * 128u);
                asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(o), "r"(h[u][0]), "r"(h[u][1]) : "memory");
                asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(o + (uint32_t)OP_BYTES), "r"(l[u][0]), "r"(l[u][1]) : "memory");
            }
            fence_proxy_async();      // generic-proxy stores -> visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(&op_full[s]);
            if (++s == a.stages) {
                s = 0;
                if (first_pass) first_pass = false;
                else empty_parity ^= 1u;
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    // MTTKRP: the kernel that adds the partial sums may be launched now (it waits for this grid to end)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, a.tmem_cols);
    }
}

static SplitPlan split_plan(int64_t K, int64_t R)
{
    using namespace split;
    SplitPlan p{};
    p.ok = false;
    if (K <= 0 || R <= 0 || K % 4 != 0 || K > MAX_K || R % 32 != 0 || R > 128) return p;
    p.kchunks = (int)((K + KC - 1) / KC);
    uint32_t cols = 32;
    while (cols < 4 * (uint32_t)R) cols *= 2;                         // two accumulators of 2R columns
    p.tmem_cols = cols;
    const size_t w_bytes = (size_t)p.kchunks * 2 * R * 128;
    const size_t fixed = 1024 + w_bytes + 512;
    const size_t budget = 227 * 1024;
    p.land = (fixed + 3 * (size_t)LAND_BYTES + 2 * STAGE_BYTES <= budget) ? 3 : 2;
    const size_t land = (size_t)p.land * LAND_BYTES;
    if (fixed + land + 2 * STAGE_BYTES > budget) return p;
    size_t st = (budget - fixed - land) / STAGE_BYTES;
    if (st > MAX_STAGES) st = MAX_STAGES;
    p.stages = (int)st;
    p.smem = fixed + land + st * STAGE_BYTES;
    p.ok = true;
    return p;
}

static st_status split_rows_launch(const float *Bp, int64_t rows, int64_t K, const float *W, int64_t R, float *out,
                                   const float *C, int64_t I, int mode, int64_t div, void *ws, size_t ws_bytes,
                                   cudaStream_t stream)
{
    using namespace split;
    const SplitPlan p = split_plan(K, R);
    if (!p.ok) return ST_ERR_UNSUPPORTED;
    if (rows > (int64_t(1) << 31) - BM) return ST_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < kWsHeaderBytes) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    const DeviceInfo di = device_info();
    if (!di.ok) return ST_ERR_CUDA;
    if (p.smem > (size_t)di.max_smem_optin) return ST_ERR_UNSUPPORTED;
    SplitArgs a;
    a.B = Bp; a.W = W; a.C = C; a.I = (int)I; a.mode = mode; a.div = div > 0 ? div : 1;
    a.out = out; a.status = (unsigned *)ws; a.rows = rows; a.K = (int)K; a.R = (int)R;
    a.kchunks = p.kchunks; a.stages = p.stages; a.tmem_cols = p.tmem_cols;
    a.ntiles = (int)((rows + BM - 1) / BM);
    if ((int64_t)a.ntiles * p.kchunks >= (int64_t(1) << 31)) return ST_ERR_UNSUPPORTED;
    const int grid = a.ntiles < di.sm_count ? a.ntiles : di.sm_count;
    if (p.land == 3) {
        if (!ensure_dynamic_smem(ttm_split_kernel<3>, p.smem)) return ST_ERR_CUDA;
        ttm_split_kernel<3><<<grid, THREADS, p.smem, stream>>>(a);
    } else {
        if (!ensure_dynamic_smem(ttm_split_kernel<2>, p.smem)) return ST_ERR_CUDA;
        ttm_split_kernel<2><<<grid, THREADS, p.smem, stream>>>(a);
    }
    return launch_status();
}

size_t ttm_split_workspace(int64_t rows, int64_t K, int64_t R)
{
    if (rows <= 0) return 0;
    return split_plan(K, R).ok ? kWsHeaderBytes : 0;
}

st_status ttm_split(const float *Bp, int64_t rows, int64_t K, const float *U, int64_t R, float *Ap, void *ws,
                    size_t ws_bytes, cudaStream_t stream)
{
    return split_rows_launch(Bp, rows, K, U, R, Ap, nullptr, 0, SP_TTM, 0, ws, ws_bytes, stream);
}

size_t mttkrp_split_workspace(int64_t rows, int64_t I, int64_t K, int64_t R)
{
    if (rows <= 0 || !split_plan(K, R).ok) return 0;
    return kWsHeaderBytes + (size_t)mttkrp_slots(rows, 32, I, 1) * R * sizeof(float);
}

// MTTKRP: W = D, the epilogue scales every fibre's result by C[j,:] and writes the sums of the runs of
// equal i to the workspace; a second kernel adds them in a fixed order (mttkrp_common.cuh).
st_status mttkrp_split(const float *Bp, const MttkrpRows &m, int64_t K, const float *C, const float *D, int64_t R,
                       float *A_full, int64_t I_full, int64_t i_off, void *ws, size_t ws_bytes, cudaStream_t stream)
{
    const size_t need = mttkrp_split_workspace(m.rows, m.I, K, R);
    if (need == 0) return ST_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < need) return ST_ERR_WORKSPACE;
    float *part = (float *)((unsigned char *)ws + kWsHeaderBytes);
    const st_status rc = split_rows_launch(Bp, m.rows, K, D, R, part, C, m.I,
                                           m.mode == MK_PACKED ? SP_MTTKRP_PACKED : SP_MTTKRP_DENSE, m.div, ws, ws_bytes,
                                           stream);
    if (rc != ST_OK) return rc;
    return mttkrp_rowsum_launch(part, A_full, I_full, i_off, m, (int)R, 32, 1, stream);
}

}  // namespace st
