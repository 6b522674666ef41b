// st_ttm_blockdiag, tensor-core path (ST_FLAG_TC_TF32): Ap[m, r] = sum_k Bp[m, k] U[k, r] over
// the fibres of the diagonal blocks only (Table 1, TTM; B is a direct sum of blocks).  In the
// packed layout the whole operation is one tall-skinny GEMM [rows, K] x [K, R]; what the
// structure buys is that the fibres of the zero blocks are never read.  HBM bound.
//
// Persistent blocks walk tiles of 128 packed fibres.  Per tile, K is streamed in slices of 32
// floats by TMA (128-byte swizzle, K-major A operand read as TF32 by the tensor core: the low
// 13 mantissa bits are ignored).  U is rounded to TF32, transposed once per block into the
// same swizzled K-major form and stays in shared memory.  The 128 x R fp32 accumulator lives
// in tensor memory, double buffered so that the epilogue of one tile overlaps the MMAs of the
// next.  Warp roles: warp 0 TMA producer, warp 1 MMA issuer / TMEM owner, warps 2..5 epilogue.
#include "tc_common.cuh"
#include "st_index.cuh"
#include "mttkrp_common.cuh"

namespace st {

namespace ttmtc {
constexpr int BM = 128;                    // fibres per tile
constexpr int KC = 32;                     // floats per k-slice (128 bytes)
constexpr int STAGE_BYTES = BM * KC * 4;   // 16 KiB
constexpr int THREADS = 192;
constexpr int MAX_STAGES = 10;
}  // namespace ttmtc

enum { TC_TTM = 0, TC_MTTKRP_PACKED = 1, TC_MTTKRP_DENSE = 2 };

struct TtmTcArgs {
    const float *U;
    const float *C;      // MTTKRP: [I, R]
    int I, mode;
    int64_t div;         // TC_MTTKRP_DENSE: fibre `row` belongs to (i, j) = (row / div, row % div)
    float *out;
    unsigned *status;
    int64_t rows;
    int K, R, kchunks, ntiles, stages;
    int reverse;         // walk the tiles from the last one down (see tc_rows_launch)
    uint32_t tmem_cols;
};

__global__ void __launch_bounds__(ttmtc::THREADS, 1)
ttm_tc_kernel(const __grid_constant__ CUtensorMap tmap, const TtmTcArgs a)
{
    using namespace ttmtc;
    using namespace tc;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int u_region = a.R * 128;                                  // bytes of one k-slice of U^T (multiple of 2048)
    unsigned char *u_smem = smem;                                    // kchunks regions
    unsigned char *stage0 = smem + (size_t)a.kchunks * u_region;
    uint64_t *bars = (uint64_t *)(stage0 + (size_t)a.stages * STAGE_BYTES);
    uint64_t *full = bars, *empty = bars + MAX_STAGES, *acc_full = bars + 2 * MAX_STAGES,
             *acc_empty = bars + 2 * MAX_STAGES + 2;
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * MAX_STAGES + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 4);     // one arrival per epilogue warp
        }
        *abort_flag = 0;
        if (blockIdx.x == 0) {
            // the status words are cleared here instead of by a separate memset; a time-out
            // report can only be written 2^24 failed polls later
            a.status[kWsStatusWord] = 0;
            a.status[kWsDetailWord] = 0;
        }
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, a.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp != 0) {
        // Warps 1..5 build U^T while warp 0 already streams fibres: U rounded to TF32, K-major with
        // the 128-byte swizzle; element (r, k) of slice k/32 goes to byte
        // r*128 + ((k%32/4) ^ (r%8))*16 + (k%4)*4 of that slice's region.
        const int nthr = THREADS - 32, t0 = threadIdx.x - 32;
        const int r4 = a.R >> 2;                                      // float4 groups per row of U
        const int total4 = a.kchunks * KC * r4;
        constexpr int UB = 16;
        for (int e0 = t0; e0 < total4; e0 += UB * nthr) {
            float4 v[UB];
#pragma unroll
            for (int u = 0; u < UB; ++u) {                            // sixteen independent loads in flight: W comes from cold memory
                const int e = e0 + u * nthr;
                const int k = e / r4;
                v[u] = (e < total4 && k < a.K) ? __ldg(reinterpret_cast<const float4 *>(a.U) + e)
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int e = e0 + u * nthr;
                if (e >= total4) continue;
                const int k = e / r4, rb = (e - k * r4) << 2;
                const int kc = k >> 5, kk = k & 31;
                const float vv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int r = rb + j;
                    uint32_t t;
                    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(t) : "f"(vv[j]));
                    const int off = r * 128 + (((kk >> 2) ^ (r & 7)) << 4) + ((kk & 3) << 2);
                    *reinterpret_cast<uint32_t *>(u_smem + (size_t)kc * u_region + off) = t;
                }
            }
        }
        fence_proxy_async();      // make the generic-proxy writes of U visible to the tensor core
        asm volatile("bar.sync 1, %0;" ::"n"(THREADS - 32) : "memory");
    }

    const int my_tiles = (a.ntiles > (int)blockIdx.x) ? (a.ntiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

    if (warp == 0) {
        if (elect_one()) {
            prefetch_tmap(&tmap);
            // ring position and barrier phase are carried in counters: a 64-bit division per stage would cost
            // this single thread a good part of the time one stage takes to arrive
            int s = 0;
            uint32_t empty_parity = 0;
            bool first_pass = true, ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                int64_t tile = blockIdx.x + (int64_t)t * gridDim.x;
                if (a.reverse) tile = a.ntiles - 1 - tile;
                const int y = (int)(tile * BM);
                for (int kc = 0; kc < a.kchunks; ++kc) {
                    if (!first_pass && !mbar_wait(&empty[s], empty_parity, abort_flag, a.status, 1)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(&full[s], STAGE_BYTES);
                    tma_load_2d(stage0 + (size_t)s * STAGE_BYTES, &tmap, &full[s], kc * KC, y);
                    if (++s == a.stages) {
                        s = 0;
                        if (first_pass) first_pass = false;
                        else empty_parity ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            const uint32_t idesc = make_idesc(2, 0, 0, BM, (uint32_t)a.R);
            int s = 0;
            uint32_t full_parity = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int buf = t & 1;
                const int use = t >> 1;
                if (use > 0 && !mbar_wait(&acc_empty[buf], (uint32_t)((use - 1) & 1), abort_flag, a.status, 2)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * a.R);
                for (int kc = 0; kc < a.kchunks; ++kc) {
                    if (!mbar_wait(&full[s], full_parity, abort_flag, a.status, 3)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(stage0 + (size_t)s * STAGE_BYTES);
                    const uint32_t sb = smem_u32(u_smem + (size_t)kc * u_region);
#pragma unroll
                    for (int kk = 0; kk < KC / 8; ++kk) {
                        const uint64_t adesc = make_smem_desc(sa + kk * 32, 16, 1024);
                        const uint64_t bdesc = make_smem_desc(sb + kk * 32, 16, 1024);
                        mma_tf32(d_tmem, adesc, bdesc, idesc, (kc > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit(&empty[s]);
                    if (++s == a.stages) {
                        s = 0;
                        full_parity ^= 1u;
                    }
                }
                tc_commit(&acc_full[buf]);
            }
        }
    } else {
        const int q = warp & 3;
        for (int t = 0; t < my_tiles; ++t) {
            const int buf = t & 1;
            int64_t tile = blockIdx.x + (int64_t)t * gridDim.x;
            if (a.reverse) tile = a.ntiles - 1 - tile;
            const int64_t row = tile * BM + q * 32 + lane;
            // MTTKRP: the fibre's (i, j) and, for R = 32, its row of C are fetched before the accumulator is
            // waited for -- with the memory system saturated by the fibre stream a dependent load costs
            // microseconds
            const bool valid = row < a.rows;
            int64_t gi = -1, gj = 0;
            WarpRuns runs{0u, 0u};
            float4 cpre[8];
            const bool pre = a.mode != TC_TTM && a.R == 32;
            if (a.mode != TC_TTM) {
                if (valid) {
                    if (a.mode == TC_MTTKRP_PACKED) tri_decode(a.I, row, gi, gj);
                    else { gi = row / a.div; gj = row - gi * a.div; }
                }
                runs = warp_runs(valid, (int)gi, lane);
                if (pre) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        cpre[e] = valid ? __ldg(reinterpret_cast<const float4 *>(a.C + gj * a.R) + e) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            if (!mbar_wait(&acc_full[buf], (uint32_t)((t >> 1) & 1), abort_flag, a.status, 4)) break;
            tc_fence_after();
            if (a.mode == TC_TTM) {
                float *dst = a.out + row * a.R;
                for (int c0 = 0; c0 < a.R; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * a.R + c0), r);
                    tmem_ld_wait();
                    if (row < a.rows) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            if (c0 + e < a.R)
                                *reinterpret_cast<uint4 *>(dst + c0 + e) = make_uint4(r[e], r[e + 1], r[e + 2], r[e + 3]);
                    }
                }
            } else {
                // MTTKRP: this lane's fibre is row (i,j); scale by C[j,:], then sum every run of fibres of
                // the warp that share i and write it to partial slot (unit + i), unit = row / 32 (see
                // mttkrp_common.cuh).  The 32 fibres of a warp are consecutive, so they usually share i:
                // one transposing shuffle reduction and one coalesced store per 32 columns.
                const int gi32 = (int)gi;
                const int64_t unit = tile * (BM / 32) + q;
                for (int c0 = 0; c0 < a.R && runs.heads != 0u; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * a.R + c0), r);
                    tmem_ld_wait();
                    float v[32];
                    if (valid) {
                        const float4 *crow = reinterpret_cast<const float4 *>(a.C + gj * a.R + c0);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float4 c = pre ? cpre[e] : __ldg(crow + e);
                            v[4 * e + 0] = c.x * __uint_as_float(r[4 * e + 0]);
                            v[4 * e + 1] = c.y * __uint_as_float(r[4 * e + 1]);
                            v[4 * e + 2] = c.z * __uint_as_float(r[4 * e + 2]);
                            v[4 * e + 3] = c.w * __uint_as_float(r[4 * e + 3]);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = 0.f;
                    }
                    warp_store_runs(v, runs, valid, gi32, unit, lane, a.out, a.R, c0, mttkrp_slots(a.rows, 32, a.I, 1));
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    }
    // MTTKRP: the kernel that adds the partial sums may be launched now (it waits for this grid to end)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, a.tmem_cols);
    }
}

struct TtmTcPlan {
    int kchunks, stages;
    uint32_t tmem_cols;
    size_t smem;
    bool ok;
};

static TtmTcPlan ttm_tc_plan(int64_t K, int64_t R)
{
    using namespace ttmtc;
    TtmTcPlan p{};
    p.ok = false;
    if (K <= 0 || R <= 0 || K % 4 != 0 || R % 16 != 0 || R > 256 || K > (1 << 20)) return p;
    p.kchunks = (int)((K + KC - 1) / KC);
    // two accumulators of R columns; the epilogue reads them with 32-column loads, so the second one
    // (which starts at column R) needs R rounded up to 32 columns behind it: 64 columns for R = 16
    uint32_t cols = 32;
    while (cols < (uint32_t)R + ((uint32_t)R + 31u) / 32u * 32u) cols *= 2;
    p.tmem_cols = cols;
    const size_t u_bytes = (size_t)p.kchunks * R * 128;
    const size_t fixed = 1024 + u_bytes + 512;
    const size_t budget = 227 * 1024;
    if (fixed + 2 * STAGE_BYTES > budget) return p;
    size_t st = (budget - fixed) / STAGE_BYTES;
    if (st > MAX_STAGES) st = MAX_STAGES;
    p.stages = (int)st;
    p.smem = fixed + st * STAGE_BYTES;
    p.ok = true;
    return p;
}

size_t ttm_tf32_tc_workspace(int64_t rows, int64_t K, int64_t R)
{
    if (rows <= 0) return 0;
    return ttm_tc_plan(K, R).ok ? kWsHeaderBytes : 0;
}

static st_status tc_rows_launch(const float *Bp, int64_t rows, int64_t K, const float *U, int64_t R, float *Ap,
                                const float *C, int64_t I, int mode, void *ws, size_t ws_bytes, cudaStream_t stream,
                                int64_t div = 0);

st_status ttm_tf32_tc(const float *Bp, int64_t rows, int64_t K, const float *U, int64_t R, float *Ap, void *ws,
                      size_t ws_bytes, cudaStream_t stream)
{
    return tc_rows_launch(Bp, rows, K, U, R, Ap, nullptr, 0, TC_TTM, ws, ws_bytes, stream);
}

size_t mttkrp_tf32_tc_workspace(int64_t rows, int64_t I, int64_t K, int64_t R)
{
    if (rows <= 0 || R % 32 != 0 || !ttm_tc_plan(K, R).ok) return 0;
    return kWsHeaderBytes + (size_t)mttkrp_slots(rows, 32, I, 1) * R * sizeof(float);
}

// MTTKRP on tensor cores: the same streaming kernel with W = D; the epilogue scales every fibre's result
// by C[j,:] and writes the sums of the runs of equal i to the workspace, a second kernel adds them in a
// fixed order (mttkrp_common.cuh).  `m` says how a row maps to (i, j); the fibres reach rows
// i_off .. i_off + m.I - 1 of A_full, which has I_full rows.  TF32 operands, 5e-3 tolerance.
st_status mttkrp_tf32_tc(const float *Bp, const MttkrpRows &m, int64_t K, const float *C, const float *D, int64_t R,
                         float *A_full, int64_t I_full, int64_t i_off, void *ws, size_t ws_bytes, cudaStream_t stream)
{
    if (R % 32 != 0) return ST_ERR_UNSUPPORTED;
    const size_t need = mttkrp_tf32_tc_workspace(m.rows, m.I, K, R);
    if (need == 0) return ST_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < need) return ST_ERR_WORKSPACE;
    float *part = (float *)((unsigned char *)ws + kWsHeaderBytes);
    const st_status rc = tc_rows_launch(Bp, m.rows, K, D, R, part, C, m.I, m.mode == MK_PACKED ? TC_MTTKRP_PACKED : TC_MTTKRP_DENSE,
                                        ws, ws_bytes, stream, m.div);
    if (rc != ST_OK) return rc;
    return mttkrp_rowsum_launch(part, A_full, I_full, i_off, m, (int)R, 32, 1, stream);
}

static st_status tc_rows_launch(const float *Bp, int64_t rows, int64_t K, const float *U, int64_t R, float *Ap,
                                const float *C, int64_t I, int mode, void *ws, size_t ws_bytes, cudaStream_t stream,
                                int64_t div)
{
    using namespace ttmtc;
    const TtmTcPlan p = ttm_tc_plan(K, R);
    if (!p.ok) return ST_ERR_UNSUPPORTED;
    if (rows > (int64_t(1) << 31) - BM) return ST_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < kWsHeaderBytes) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    const DeviceInfo di = device_info();
    if (!di.ok) return ST_ERR_CUDA;
    if (p.smem > (size_t)di.max_smem_optin) return ST_ERR_UNSUPPORTED;
    CUtensorMap tmap;
    if (!tc::make_tmap_2d(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Bp, (uint64_t)rows, (uint64_t)K, (uint64_t)K * 4, KC,
                          BM))
        return ST_ERR_CUDA;
    TtmTcArgs a;
    a.U = U; a.C = C; a.I = (int)I; a.mode = mode; a.div = div > 0 ? div : (I > 0 ? I : 1); a.out = Ap; a.status = (unsigned *)ws; a.rows = rows; a.K = (int)K; a.R = (int)R;
    a.kchunks = p.kchunks; a.stages = p.stages; a.tmem_cols = p.tmem_cols;
    a.ntiles = (int)((rows + BM - 1) / BM);
    // MTTKRP usually runs right after the call that produced its packed operand (st_pack, or a kernel
    // that writes packed output).  The end of that operand is then still in L2, so the tiles are walked
    // from the last one down: what was written last is read first, before later fills evict it.
    a.reverse = mode != TC_TTM ? 1 : 0;
    if (!ensure_dynamic_smem(ttm_tc_kernel, p.smem)) return ST_ERR_CUDA;
    const int grid = a.ntiles < di.sm_count ? a.ntiles : di.sm_count;
    ttm_tc_kernel<<<grid, THREADS, p.smem, stream>>>(tmap, a);
    return launch_status();
}

}  // namespace st
