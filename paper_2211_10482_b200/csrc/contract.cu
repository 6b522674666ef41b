// st_ttm_blockdiag and st_mttkrp_tri, fp32 FMA path (Table 1: TTM, MTTKRP).
//
// In the packed layouts both kernels contract the trailing dense mode k of a tall matrix of
// fibres with a small dense factor W[K,R]:
//     Y[m, r] = sum_k Bp[m, k] * W[k, r]
//   TTM     m runs over the fibres of the diagonal blocks only; Y is the packed output
//           (the zero blocks of the direct sum are never touched: A_U(i,j,r) = B_U(i,j,.)).
//   MTTKRP  m = p(i,j) runs over i<=j only; W = D; then A[i,r] += C[j,r] * Y[m,r], the
//           product with C hoisted out of the k loop (Section 5.5, loop-invariant code motion).
//
// A warp owns a unit of consecutive fibres (32 for R >= 32, 64 below) and each of its threads keeps
// 8 x 8 sums (4 x 8 for R = 32, where the finer units balance the SMs better than the larger tile pays; fewer
// rows still below) in registers.  That shape is set by what limits an fp32 FMA kernel that is
// fed from shared memory on this GPU: an SM can issue 128 FMAs but deliver only 32 words from shared memory to its
// registers per cycle, broadcasts included (an inner-loop probe ran at 0.87 of the FMA peak on registers alone,
// 0.73 with an 8 x 8 tile, 0.67 with 8 x 4), so a thread must not read more than 16 words per 64 FMAs.
// The units are dealt to the thread blocks in equal contiguous ranges; a block walks its range 16 units at
// a time (in a last, partial step the warps without a unit skip the arithmetic).  Fibres stream through a cp.async
// pipeline in stages of 16 k-values, each stage together with its 16 rows of W, so neither K nor R is limited by
// the shared memory.  The sum over j of MTTKRP is taken in a fixed order: every warp adds the fibres of its unit
// that share a row of A (i-slots in the thread, then a shuffle butterfly) and writes the sum to the partial slot
// (unit + row); a second kernel adds the slots of every row of A (mttkrp_common.cuh).
#include "st_common.cuh"
#include "st_index.cuh"
#include "mttkrp_common.cuh"

namespace st {

st_status ttm_tf32_tc(const float *Bp, int64_t rows, int64_t K, const float *U, int64_t R, float *Ap, void *ws,
                      size_t ws_bytes, cudaStream_t stream);
st_status mttkrp_tf32_tc(const float *Bp, const MttkrpRows &m, int64_t K, const float *C, const float *D, int64_t R,
                         float *A_full, int64_t I_full, int64_t i_off, void *ws, size_t ws_bytes, cudaStream_t stream);
size_t mttkrp_tf32_tc_workspace(int64_t rows, int64_t I, int64_t K, int64_t R);
st_status ttm_split(const float *Bp, int64_t rows, int64_t K, const float *U, int64_t R, float *Ap, void *ws,
                    size_t ws_bytes, cudaStream_t stream);
st_status mttkrp_split(const float *Bp, const MttkrpRows &m, int64_t K, const float *C, const float *D, int64_t R,
                       float *A_full, int64_t I_full, int64_t i_off, void *ws, size_t ws_bytes, cudaStream_t stream);
size_t mttkrp_split_workspace(int64_t rows, int64_t I, int64_t K, int64_t R);

// The fp32 kernels need no workspace; when the caller passes one anyway its status word is set to "ok".
static inline unsigned *ws_status(void *ws, size_t ws_bytes)
{
    return (ws && ws_bytes >= kWsHeaderBytes && aligned256(ws)) ? (unsigned *)ws : nullptr;
}

constexpr int RG_THREADS = 512;
constexpr int RG_KC = 16;         // k-values per stage: one fibre contributes 64 bytes = four 16-byte chunks

enum { RG_TTM = 0, RG_MTTKRP_PACKED = 1, RG_MTTKRP_DENSE = 2 };

__device__ __forceinline__ void rg_cp_async16(void *smem, const void *gmem, bool valid)
{
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    const int sz = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(sz));
}

struct RgArgs {
    const float *B;      // [rows, K]
    const float *W;      // [K, R]
    const float *C;      // MTTKRP: [I, R]
    float *out;          // TTM: [rows, R];  MTTKRP: partial slots [slots, R]
    int64_t rows;
    int K, R, I;         // I: rows of A reachable from `out`
    int64_t div;         // RG_MTTKRP_DENSE: fibre `row` belongs to (i, j) = (row / div, row % div)
    int kchunks;
    int64_t units, units_per_block;   // a unit = the consecutive fibres of one warp; block b owns units b*upb .. (b+1)*upb-1
    unsigned *status;    // workspace header, or NULL
};

// R = 8 CT columns.  A warp owns WR = TM * (32 / CT) consecutive fibres: lane (fib, tc) holds, for each of its TM
// "i-slots", fibre i * US + fib and the eight columns 4tc .. 4tc+3, R/2 + 4tc .. R/2 + 4tc+3.  What a thread reads
// from shared memory per FMA decides the speed of this kernel (an SM returns 32 words per cycle to its registers and
// can issue 128 FMAs): TM + 8 words per 8 TM FMAs.  A stage holds 16 k-values of every fibre of the tile without
// padding; the four 16-byte chunks of a fibre are permuted by (fibre >> 1) so that the fibres of one load
// instruction (consecutive `fib`) fall into different banks.
template <int TM, int CT, int RG_STAGES, int MODE>
__global__ void __launch_bounds__(RG_THREADS, 1) rowgemm_kernel(const RgArgs a)
{
    constexpr int R_ = CT * 8;
    constexpr int US = 32 / CT;                         // fibres of one i-slot in a warp
    constexpr int WR = TM * US;                         // consecutive fibres of a warp
    constexpr int RG_ROWS = (RG_THREADS / 32) * WR;
    constexpr int SWMASK = US >= 8 ? 3 : 1;             // chunk c of fibre f sits at chunk c ^ ((f >> 1) & SWMASK)
    extern __shared__ __align__(16) float smem[];
    constexpr int STAGE = RG_ROWS * RG_KC + RG_KC * R_; // floats of a stage: fibres [RG_ROWS][RG_KC], then W [RG_KC][R]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tc = lane % CT, fib = lane / CT;

    if (a.status && blockIdx.x == 0 && tid == 0) {      // no bounded waits in this kernel: the status is "ok"
        a.status[kWsStatusWord] = 0;
        a.status[kWsDetailWord] = 0;
    }
    // The block owns a contiguous range of units and walks it in tiles of 16 (one unit per warp); in the last
    // tile the warps without a unit skip the arithmetic, so a partial tile costs what its units cost.  The
    // (tile, k-chunk) steps form one sequence; the loader runs RG_STAGES - 1 steps ahead of the arithmetic.
    const int64_t u0 = (int64_t)blockIdx.x * a.units_per_block;
    int64_t u1 = u0 + a.units_per_block;
    if (u1 > a.units) u1 = a.units;
    int64_t row_end = u1 * WR;
    if (row_end > a.rows) row_end = a.rows;
    const int my_items = u1 > u0 ? (int)((u1 - u0 + RG_THREADS / 32 - 1) / (RG_THREADS / 32)) : 0;
    int ld_it = 0, ld_kcl = 0, ld_slot = 0;

    auto issue = [&]() {
        if (ld_it < my_items) {
            const int kc = ld_kcl;
            const int q = tid & 3, r0 = tid >> 2;
            const int k = kc * RG_KC + q * 4;
            const bool kok = k < a.K;
            int64_t row = (u0 + (int64_t)ld_it * (RG_THREADS / 32)) * WR + r0;
            const float *src = a.B + row * a.K + k;
            // rows advance by 128 per pass, so (row >> 1) & SWMASK stays what it is for r0
            float *stage = smem + ld_slot * STAGE;
            float *dst = stage + r0 * RG_KC + ((q ^ ((r0 >> 1) & SWMASK)) << 2);
#pragma unroll
            for (int u = 0; u < RG_ROWS / (RG_THREADS / 4); ++u) {
                const bool ok = kok && row < row_end;
                rg_cp_async16(dst, ok ? src : a.B, ok);
                row += RG_THREADS / 4;
                src += (int64_t)(RG_THREADS / 4) * a.K;
                dst += (RG_THREADS / 4) * RG_KC;
            }
            // the 16 rows of W that go with this k-chunk (from L2 after the first tile); rows >= K are zero
            if (tid < RG_KC * R_ / 4) {
                const bool wok = kc * RG_KC + tid / (R_ / 4) < a.K;
                rg_cp_async16(stage + RG_ROWS * RG_KC + tid * 4, wok ? a.W + (size_t)kc * RG_KC * R_ + tid * 4 : a.W, wok);
            }
            if (++ld_kcl == a.kchunks) { ld_kcl = 0; ++ld_it; }
            if (++ld_slot == RG_STAGES) ld_slot = 0;
        }
        asm volatile("cp.async.commit_group;\n" ::);
    };

    for (int s = 0; s < RG_STAGES - 1; ++s) issue();

    float acc[TM][8];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    const int sw = (fib >> 1) & SWMASK;
    int slot = 0;
    for (int it = 0; it < my_items; ++it) {
        const int64_t unit = u0 + (int64_t)it * (RG_THREADS / 32) + warp;
        const bool active = unit < u1;
        for (int kc = 0; kc < a.kchunks; ++kc) {
            asm volatile("cp.async.wait_group %0;\n" ::"n"(RG_STAGES - 2));
            __syncthreads();                       // this step's stage landed; the stage of the step before is free again
            issue();
            const float *bs = smem + slot * STAGE + (warp * WR + fib) * RG_KC;
            const float *ws = smem + slot * STAGE + RG_ROWS * RG_KC + tc * 4;
            if (++slot == RG_STAGES) slot = 0;
            if (!active) continue;
#pragma unroll
            for (int c = 0; c < RG_KC / 4; ++c) {
                float4 b[TM];
#pragma unroll
                for (int i = 0; i < TM; ++i)
                    b[i] = *reinterpret_cast<const float4 *>(bs + i * (US * RG_KC) + ((c ^ sw) << 2));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    // k beyond K: the fibre slice was zero-filled and the rows of Ws are zero
                    const float4 w0 = *reinterpret_cast<const float4 *>(ws + (4 * c + kk) * R_);
                    const float4 w1 = *reinterpret_cast<const float4 *>(ws + (4 * c + kk) * R_ + R_ / 2);
                    const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
                    for (int i = 0; i < TM; ++i) {
                        const float bv = kk == 0 ? b[i].x : kk == 1 ? b[i].y : kk == 2 ? b[i].z : b[i].w;
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(bv, wv[j], acc[i][j]);
                    }
                }
            }
        }
        // ---- epilogue of this work item
        const int64_t wbase = unit * WR;                             // first fibre of this warp
        if (!active) continue;
        if (MODE == RG_TTM) {
#pragma unroll
            for (int i = 0; i < TM; ++i) {
                const int64_t row = wbase + i * US + fib;
                if (row < a.rows) {
                    float *o = a.out + row * R_ + 4 * tc;
                    *reinterpret_cast<float4 *>(o) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                    *reinterpret_cast<float4 *>(o + R_ / 2) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
                }
            }
        } else {
            // The warp's WR fibres are one unit.  Every run of fibres of the unit that share the row g of A is summed
            // in a fixed order (i-slots in the thread, then a shuffle butterfly over the fibres of a slot) and written
            // to partial slot (unit + g); rows are sorted by g, so the runs are g0 .. g1.
            int64_t wlast = wbase + WR - 1;
            if (wlast >= a.rows) wlast = a.rows - 1;
            int64_t g0, j0, g1, j1;
            if (MODE == RG_MTTKRP_PACKED) {
                tri_decode(a.I, wbase, g0, j0);
                tri_decode(a.I, wlast, g1, j1);
            } else {
                g0 = wbase / a.div; j0 = wbase - g0 * a.div;
                g1 = wlast / a.div; j1 = wlast - g1 * a.div;
            }
            (void)j1;
            int gi[TM];
#pragma unroll
            for (int i = 0; i < TM; ++i) {
                const int64_t row = wbase + i * US + fib;
                int64_t g = -1, j = 0;
                if (row < a.rows) {
                    if (g0 == g1) { g = g0; j = j0 + (row - wbase); }
                    else if (MODE == RG_MTTKRP_PACKED) tri_decode(a.I, row, g, j);
                    else { g = row / a.div; j = row - g * a.div; }
                    const float4 c0 = *reinterpret_cast<const float4 *>(a.C + j * R_ + 4 * tc);
                    const float4 c1 = *reinterpret_cast<const float4 *>(a.C + j * R_ + R_ / 2 + 4 * tc);
                    acc[i][0] *= c0.x; acc[i][1] *= c0.y; acc[i][2] *= c0.z; acc[i][3] *= c0.w;
                    acc[i][4] *= c1.x; acc[i][5] *= c1.y; acc[i][6] *= c1.z; acc[i][7] *= c1.w;
                }
                gi[i] = (int)g;
            }
            for (int g = (int)g0; g <= (int)g1; ++g) {
                float w[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int i = 0; i < TM; ++i)
                    if (gi[i] == g) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) w[c] += acc[i][c];
                    }
#pragma unroll
                for (int off = CT; off < 32; off <<= 1)
#pragma unroll
                    for (int c = 0; c < 8; ++c) w[c] += __shfl_xor_sync(0xffffffffu, w[c], off);
                if (lane < CT && ST_BOUNDS_OK(unit + g, mttkrp_slots(a.rows, WR, a.I, 1), 5)) {
                    float *o = a.out + (unit + g) * R_ + 4 * tc;
                    *reinterpret_cast<float4 *>(o) = make_float4(w[0], w[1], w[2], w[3]);
                    *reinterpret_cast<float4 *>(o + R_ / 2) = make_float4(w[4], w[5], w[6], w[7]);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
    }
    asm volatile("cp.async.wait_group 0;\n" ::);
    if (MODE != RG_TTM) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the row sums may be launched
}

// Second pass of MTTKRP: one warp per row of A adds the partial slots of that row in increasing
// order (units, then k-splits) and writes the row; rows the fibres do not reach are zero.
__global__ void __launch_bounds__(256)
mttkrp_rowsum_kernel(const float *__restrict__ part, float *__restrict__ A, int64_t I_full, int64_t i_off, MttkrpRows m,
                     int R, int unit_rows, int ksplit)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");      // launched early: wait for the kernel that wrote the partials
    const int lane = threadIdx.x & 31;
    const int64_t ii = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (ii >= I_full) return;
    const int64_t i = ii - i_off;
    float *dst = A + ii * R;
    if (i < 0 || i >= m.I) {
        for (int r = lane; r < R; r += 32) dst[r] = 0.f;
        return;
    }
    int64_t s, e;
    if (m.mode == MK_PACKED) { s = tri_row_start(m.I, i); e = s + (m.I - i); }
    else { s = i * m.div; e = s + m.div; }
    if (e > m.rows) e = m.rows;
    const int64_t u0 = s / unit_rows, u1 = (e - 1) / unit_rows;
    for (int r = lane; r < R; r += 32) {
        float sum = 0.f;
        if (e > s) {
            const float *p = part + ((u0 + i) * ksplit) * R + r;
            const int64_t n = (u1 - u0 + 1) * ksplit;
            if (!ST_BOUNDS_OK((u0 + i) * ksplit + n - 1, mttkrp_slots(m.rows, unit_rows, m.I, ksplit), 6)) continue;
            int64_t k = 0;
            for (; k + 8 <= n; k += 8) {               // eight independent loads in flight
                float t[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) t[u] = __ldcg(p + (k + u) * R);
#pragma unroll
                for (int u = 0; u < 8; ++u) sum += t[u];
            }
            for (; k < n; ++k) sum += __ldcg(p + k * R);
        }
        dst[r] = sum;
    }
}

st_status mttkrp_rowsum_launch(const float *part, float *A_full, int64_t I_full, int64_t i_off, const MttkrpRows &m,
                               int R, int unit_rows, int ksplit, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((I_full + 7) / 8));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, mttkrp_rowsum_kernel, part, A_full, I_full, i_off, m, R, unit_rows, ksplit) != cudaSuccess) {
        (void)cudaGetLastError();
        return ST_ERR_CUDA;
    }
    return ST_OK;
}

// tile shape by R: {TM, stages}; a warp owns TM * 32 / (R/8) consecutive fibres, a tile is the block's 16 warps
static void rowgemm_shape(int64_t R, int &tm, int &stages)
{
    // measured at the benchmark sizes: R = 64 runs 213 / 205 / 208 us with 6 / 4 / 3 stages; R = 32 runs 151 us with
    // 8 fibres per thread (14 units of 64 fibres per SM: 3.5 per scheduler) and 136 us with 4 (28 units of 32), whatever
    // the stage count from 2 to 6
    if (R == 64) { tm = 8; stages = 4; }          // 512 fibres per tile, 36 KiB per stage
    else if (R == 32) { tm = 4; stages = 4; }     // 512 fibres per tile, 34 KiB per stage
    else { tm = (int)R / 4; stages = 3; }         // 1024 fibres per tile
}
static int64_t rowgemm_warp_rows(int64_t R)
{
    int tm, stages;
    rowgemm_shape(R, tm, stages);
    return (int64_t)tm * (32 / (R / 8));
}

static size_t rowgemm_smem(int64_t K, int64_t R)
{
    int tm, stages;
    rowgemm_shape(R, tm, stages);
    const size_t rows = (size_t)(RG_THREADS / 32) * rowgemm_warp_rows(R);
    (void)K;
    return (size_t)stages * (rows * RG_KC + (size_t)RG_KC * R) * sizeof(float);
}

struct RgPlan {
    int kchunks, unit_rows, grid;
    int64_t units, units_per_block;
};

// Units of consecutive fibres (one per warp and tile step) dealt to the blocks in equal contiguous ranges.
static RgPlan rowgemm_plan(int64_t rows, int64_t K, int64_t R)
{
    RgPlan p;
    p.unit_rows = (int)rowgemm_warp_rows(R);
    p.kchunks = (int)((K + RG_KC - 1) / RG_KC);
    p.units = (rows + p.unit_rows - 1) / p.unit_rows;
    const int sms = sm_count_or_default();
    p.units_per_block = (p.units + sms - 1) / sms;
    p.grid = (int)((p.units + p.units_per_block - 1) / p.units_per_block);
    return p;
}

template <int MODE>
static st_status rowgemm_launch(const RgArgs &a0, cudaStream_t stream)
{
    RgArgs a = a0;
    const DeviceInfo di = device_info();
    if (!di.ok) return ST_ERR_CUDA;
    const size_t smem = rowgemm_smem(a.K, a.R);
    if (smem > (size_t)di.max_smem_optin) return ST_ERR_UNSUPPORTED;
    const RgPlan p = rowgemm_plan(a.rows, a.K, a.R);
    a.kchunks = p.kchunks;
    a.units = p.units;
    a.units_per_block = p.units_per_block;
    const int grid = p.grid;
    auto run = [&](auto kernel) -> st_status {
        if (!ensure_dynamic_smem(kernel, smem)) return ST_ERR_CUDA;
        kernel<<<grid, RG_THREADS, smem, stream>>>(a);
        return launch_status();
    };
    switch (a.R) {
    case 8: return run(rowgemm_kernel<2, 1, 3, MODE>);
    case 16: return run(rowgemm_kernel<4, 2, 3, MODE>);
    case 32: return run(rowgemm_kernel<4, 4, 4, MODE>);
    case 64: return run(rowgemm_kernel<8, 8, 4, MODE>);
    default: return ST_ERR_UNSUPPORTED;
    }
}

static bool rowgemm_r_ok(int64_t R) { return R == 8 || R == 16 || R == 32 || R == 64; }

// Workspace of MTTKRP over `rows` fibres that reach `I` rows of A: the header and the partial slots.
size_t mttkrp_workspace(int64_t rows, int64_t I, int64_t K, int64_t R, unsigned flags)
{
    if (rows <= 0 || I <= 0 || K <= 0 || R <= 0 || K % 4 != 0) return 0;
    if ((flags & ST_FLAG_TC_TF32) && (flags & ST_FLAG_TC_SPLIT)) return 0;
    if (flags & ST_FLAG_TC_TF32) return mttkrp_tf32_tc_workspace(rows, I, K, R);
    if (flags & ST_FLAG_TC_SPLIT) return mttkrp_split_workspace(rows, I, K, R);
    if (!rowgemm_r_ok(R)) return 0;
    const RgPlan p = rowgemm_plan(rows, K, R);
    return kWsHeaderBytes + (size_t)mttkrp_slots(rows, p.unit_rows, I, 1) * R * sizeof(float);
}

// Both passes of MTTKRP; `m` says how a row maps to (i, j), the fibres reach rows i_off .. of A_full.
static st_status mttkrp_run(const float *Bp, const MttkrpRows &m, int64_t K, const float *C, const float *D, int64_t R,
                            float *A_full, int64_t I_full, int64_t i_off, void *ws, size_t ws_bytes, unsigned flags,
                            cudaStream_t stream)
{
    if (flags & ST_FLAG_TC_TF32)
        return mttkrp_tf32_tc(Bp, m, K, C, D, R, A_full, I_full, i_off, ws, ws_bytes, stream);
    if (flags & ST_FLAG_TC_SPLIT)
        return mttkrp_split(Bp, m, K, C, D, R, A_full, I_full, i_off, ws, ws_bytes, stream);
    if (!rowgemm_r_ok(R)) return ST_ERR_UNSUPPORTED;
    const size_t need = mttkrp_workspace(m.rows, m.I, K, R, flags);
    if (!ws || ws_bytes < need) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    const RgPlan p = rowgemm_plan(m.rows, K, R);
    RgArgs a{};
    a.B = Bp; a.W = D; a.C = C; a.out = (float *)((unsigned char *)ws + kWsHeaderBytes);
    a.K = (int)K; a.R = (int)R; a.I = m.I; a.rows = m.rows; a.div = m.div;
    a.status = (unsigned *)ws;
    const st_status rc = m.mode == MK_PACKED ? rowgemm_launch<RG_MTTKRP_PACKED>(a, stream)
                                             : rowgemm_launch<RG_MTTKRP_DENSE>(a, stream);
    if (rc != ST_OK) return rc;
    return mttkrp_rowsum_launch(a.out, A_full, I_full, i_off, m, (int)R, p.unit_rows, 1, stream);
}

}  // namespace st

extern "C" {

st_status st_ttm_blockdiag(const float *Bp, int64_t nblocks, int64_t bs, int64_t K, const float *U, int64_t R,
                           float *Ap, void *ws, size_t ws_bytes, unsigned flags, void *stream)
{
    using namespace st;
    if (!Bp || !U || !Ap) return ST_ERR_NULL;
    if (nblocks <= 0 || bs <= 0 || K <= 0 || R <= 0) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_DENSE_CONTROL | ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if ((flags & ST_FLAG_TC_TF32) && (flags & ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if (!aligned16(Bp) || !aligned16(U) || !aligned16(Ap)) return ST_ERR_ALIGN;
    if (nblocks > (int64_t(1) << 24) || bs > (int64_t(1) << 15) || K > (1 << 20)) return ST_ERR_UNSUPPORTED;
    const int64_t d = nblocks * bs;
    const int64_t rows = (flags & ST_FLAG_DENSE_CONTROL) ? d * d : nblocks * bs * bs;
    if (rows / 256 + 1 > (int64_t(1) << 28)) return ST_ERR_UNSUPPORTED;
    if (flags & ST_FLAG_TC_TF32) return ttm_tf32_tc(Bp, rows, K, U, R, Ap, ws, ws_bytes, (cudaStream_t)stream);
    if (flags & ST_FLAG_TC_SPLIT) return ttm_split(Bp, rows, K, U, R, Ap, ws, ws_bytes, (cudaStream_t)stream);
    if (K % 4 != 0) return ST_ERR_UNSUPPORTED;
    if (R != 8 && R != 16 && R != 32 && R != 64) return ST_ERR_UNSUPPORTED;
    RgArgs a{};
    a.B = Bp; a.W = U; a.C = nullptr; a.out = Ap; a.rows = rows; a.K = (int)K; a.R = (int)R; a.I = 0;
    a.status = ws_status(ws, ws_bytes);
    return rowgemm_launch<RG_TTM>(a, (cudaStream_t)stream);
}

st_status st_ttm_packed(const st_layout *layout, const float *Bp, const float *U, int64_t R, float *Ap, void *ws,
                        size_t ws_bytes, unsigned flags, void *stream)
{
    using namespace st;
    if (!layout || !Bp || !U || !Ap) return ST_ERR_NULL;
    if (R <= 0) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if ((flags & ST_FLAG_TC_TF32) && (flags & ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if (!aligned16(Bp) || !aligned16(U) || !aligned16(Ap)) return ST_ERR_ALIGN;
    const int64_t K = layout->inner;
    const int64_t elems = st_packed_elems(layout);      // validates the layout
    if (elems <= 0 || K <= 0) return ST_ERR_SHAPE;
    const int64_t rows = elems / K;                      // one fibre along k per packed position
    if (K > (1 << 20) || rows / 256 + 1 > (int64_t(1) << 28)) return ST_ERR_UNSUPPORTED;
    if (flags & ST_FLAG_TC_TF32) return ttm_tf32_tc(Bp, rows, K, U, R, Ap, ws, ws_bytes, (cudaStream_t)stream);
    if (flags & ST_FLAG_TC_SPLIT) return ttm_split(Bp, rows, K, U, R, Ap, ws, ws_bytes, (cudaStream_t)stream);
    if (K % 4 != 0) return ST_ERR_UNSUPPORTED;
    if (R != 8 && R != 16 && R != 32 && R != 64) return ST_ERR_UNSUPPORTED;
    RgArgs a{};
    a.B = Bp; a.W = U; a.C = nullptr; a.out = Ap; a.rows = rows; a.K = (int)K; a.R = (int)R; a.I = 0;
    a.status = ws_status(ws, ws_bytes);
    return rowgemm_launch<RG_TTM>(a, (cudaStream_t)stream);
}

st_status st_mttkrp_tri(const float *Bp, int64_t I, int64_t K, const float *C, const float *D, int64_t R,
                        float *A, void *ws, size_t ws_bytes, unsigned flags, void *stream)
{
    using namespace st;
    if (!Bp || !C || !D || !A) return ST_ERR_NULL;
    if (I <= 0 || K <= 0 || R <= 0) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_DENSE_CONTROL | ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if ((flags & ST_FLAG_TC_TF32) && (flags & ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if (!aligned16(Bp) || !aligned16(C) || !aligned16(D) || !aligned16(A)) return ST_ERR_ALIGN;
    if (I > (1 << 15) || K > (1 << 20) || K % 4 != 0) return ST_ERR_UNSUPPORTED;
    const bool dense = (flags & ST_FLAG_DENSE_CONTROL) != 0;
    MttkrpRows m;
    m.mode = dense ? MK_DENSE : MK_PACKED;
    m.I = (int)I;
    m.div = I;
    m.rows = dense ? I * I : tri_rows(I);
    return mttkrp_run(Bp, m, K, C, D, R, A, I, 0, ws, ws_bytes, flags, (cudaStream_t)stream);
}

st_status st_mttkrp_slice(const float *Bp, int64_t I, int64_t J, int64_t K, int64_t fixed_i, int64_t fixed_j,
                          const float *C, const float *D, int64_t R, float *A, void *ws, size_t ws_bytes,
                          unsigned flags, void *stream)
{
    using namespace st;
    if (!Bp || !C || !D || !A) return ST_ERR_NULL;
    if (I <= 0 || J <= 0 || K <= 0 || R <= 0) return ST_ERR_SHAPE;
    if (fixed_i >= I || fixed_j >= J || (fixed_i < 0 && fixed_j < 0)) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if ((flags & ST_FLAG_TC_TF32) && (flags & ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if (!aligned16(Bp) || !aligned16(C) || !aligned16(D) || !aligned16(A)) return ST_ERR_ALIGN;
    if (I > (1 << 24) || J > (1 << 24) || K > (1 << 20) || K % 4 != 0 || R % 4 != 0) return ST_ERR_UNSUPPORTED;
    // The fibres of the slice are the packed rows.  With (i, j) = (row / div, row % div):
    //   fixed j: row = i, div = 1, C starts at row j0              -> (i, 0)
    //   fixed i: row = j, div = J, A starts at row i0 (one row)     -> (0, j)
    //   both   : one fibre, both shifts
    const int64_t rows = fixed_i >= 0 ? (fixed_j >= 0 ? 1 : J) : I;
    const int64_t div = fixed_i >= 0 ? (fixed_j >= 0 ? 1 : J) : 1;
    const float *Cs = fixed_j >= 0 ? C + fixed_j * R : C;
    MttkrpRows m;
    m.mode = MK_DENSE;
    m.I = (int)(fixed_i >= 0 ? 1 : I);
    m.div = div;
    m.rows = rows;
    // the fibres reach row fixed_i of A only (fixed i), or every row; the second pass writes the others as zero
    return mttkrp_run(Bp, m, K, Cs, D, R, A, I, fixed_i >= 0 ? fixed_i : 0, ws, ws_bytes, flags, (cudaStream_t)stream);
}

}  // extern "C"
