// st_ttm_blockdiag and st_mttkrp_tri, fp32 FMA path (Table 1: TTM, MTTKRP).
//
// In the packed layouts both kernels contract the trailing dense mode k of a tall matrix of
// fibres with a small dense factor W[K,R] that stays in shared memory:
//     Y[m, r] = sum_k Bp[m, k] * W[k, r]
//   TTM     m runs over the fibres of the diagonal blocks only; Y is the packed output
//           (the zero blocks of the direct sum are never touched: A_U(i,j,r) = B_U(i,j,.)).
//   MTTKRP  m = p(i,j) runs over i<=j only; W = D; then A[i,r] += C[j,r] * Y[m,r], the
//           product with C hoisted out of the k loop (Section 5.5, loop-invariant code motion).
//
// A thread block owns tiles of consecutive fibres (256 for R=64 and R<=16, 512 for R=32); 256
// threads each keep TM x 8 sums in registers (TM = 8 for R >= 32).  Fibres are streamed through
// a cp.async pipeline in slices of 32 k-values; work items (tile, k-split) are walked in one flattened loop so the
// pipeline never drains between tiles.  MTTKRP splits k over work items when that evens out
// the load (its output is a sum over k anyway); the sum over j is taken in a fixed order: every
// warp writes the sums of its runs of fibres with equal i to partial slots and a second kernel
// adds the slots of every row of A (mttkrp_common.cuh).
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

constexpr int RG_THREADS = 256;
constexpr int RG_KC = 32;         // k-values per stage
constexpr int RG_LD = RG_KC + 4;  // padded row stride (floats) of a stage

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
    int tiles, ksplit, kchunks_per_split, kchunks;
    unsigned *status;    // workspace header, or NULL
};

// TM rows x 8 columns per thread, CT column threads (R = 8*CT), RG_ROWS = 256/CT*TM fibres per tile.
template <int TM, int CT, int RG_STAGES, int MODE>
__global__ void __launch_bounds__(RG_THREADS, 1) rowgemm_kernel(const RgArgs a)
{
    constexpr int RG_ROWS = RG_THREADS / CT * TM;
    extern __shared__ __align__(16) float smem[];
    float *Ws = smem;                                   // [kchunks*RG_KC][R], rows >= K are zero
    float *Bs = Ws + (size_t)a.kchunks * RG_KC * a.R;   // RG_STAGES x [RG_ROWS][RG_LD]
    constexpr int R_ = CT * 8;
    constexpr int RT = RG_THREADS / CT;                 // row threads; thread rows = tr + a*RT
    const int tid = threadIdx.x;
    const int tc = tid % CT, tr = tid / CT;

    if (a.status && blockIdx.x == 0 && tid == 0) {      // no bounded waits in this kernel: the status is "ok"
        a.status[kWsStatusWord] = 0;
        a.status[kWsDetailWord] = 0;
    }
    for (int e = tid; e < a.kchunks * RG_KC * a.R / 4; e += RG_THREADS)
        reinterpret_cast<float4 *>(Ws)[e] =
            (e < a.K * a.R / 4) ? reinterpret_cast<const float4 *>(a.W)[e] : make_float4(0.f, 0.f, 0.f, 0.f);

    const int items = a.tiles * a.ksplit;
    // flattened (item, k-chunk) sequence of this block
    const int my_items = (items > (int)blockIdx.x) ? (items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int64_t total_steps = (int64_t)my_items * a.kchunks_per_split;

    auto issue = [&](int64_t step) {
        if (step < total_steps) {
            const int it = (int)(step / a.kchunks_per_split);
            const int kc_local = (int)(step - (int64_t)it * a.kchunks_per_split);
            const int item = blockIdx.x + it * gridDim.x;
            const int tile = item / a.ksplit, ks = item - tile * a.ksplit;
            const int kc = ks * a.kchunks_per_split + kc_local;
            float *dst = Bs + (int)(step % RG_STAGES) * (RG_ROWS * RG_LD);
            const int64_t row0 = (int64_t)tile * RG_ROWS;
            for (int c = tid; c < RG_ROWS * (RG_KC / 4); c += RG_THREADS) {
                const int r = c >> 3, q = c & 7;
                const int64_t row = row0 + r;
                const int k = kc * RG_KC + q * 4;
                const bool ok = row < a.rows && k < a.K && kc < a.kchunks;
                rg_cp_async16(dst + r * RG_LD + q * 4, a.B + (ok ? row * a.K + k : 0), ok);
            }
        }
        asm volatile("cp.async.commit_group;\n" ::);
    };

    for (int s = 0; s < RG_STAGES - 1; ++s) issue(s);

    float acc[TM][8];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    for (int64_t step = 0; step < total_steps; ++step) {
        asm volatile("cp.async.wait_group %0;\n" ::"n"(RG_STAGES - 2));
        __syncthreads();                       // stage `step` landed; stage step-1 is free again
        issue(step + RG_STAGES - 1);
        const int it = (int)(step / a.kchunks_per_split);
        const int kc_local = (int)(step - (int64_t)it * a.kchunks_per_split);
        const int item = blockIdx.x + it * gridDim.x;
        const int tile = item / a.ksplit, ks = item - tile * a.ksplit;
        const int kc = ks * a.kchunks_per_split + kc_local;
        const float *bs = Bs + (int)(step % RG_STAGES) * (RG_ROWS * RG_LD);
        const float *ws = Ws + (size_t)kc * RG_KC * R_ + tc * 8;
        if (kc < a.kchunks) {
#pragma unroll 2
            for (int k4 = 0; k4 < RG_KC; k4 += 4) {
                float4 b[TM];
#pragma unroll
                for (int i = 0; i < TM; ++i)
                    b[i] = *reinterpret_cast<const float4 *>(bs + (tr + i * RT) * RG_LD + k4);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    // k beyond K: the fibre slice was zero-filled and the rows of Ws are zero
                    const float4 w0 = *reinterpret_cast<const float4 *>(ws + (k4 + kk) * R_);
                    const float4 w1 = *reinterpret_cast<const float4 *>(ws + (k4 + kk) * R_ + 4);
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
        if (kc_local == a.kchunks_per_split - 1) {
            // ---- epilogue of this work item
            const int64_t row0 = (int64_t)tile * RG_ROWS;
            if (MODE == RG_TTM) {
#pragma unroll
                for (int i = 0; i < TM; ++i) {
                    const int64_t row = row0 + tr + i * RT;
                    if (row < a.rows) {
                        float4 *o = reinterpret_cast<float4 *>(a.out + row * R_ + tc * 8);
                        o[0] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                        o[1] = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
                    }
                }
            } else {
                // A warp holds, for each i-slot, US = 32/CT consecutive fibres (8 columns per lane): one unit.
                // Every run of fibres of the unit that share the row of A is summed with a shuffle butterfly
                // (masked when the unit holds several runs) and written to partial slot (unit + row of A).
                constexpr int US = 32 / CT;
                const int lane = tid & 31;
                const int fib = lane / CT;                 // fibre of this lane within the unit
#pragma unroll
                for (int i = 0; i < TM; ++i) {
                    const int64_t row = row0 + tr + i * RT;
                    const bool valid = row < a.rows;
                    int64_t gi = -1, gj = 0;
                    if (valid) {
                        if (MODE == RG_MTTKRP_PACKED) tri_decode(a.I, row, gi, gj);
                        else { gi = row / a.div; gj = row - gi * a.div; }
                    }
                    float v[8];
                    if (valid) {
                        const float4 c0 = *reinterpret_cast<const float4 *>(a.C + gj * R_ + tc * 8);
                        const float4 c1 = *reinterpret_cast<const float4 *>(a.C + gj * R_ + tc * 8 + 4);
                        const float cv[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
                        for (int j = 0; j < 8; ++j) v[j] = cv[j] * acc[i][j];
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) v[j] = 0.f;
                    }
                    const int gi32 = (int)gi;
                    const int prev = __shfl_up_sync(0xffffffffu, gi32, CT);
                    // one bit per fibre (taken from the lanes with tc == 0)
                    const unsigned heads = __ballot_sync(0xffffffffu, valid && tc == 0 && (fib == 0 || prev != gi32));
                    const unsigned vmask = __ballot_sync(0xffffffffu, valid && tc == 0);
                    if (heads == 0u) continue;             // no fibre of this unit exists
                    const int64_t unit = (row - fib) / US; // the unit's first row is a multiple of US
                    const int64_t unit0 = __shfl_sync(0xffffffffu, (long long)unit, 0);
                    auto store = [&](int64_t slot, const float (&w)[8]) {
                        float4 *dst = reinterpret_cast<float4 *>(a.out + (slot * a.ksplit + ks) * R_ + tc * 8);
                        dst[0] = make_float4(w[0], w[1], w[2], w[3]);
                        dst[1] = make_float4(w[4], w[5], w[6], w[7]);
                    };
                    const int gi0 = __shfl_sync(0xffffffffu, gi32, 0);
                    if (heads == 1u) {
#pragma unroll
                        for (int off = CT; off < 32; off <<= 1)
#pragma unroll
                            for (int j = 0; j < 8; ++j) v[j] += __shfl_xor_sync(0xffffffffu, v[j], off);
                        if (lane < CT) store(unit0 + gi0, v);
                    } else if (heads == vmask) {
                        if (valid) store(unit0 + gi, v);
                    } else {
                        unsigned h = heads;
                        while (h) {
                            const int l0 = __ffs(h) - 1;
                            h &= h - 1;
                            const int l1 = h ? __ffs(h) - 1 : 32;
                            const bool in = lane >= l0 && lane < l1;
                            float w[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) w[j] = in ? v[j] : 0.f;
#pragma unroll
                            for (int off = CT; off < 32; off <<= 1)
#pragma unroll
                                for (int j = 0; j < 8; ++j) w[j] += __shfl_xor_sync(0xffffffffu, w[j], off);
                            const int gis = __shfl_sync(0xffffffffu, gi32, l0);
                            if (lane < CT) store(unit0 + gis, w);
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
        }
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

// tile shape by R: {TM, stages}; rows per tile = 256 / (R/8) * TM
static void rowgemm_shape(int64_t R, int &tm, int &stages)
{
    if (R == 64) { tm = 8; stages = 3; }
    else if (R == 32) { tm = 8; stages = 2; }
    else { tm = (int)R / 8; stages = 3; }
}

static size_t rowgemm_smem(int64_t K, int64_t R)
{
    int tm, stages;
    rowgemm_shape(R, tm, stages);
    const size_t rows = (size_t)RG_THREADS / (R / 8) * tm;
    const size_t kpad = (size_t)((K + RG_KC - 1) / RG_KC) * RG_KC;
    return (kpad * R + (size_t)stages * rows * RG_LD) * sizeof(float);
}

struct RgPlan {
    int tiles, ksplit, kchunks, unit_rows;
};

// Tiles and, for MTTKRP, the k-split that wastes the fewest SM slots in the last wave.
static RgPlan rowgemm_plan(int64_t rows, int64_t K, int64_t R, bool mttkrp)
{
    RgPlan p;
    int tm, stages;
    rowgemm_shape(R, tm, stages);
    const int64_t tile_rows = (int64_t)RG_THREADS / (R / 8) * tm;
    p.tiles = (int)((rows + tile_rows - 1) / tile_rows);
    p.kchunks = (int)((K + RG_KC - 1) / RG_KC);
    p.unit_rows = (int)(32 / (R / 8));
    p.ksplit = 1;
    if (mttkrp) {
        const int sms = sm_count_or_default();
        double best = -1.0;
        for (int ks = 1; ks <= 4; ks *= 2) {
            if (p.kchunks % ks) continue;
            const int64_t items = (int64_t)p.tiles * ks;
            const int64_t waves = (items + sms - 1) / sms;
            const double eff = (double)items / (double)(waves * sms);
            if (eff > best + 0.02) { best = eff; p.ksplit = ks; }
        }
    }
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
    const RgPlan p = rowgemm_plan(a.rows, a.K, a.R, MODE != RG_TTM);
    a.kchunks = p.kchunks;
    a.tiles = p.tiles;
    a.ksplit = p.ksplit;
    a.kchunks_per_split = a.kchunks / a.ksplit;
    const int64_t items = (int64_t)a.tiles * a.ksplit;
    const int grid = (int)(items < di.sm_count ? items : di.sm_count);
    auto run = [&](auto kernel) -> st_status {
        if (!ensure_dynamic_smem(kernel, smem)) return ST_ERR_CUDA;
        kernel<<<grid, RG_THREADS, smem, stream>>>(a);
        return launch_status();
    };
    switch (a.R) {
    case 8: return run(rowgemm_kernel<1, 1, 3, MODE>);
    case 16: return run(rowgemm_kernel<2, 2, 3, MODE>);
    case 32: return run(rowgemm_kernel<8, 4, 2, MODE>);
    case 64: return run(rowgemm_kernel<8, 8, 3, MODE>);
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
    const RgPlan p = rowgemm_plan(rows, K, R, true);
    return kWsHeaderBytes + (size_t)mttkrp_slots(rows, p.unit_rows, I, p.ksplit) * R * sizeof(float);
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
    const RgPlan p = rowgemm_plan(m.rows, K, R, true);
    RgArgs a{};
    a.B = Bp; a.W = D; a.C = C; a.out = (float *)((unsigned char *)ws + kWsHeaderBytes);
    a.K = (int)K; a.R = (int)R; a.I = m.I; a.rows = m.rows; a.div = m.div;
    a.status = (unsigned *)ws;
    const st_status rc = m.mode == MK_PACKED ? rowgemm_launch<RG_MTTKRP_PACKED>(a, stream)
                                             : rowgemm_launch<RG_MTTKRP_DENSE>(a, stream);
    if (rc != ST_OK) return rc;
    return mttkrp_rowsum_launch(a.out, A_full, I_full, i_off, m, (int)R, p.unit_rows, p.ksplit, stream);
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
