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
// the load (its output is a sum over k anyway) and reduces over j with shared-memory
// accumulators per tile followed by one global atomic per (i,r).
#include "st_common.cuh"
#include "st_index.cuh"

namespace st {

st_status ttm_tf32_tc(const float *Bp, int64_t rows, int64_t K, const float *U, int64_t R, float *Ap, void *ws,
                      size_t ws_bytes, cudaStream_t stream);
st_status mttkrp_slice_tf32_tc(const float *Bp, int64_t rows, int64_t div, int64_t K, const float *C, const float *D,
                               int64_t R, float *A, void *zero, size_t zero_bytes, void *ws, size_t ws_bytes,
                               cudaStream_t stream);
st_status mttkrp_tf32_tc(const float *Bp, int64_t I, int64_t K, const float *C, const float *D, int64_t R, float *A,
                         bool dense, void *ws, size_t ws_bytes, cudaStream_t stream);

// The fp32 kernels need no workspace; when the caller passes one anyway its status word is set to "ok".
static inline unsigned *ws_status(void *ws, size_t ws_bytes)
{
    return (ws && ws_bytes >= kWsHeaderBytes && aligned256(ws)) ? (unsigned *)ws : nullptr;
}

constexpr int RG_THREADS = 256;
constexpr int RG_KC = 32;         // k-values per stage
constexpr int RG_LD = RG_KC + 4;  // padded row stride (floats) of a stage
constexpr int RG_NI = 40;         // rows of A accumulated in shared memory per tile

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
    float *out;          // TTM: [rows, R];  MTTKRP: A [I, R] (zeroed before the launch)
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
    float *As = Bs + RG_STAGES * RG_ROWS * RG_LD;       // MTTKRP: [RG_NI][R]
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
                // first row of A touched by this tile
                int64_t i_first, j_first;
                if (MODE == RG_MTTKRP_PACKED) tri_decode(a.I, row0, i_first, j_first);
                else { i_first = row0 / a.div; j_first = 0; }
                (void)j_first;
                for (int e = tid; e < RG_NI * R_; e += RG_THREADS) As[e] = 0.f;
                __syncthreads();
                // A warp holds, for each i, 32/CT consecutive fibres (8 columns per lane).  When they
                // all belong to one row of A (the usual case: a row of A owns I-i consecutive fibres)
                // they are summed with shuffles and one lane per column group adds the result to the
                // shared accumulator; otherwise every lane adds its own fibre.
                const int lane = tid & 31;
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
                    const int gi_first = __shfl_sync(0xffffffffu, gi32, 0);
                    const int gi_last = __shfl_sync(0xffffffffu, gi32, 31);
                    const bool uniform = (gi_first == gi_last) && gi_first >= 0;
                    if (uniform) {
#pragma unroll
                        for (int off = CT; off < 32; off <<= 1)
#pragma unroll
                            for (int j = 0; j < 8; ++j) v[j] += __shfl_xor_sync(0xffffffffu, v[j], off);
                    }
                    if (valid && (!uniform || lane < CT)) {
                        const int li = (int)(gi - i_first);
                        if (li < RG_NI) {
                            float *dst = As + li * R_ + tc * 8;
#pragma unroll
                            for (int j = 0; j < 8; ++j) atomicAdd(dst + j, v[j]);
                        } else {
                            float *dst = a.out + gi * R_ + tc * 8;
#pragma unroll
                            for (int j = 0; j < 8; ++j) atomicAdd(dst + j, v[j]);
                        }
                    }
                }
                __syncthreads();
                for (int e = tid; e < RG_NI * R_; e += RG_THREADS) {
                    const int li = e / R_;
                    const float v = As[e];
                    if (i_first + li < a.I && v != 0.f) atomicAdd(a.out + (i_first + li) * R_ + (e - li * R_), v);
                }
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
        }
    }
    asm volatile("cp.async.wait_group 0;\n" ::);
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
    return (kpad * R + (size_t)stages * rows * RG_LD + (size_t)RG_NI * R) * sizeof(float);
}

// `zero` (MTTKRP: the output A, which the kernel adds into) is cleared right before the launch, after
// every check that can still reject the call.
template <int MODE>
static st_status rowgemm_launch(const RgArgs &a0, cudaStream_t stream, void *zero = nullptr, size_t zero_bytes = 0)
{
    RgArgs a = a0;
    const DeviceInfo di = device_info();
    if (!di.ok) return ST_ERR_CUDA;
    const size_t smem = rowgemm_smem(a.K, a.R);
    if (smem > (size_t)di.max_smem_optin) return ST_ERR_UNSUPPORTED;
    a.kchunks = (a.K + RG_KC - 1) / RG_KC;
    int tm, stages;
    rowgemm_shape(a.R, tm, stages);
    const int64_t tile_rows = (int64_t)RG_THREADS / (a.R / 8) * tm;
    a.tiles = (int)((a.rows + tile_rows - 1) / tile_rows);
    a.ksplit = 1;
    if (MODE != RG_TTM) {
        // pick the k-split that wastes the fewest SM slots in the last wave
        double best = -1.0;
        for (int ks = 1; ks <= 4; ks *= 2) {
            if (a.kchunks % ks) continue;
            const int64_t items = (int64_t)a.tiles * ks;
            const int64_t waves = (items + di.sm_count - 1) / di.sm_count;
            const double eff = (double)items / (double)(waves * di.sm_count);
            if (eff > best + 0.02) { best = eff; a.ksplit = ks; }
        }
    }
    a.kchunks_per_split = a.kchunks / a.ksplit;
    const int64_t items = (int64_t)a.tiles * a.ksplit;
    const int grid = (int)(items < di.sm_count ? items : di.sm_count);
    auto run = [&](auto kernel) -> st_status {
        if (!ensure_dynamic_smem(kernel, smem)) return ST_ERR_CUDA;
        if (zero && cudaMemsetAsync(zero, 0, zero_bytes, stream) != cudaSuccess) return ST_ERR_CUDA;
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

}  // namespace st

extern "C" {

st_status st_ttm_blockdiag(const float *Bp, int64_t nblocks, int64_t bs, int64_t K, const float *U, int64_t R,
                           float *Ap, void *ws, size_t ws_bytes, unsigned flags, void *stream)
{
    using namespace st;
    if (!Bp || !U || !Ap) return ST_ERR_NULL;
    if (nblocks <= 0 || bs <= 0 || K <= 0 || R <= 0) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_DENSE_CONTROL | ST_FLAG_TC_TF32)) return ST_ERR_UNSUPPORTED;
    if (!aligned16(Bp) || !aligned16(U) || !aligned16(Ap)) return ST_ERR_ALIGN;
    if (nblocks > (int64_t(1) << 24) || bs > (int64_t(1) << 15) || K > (1 << 20)) return ST_ERR_UNSUPPORTED;
    const int64_t d = nblocks * bs;
    const int64_t rows = (flags & ST_FLAG_DENSE_CONTROL) ? d * d : nblocks * bs * bs;
    if (rows / 256 + 1 > (int64_t(1) << 28)) return ST_ERR_UNSUPPORTED;
    if (flags & ST_FLAG_TC_TF32) return ttm_tf32_tc(Bp, rows, K, U, R, Ap, ws, ws_bytes, (cudaStream_t)stream);
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
    if (flags & ~(ST_FLAG_TC_TF32)) return ST_ERR_UNSUPPORTED;
    if (!aligned16(Bp) || !aligned16(U) || !aligned16(Ap)) return ST_ERR_ALIGN;
    const int64_t K = layout->inner;
    const int64_t elems = st_packed_elems(layout);      // validates the layout
    if (elems <= 0 || K <= 0) return ST_ERR_SHAPE;
    const int64_t rows = elems / K;                      // one fibre along k per packed position
    if (K > (1 << 20) || rows / 256 + 1 > (int64_t(1) << 28)) return ST_ERR_UNSUPPORTED;
    if (flags & ST_FLAG_TC_TF32) return ttm_tf32_tc(Bp, rows, K, U, R, Ap, ws, ws_bytes, (cudaStream_t)stream);
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
    if (flags & ~(ST_FLAG_DENSE_CONTROL | ST_FLAG_TC_TF32)) return ST_ERR_UNSUPPORTED;
    if (!aligned16(Bp) || !aligned16(C) || !aligned16(D) || !aligned16(A)) return ST_ERR_ALIGN;
    if (I > (1 << 15) || K > (1 << 20) || K % 4 != 0) return ST_ERR_UNSUPPORTED;
    if (flags & ST_FLAG_TC_TF32)
        return mttkrp_tf32_tc(Bp, I, K, C, D, R, A, (flags & ST_FLAG_DENSE_CONTROL) != 0, ws, ws_bytes,
                              (cudaStream_t)stream);
    if (R != 8 && R != 16 && R != 32 && R != 64) return ST_ERR_UNSUPPORTED;
    const bool dense = (flags & ST_FLAG_DENSE_CONTROL) != 0;
    RgArgs a{};
    a.B = Bp; a.W = D; a.C = C; a.out = A; a.K = (int)K; a.R = (int)R; a.I = (int)I;
    a.rows = dense ? I * I : tri_rows(I);
    a.div = I;
    a.status = ws_status(ws, ws_bytes);
    const size_t a_bytes = (size_t)I * R * sizeof(float);
    return dense ? rowgemm_launch<RG_MTTKRP_DENSE>(a, (cudaStream_t)stream, A, a_bytes)
                 : rowgemm_launch<RG_MTTKRP_PACKED>(a, (cudaStream_t)stream, A, a_bytes);
}

st_status st_mttkrp_slice(const float *Bp, int64_t I, int64_t J, int64_t K, int64_t fixed_i, int64_t fixed_j,
                          const float *C, const float *D, int64_t R, float *A, void *ws, size_t ws_bytes,
                          unsigned flags, void *stream)
{
    using namespace st;
    if (!Bp || !C || !D || !A) return ST_ERR_NULL;
    if (I <= 0 || J <= 0 || K <= 0 || R <= 0) return ST_ERR_SHAPE;
    if (fixed_i >= I || fixed_j >= J || (fixed_i < 0 && fixed_j < 0)) return ST_ERR_SHAPE;
    if (flags & ~(ST_FLAG_TC_TF32)) return ST_ERR_UNSUPPORTED;
    if (!aligned16(Bp) || !aligned16(C) || !aligned16(D) || !aligned16(A)) return ST_ERR_ALIGN;
    if (I > (1 << 24) || J > (1 << 24) || K > (1 << 20) || K % 4 != 0 || R % 4 != 0) return ST_ERR_UNSUPPORTED;
    // The fibres of the slice are the packed rows.  With (i, j) = (row / div, row % div):
    //   fixed j: row = i, div = 1, C starts at row j0              -> (i, 0)
    //   fixed i: row = j, div = J, A starts at row i0 (one row)     -> (0, j)
    //   both   : one fibre, both shifts
    const int64_t rows = fixed_i >= 0 ? (fixed_j >= 0 ? 1 : J) : I;
    const int64_t div = fixed_i >= 0 ? (fixed_j >= 0 ? 1 : J) : 1;
    const float *Cs = fixed_j >= 0 ? C + fixed_j * R : C;
    float *As = fixed_i >= 0 ? A + fixed_i * R : A;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t a_bytes = (size_t)I * R * sizeof(float);
    if (flags & ST_FLAG_TC_TF32) return mttkrp_slice_tf32_tc(Bp, rows, div, K, Cs, D, R, As, A, a_bytes, ws, ws_bytes, s);
    if (R != 8 && R != 16 && R != 32 && R != 64) return ST_ERR_UNSUPPORTED;
    RgArgs a{};
    a.B = Bp; a.W = D; a.C = Cs; a.out = As; a.K = (int)K; a.R = (int)R;
    a.I = (int)(fixed_i >= 0 ? 1 : I);
    a.rows = rows;
    a.div = div;
    a.status = ws_status(ws, ws_bytes);
    return rowgemm_launch<RG_MTTKRP_DENSE>(a, s, A, a_bytes);
}

}  // extern "C"
