// st_sym_moment2, fp32 FMA path: out[p(i,j)] = sum_n X[n,i] X[n,j] over the unique set
// 0<=i<=j<d of the symmetric output (Section 3, M1; Section 5.5, y_U = 0<=i<=j<n).
//
// The upper triangle is cut into 64x64 output tiles (bi<=bj); tiles below the diagonal are
// never launched, and on diagonal tiles only the 136 of 256 4x4 register blocks that touch
// i<=j are computed.  The samples are split over gridDim.y; every CTA stages 32-row slices
// of its two column panels in shared memory, accumulates a 4x4 block per thread, and
// writes a partial tile to the workspace.  A second kernel adds the partials of every tile in
// a fixed order (deterministic result) and writes the packed output.
//
// Two main kernels.  moment2_gemm_kernel (d >= 128 with 16-byte aligned rows): 128x128 output
// tiles, 8x8 register blocks as four 4x4 quadrants, packed fp32 FMAs, samples streamed through a
// four-stage cp.async pipeline; on diagonal tiles the quadrant that lies wholly below the
// diagonal is not computed.  moment2_f32_kernel: the plain 64x64-tile kernel for everything else.
#include "st_common.cuh"
#include "st_index.cuh"
#include <type_traits>

namespace st {

st_status moment2_bf16_tc(const void *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws,
                          size_t ws_bytes, unsigned flags, cudaStream_t stream);
size_t moment2_bf16_tc_workspace(int64_t N, int64_t d, unsigned flags);
st_status moment2_tf32_tc(const void *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws,
                          size_t ws_bytes, unsigned flags, cudaStream_t stream);
size_t moment2_tf32_tc_workspace(int64_t N, int64_t d, unsigned flags);
st_status moment2_split_tc(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                           unsigned flags, cudaStream_t stream);
size_t moment2_split_tc_workspace(int64_t N, int64_t d, unsigned flags);
bool moment2_small_applies(int64_t N, int64_t d);
size_t moment2_small_workspace(int64_t N, int64_t d, unsigned flags);
st_status moment2_small(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                        unsigned flags, cudaStream_t stream);

constexpr int M2_T = 64;    // output tile edge
constexpr int M2_KC = 64;   // sample rows staged per step

struct M2Plan {
    int nt;          // tiles per edge
    int ntiles;      // launched tiles
    int nsplit;      // splits of the sample range
    int64_t rows_per_split;
    size_t ticket_bytes, partial_bytes;
};

static M2Plan moment2_plan(int64_t N, int64_t d, unsigned flags)
{
    M2Plan p;
    p.nt = (int)((d + M2_T - 1) / M2_T);
    p.ntiles = (flags & ST_FLAG_DENSE_CONTROL) ? p.nt * p.nt : p.nt * (p.nt + 1) / 2;
    const int sms = sm_count_or_default();
    int64_t want = (2 * (int64_t)sms + p.ntiles - 1) / p.ntiles;   // about two CTAs per SM
    int64_t max_split = (N + M2_KC - 1) / M2_KC;                   // at least one stage of rows per split
    if (want > max_split) want = max_split;
    if (want > 128) want = 128;
    if (want < 1) want = 1;
    int64_t rows = (N + want - 1) / want;
    rows = (rows + M2_KC - 1) / M2_KC * M2_KC;
    p.rows_per_split = rows;
    p.nsplit = (int)((N + rows - 1) / rows);
    p.ticket_bytes = round_up((size_t)p.ntiles * sizeof(unsigned), 256);
    p.partial_bytes = (size_t)p.ntiles * p.nsplit * M2_T * M2_T * sizeof(float);
    return p;
}

template <bool DENSE>
__global__ void __launch_bounds__(256)
moment2_f32_kernel(const float *__restrict__ X, int64_t N, int d, int64_t ldx, float *__restrict__ out,
                   float *__restrict__ partials, int nt, int nsplit, int64_t rows_per_split, unsigned *status)
{
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {   // no bounded waits here: the status is "ok"
        status[kWsStatusWord] = 0;
        status[kWsDetailWord] = 0;
    }
    __shared__ __align__(16) float As[M2_KC][M2_T];
    __shared__ __align__(16) float Bs[M2_KC][M2_T];

    const int tile = blockIdx.x;
    int bi, bj;
    if (DENSE) {
        bi = tile / nt;
        bj = tile - bi * nt;
    } else {
        int64_t a, b;
        tri_decode(nt, tile, a, b);
        bi = (int)a;
        bj = (int)b;
    }
    const bool diag = (bi == bj);
    const int tid = threadIdx.x;

    // register block of this thread: rows ty*4.., columns tx*4.. of the tile
    int ty, tx;
    bool active = true;
    if (!DENSE && diag) {
        if (tid < 136) {
            int64_t a, b;
            tri_decode(16, tid, a, b);
            ty = (int)a;
            tx = (int)b;
        } else {
            ty = tx = 0;
            active = false;
        }
    } else {
        ty = tid >> 4;
        tx = tid & 15;
    }

    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;

    const int64_t n_begin = (int64_t)blockIdx.y * rows_per_split;
    int64_t n_end = n_begin + rows_per_split;
    if (n_end > N) n_end = N;
    const int col_a = bi * M2_T, col_b = bj * M2_T;
    const float(*Bp)[M2_T] = diag ? As : Bs;

    for (int64_t n0 = n_begin; n0 < n_end; n0 += M2_KC) {
        // stage rows n0..n0+31 of both column panels (zero beyond N and beyond d)
        for (int e = tid; e < M2_KC * M2_T; e += 256) {
            const int r = e >> 6, c = e & 63;   // M2_T == 64
            const int64_t n = n0 + r;
            const bool row_ok = n < n_end;
            As[r][c] = (row_ok && col_a + c < d) ? X[n * ldx + col_a + c] : 0.f;
            if (!diag) Bs[r][c] = (row_ok && col_b + c < d) ? X[n * ldx + col_b + c] : 0.f;
        }
        __syncthreads();
        if (active) {
#pragma unroll 8
            for (int r = 0; r < M2_KC; ++r) {
                const float4 a = *reinterpret_cast<const float4 *>(&As[r][ty * 4]);
                const float4 b = *reinterpret_cast<const float4 *>(&Bp[r][tx * 4]);
                const float av[4] = {a.x, a.y, a.z, a.w};
                const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
            }
        }
        __syncthreads();
    }

    float *mine = partials + ((size_t)tile * nsplit + blockIdx.y) * (M2_T * M2_T);
    if (active) {
#pragma unroll
        for (int r = 0; r < 4; ++r)
            *reinterpret_cast<float4 *>(&mine[(ty * 4 + r) * M2_T + tx * 4]) =
                make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
    }
}

// out[p(i,j)] = sum over the splits of a tile, in split order; i <= j only.  T: tile edge.
template <int T>
__global__ void __launch_bounds__(256)
moment2_f32_reduce_kernel(const float *__restrict__ partials, float *__restrict__ out, int d, int nt, int nsplit,
                          int dense)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");   // may be launched as a programmatic dependent of the main kernel
    const int tile = blockIdx.x;
    int bi, bj;
    if (dense) {
        bi = tile / nt;
        bj = tile - bi * nt;
    } else {
        int64_t a, b;
        tri_decode(nt, tile, a, b);
        bi = (int)a;
        bj = (int)b;
    }
    if (bi > bj) return;                                        // dense control: lower tiles are discarded
    const int col_a = bi * T, col_b = bj * T;
    const float *base = partials + (size_t)tile * nsplit * (T * T);
    // one output per thread and up to 32 independent loads in flight: after the other kernels of
    // a pipeline have streamed gigabytes, every dependent round trip to memory costs microseconds
    for (int e = blockIdx.y * 256 + threadIdx.x; e < T * T; e += gridDim.y * 256) {
        const int r = e / T, c = e - r * T;
        const int gi = col_a + r, gj = col_b + c;
        if (gi >= d || gj >= d || gi > gj) continue;
        float s = 0.f;
        const float *p1 = base + e;
        for (int k0 = 0; k0 < nsplit; k0 += 32) {
            float v[32];
#pragma unroll
            for (int u = 0; u < 32; ++u) v[u] = (k0 + u < nsplit) ? __ldcg(p1 + (size_t)(k0 + u) * (T * T)) : 0.f;
#pragma unroll
            for (int u = 0; u < 32; ++u) s += v[u];
        }
        if (ST_BOUNDS_OK(tri_encode(d, gi, gj), tri_rows(d), 2)) out[tri_encode(d, gi, gj)] = s;
    }
}

// ---- large d: 128 x 128 tiles -------------------------------------------------------------
constexpr int MG_T = 128;       // output tile edge
constexpr int MG_KC = 16;       // sample rows per stage
constexpr int MG_STAGES = 4;
constexpr size_t MG_SMEM = (size_t)MG_STAGES * 2 * MG_KC * MG_T * sizeof(float);   // 64 KiB

struct MgPlan {
    int nt, ntiles, nsplit;
    int64_t rows_per_split;
    size_t partial_bytes;
};

static MgPlan moment2_gemm_plan(int64_t N, int64_t d, unsigned flags)
{
    MgPlan p;
    p.nt = (int)((d + MG_T - 1) / MG_T);
    p.ntiles = (flags & ST_FLAG_DENSE_CONTROL) ? p.nt * p.nt : p.nt * (p.nt + 1) / 2;
    // two thread blocks fit on an SM: the number of sample splits is the one whose blocks fill whole waves
    // of 2 x SMs best (time ~ waves / splits), the smallest such number within 3 %
    const int64_t slots = 2 * (int64_t)sm_count_or_default();
    int64_t max_split = (N + 8 * MG_KC - 1) / (8 * MG_KC);            // at least eight stages of rows per split
    if (max_split > 256) max_split = 256;
    if (max_split < 1) max_split = 1;
    int64_t want = 1;
    double best = 1e30;
    for (int64_t w = 1; w <= max_split; ++w) {
        const double t = (double)((p.ntiles * w + slots - 1) / slots) / (double)w;
        if (t < best * 0.97) { best = t; want = w; }
    }
    int64_t rows = (N + want - 1) / want;
    rows = (rows + MG_KC - 1) / MG_KC * MG_KC;
    p.rows_per_split = rows;
    p.nsplit = (int)((N + rows - 1) / rows);
    p.partial_bytes = (size_t)p.ntiles * p.nsplit * MG_T * MG_T * sizeof(float);
    return p;
}

__device__ __forceinline__ uint64_t mg_pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ uint64_t mg_ffma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// Thread (ty, tx) of the 16 x 16 thread grid owns rows 4ty..4ty+3 and 64+4ty.., columns 4tx.. and 64+4tx..
// of the tile: quadrant (h, g) = rows of half h, columns of half g.  acc[h][g][r][c2] holds columns 2c2, 2c2+1.
template <bool DENSE>
__global__ void __launch_bounds__(256, 2)
moment2_gemm_kernel(const float *__restrict__ X, int64_t N, int d, int64_t ldx, float *__restrict__ partials, int nt,
                    int nsplit, int64_t rows_per_split, unsigned *status)
{
    extern __shared__ __align__(16) float smem[];     // MG_STAGES x { As[MG_KC][MG_T], Bs[MG_KC][MG_T] }
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {   // no bounded waits here: the status is "ok"
        status[kWsStatusWord] = 0;
        status[kWsDetailWord] = 0;
    }
    const int tile = blockIdx.x;
    int bi, bj;
    if (DENSE) {
        bi = tile / nt;
        bj = tile - bi * nt;
    } else {
        int64_t a, b;
        tri_decode(nt, tile, a, b);
        bi = (int)a;
        bj = (int)b;
    }
    const bool diag = (bi == bj);
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int col_a = bi * MG_T, col_b = bj * MG_T;
    const int64_t n_begin = (int64_t)blockIdx.y * rows_per_split;
    int64_t n_end = n_begin + rows_per_split;
    if (n_end > N) n_end = N;
    const int nstages = n_end > n_begin ? (int)((n_end - n_begin + MG_KC - 1) / MG_KC) : 0;

    uint64_t acc[2][2][4][2];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[h][g][r][0] = acc[h][g][r][1] = 0ull;

    // a stage: MG_KC rows of the two column panels; 16-byte chunks, zero-filled past N and past d
    auto load_stage = [&](int s) {
        if (s < nstages) {
            float *As = smem + (size_t)(s % MG_STAGES) * (2 * MG_KC * MG_T), *Bs = As + MG_KC * MG_T;
            const int64_t n0 = n_begin + (int64_t)s * MG_KC;
            for (int c = tid; c < 2 * MG_KC * (MG_T / 4); c += 256) {
                const int panel = c / (MG_KC * (MG_T / 4)), e = c - panel * (MG_KC * (MG_T / 4));
                const int r = e / (MG_T / 4), q = e - r * (MG_T / 4);
                const int col = (panel ? col_b : col_a) + 4 * q;
                const int64_t n = n0 + r;
                const bool in = n < n_end && col < d;
                const unsigned dst = (unsigned)__cvta_generic_to_shared((panel ? Bs : As) + r * MG_T + 4 * q);
                const int sz = in ? 16 : 0;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(in ? X + n * ldx + col : X), "r"(sz));
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    for (int s = 0; s < MG_STAGES - 1; ++s) load_stage(s);
    const bool skip_low = !DENSE && diag;       // quadrant (1, 0) of a diagonal tile lies below the diagonal
    auto run = [&](auto skip_tag) {              // two instances of the loop: the skip is a compile-time fact in each
    constexpr bool SKIP = decltype(skip_tag)::value;
    for (int s = 0; s < nstages; ++s) {
        asm volatile("cp.async.wait_group %0;" ::"n"(MG_STAGES - 2) : "memory");
        __syncthreads();                         // stage s has landed; the buffer of stage s-1 is free
        load_stage(s + MG_STAGES - 1);
        const float *As = smem + (size_t)(s % MG_STAGES) * (2 * MG_KC * MG_T), *Bs = As + MG_KC * MG_T;
#pragma unroll 4
        for (int k = 0; k < MG_KC; ++k) {
            const float4 a0 = *reinterpret_cast<const float4 *>(As + k * MG_T + 4 * ty);
            const float4 a1 = *reinterpret_cast<const float4 *>(As + k * MG_T + 64 + 4 * ty);
            const float4 b0 = *reinterpret_cast<const float4 *>(Bs + k * MG_T + 4 * tx);
            const float4 b1 = *reinterpret_cast<const float4 *>(Bs + k * MG_T + 64 + 4 * tx);
            const float av[2][4] = {{a0.x, a0.y, a0.z, a0.w}, {a1.x, a1.y, a1.z, a1.w}};
            const uint64_t bv[2][2] = {{mg_pack2(b0.x, b0.y), mg_pack2(b0.z, b0.w)}, {mg_pack2(b1.x, b1.y), mg_pack2(b1.z, b1.w)}};
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const uint64_t aa = mg_pack2(av[h][r], av[h][r]);
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        if (h == 1 && g == 0 && SKIP) continue;
                        acc[h][g][r][0] = mg_ffma2(aa, bv[g][0], acc[h][g][r][0]);
                        acc[h][g][r][1] = mg_ffma2(aa, bv[g][1], acc[h][g][r][1]);
                    }
                }
        }
    }
    };
    if (skip_low) run(std::true_type{});
    else run(std::false_type{});
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    float *mine = partials + ((size_t)tile * nsplit + blockIdx.y) * (MG_T * MG_T);
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                if (h == 1 && g == 0 && skip_low) continue;          // never read: the reduction keeps i <= j only
                float4 v;
                asm("mov.b64 {%0, %1}, %2;" : "=f"(v.x), "=f"(v.y) : "l"(acc[h][g][r][0]));
                asm("mov.b64 {%0, %1}, %2;" : "=f"(v.z), "=f"(v.w) : "l"(acc[h][g][r][1]));
                *reinterpret_cast<float4 *>(&mine[(64 * h + 4 * ty + r) * MG_T + 64 * g + 4 * tx]) = v;
            }
}

static bool moment2_gemm_applies(const float *X, int64_t d, int64_t ldx)
{
    return d >= 128 && d % 4 == 0 && ldx % 4 == 0 && aligned16(X);
}

static st_status moment2_gemm(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                              unsigned flags, cudaStream_t stream)
{
    const MgPlan p = moment2_gemm_plan(N, d, flags);
    if (!ws || ws_bytes < kWsHeaderBytes + p.partial_bytes) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    float *partials = (float *)((unsigned char *)ws + kWsHeaderBytes);
    const dim3 grid(p.ntiles, p.nsplit);
    const int dense = (flags & ST_FLAG_DENSE_CONTROL) ? 1 : 0;
    if (dense) {
        if (!ensure_dynamic_smem(moment2_gemm_kernel<true>, MG_SMEM)) return ST_ERR_CUDA;
        moment2_gemm_kernel<true><<<grid, 256, MG_SMEM, stream>>>(X, N, (int)d, ldx, partials, p.nt, p.nsplit, p.rows_per_split,
                                                                    (unsigned *)ws);
    } else {
        if (!ensure_dynamic_smem(moment2_gemm_kernel<false>, MG_SMEM)) return ST_ERR_CUDA;
        moment2_gemm_kernel<false><<<grid, 256, MG_SMEM, stream>>>(X, N, (int)d, ldx, partials, p.nt, p.nsplit, p.rows_per_split,
                                                                     (unsigned *)ws);
    }
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.ntiles, 32);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float *cpart = partials;
    const int di = (int)d;
    if (cudaLaunchKernelEx(&cfg, moment2_f32_reduce_kernel<MG_T>, cpart, out, di, p.nt, p.nsplit, dense) != cudaSuccess) {
        (void)cudaGetLastError();
        return ST_ERR_CUDA;
    }
    return ST_OK;
}

static st_status moment2_f32(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws,
                             size_t ws_bytes, unsigned flags, cudaStream_t stream)
{
    if (d > 32768) return ST_ERR_UNSUPPORTED;
    // few features, many samples: the register-tile kernel of moment2_small.cu
    if (moment2_small_applies(N, d) && ldx % 4 == 0) return moment2_small(X, N, d, ldx, out, ws, ws_bytes, flags, stream);
    if (moment2_gemm_applies(X, d, ldx)) return moment2_gemm(X, N, d, ldx, out, ws, ws_bytes, flags, stream);
    const M2Plan p = moment2_plan(N, d, flags);
    const size_t need = kWsHeaderBytes + p.ticket_bytes + p.partial_bytes;
    if (!ws || ws_bytes < need) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    unsigned char *w = (unsigned char *)ws;
    float *partials = (float *)(w + kWsHeaderBytes + p.ticket_bytes);
    dim3 grid(p.ntiles, p.nsplit);
    const int dense = (flags & ST_FLAG_DENSE_CONTROL) ? 1 : 0;
    if (dense)
        moment2_f32_kernel<true><<<grid, 256, 0, stream>>>(X, N, (int)d, ldx, out, partials, p.nt, p.nsplit,
                                                           p.rows_per_split, (unsigned *)ws);
    else
        moment2_f32_kernel<false><<<grid, 256, 0, stream>>>(X, N, (int)d, ldx, out, partials, p.nt, p.nsplit,
                                                            p.rows_per_split, (unsigned *)ws);
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    moment2_f32_reduce_kernel<M2_T><<<dim3(p.ntiles, 16), 256, 0, stream>>>(partials, out, (int)d, p.nt, p.nsplit, dense);
    return launch_status();
}

size_t moment2_workspace(int64_t N, int64_t d, int xdt, unsigned flags)
{
    if (N <= 0 || d <= 0) return 0;
    const unsigned tc = flags & (ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT);
    if (tc == (ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT)) return 0;
    if (xdt == ST_BF16) return tc ? 0 : moment2_bf16_tc_workspace(N, d, flags);
    if (xdt == ST_F32 && (flags & ST_FLAG_TC_TF32)) return moment2_tf32_tc_workspace(N, d, flags & ~ST_FLAG_TC_TF32);
    if (xdt == ST_F32 && (flags & ST_FLAG_TC_SPLIT)) return moment2_split_tc_workspace(N, d, flags & ~ST_FLAG_TC_SPLIT);
    if (xdt != ST_F32 || d > 32768) return 0;
    const M2Plan p = moment2_plan(N, d, flags);
    size_t need = kWsHeaderBytes + p.ticket_bytes + p.partial_bytes;
    if (d >= 128) {                        // which kernel runs depends on ldx and the alignment of X: size for either
        const size_t g = kWsHeaderBytes + moment2_gemm_plan(N, d, flags).partial_bytes;
        if (g > need) need = g;
    }
    if (moment2_small_applies(N, d)) {     // which kernel runs depends on ldx: size for either
        const size_t small = moment2_small_workspace(N, d, flags);
        if (small > need) need = small;
    }
    return need;
}

}  // namespace st

extern "C" st_status st_sym_moment2(const void *X, st_dtype xdt, int64_t N, int64_t d, int64_t ldx,
                                    float *out_packed, void *ws, size_t ws_bytes, unsigned flags, void *stream)
{
    if (!X || !out_packed) return ST_ERR_NULL;
    if (N <= 0 || d <= 0 || ldx < d) return ST_ERR_SHAPE;
    if (xdt != ST_F32 && xdt != ST_BF16) return ST_ERR_DTYPE;
    if (flags & ~(ST_FLAG_DENSE_CONTROL | ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if ((flags & (ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT)) && xdt != ST_F32) return ST_ERR_UNSUPPORTED;
    if ((flags & ST_FLAG_TC_TF32) && (flags & ST_FLAG_TC_SPLIT)) return ST_ERR_UNSUPPORTED;
    if (!st::aligned16(X) || !st::aligned16(out_packed)) return ST_ERR_ALIGN;
    if (xdt == ST_BF16)
        return st::moment2_bf16_tc(X, N, d, ldx, out_packed, ws, ws_bytes, flags, (cudaStream_t)stream);
    if (flags & ST_FLAG_TC_TF32)
        return st::moment2_tf32_tc(X, N, d, ldx, out_packed, ws, ws_bytes, flags & ~ST_FLAG_TC_TF32, (cudaStream_t)stream);
    if (flags & ST_FLAG_TC_SPLIT)
        return st::moment2_split_tc((const float *)X, N, d, ldx, out_packed, ws, ws_bytes, flags & ~ST_FLAG_TC_SPLIT,
                                    (cudaStream_t)stream);
    return st::moment2_f32((const float *)X, N, d, ldx, out_packed, ws, ws_bytes, flags, (cudaStream_t)stream);
}
