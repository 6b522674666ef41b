// st_sym_moment2, fp32 FMA path: out[p(i,j)] = sum_n X[n,i] X[n,j] over the unique set
// 0<=i<=j<d of the symmetric output (Section 3, M1; Section 5.5, y_U = 0<=i<=j<n).
//
// The upper triangle is cut into 64x64 output tiles (bi<=bj); tiles below the diagonal are
// never launched, and on diagonal tiles only the 136 of 256 4x4 register blocks that touch
// i<=j are computed.  The samples are split over gridDim.y; every CTA stages 32-row slices
// of its two column panels in shared memory, accumulates a 4x4 block per thread, and
// writes a partial tile to the workspace.  A second kernel adds the partials of every tile in
// a fixed order (deterministic result) and writes the packed output.
#include "st_common.cuh"
#include "st_index.cuh"

namespace st {

st_status moment2_bf16_tc(const void *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws,
                          size_t ws_bytes, unsigned flags, cudaStream_t stream);
size_t moment2_bf16_tc_workspace(int64_t N, int64_t d, unsigned flags);
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

// out[p(i,j)] = sum over the splits of a tile, in split order; i <= j only.
__global__ void __launch_bounds__(256)
moment2_f32_reduce_kernel(const float *__restrict__ partials, float *__restrict__ out, int d, int nt, int nsplit,
                          int dense)
{
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
    const int col_a = bi * M2_T, col_b = bj * M2_T;
    const float *base = partials + (size_t)tile * nsplit * (M2_T * M2_T);
    // one output per thread and up to 32 independent loads in flight: after the other kernels of
    // a pipeline have streamed gigabytes, every dependent round trip to memory costs microseconds
    for (int e = blockIdx.y * 256 + threadIdx.x; e < M2_T * M2_T; e += gridDim.y * 256) {
        const int r = e >> 6, c = e & 63;
        const int gi = col_a + r, gj = col_b + c;
        if (gi >= d || gj >= d || gi > gj) continue;
        float s = 0.f;
        const float *p1 = base + e;
        for (int k0 = 0; k0 < nsplit; k0 += 32) {
            float v[32];
#pragma unroll
            for (int u = 0; u < 32; ++u) v[u] = (k0 + u < nsplit) ? __ldcg(p1 + (size_t)(k0 + u) * (M2_T * M2_T)) : 0.f;
#pragma unroll
            for (int u = 0; u < 32; ++u) s += v[u];
        }
        out[tri_encode(d, gi, gj)] = s;
    }
}

static st_status moment2_f32(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws,
                             size_t ws_bytes, unsigned flags, cudaStream_t stream)
{
    if (d > 32768) return ST_ERR_UNSUPPORTED;
    // few features, many samples: the register-tile kernel of moment2_small.cu
    if (moment2_small_applies(N, d) && ldx % 4 == 0) return moment2_small(X, N, d, ldx, out, ws, ws_bytes, flags, stream);
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
    moment2_f32_reduce_kernel<<<dim3(p.ntiles, 16), 256, 0, stream>>>(partials, out, (int)d, p.nt, p.nsplit, dense);
    return launch_status();
}

size_t moment2_workspace(int64_t N, int64_t d, int xdt, unsigned flags)
{
    if (N <= 0 || d <= 0) return 0;
    if (xdt == ST_BF16) return moment2_bf16_tc_workspace(N, d, flags);
    if (xdt != ST_F32 || d > 32768) return 0;
    const M2Plan p = moment2_plan(N, d, flags);
    size_t need = kWsHeaderBytes + p.ticket_bytes + p.partial_bytes;
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
    if (flags & ~(ST_FLAG_DENSE_CONTROL)) return ST_ERR_UNSUPPORTED;
    if (!st::aligned16(X) || !st::aligned16(out_packed)) return ST_ERR_ALIGN;
    if (xdt == ST_BF16)
        return st::moment2_bf16_tc(X, N, d, ldx, out_packed, ws, ws_bytes, flags, (cudaStream_t)stream);
    return st::moment2_f32((const float *)X, N, d, ldx, out_packed, ws, ws_bytes, flags, (cudaStream_t)stream);
}
