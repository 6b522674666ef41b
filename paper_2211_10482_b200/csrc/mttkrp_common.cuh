// Fixed-order reduction over j of MTTKRP (Table 1): A[i,r] = sum_j C[j,r] * Y[(i,j), r], where
// Y = sum_k B[(i,j),k] D[k,r] is what the fibre kernels compute.
//
// The fibres (i,j) are the rows of a tall matrix in which i never decreases (packed upper half
// cube: row p(i,j); dense and slice forms: row = i * div + j).  The fibre kernels cut the rows into
// units of `unit_rows` consecutive rows (the rows one warp reduces with shuffles) and, for every
// maximal run of rows of one unit that share i, write the sum of the run to partial slot
//     slot(unit, i) = unit + i        (times ksplit, plus the k-split index, when k is split).
// Walking the rows, every new run increments unit, i or both, so unit + i is strictly increasing:
// the slots of different runs differ, and the runs of one i occupy consecutive slots.  The second
// pass adds the slots of every i in increasing order and writes A, every element exactly once:
// no atomics, no zeroing of A, and the same bits on every call.
#pragma once
#include "st_common.cuh"
#include "st_index.cuh"

namespace st {

enum { MK_PACKED = 1, MK_DENSE = 2 };      // how a row maps to (i, j)

struct MttkrpRows {
    int mode;            // MK_PACKED: row = p(i,j) of a triangle of side I;  MK_DENSE: (i, j) = (row / div, row % div)
    int I;               // rows of A that the fibres reach (MK_PACKED: side of the triangle)
    int64_t div;
    int64_t rows;
};

__host__ __device__ inline int64_t mttkrp_slots(int64_t rows, int unit_rows, int64_t I, int ksplit)
{
    return ((rows + unit_rows - 1) / unit_rows + I) * ksplit;
}

// Second pass.  A_full has I_full rows; the fibres reach rows i_off .. i_off + m.I - 1 of it, the
// other rows are written as zero.
st_status mttkrp_rowsum_launch(const float *part, float *A_full, int64_t I_full, int64_t i_off, const MttkrpRows &m,
                               int R, int unit_rows, int ksplit, cudaStream_t stream);

#if defined(__CUDACC__)
// Transposing shuffle reduction of 32 columns held by every lane (one fibre per lane): after the
// step with offset o a lane keeps the half of its columns selected by bit o of its lane index; at
// the end lane l holds the sum of column l over the warp.  The order of the additions is fixed.
__device__ __forceinline__ float warp_transpose_sum32(float (&v)[32], int lane)
{
#define ST_TR_STEP(OFF)                                                                       \
    {                                                                                         \
        const bool up = (lane & OFF) != 0;                                                    \
        _Pragma("unroll") for (int j = 0; j < OFF; ++j) {                                     \
            const float send = up ? v[j] : v[j + OFF];                                        \
            const float keep = up ? v[j + OFF] : v[j];                                        \
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, OFF);                            \
        }                                                                                     \
    }
    ST_TR_STEP(16) ST_TR_STEP(8) ST_TR_STEP(4) ST_TR_STEP(2) ST_TR_STEP(1)
#undef ST_TR_STEP
    return v[0];
}

// The same for 16 columns: every lane ends with the sum of column (lane % 16) over the warp.
__device__ __forceinline__ float warp_transpose_sum16(float (&v)[16], int lane)
{
#define ST_TR_STEP(OFF)                                                                       \
    {                                                                                         \
        const bool up = (lane & OFF) != 0;                                                    \
        _Pragma("unroll") for (int j = 0; j < OFF; ++j) {                                     \
            const float send = up ? v[j] : v[j + OFF];                                        \
            const float keep = up ? v[j + OFF] : v[j];                                        \
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, OFF);                            \
        }                                                                                     \
    }
    ST_TR_STEP(8) ST_TR_STEP(4) ST_TR_STEP(2) ST_TR_STEP(1)
#undef ST_TR_STEP
    return v[0] + __shfl_xor_sync(0xffffffffu, v[0], 16);
}

// How the fibres of a warp (one per lane, consecutive rows) fall into runs of equal i.
struct WarpRuns {
    unsigned heads;      // lanes that start a run
    unsigned vmask;      // lanes that hold a fibre
};
__device__ __forceinline__ WarpRuns warp_runs(bool valid, int gi32, int lane)
{
    WarpRuns w;
    const int prev = __shfl_up_sync(0xffffffffu, gi32, 1);
    w.heads = __ballot_sync(0xffffffffu, valid && (lane == 0 || prev != gi32));
    w.vmask = __ballot_sync(0xffffffffu, valid);
    return w;
}

// Writes the sums of the warp's runs for the 32 columns c0.. held in v (v[c] = C[j,c0+c] * Y[fibre,c0+c],
// zeros in lanes without a fibre) to the partial slots (unit + i).  Call with all 32 lanes.
// nslots: number of partial slots behind `part` (read by the range checks of the debug build only).
__device__ __forceinline__ void warp_store_runs(float (&v)[32], const WarpRuns &w, bool valid, int gi32, int64_t unit,
                                                int lane, float *part, int R, int c0, int64_t nslots)
{
    if (w.heads == 0u) return;                 // no fibre in this warp
    if (w.heads == 1u) {                       // one run: the whole warp
        const float sum = warp_transpose_sum32(v, lane);
        const int64_t slot = unit + __shfl_sync(0xffffffffu, gi32, 0);
        if (ST_BOUNDS_OK(slot, nslots, 5)) part[slot * R + c0 + lane] = sum;
    } else if (w.heads == w.vmask) {           // every fibre is a run of its own
        if (valid && ST_BOUNDS_OK(unit + gi32, nslots, 5)) {
            float4 *dst = reinterpret_cast<float4 *>(part + (unit + gi32) * R + c0);
#pragma unroll
            for (int e = 0; e < 8; ++e) dst[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
        }
    } else {                                   // several runs: one masked reduction per run
        unsigned h = w.heads;
        while (h) {
            const int s0 = __ffs(h) - 1;
            h &= h - 1;
            const int s1 = h ? __ffs(h) - 1 : 32;
            const bool in = lane >= s0 && lane < s1;
            float t[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) t[e] = in ? v[e] : 0.f;
            const float sum = warp_transpose_sum32(t, lane);
            const int64_t slot = unit + __shfl_sync(0xffffffffu, gi32, s0);
            if (ST_BOUNDS_OK(slot, nslots, 5)) part[slot * R + c0 + lane] = sum;
        }
    }
}

// The same for the 16 columns c0.. held in v.
__device__ __forceinline__ void warp_store_runs16(float (&v)[16], const WarpRuns &w, bool valid, int gi32, int64_t unit,
                                                  int lane, float *part, int R, int c0, int64_t nslots)
{
    if (w.heads == 0u) return;
    if (w.heads == 1u) {
        const float sum = warp_transpose_sum16(v, lane);
        const int gi0 = __shfl_sync(0xffffffffu, gi32, 0);
        if (lane < 16 && ST_BOUNDS_OK(unit + gi0, nslots, 5)) part[(unit + gi0) * R + c0 + lane] = sum;
    } else if (w.heads == w.vmask) {
        if (valid && ST_BOUNDS_OK(unit + gi32, nslots, 5)) {
            float4 *dst = reinterpret_cast<float4 *>(part + (unit + gi32) * R + c0);
#pragma unroll
            for (int e = 0; e < 4; ++e) dst[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
        }
    } else {
        unsigned h = w.heads;
        while (h) {
            const int s0 = __ffs(h) - 1;
            h &= h - 1;
            const int s1 = h ? __ffs(h) - 1 : 32;
            const bool in = lane >= s0 && lane < s1;
            float t[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) t[e] = in ? v[e] : 0.f;
            const float sum = warp_transpose_sum16(t, lane);
            const int gis = __shfl_sync(0xffffffffu, gi32, s0);
            if (lane < 16 && ST_BOUNDS_OK(unit + gis, nslots, 5)) part[(unit + gis) * R + c0 + lane] = sum;
        }
    }
}
#endif

}  // namespace st
