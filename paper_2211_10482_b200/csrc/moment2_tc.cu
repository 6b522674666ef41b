// st_sym_moment2, tensor-core path: out[p(i,j)] = sum_n X[n,i] X[n,j], X in bfloat16, fp32
// accumulation (Section 3, M1; the outer product summed over samples is a symmetric
// rank-N update, i.e. a triangular tile GEMM X^T X).
//
// Output tiles are 128 rows (i) x 256 columns (j).  Only tiles that contain an entry with
// i <= j are launched; tiles wholly below the diagonal are never issued, and of a tile whose
// left 128 columns lie below the diagonal only the right 128 x 128 half is issued (N = 128).
// The sample range of every tile is split over the same number of blocks, so that the blocks of
// one sample range run in step and share X through L2; every block accumulates its tile
// over its samples in tensor memory and keeps an fp32 partial tile; a second kernel adds
// the partials of a tile in fixed order and writes the packed upper triangle.
//
// The tensor core adds into its fp32 accumulator without round-to-nearest, so a chain of
// many thousands of accumulating MMAs drifts low (measured: -7.7e-4 relative on all-positive
// sums of 150k terms).  The chain is therefore cut every FLUSH_CHUNKS stages: the MMAs switch
// to the second accumulator in tensor memory while the epilogue warps add the finished one
// into the block's partial tile with ordinary fp32 additions.
//
// Both operands of X^T X are "MN-major" for the tensor core: X is [N, d] row-major, so the
// output index (i or j) is contiguous and the reduction index n strides by a row.  TMA
// loads boxes of 64 columns x 64 rows with the 128-byte swizzle, which is exactly the
// canonical MN-major layout of tcgen05 (8 rows x 128 bytes per swizzle atom).  When the
// 128 columns of the A panel lie inside the columns of the B panel (tiles on the diagonal)
// only the B panel is loaded and A aliases it.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (TMEM -> registers -> global), one per 32-lane quarter of TMEM.
#include "tc_common.cuh"
#include "st_index.cuh"
#include <cuda_bf16.h>

namespace st {

namespace m2tc {
constexpr int BM = 128, BN = 256;
constexpr int KROWS = 64;                       // sample rows per pipeline stage
constexpr int BOXC = 64;                        // columns per TMA box (128 bytes of bf16)
constexpr int BOX_BYTES = BOXC * KROWS * 2;     // 8 KiB
constexpr int NBOX_A = BM / BOXC, NBOX_B = BN / BOXC;
constexpr int STAGE_BYTES = (NBOX_A + NBOX_B) * BOX_BYTES;   // 48 KiB
constexpr int STAGES = 4;
constexpr int THREADS = 192;
constexpr int MAX_TILES = 288;
constexpr int MAX_BLOCKS = 448;
constexpr uint32_t TMEM_COLS = 512;              // two 128 x 256 fp32 accumulators
constexpr int FLUSH_CHUNKS = 64;                 // stages (of 64 samples) per accumulator phase
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;

struct TileTable {
    int ntiles, nblocks;
    unsigned short tm[MAX_TILES];          // tile row (units of 128)
    unsigned short tn[MAX_TILES];          // tile column (units of 256)
    unsigned char half[MAX_TILES];         // 1: only columns 128..255 of the tile are issued
    unsigned short nsplit[MAX_TILES];      // blocks that share the samples of this tile
    unsigned short first_block[MAX_TILES];
    unsigned short blk_tile[MAX_BLOCKS];   // block -> tile
};
}  // namespace m2tc

__global__ void __launch_bounds__(m2tc::THREADS, 1)
moment2_tc_kernel(const __grid_constant__ CUtensorMap tmap, float *__restrict__ partials, unsigned *status,
                  int chunks_total, const __grid_constant__ m2tc::TileTable tab)
{
    using namespace m2tc;
    using namespace tc;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + (size_t)STAGES * STAGE_BYTES);
    uint64_t *full = bars, *empty = bars + STAGES, *acc_full = bars + 2 * STAGES, *acc_empty = bars + 2 * STAGES + 2;
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * STAGES + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = tab.blk_tile[blockIdx.x];
    const int split = (int)blockIdx.x - tab.first_block[tile];
    const int nsplit = tab.nsplit[tile];
    const int tm = tab.tm[tile], tn = tab.tn[tile];
    const bool half = tab.half[tile] != 0;
    const bool a_in_b = (tm >> 1) == tn;
    const int chunks_per_split = (chunks_total + nsplit - 1) / nsplit;
    const int c_begin = split * chunks_per_split;
    int c_end = c_begin + chunks_per_split;
    if (c_end > chunks_total) c_end = chunks_total;
    const int nchunks = c_end > c_begin ? c_end - c_begin : 0;
    const int nphases = (nchunks + FLUSH_CHUNKS - 1) / FLUSH_CHUNKS;
    const int ncols = half ? BN / 2 : BN;                 // issued columns of the tile
    const int b_box0 = half ? NBOX_B / 2 : 0;             // first B box that is loaded

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
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
            status[kWsStatusWord] = 0;
            status[kWsDetailWord] = 0;
        }
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer
        if (elect_one()) {
            prefetch_tmap(&tmap);
            const int nb_boxes = NBOX_B - b_box0;
            const uint32_t tx = (uint32_t)((a_in_b ? nb_boxes : NBOX_A + nb_boxes) * BOX_BYTES);
            for (int c = 0; c < nchunks; ++c) {
                const int s = c % STAGES;
                if (c >= STAGES && !mbar_wait(&empty[s], ((c / STAGES) - 1) & 1, abort_flag, status, 1)) break;
                unsigned char *st_base = smem + (size_t)s * STAGE_BYTES;
                mbar_expect_tx(&full[s], tx);
                const int row = (c_begin + c) * KROWS;
                for (int b = b_box0; b < NBOX_B; ++b)
                    tma_load_2d(st_base + b * BOX_BYTES, &tmap, &full[s], tn * BN + b * BOXC, row);
                if (!a_in_b)
                    for (int b = 0; b < NBOX_A; ++b)
                        tma_load_2d(st_base + (NBOX_B + b) * BOX_BYTES, &tmap, &full[s], tm * BM + b * BOXC, row);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (elect_one()) {
            const uint32_t idesc = half ? make_idesc(1, 1, 1, BM, BN / 2) : make_idesc(1, 1, 1, BM, BN);
            const uint32_t a_off = a_in_b ? (uint32_t)((tm & 1) * NBOX_A * BOX_BYTES) : (uint32_t)(NBOX_B * BOX_BYTES);
            const uint32_t b_off = (uint32_t)(b_box0 * BOX_BYTES);
            // descriptors of k-step 0 of every stage; a k-step of 16 rows advances the start
            // address by two swizzle atoms (2048 bytes = 128 in descriptor units)
            const uint32_t sb0 = smem_u32(smem);
            const uint64_t adesc_base = make_smem_desc(sb0 + a_off, BOX_BYTES, 1024);
            const uint64_t bdesc_base = make_smem_desc(sb0 + b_off, BOX_BYTES, 1024);
            bool ok = true;
            int c = 0;
            for (int ph = 0; ph < nphases && ok; ++ph) {
                const int buf = ph & 1;
                if (ph >= 2 && !mbar_wait(&acc_empty[buf], (uint32_t)(((ph >> 1) - 1) & 1), abort_flag, status, 4)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                const int ce = (c + FLUSH_CHUNKS < nchunks) ? c + FLUSH_CHUNKS : nchunks;
                uint32_t accumulate = 0;
                for (; c < ce; ++c) {
                    const int s = c % STAGES;
                    if (!mbar_wait(&full[s], (c / STAGES) & 1, abort_flag, status, 2)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t ad = adesc_base + (uint64_t)(s * (STAGE_BYTES >> 4));
                    const uint64_t bd = bdesc_base + (uint64_t)(s * (STAGE_BYTES >> 4));
#pragma unroll
                    for (int k = 0; k < KROWS / 16; ++k) {
                        mma_bf16(d_tmem, ad + (uint64_t)(k * 128), bd + (uint64_t)(k * 128), idesc, accumulate);
                        accumulate = 1;
                    }
                    tc_commit(&empty[s]);          // frees the stage when these MMAs have read it
                }
                tc_commit(&acc_full[buf]);         // this accumulator phase is complete
            }
        }
    } else {
        // ---------------- epilogue: TMEM lanes 32q..32q+31 belong to warp q = warp % 4
        const int q = warp & 3;
        float *dst = partials + ((size_t)blockIdx.x * BM + (q * 32 + lane)) * BN;
        if (nphases == 0) {
            for (int c0 = 0; c0 < ncols; c0 += 4) *reinterpret_cast<float4 *>(dst + c0) = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int ph = 0; ph < nphases; ++ph) {
            const int buf = ph & 1;
            if (!mbar_wait(&acc_full[buf], (uint32_t)((ph >> 1) & 1), abort_flag, status, 3)) break;
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < ncols; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), r);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    float4 v = make_float4(__uint_as_float(r[e]), __uint_as_float(r[e + 1]), __uint_as_float(r[e + 2]),
                                           __uint_as_float(r[e + 3]));
                    float4 *p = reinterpret_cast<float4 *>(dst + c0 + e);
                    if (ph > 0) {
                        const float4 o = *p;        // written by this same thread in the previous phase
                        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                    }
                    *p = v;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// out[p(i,j)] = sum over splits of the partial tiles, i <= j only.
__global__ void __launch_bounds__(256)
moment2_tc_reduce_kernel(const float *__restrict__ partials, float *__restrict__ out, int d,
                         const __grid_constant__ m2tc::TileTable tab)
{
    using namespace m2tc;
    const int tile = blockIdx.x;
    const int tm = tab.tm[tile], tn = tab.tn[tile], nsplit = tab.nsplit[tile];
    const int ncols = tab.half[tile] ? BN / 2 : BN;
    const int col0 = tn * BN + (tab.half[tile] ? BN / 2 : 0);
    const float *base = partials + (size_t)tab.first_block[tile] * (BM * BN);
    for (int e = blockIdx.y * 256 + threadIdx.x; e < BM * BN; e += gridDim.y * 256) {
        const int r = e / BN, c = e - r * BN;
        const int gi = tm * BM + r, gj = col0 + c;
        if (c < ncols && gi < d && gj < d && gi <= gj) {
            float s = 0.f;
            for (int k0 = 0; k0 < nsplit; k0 += 8) {
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = (k0 + u < nsplit) ? __ldcg(&base[(size_t)(k0 + u) * (BM * BN) + e]) : 0.f;
#pragma unroll
                for (int u = 0; u < 8; ++u) s += v[u];
            }
            if (ST_BOUNDS_OK(tri_encode(d, gi, gj), tri_rows(d), 2)) out[tri_encode(d, gi, gj)] = s;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Two-block variant (d >= 512): a cluster of two blocks owns a 256 x 256 tile.  Block r stages
// columns 256*TM+128r.. (its 128 rows of the A operand) and columns 256*TN+128r.. (its half of
// the B operand); on diagonal tiles the two coincide and are loaded once.  The leader block
// issues one MMA of M = 256, N = 256 for the pair; each block keeps the accumulator of its 128
// rows in its own tensor memory.  Per MMA cycle a block now fetches a third less from L2 than in
// the one-block kernel (whose tensor pipe idled ~30% of the time waiting for operands).  Four
// stages of 64 samples are the measured optimum: with 6 or 7 stages the blocks of a sample range
// drift apart, share less of X in L2 and the kernel gets 5-12% slower; with 3 it starves.
//
// The same kernel reads an fp32 X as TF32 (template argument): the tensor core takes the upper 19 bits of every
// fp32 word, so the boxes are 32 columns (128 bytes) wide, a stage holds 32 samples and an MMA spans 8 of them;
// the bytes per stage, the MMAs per stage and everything after the accumulator are the same.  An MN-major
// operand of 32-bit elements has one legal shared-memory form, the 128-byte swizzle of 32-byte units, which
// the copies write (tensor-map swizzle "128B, atom 32B") and the descriptors name.
namespace m2tc2 {
constexpr int BM = 256, BN = 256;               // tile of the pair
constexpr int HALF = 128;                       // rows / B columns staged per block
constexpr int STAGE_BYTES = 32768;              // HALF columns of A and of B over the sample rows of one stage
constexpr int STAGES = 4;
constexpr int THREADS = 192;
constexpr int MAX_TILES = 160;
constexpr uint32_t TMEM_COLS = 512;
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 + 256;
template <bool TF32> struct Shape {
    static constexpr int ELEM = TF32 ? 4 : 2;
    static constexpr int KROWS = TF32 ? 32 : 64;            // sample rows per stage
    static constexpr int KMMA = TF32 ? 8 : 16;              // sample rows per MMA
    static constexpr int BOXC = 128 / ELEM;                 // columns per TMA box (128 bytes)
    static constexpr int BOX_BYTES = 128 * KROWS;
    static constexpr int NBOX = HALF / BOXC;                // boxes per operand per block
    static constexpr int FLUSH_CHUNKS = 4096 / KROWS;       // 4096 samples (256 or 512 MMAs) per accumulator phase
    static_assert(2 * NBOX * BOX_BYTES == STAGE_BYTES, "stage size");
};

struct TileTable {
    int ntiles, nsplit;
    unsigned char tm[MAX_TILES];   // units of 256
    unsigned char tn[MAX_TILES];
};
}  // namespace m2tc2

template <bool TF32>
__global__ void __launch_bounds__(m2tc2::THREADS, 1)
moment2_tc_pair_kernel(const __grid_constant__ CUtensorMap tmap, float *__restrict__ partials, unsigned *status,
                       int chunks_total, const __grid_constant__ m2tc2::TileTable tab, int seg_chunks, int lo_row0)
{
    // seg_chunks > 0: the rows of the tensor are [hi part of X; lo part of X] (lo_row0 = first row of the lo part)
    // and the sample loop runs over three segments of seg_chunks stages: A and B from hi, A from hi and B from lo,
    // A from lo and B from hi -- the sum is hi^T hi + hi^T lo + lo^T hi, symmetric, so the tiles stay the upper ones.
    using namespace m2tc2;
    using namespace tc;
    using S = Shape<TF32>;
    constexpr int KROWS = S::KROWS, BOXC = S::BOXC, BOX_BYTES = S::BOX_BYTES, NBOX = S::NBOX, FLUSH_CHUNKS = S::FLUSH_CHUNKS;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + (size_t)STAGES * STAGE_BYTES);
    uint64_t *full = bars, *empty = bars + STAGES, *acc_full = bars + 2 * STAGES, *acc_empty = bars + 2 * STAGES + 2;
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * STAGES + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = leader
    const int cluster = blockIdx.x >> 1;
    const int tile = cluster / tab.nsplit, split = cluster - tile * tab.nsplit;
    const int tm = tab.tm[tile], tn = tab.tn[tile];
    const bool diag = (tm == tn) && seg_chunks == 0;    // A columns == B columns (and rows) in every block: one load serves both
    const int chunks_per_split = (chunks_total + tab.nsplit - 1) / tab.nsplit;
    const int c_begin = split * chunks_per_split;
    int c_end = c_begin + chunks_per_split;
    if (c_end > chunks_total) c_end = chunks_total;
    const int nchunks = c_end > c_begin ? c_end - c_begin : 0;
    const int nphases = (nchunks + FLUSH_CHUNKS - 1) / FLUSH_CHUNKS;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);          // leader's producer arrives once and announces the bytes of both blocks
            mbar_init(&empty[s], 1);         // one commit per use, delivered to both blocks
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 8);     // four epilogue warps in each of the two blocks (leader's copy is used)
        }
        *abort_flag = 0;
        if (blockIdx.x == 0) {
            // the status words are cleared here instead of by a separate memset; a time-out
            // report can only be written 2^24 failed polls later
            status[kWsStatusWord] = 0;
            status[kWsDetailWord] = 0;
        }
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // both blocks' barriers exist before anything is signalled across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer (both blocks): own boxes, completion counted on the leader's barrier
        if (elect_one()) {
            prefetch_tmap(&tmap);
            const uint32_t own_tx = (uint32_t)((diag ? NBOX : 2 * NBOX) * BOX_BYTES);
            for (int c = 0; c < nchunks; ++c) {
                const int s = c % STAGES;
                if (c >= STAGES && !mbar_wait(&empty[s], ((c / STAGES) - 1) & 1, abort_flag, status, 1)) break;
                unsigned char *st_base = smem + (size_t)s * STAGE_BYTES;
                if (rank == 0) mbar_expect_tx(&full[s], 2 * own_tx);
                const uint32_t bar = map_to_cta(smem_u32(&full[s]), 0);
                int row_a = (c_begin + c) * KROWS, row_b = row_a;
                if (seg_chunks > 0) {
                    const int gc = c_begin + c, seg = gc / seg_chunks;
                    row_a = row_b = (gc - seg * seg_chunks) * KROWS;
                    if (seg == 1) row_b += lo_row0;
                    if (seg == 2) row_a += lo_row0;
                }
                for (int b = 0; b < NBOX; ++b)          // B half (and A on diagonal tiles)
                    tma_load_2d_pair(st_base + b * BOX_BYTES, &tmap, bar, tn * BN + (int)rank * HALF + b * BOXC, row_b);
                if (!diag)
                    for (int b = 0; b < NBOX; ++b)      // A rows of this block
                        tma_load_2d_pair(st_base + (NBOX + b) * BOX_BYTES, &tmap, bar, tm * BM + (int)rank * HALF + b * BOXC, row_a);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader only)
        if (rank == 0 && elect_one()) {
            constexpr uint32_t idesc = make_idesc(TF32 ? 2 : 1, 1, 1, BM, BN);
            const uint32_t a_off = diag ? 0u : (uint32_t)(NBOX * BOX_BYTES);
            const uint32_t sb0 = smem_u32(smem);
            // bf16: groups of 8 sample rows, 16-byte swizzle units; fp32 read as TF32: groups of 4, 32-byte units
            const uint64_t adesc_base = make_smem_desc(sb0 + a_off, BOX_BYTES, TF32 ? 512 : 1024, TF32 ? 1 : 2);
            const uint64_t bdesc_base = make_smem_desc(sb0, BOX_BYTES, TF32 ? 512 : 1024, TF32 ? 1 : 2);
            bool ok = true;
            int c = 0;
            for (int ph = 0; ph < nphases && ok; ++ph) {
                const int buf = ph & 1;
                if (ph >= 2 && !mbar_wait(&acc_empty[buf], (uint32_t)(((ph >> 1) - 1) & 1), abort_flag, status, 4)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                const int ce = (c + FLUSH_CHUNKS < nchunks) ? c + FLUSH_CHUNKS : nchunks;
                uint32_t accumulate = 0;
                for (; c < ce; ++c) {
                    const int s = c % STAGES;
                    if (!mbar_wait(&full[s], (c / STAGES) & 1, abort_flag, status, 2)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t ad = adesc_base + (uint64_t)(s * (STAGE_BYTES >> 4));
                    const uint64_t bd = bdesc_base + (uint64_t)(s * (STAGE_BYTES >> 4));
#pragma unroll
                    for (int k = 0; k < KROWS / S::KMMA; ++k) {
                        // one MMA spans KMMA sample rows of 128 bytes: 2048 bytes (bf16) or 1024 bytes (TF32) further on
                        constexpr int STEP = S::KMMA * 128 / 16;
                        if (TF32) mma_tf32_pair(d_tmem, ad + (uint64_t)(k * STEP), bd + (uint64_t)(k * STEP), idesc, accumulate);
                        else mma_bf16_pair(d_tmem, ad + (uint64_t)(k * STEP), bd + (uint64_t)(k * STEP), idesc, accumulate);
                        accumulate = 1;
                    }
                    tc_commit_pair(&empty[s]);
                }
                tc_commit_pair(&acc_full[buf]);
            }
        }
    } else {
        // ---------------- epilogue (both blocks): own 128 rows of the tile
        const int q = warp & 3;
        float *dst = partials + ((size_t)blockIdx.x * HALF + (q * 32 + lane)) * BN;
        const uint32_t leader_acc_empty0 = map_to_cta(smem_u32(&acc_empty[0]), 0);
        if (nphases == 0) {
            for (int c0 = 0; c0 < BN; c0 += 4) *reinterpret_cast<float4 *>(dst + c0) = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int ph = 0; ph < nphases; ++ph) {
            const int buf = ph & 1;
            if (!mbar_wait(&acc_full[buf], (uint32_t)((ph >> 1) & 1), abort_flag, status, 3)) break;
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), r);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    float4 v = make_float4(__uint_as_float(r[e]), __uint_as_float(r[e + 1]), __uint_as_float(r[e + 2]),
                                           __uint_as_float(r[e + 3]));
                    float4 *p = reinterpret_cast<float4 *>(dst + c0 + e);
                    if (ph > 0) {
                        const float4 o = *p;
                        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                    }
                    *p = v;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_acc_empty0 + (uint32_t)(buf * sizeof(uint64_t)));
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // no block leaves while its peer may still signal it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

__global__ void __launch_bounds__(256)
moment2_tc_pair_reduce_kernel(const float *__restrict__ partials, float *__restrict__ out, int d,
                              const __grid_constant__ m2tc2::TileTable tab)
{
    using namespace m2tc2;
    const int tile = blockIdx.x;
    const int tm = tab.tm[tile], tn = tab.tn[tile], nsplit = tab.nsplit;
    // partial of (tile, split, block r) lives in slot 2*(tile*nsplit+split)+r, a [128][256] array
    for (int e = blockIdx.y * 256 + threadIdx.x; e < BM * BN; e += gridDim.y * 256) {
        const int r = e / BN, c = e - r * BN;
        const int gi = tm * BM + r, gj = tn * BN + c;
        if (gi < d && gj < d && gi <= gj) {
            const float *base = partials + ((size_t)(2 * tile * nsplit + (r >> 7)) * HALF + (r & 127)) * BN + c;
            const size_t stride = (size_t)2 * HALF * BN;
            float s = 0.f;
            for (int k0 = 0; k0 < nsplit; k0 += 8) {
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = (k0 + u < nsplit) ? __ldcg(base + (size_t)(k0 + u) * stride) : 0.f;
#pragma unroll
                for (int u = 0; u < 8; ++u) s += v[u];
            }
            if (ST_BOUNDS_OK(tri_encode(d, gi, gj), tri_rows(d), 2)) out[tri_encode(d, gi, gj)] = s;
        }
    }
}

struct M2Tc2Plan {
    m2tc2::TileTable tab;
    int chunks_total;
    size_t partial_bytes;
    bool ok;
};

static M2Tc2Plan m2tc2_plan(int64_t N, int64_t d, unsigned flags, bool tf32 = false, int segments = 1)
{
    using namespace m2tc2;
    const int KROWS = tf32 ? Shape<true>::KROWS : Shape<false>::KROWS;
    M2Tc2Plan p;
    p.ok = false;
    const bool dense = (flags & ST_FLAG_DENSE_CONTROL) != 0;
    const int nt = (int)((d + BM - 1) / BM);
    int n = 0;
    for (int tn = 0; tn < nt; ++tn)
        for (int tm = 0; tm < nt; ++tm) {
            if (tm > tn && !dense) continue;
            if (n >= MAX_TILES) return p;
            p.tab.tm[n] = (unsigned char)tm;
            p.tab.tn[n] = (unsigned char)tn;
            ++n;
        }
    for (int i = n; i < MAX_TILES; ++i) p.tab.tm[i] = p.tab.tn[i] = 0;
    p.tab.ntiles = n;
    const int64_t chunks = segments * ((N + KROWS - 1) / KROWS);
    if (chunks > (int64_t(1) << 30)) return p;
    p.chunks_total = (int)chunks;
    int64_t per = (sm_count_or_default() / 2) / n;   // clusters per tile: equal, so that sample ranges run in step
    if (per < 1) per = 1;
    if (per > chunks) per = chunks;
    p.tab.nsplit = (int)per;
    p.partial_bytes = (size_t)2 * n * per * HALF * BN * sizeof(float);
    p.ok = true;
    return p;
}

static bool m2_use_pair(int64_t d) { return d >= 512; }

struct M2TcPlan {
    m2tc::TileTable tab;
    int chunks_total;
    size_t partial_bytes;
    bool ok;
};

static M2TcPlan m2tc_plan(int64_t N, int64_t d, unsigned flags)
{
    using namespace m2tc;
    M2TcPlan p;
    p.ok = false;
    const bool dense = (flags & ST_FLAG_DENSE_CONTROL) != 0;
    const int ntm = (int)((d + BM - 1) / BM), ntn = (int)((d + BN - 1) / BN);
    int n = 0;
    for (int tn = 0; tn < ntn; ++tn)
        for (int tm = 0; tm < ntm; ++tm) {
            const bool touches_upper = (int64_t)tm * BM <= (int64_t)tn * BN + BN - 1;
            if (!touches_upper && !dense) continue;
            if (n >= MAX_TILES) return p;
            p.tab.tm[n] = (unsigned short)tm;
            p.tab.tn[n] = (unsigned short)tn;
            // rows 128*tm.. against columns 256*tn..256*tn+127: all below the diagonal when tm == 2*tn+1
            const bool half = !dense && tm == 2 * tn + 1;
            p.tab.half[n] = half ? 1 : 0;
            ++n;
        }
    p.tab.ntiles = n;
    for (int i = n; i < MAX_TILES; ++i) {
        p.tab.tm[i] = p.tab.tn[i] = p.tab.nsplit[i] = p.tab.first_block[i] = 0;
        p.tab.half[i] = 0;
    }
    const int64_t chunks = (N + KROWS - 1) / KROWS;
    if (chunks > (int64_t(1) << 30)) return p;
    p.chunks_total = (int)chunks;
    // splits: the same number for every tile.  Blocks that work on the same sample range then run
    // in step and share the rows of X through L2 (X is read from HBM once); unequal splits were
    // measured 12-20% slower although they use more SMs.
    const int sms = sm_count_or_default();
    int64_t per = sms / n;
    if (per < 1) per = 1;
    if (per > chunks) per = chunks;
    for (int i = 0; i < n; ++i) p.tab.nsplit[i] = (unsigned short)per;
    const int blocks = (int)per * n;
    if (blocks > MAX_BLOCKS) return p;
    int b = 0;
    for (int i = 0; i < n; ++i) {
        p.tab.first_block[i] = (unsigned short)b;
        for (int s = 0; s < p.tab.nsplit[i]; ++s) p.tab.blk_tile[b++] = (unsigned short)i;
    }
    for (int i = b; i < MAX_BLOCKS; ++i) p.tab.blk_tile[i] = 0;
    p.tab.nblocks = b;
    p.partial_bytes = (size_t)b * BM * BN * sizeof(float);
    p.ok = true;
    return p;
}

// Launches the pair kernel and the sum of its partial tiles.
template <bool TF32>
static st_status m2_pair_launch(const M2Tc2Plan &q, const void *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws,
                                cudaStream_t stream, size_t part_off = kWsHeaderBytes, int seg_chunks = 0, int lo_row0 = 0)
{
    using S = m2tc2::Shape<TF32>;
    CUtensorMap tm2;
    if (!tc::make_tmap_2d(&tm2, TF32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, X, (uint64_t)N,
                          (uint64_t)d, (uint64_t)ldx * S::ELEM, S::BOXC, S::KROWS,
                          TF32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B))
        return ST_ERR_CUDA;
    float *part2 = (float *)((unsigned char *)ws + part_off);
    if (!ensure_dynamic_smem(moment2_tc_pair_kernel<TF32>, m2tc2::SMEM_BYTES)) return ST_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * q.tab.ntiles * q.tab.nsplit);
    cfg.blockDim = dim3(m2tc2::THREADS);
    cfg.dynamicSmemBytes = m2tc2::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, moment2_tc_pair_kernel<TF32>, tm2, part2, (unsigned *)ws, q.chunks_total, q.tab, seg_chunks,
                           lo_row0) != cudaSuccess) {
        (void)cudaGetLastError();
        return ST_ERR_CUDA;
    }
    moment2_tc_pair_reduce_kernel<<<dim3(q.tab.ntiles, 64), 256, 0, stream>>>(part2, out, (int)d, q.tab);
    return launch_status();
}

// fp32 input read as TF32 by the pair kernel (any d that is a multiple of 4: tiles beyond d are zero-filled by the copies)
size_t moment2_tf32_tc_workspace(int64_t N, int64_t d, unsigned flags)
{
    if (N <= 0 || d <= 0 || d % 4 != 0 || d > 4096 || N > (int64_t(1) << 31) - 64) return 0;
    const M2Tc2Plan q = m2tc2_plan(N, d, flags, true);
    return q.ok ? kWsHeaderBytes + q.partial_bytes : 0;
}

st_status moment2_tf32_tc(const void *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                          unsigned flags, cudaStream_t stream)
{
    if (d % 4 != 0 || ldx % 4 != 0) return ST_ERR_ALIGN;
    if (d > 4096 || N > (int64_t(1) << 31) - 64) return ST_ERR_UNSUPPORTED;
    const M2Tc2Plan q = m2tc2_plan(N, d, flags, true);
    if (!q.ok) return ST_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < kWsHeaderBytes + q.partial_bytes) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    return m2_pair_launch<true>(q, X, N, d, ldx, out, ws, stream);
}

// ---------------------------------------------------------------------------------------------
// fp32 input at the fp32 tolerance on the tensor cores (ST_FLAG_TC_SPLIT): every x is written once as
// hi = bf16(x) and lo = bf16(x - hi) (x - hi - lo is below 2^-16 |x|), and the pair kernel adds
// hi^T hi + hi^T lo + lo^T hi over three passes of the samples (lo^T lo is below 2^-16 of the result).
// The split pass reads X once and writes the same number of bytes; the three passes then run at the bf16 rate.
__global__ void __launch_bounds__(256)
moment2_split_rows_kernel(const float *__restrict__ X, int64_t N, int64_t Np, int d, int64_t ldx, __nv_bfloat16 *__restrict__ Z)
{
    // Z: [2 Np, d]; rows 0 .. Np-1 hi, rows Np .. 2Np-1 lo; rows N .. Np-1 of either part are zero
    const int64_t quads = (int64_t)Np * (d / 4);
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < quads; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t n = e / (d / 4);
        const int c = (int)(e - n * (d / 4)) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (n < N) x = __ldcs(reinterpret_cast<const float4 *>(X + n * ldx + c));
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(x.x, x.y), h1 = __floats2bfloat162_rn(x.z, x.w);
        const float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
        const __nv_bfloat162 l0 = __floats2bfloat162_rn(x.x - f0.x, x.y - f0.y), l1 = __floats2bfloat162_rn(x.z - f1.x, x.w - f1.y);
        *reinterpret_cast<uint2 *>(Z + n * d + c) =
            make_uint2(*reinterpret_cast<const uint32_t *>(&h0), *reinterpret_cast<const uint32_t *>(&h1));
        *reinterpret_cast<uint2 *>(Z + (Np + n) * d + c) =
            make_uint2(*reinterpret_cast<const uint32_t *>(&l0), *reinterpret_cast<const uint32_t *>(&l1));
    }
}

struct M2SplitPlan {
    M2Tc2Plan q;
    int64_t Np;
    size_t z_off, part_off, total;
    bool ok;
};

static M2SplitPlan m2_split_plan(int64_t N, int64_t d, unsigned flags)
{
    M2SplitPlan p{};
    p.ok = false;
    if (N <= 0 || d <= 0 || d % 8 != 0 || d > 4096 || N > (int64_t(1) << 29)) return p;
    const int KROWS = m2tc2::Shape<false>::KROWS;
    p.Np = (N + KROWS - 1) / KROWS * KROWS;
    p.q = m2tc2_plan(N, d, flags, false, 3);
    if (!p.q.ok) return p;
    p.z_off = kWsHeaderBytes;
    p.part_off = round_up(p.z_off + (size_t)2 * p.Np * d * sizeof(__nv_bfloat16), 256);
    p.total = p.part_off + p.q.partial_bytes;
    p.ok = true;
    return p;
}

// The three-segment product for a caller that has written the parts itself (the fourth moment makes its pair
// features straight into this form): Z = [hi rows; lo rows], each part N rounded up to 64 rows with zero rows
// at the end, d columns, bf16.
int64_t moment2_split_part_rows(int64_t N) { return (N + 63) / 64 * 64; }

size_t moment2_split_parts_workspace(int64_t N, int64_t d)
{
    const M2SplitPlan p = m2_split_plan(N, d, 0);
    return p.ok ? kWsHeaderBytes + p.q.partial_bytes : 0;
}

st_status moment2_split_tc_parts(const void *Z, int64_t N, int64_t d, float *out, void *ws, size_t ws_bytes, cudaStream_t stream)
{
    const M2SplitPlan p = m2_split_plan(N, d, 0);
    if (!p.ok) return ST_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < kWsHeaderBytes + p.q.partial_bytes) return ST_ERR_WORKSPACE;
    if (!aligned256(ws) || !aligned16(Z)) return ST_ERR_ALIGN;
    return m2_pair_launch<false>(p.q, Z, 2 * p.Np, d, d, out, ws, stream, kWsHeaderBytes, p.q.chunks_total / 3, (int)p.Np);
}

size_t moment2_split_tc_workspace(int64_t N, int64_t d, unsigned flags)
{
    const M2SplitPlan p = m2_split_plan(N, d, flags);
    return p.ok ? p.total : 0;
}

st_status moment2_split_tc(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                           unsigned flags, cudaStream_t stream)
{
    if (d % 8 != 0 || ldx % 4 != 0) return ST_ERR_ALIGN;
    const M2SplitPlan p = m2_split_plan(N, d, flags);
    if (!p.ok) return ST_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < p.total) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    __nv_bfloat16 *Z = (__nv_bfloat16 *)((unsigned char *)ws + p.z_off);
    const int64_t quads = p.Np * (d / 4);
    const int64_t want = (quads + 255) / 256;
    const int64_t cap = (int64_t)sm_count_or_default() * 16;
    moment2_split_rows_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, stream>>>(X, N, p.Np, (int)d, ldx, Z);
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    return m2_pair_launch<false>(p.q, Z, 2 * p.Np, d, d, out, ws, stream, p.part_off, p.q.chunks_total / 3, (int)p.Np);
}

size_t moment2_bf16_tc_workspace(int64_t N, int64_t d, unsigned flags)
{
    if (N <= 0 || d <= 0 || d % 8 != 0 || d > 4096 || N > (int64_t(1) << 31) - 64) return 0;
    if (m2_use_pair(d)) {
        const M2Tc2Plan q = m2tc2_plan(N, d, flags);
        return q.ok ? kWsHeaderBytes + q.partial_bytes : 0;
    }
    const M2TcPlan p = m2tc_plan(N, d, flags);
    return p.ok ? kWsHeaderBytes + p.partial_bytes : 0;
}

st_status moment2_bf16_tc(const void *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                          unsigned flags, cudaStream_t stream)
{
    using namespace m2tc;
    if (d % 8 != 0 || ldx % 8 != 0) return ST_ERR_ALIGN;
    if (d > 4096 || N > (int64_t(1) << 31) - 64) return ST_ERR_UNSUPPORTED;
    if (m2_use_pair(d)) {
        const M2Tc2Plan q = m2tc2_plan(N, d, flags);
        if (!q.ok) return ST_ERR_UNSUPPORTED;
        if (!ws || ws_bytes < kWsHeaderBytes + q.partial_bytes) return ST_ERR_WORKSPACE;
        if (!aligned256(ws)) return ST_ERR_ALIGN;
        return m2_pair_launch<false>(q, X, N, d, ldx, out, ws, stream);
    }
    const M2TcPlan p = m2tc_plan(N, d, flags);
    if (!p.ok) return ST_ERR_UNSUPPORTED;
    const size_t need = kWsHeaderBytes + p.partial_bytes;
    if (!ws || ws_bytes < need) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    CUtensorMap tmap;
    if (!tc::make_tmap_2d(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, X, (uint64_t)N, (uint64_t)d, (uint64_t)ldx * 2,
                          BOXC, KROWS))
        return ST_ERR_CUDA;
    float *partials = (float *)((unsigned char *)ws + kWsHeaderBytes);
    if (!ensure_dynamic_smem(moment2_tc_kernel, SMEM_BYTES)) return ST_ERR_CUDA;
    moment2_tc_kernel<<<p.tab.nblocks, THREADS, SMEM_BYTES, stream>>>(tmap, partials, (unsigned *)ws, p.chunks_total,
                                                                      p.tab);
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    moment2_tc_reduce_kernel<<<dim3(p.tab.ntiles, 32), 256, 0, stream>>>(partials, out, (int)d, p.tab);
    return launch_status();
}

}  // namespace st
