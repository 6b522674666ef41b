// st_sym_moment3, tensor-core path (ST_FLAG_TC_TF32 / ST_FLAG_TC_BF16):
//     out[q(i,j,k)] = sum_n X[n,i] X[n,j] X[n,k]   for 0 <= i <= j <= k < d
// (Section 3, M2 = f (x) vec(f (x) f) summed over samples; unique elements i<=j<=k, Section 2
// "Tensor Structures").  With the pair product hoisted out of the k loop (loop-invariant code
// motion, Section 5.5) the sum is a contraction over the samples,
//     out[(i,j), k] = sum_n P[n,(i,j)] X[n,k],      P[n,(i,j)] = X[n,i] X[n,j]   (i <= j),
// that is a GEMM [pairs x samples] x [samples x d] whose left operand exists nowhere in memory.
// This kernel makes P on the fly.  A loader warp writes slices of 32 (TF32) or 64 (bf16) samples of X^T,
// rounded, into shared memory in the K-major 128-byte-swizzled form the tensor core reads (lane =
// sample).  Producer warps read their lane's x_i and x_j back from that slice, multiply the
// pairs of one tile (8 values of i x 16 values of j) and store the products, rounded to TF32, in
// the same form as the left operand of the tile's MMA.  A tile with j >= 16*JB needs the
// columns k >= 16*JB only: its MMA has N = d - 16*JB, so the part k < j of the iteration space
// is (up to that granularity) never issued, and tiles with i > j everywhere do not exist.
// Accumulators of all tiles of a block stay in tensor memory for the block's whole sample
// range; at d = 64 they need 640 columns, so two blocks ("groups") share one sample range.
//
// What bounds it: an MMA of M = 128 takes about 49 ns whatever N <= 128 is, and N <= d <= 64 here, so the
// time goes with the number of MMAs (4 per tile and slice) and with what the issuing threads do between them
// (a barrier poll behind tcgen05.mma instructions of the same thread returns only as they drain: two issuer
// warps take alternate stages), not with the tensor arithmetic.  bf16 halves the number of MMAs
// (64 samples per slice instead of 32).  Products and x_k rounded to TF32 / bf16, fp32 accumulation: 5e-3
// tolerance (bf16: for N >= 1000).
#include "tc_common.cuh"
#include "st_index.cuh"

namespace st {

st_status sum_slices_launch(const float *partials, float *out, int64_t elems, int slices, cudaStream_t stream);

namespace m3tc {
constexpr int DP = 64;                       // largest d
constexpr int TI = 8, TJ = 16;               // a tile holds the pairs (8 IB + a, 16 JB + b)
constexpr int BM = TI * TJ;                  // 128 pairs = rows of the MMA
constexpr int ROW_BYTES = 128;               // one swizzled row: 32 TF32 or 64 bf16 samples
constexpr int A_STAGE_BYTES = BM * ROW_BYTES; // 16 KiB
constexpr int B_STAGE_BYTES = DP * ROW_BYTES; // 8 KiB
constexpr int NA_MAX = 10;                   // A stages in flight (TF32: 10, bf16: 8; even: see the issuers)
constexpr int NB = 4;                        // X^T slices in flight
constexpr int X32_STAGE_BYTES = DP * 64 * 4; // bf16 path: fp32 copy of a slice of X^T for the producers (16 KiB)
constexpr int PRODUCERS = 8;                 // producer warps (also the epilogue warps)
constexpr int MMA_WARPS = 2;                 // issuer w takes the stages q = w (mod 2): while one polls, the other's MMAs run
constexpr int MMA_WARP = PRODUCERS, LOAD_WARP = PRODUCERS + MMA_WARPS;
constexpr int LOAD_WARPS = 1;                // one loader: slices are filled in order
constexpr int THREADS = 32 * (PRODUCERS + MMA_WARPS + LOAD_WARPS);
constexpr uint32_t TMEM_COLS = 512;
constexpr int MAX_GROUP_TILES = 12;
constexpr int EPI_PITCH = DP + 1;             // floats per row of the epilogue's transposing buffer
constexpr size_t smem_bytes(bool bf16)
{
    return 1024 + (size_t)(bf16 ? 8 : 10) * A_STAGE_BYTES + (size_t)NB * B_STAGE_BYTES +
           (bf16 ? (size_t)NB * X32_STAGE_BYTES : 0) + 512;
}

struct Tile {
    unsigned char ib, jb;
    unsigned short col;                      // first tensor-memory column of the tile's accumulator
};

struct Args {
    const float *X;
    float *partials;
    unsigned *status;
    int64_t N, ldx, rows_per_slice;
    int d, dcols, out_elems, vec;            // dcols = d rounded up to a multiple of 16
    int ntiles[2];
    Tile tiles[2][MAX_GROUP_TILES];
};

// byte offset of the 4-byte word `lane` (one TF32 sample, or two bf16 samples) inside a 128-byte row whose
// index has (row & 7) == m
__device__ __forceinline__ uint32_t swz(int lane, int m) { return (uint32_t)((((lane >> 2) ^ m) << 4) + ((lane & 3) << 2)); }

template <bool BF16>
__global__ void __launch_bounds__(THREADS, 1)
moment3_tc_kernel(const __grid_constant__ Args a)
{
    using namespace tc;
    constexpr int KS = BF16 ? 64 : 32;           // samples per slice
    constexpr int NA = BF16 ? 8 : 10;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *a_stage0 = smem;
    unsigned char *b_stage0 = smem + (size_t)NA * A_STAGE_BYTES;
    unsigned char *x32_stage0 = b_stage0 + (size_t)NB * B_STAGE_BYTES;   // bf16 path only
    uint64_t *bars = (uint64_t *)(x32_stage0 + (BF16 ? (size_t)NB * X32_STAGE_BYTES : 0));
    uint64_t *a_full = bars, *a_empty = bars + NA_MAX, *b_full = bars + 2 * NA_MAX, *b_empty = bars + 2 * NA_MAX + NB,
             *acc_full = bars + 2 * NA_MAX + 2 * NB;
    uint64_t *iss_sync = acc_full + 1;
    uint32_t *tmem_slot = (uint32_t *)(acc_full + 2);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int group = blockIdx.x;
    const int tg = a.ntiles[group];                          // tiles of this block
    const Tile *tiles = a.tiles[group];

    if (threadIdx.x == 0) {
        for (int s = 0; s < NA; ++s) {
            mbar_init(&a_full[s], 1);
            mbar_init(&a_empty[s], 1);
        }
        for (int s = 0; s < NB; ++s) {
            mbar_init(&b_full[s], 1);
            mbar_init(&b_empty[s], MMA_WARPS);
        }
        mbar_init(acc_full, MMA_WARPS);
        mbar_init(iss_sync, MMA_WARPS);
        *abort_flag = 0;
        if (blockIdx.x == 0 && blockIdx.y == 0) {
            a.status[kWsStatusWord] = 0;
            a.status[kWsDetailWord] = 0;
        }
        fence_barrier_init();
    }
    if (warp == MMA_WARP) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int64_t n_begin = (int64_t)blockIdx.y * a.rows_per_slice;
    int64_t n_end = n_begin + a.rows_per_slice;
    if (n_end > a.N) n_end = a.N;
    const int nslices = n_end > n_begin ? (int)((n_end - n_begin + KS - 1) / KS) : 0;
    const int64_t nstages = (int64_t)nslices * tg;

    uint32_t sw[8];
#pragma unroll
    for (int m = 0; m < 8; ++m) sw[m] = swz(lane, m);

    if (warp < PRODUCERS) {
        // ---- producers: A stage q = slice * tg + tile is made by warp q % PRODUCERS -------------
        // A wait names a phase by its parity only, so a waiter must never be two phases ahead of its
        // barrier: with stages dealt round-robin to `nprod` warps that holds when nprod <= NA (slots of
        // the A ring) and nprod <= NB * tg (stages covered by the slices of the X^T ring).
        const int nprod = min(min(PRODUCERS, NA), NB * tg);
        bool ok = true;
        for (int64_t q = warp; q < nstages && ok && warp < nprod; q += nprod) {
            const int slice = (int)(q / tg), ti = (int)(q - (int64_t)slice * tg);
            const int bs = slice % NB;
            if (!mbar_wait(&b_full[bs], (uint32_t)((slice / NB) & 1), abort_flag, a.status, 11)) break;
            // this lane's sample: x_i for the tile's 8 values of i, x_j for its 16 values of j
            const unsigned char *bst = b_stage0 + (size_t)bs * B_STAGE_BYTES;
            const Tile t = tiles[ti];
            // TF32: the rounded values of the MMA's own slice; bf16: the fp32 copy, two samples per lane,
            // so that every product is rounded once
            float xi[TI][BF16 ? 2 : 1], xj[TJ][BF16 ? 2 : 1];
            if (BF16) {
                const unsigned char *xst = x32_stage0 + (size_t)bs * X32_STAGE_BYTES + 8 * lane;
#pragma unroll
                for (int e = 0; e < TI; ++e) {
                    const float2 v = *reinterpret_cast<const float2 *>(xst + (TI * t.ib + e) * 256);
                    xi[e][0] = v.x; xi[e][BF16 ? 1 : 0] = v.y;
                }
#pragma unroll
                for (int e = 0; e < TJ; ++e) {
                    const float2 v = *reinterpret_cast<const float2 *>(xst + (TJ * t.jb + e) * 256);
                    xj[e][0] = v.x; xj[e][BF16 ? 1 : 0] = v.y;
                }
            } else {
#pragma unroll
                for (int e = 0; e < TI; ++e)
                    xi[e][0] = *reinterpret_cast<const float *>(bst + (TI * t.ib + e) * 128 + sw[e & 7]);
#pragma unroll
                for (int e = 0; e < TJ; ++e)
                    xj[e][0] = *reinterpret_cast<const float *>(bst + (TJ * t.jb + e) * 128 + sw[e & 7]);
            }
            const int as = (int)(q % NA);
            const int64_t use = q / NA;
            if (use > 0 && !mbar_wait(&a_empty[as], (uint32_t)((use - 1) & 1), abort_flag, a.status, 12)) {
                ok = false;
                break;
            }
            unsigned char *ast = a_stage0 + (size_t)as * A_STAGE_BYTES;
#pragma unroll
            for (int e = 0; e < TI; ++e)
#pragma unroll
                for (int f = 0; f < TJ; ++f) {
                    // row e*16+f of the tile
                    uint32_t v;
                    if (BF16) {
                        // two samples per word, each product rounded once to bf16 (first sample in the low half)
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(v) : "f"(xi[e][BF16 ? 1 : 0] * xj[f][BF16 ? 1 : 0]), "f"(xi[e][0] * xj[f][0]));
                    } else {
                        // round to nearest TF32 (ties away from zero): the tensor core ignores the low 13 bits
                        v = __float_as_uint(xi[e][0] * xj[f][0]) + 0x1000u;
                    }
                    *reinterpret_cast<uint32_t *>(ast + (e * TJ + f) * 128 + sw[f & 7]) = v;
                }
            fence_proxy_async();      // generic-proxy stores must be visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(&a_full[as]);
        }

        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the slice sums may be launched; they wait for this grid to end
        // ---- epilogue: tensor memory -> this slice's partial sums ---------------------------------
        if (nstages > 0 && mbar_wait(acc_full, 0u, abort_flag, a.status, 13)) {
            tc_fence_after();
            float *__restrict__ mine = a.partials + (size_t)blockIdx.y * a.out_elems;
            // All MMAs are complete, so the A ring is free: every warp takes EPI_PITCH x 32 floats of it
            // to turn "one thread = one pair, registers = k" into rows of consecutive k.  In the packed
            // order the rows (i, j, k >= j) of one i and consecutive j follow each other, so the 16 rows of
            // one i of a tile form one contiguous run in memory.
            float *tr = reinterpret_cast<float *>(a_stage0) + (size_t)warp * (32 * EPI_PITCH);
            const int q4 = warp & 3;                                // lanes 32*q4 .. 32*q4+31 of tensor memory
            for (int ti = warp >> 2; ti < tg; ti += PRODUCERS / 4) {
                const Tile t = tiles[ti];
                const int kstart = TJ * t.jb, ncols = a.dcols - kstart;
                uint32_t v[DP];
#pragma unroll
                for (int c0 = 0; c0 < DP; c0 += 16)                 // all loads of the tile in flight, one wait
                    if (c0 < ncols)
                        tmem_ld_32x16(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(t.col + c0), v + c0);
                tmem_ld_wait();
#pragma unroll
                for (int c0 = 0; c0 < DP; c0 += 16)
                    if (c0 < ncols) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) tr[lane * EPI_PITCH + c0 + e] = __uint_as_float(v[c0 + e]);
                    }
                __syncwarp();
                // lane rr describes row rr: first output element and (shift, length) of its run of k
                int my_base = 0, my_run = 0;
                {
                    const int r = q4 * 32 + lane;
                    const int i = TI * t.ib + r / TJ, j = TJ * t.jb + r % TJ;
                    if (i <= j && j < a.d) {
                        // first element of row (i, j, k = j ..) of the packed tetrahedron, in 32-bit arithmetic
                        const int m = a.d - i, jj = j - i;
                        my_base = a.out_elems - m * (m + 1) * (m + 2) / 6 + jj * (2 * m - jj + 1) / 2;
                        my_run = ((j - kstart) << 8) | (a.d - j);
                    }
                }
                for (int rr0 = 0; rr0 < 32; rr0 += 8) {             // eight rows: all loads, then all stores
                    float v0[8], v1[8];
                    int base[8], len[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        base[u] = __shfl_sync(0xffffffffu, my_base, rr0 + u);
                        const int run = __shfl_sync(0xffffffffu, my_run, rr0 + u);
                        len[u] = run & 255;
                        const float *src = tr + (rr0 + u) * EPI_PITCH + (run >> 8);
                        v0[u] = lane < len[u] ? src[lane] : 0.f;
                        v1[u] = lane + 32 < len[u] ? src[lane + 32] : 0.f;
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (lane < len[u] && ST_BOUNDS_OK(base[u] + lane, a.out_elems, 4)) mine[base[u] + lane] = v0[u];
                        if (lane + 32 < len[u] && ST_BOUNDS_OK(base[u] + lane + 32, a.out_elems, 4)) mine[base[u] + lane + 32] = v1[u];
                    }
                }
                __syncwarp();
            }
        }
    } else if (warp < LOAD_WARP) {
        // ---- MMA issuers: two warps.  A barrier poll issued behind tcgen05.mma instructions of the same thread
        // returns only as they drain, so one issuer alone leaves the tensor pipe idle while it polls.
        // A ring slot q % NA has the parity of q (NA is even), so every slot has one issuer and its uses are polled in
        // order.  The MMAs of slice 0 overwrite the accumulators: both issuers wait until all of them are complete
        // before either adds slice 1, after which the order of the additions into a tile is free.
        const int iw = warp - MMA_WARP;
        if (elect_one()) {
            bool ok = true;
            for (int slice = 0; slice < nslices && ok; ++slice) {
                const int bs = slice % NB;
                if (!mbar_wait(&b_full[bs], (uint32_t)((slice / NB) & 1), abort_flag, a.status, 14)) break;
                const uint32_t sb = smem_u32(b_stage0 + (size_t)bs * B_STAGE_BYTES);
                for (int ti = 0; ti < tg; ++ti) {
                    const int64_t q = (int64_t)slice * tg + ti;
                    if ((int)(q & 1) != iw) continue;
                    const Tile t = tiles[ti];
                    const int kstart = TJ * t.jb, ncols = a.dcols - kstart;
                    const int as = (int)(q % NA);
                    if (!mbar_wait(&a_full[as], (uint32_t)((q / NA) & 1), abort_flag, a.status, 15)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(a_stage0 + (size_t)as * A_STAGE_BYTES);
                    const uint32_t idesc = make_idesc(BF16 ? 1 : 2, 0, 0, BM, (uint32_t)ncols);
#pragma unroll
                    for (int kk = 0; kk < ROW_BYTES / 32; ++kk) {             // 32 bytes of K per MMA
                        const uint64_t adesc = make_smem_desc(sa + kk * 32, 16, 1024);
                        const uint64_t bdesc = make_smem_desc(sb + kstart * 128 + kk * 32, 16, 1024);
                        if (BF16) mma_bf16(tmem_base + (uint32_t)t.col, adesc, bdesc, idesc, (slice > 0 || kk > 0) ? 1u : 0u);
                        else mma_tf32(tmem_base + (uint32_t)t.col, adesc, bdesc, idesc, (slice > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit(&a_empty[as]);
                }
                if (!ok) break;
                tc_commit(&b_empty[bs]);
                if (slice == 0 && nslices > 1) {
                    tc_commit(iss_sync);
                    if (!mbar_wait(iss_sync, 0u, abort_flag, a.status, 17)) break;
                    tc_fence_after();
                }
                if (slice == nslices - 1) tc_commit(acc_full);
            }
        }
    } else {
        // ---- loader: slices of X^T (row = column c of X), rounded to TF32 or bf16.  A lane owns one
        // 4-byte word of every row: sample `lane` (TF32) or samples 2*lane, 2*lane+1 (bf16).
        constexpr int SPL = BF16 ? 2 : 1;                            // samples per lane
        constexpr int CH = 32;                                       // columns per pass
        constexpr int PF_AHEAD = 4;                                  // slices of L2 prefetch distance
        for (int slice = 0; slice < nslices; ++slice) {
            const int bs = slice % NB, use = slice / NB;
            unsigned char *bst = b_stage0 + (size_t)bs * B_STAGE_BYTES;
            bool waited = false;
            // pull the rows of later slices into L2 while this one is worked on
            for (int ahead = (slice == 0 ? 1 : PF_AHEAD); ahead <= PF_AHEAD; ++ahead)
#pragma unroll
                for (int u = 0; u < SPL; ++u) {
                    const int64_t n = n_begin + (int64_t)(slice + ahead) * KS + SPL * lane + u;
                    if (n < n_end) {
                        const char *pf = reinterpret_cast<const char *>(a.X + n * a.ldx);
                        for (int o = 0; o < a.d * 4; o += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(pf + o));
                    }
                }
            for (int c0 = 0; c0 < DP; c0 += CH) {
                float x[SPL][CH];
#pragma unroll
                for (int u = 0; u < SPL; ++u) {
                    const int64_t n = n_begin + (int64_t)slice * KS + SPL * lane + u;
                    const bool row_ok = n < n_end;
                    if (a.vec) {
                        const float4 *src = reinterpret_cast<const float4 *>(a.X + (row_ok ? n : n_begin) * a.ldx + c0);
#pragma unroll
                        for (int c = 0; c < CH / 4; ++c) {
                            const float4 v = (row_ok && c0 + 4 * c < a.d) ? __ldg(src + c) : make_float4(0.f, 0.f, 0.f, 0.f);
                            x[u][4 * c] = v.x; x[u][4 * c + 1] = v.y; x[u][4 * c + 2] = v.z; x[u][4 * c + 3] = v.w;
                        }
                    } else {
                        const float *src = a.X + (row_ok ? n : n_begin) * a.ldx + c0;
#pragma unroll
                        for (int c = 0; c < CH; ++c) x[u][c] = (row_ok && c0 + c < a.d) ? __ldg(src + c) : 0.f;
                    }
                }
                if (!waited) {
                    if (use > 0 && !mbar_wait(&b_empty[bs], (uint32_t)((use - 1) & 1), abort_flag, a.status, 16)) break;
                    waited = true;
                }
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    uint32_t t;
                    if (BF16) {
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(t) : "f"(x[SPL - 1][c]), "f"(x[0][c]));
                        *reinterpret_cast<float2 *>(x32_stage0 + (size_t)bs * X32_STAGE_BYTES + (c0 + c) * 256 + 8 * lane) =
                            make_float2(x[0][c], x[SPL - 1][c]);
                    } else {
                        asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(t) : "f"(x[0][c]));
                    }
                    *reinterpret_cast<uint32_t *>(bst + (c0 + c) * 128 + sw[c & 7]) = t;
                }
            }
            if (!waited) break;
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&b_full[bs]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

struct Plan {
    int groups, slices, dcols;
    int ntiles[2];
    Tile tiles[2][MAX_GROUP_TILES];
    int64_t rows_per_slice, out_elems;
    bool ok;
};

static Plan plan(int64_t N, int64_t d, bool bf16)
{
    const int KS = bf16 ? 64 : 32;
    Plan p{};
    p.ok = false;
    if (N <= 0 || d < 1 || d > DP) return p;
    p.out_elems = tet_rows(d);
    p.dcols = (int)((d + 15) / 16 * 16);
    // tiles in the order (JB, IB); a tile exists when it holds some i <= j < d
    Tile all[2 * MAX_GROUP_TILES];
    int cols[2 * MAX_GROUP_TILES], n = 0, total_cols = 0;
    for (int jb = 0; jb * TJ < d; ++jb)
        for (int ib = 0; ib * TI < d && ib * TI <= jb * TJ + TJ - 1; ++ib) {
            if (n >= 2 * MAX_GROUP_TILES) return p;
            all[n].ib = (unsigned char)ib;
            all[n].jb = (unsigned char)jb;
            cols[n] = p.dcols - jb * TJ;
            total_cols += cols[n];
            ++n;
        }
    p.groups = total_cols > (int)TMEM_COLS ? 2 : 1;
    const int first = p.groups == 1 ? n : (n + 1) / 2;      // equal numbers of tiles: the stores of P are the bound
    if (first > MAX_GROUP_TILES || n - first > MAX_GROUP_TILES) return p;
    for (int g = 0; g < p.groups; ++g) {
        const int lo = g == 0 ? 0 : first, hi = g == 0 ? first : n;
        int col = 0;
        for (int t = lo; t < hi; ++t) {
            p.tiles[g][t - lo] = all[t];
            p.tiles[g][t - lo].col = (unsigned short)col;
            col += cols[t];
        }
        if (col > (int)TMEM_COLS) return p;
        p.ntiles[g] = hi - lo;
    }
    const int sms = sm_count_or_default();
    int64_t slices = sms / p.groups;
    if (slices < 1) slices = 1;
    int64_t rps = (N + slices - 1) / slices;
    rps = (rps + KS - 1) / KS * KS;                        // whole MMA slices
    p.rows_per_slice = rps;
    p.slices = (int)((N + rps - 1) / rps);
    p.ok = true;
    return p;
}

}  // namespace m3tc

size_t moment3_tc_workspace(int64_t N, int64_t d, bool bf16)
{
    const m3tc::Plan p = m3tc::plan(N, d, bf16);
    if (!p.ok) return 0;
    return kWsHeaderBytes + (size_t)p.slices * p.out_elems * sizeof(float);
}

st_status moment3_tc(const float *X, int64_t N, int64_t d, int64_t ldx, float *out, void *ws, size_t ws_bytes,
                     bool bf16, cudaStream_t stream)
{
    using namespace m3tc;
    const Plan p = plan(N, d, bf16);
    if (!p.ok) return ST_ERR_UNSUPPORTED;
    const size_t need = kWsHeaderBytes + (size_t)p.slices * p.out_elems * sizeof(float);
    if (!ws || ws_bytes < need) return ST_ERR_WORKSPACE;
    if (!aligned256(ws)) return ST_ERR_ALIGN;
    const DeviceInfo di = device_info();
    if (!di.ok) return ST_ERR_CUDA;
    if (smem_bytes(bf16) > (size_t)di.max_smem_optin) return ST_ERR_UNSUPPORTED;
    Args a;
    a.X = X;
    a.partials = (float *)((unsigned char *)ws + kWsHeaderBytes);
    a.status = (unsigned *)ws;
    a.N = N; a.ldx = ldx; a.rows_per_slice = p.rows_per_slice;
    a.d = (int)d; a.dcols = p.dcols; a.out_elems = (int)p.out_elems;
    a.vec = (ldx % 4 == 0 && d % 4 == 0) ? 1 : 0;
    for (int g = 0; g < 2; ++g) {
        a.ntiles[g] = p.ntiles[g];
        for (int t = 0; t < MAX_GROUP_TILES; ++t) a.tiles[g][t] = p.tiles[g][t];
    }
    if (bf16) {
        if (!ensure_dynamic_smem(moment3_tc_kernel<true>, smem_bytes(true))) return ST_ERR_CUDA;
        moment3_tc_kernel<true><<<dim3(p.groups, p.slices), THREADS, smem_bytes(true), stream>>>(a);
    } else {
        if (!ensure_dynamic_smem(moment3_tc_kernel<false>, smem_bytes(false))) return ST_ERR_CUDA;
        moment3_tc_kernel<false><<<dim3(p.groups, p.slices), THREADS, smem_bytes(false), stream>>>(a);
    }
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    return sum_slices_launch(a.partials, out, p.out_elems, p.slices, stream);
}

}  // namespace st
