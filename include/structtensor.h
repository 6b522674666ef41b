/*
 * structtensor.h -- C ABI of the structured-tensor hot path for NVIDIA B200 (sm_100a).
 *
 * The library executes tensor contractions only over the iteration space that is
 * left once the sparsity structure T_U (unique set) and the redundancy structure
 * T_R (redundancy map) of "Compiling Structured Tensor Algebra" (StructTensor,
 * arXiv 2211.10482) are applied, and it reads and writes tensors in packed layouts
 * that hold T_C = T * T_U contiguously (Section 4, "Compressed Tensor").
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers owned by the caller.  The library
 *     never allocates, frees or keeps them.  Base pointers must be 16-byte aligned.
 *   - Everything is row-major; extents are int64_t.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls are asynchronous on that stream and do not synchronise, except
 *     st_check_status.
 *   - Outputs are overwritten, not accumulated into.
 *   - `ws` is caller-provided scratch of at least st_workspace_bytes(...) bytes,
 *     256-byte aligned.  It needs no initialisation.  Two calls that share one
 *     workspace must be ordered on the same stream.
 *   - Argument errors are found on the host and returned before anything is
 *     launched.  There is no CPU fallback: a shape a kernel does not support
 *     returns ST_ERR_UNSUPPORTED.
 *
 * Packed layouts (lexicographic order of the unique set; `inner` = length of a
 * trailing dense mode carried by every position, 1 if there is none):
 *   ST_TRI_UPPER  T_U(i,j) = 0<=i<=j<d (Section 4, upper-triangular example;
 *                 Figure "structures in STUR", symmetric):
 *                 row p(i,j) = i(2d-i+1)/2 + (j-i);  d(d+1)/2 rows.
 *   ST_TET        T_U(i,j,k) = 0<=i<=j<=k<d (Section 2, "Tensor Structures"):
 *                 all (j,k) of slab i follow those of slab i-1; d(d+1)(d+2)/6 rows.
 *   ST_BAND       T_U(i,j) = i-kl<=j<=i+ku: fixed width kl+ku+1 per row, slot
 *                 (i, j-i+kl); slots outside the matrix are written as zero bytes
 *                 by st_pack and ignored by st_unpack.
 *   ST_BLOCKDIAG  direct sum of nblocks square blocks of size bs (Figure
 *                 "operations in STUR", e1 (+) e2): row (b*bs+i')*bs+j'.
 *   ST_FIXED_ROW  T_U(i,j) = (i = r), ST_FIXED_COL T_U(i,j) = (j = c): the row / column structures R_r,
 *                 C_c of Figure "matrix structures", i.e. Table 1's "fixed i" / "fixed j" on the first
 *                 two modes; the fixed index is passed in `kl`; d rows (row j, resp. row i).
 *   ST_SIMPLEX4   T_U(i,j,k,l) = 0<=i<=j<=k<=l<d (the unique 4-tuples of M3, Section 3): slab i holds
 *                 the tetrahedron (j,k,l) of side d-i; d(d+1)(d+2)(d+3)/24 rows.
 *   The dense counterpart is [d,d,inner] (ST_TET: [d,d,d,inner], ST_SIMPLEX4: [d,d,d,d,inner]).
 */
#ifndef STRUCTTENSOR_H
#define STRUCTTENSOR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ST_OK = 0,
    ST_ERR_NULL = 1,         /* a required pointer is NULL */
    ST_ERR_SHAPE = 2,        /* non-positive or inconsistent extent */
    ST_ERR_ALIGN = 3,        /* pointer or leading dimension not aligned as required */
    ST_ERR_DTYPE = 4,        /* element type not supported by this call */
    ST_ERR_WORKSPACE = 5,    /* workspace missing or too small */
    ST_ERR_UNSUPPORTED = 6,  /* well-formed request outside what the kernels cover */
    ST_ERR_CUDA = 7,         /* a CUDA runtime / driver call failed */
    ST_ERR_DEV_TIMEOUT = 8,  /* a bounded wait inside a kernel ran out (see st_check_status) */
    ST_ERR_DEV_BOUNDS = 9,   /* a kernel-side consistency check failed */
    ST_ERR_STATIC_SCRATCH = 10 /* st_sym_moment3_static: the request needs more scratch than the
                                  built-in ST_STATIC_SCRATCH_BYTES */
} st_status;

typedef enum { ST_F32 = 0, ST_BF16 = 1, ST_F64 = 2 } st_dtype;
typedef enum { ST_TRI_UPPER = 0, ST_TET = 1, ST_BAND = 2, ST_BLOCKDIAG = 3, ST_FIXED_ROW = 4, ST_FIXED_COL = 5,
               ST_SIMPLEX4 = 6 } st_kind;
typedef enum { ST_FILL_ZERO = 0, ST_FILL_SYMMETRIC = 1 } st_fill;
typedef enum { ST_OP_SYM_MOMENT2 = 0, ST_OP_SYM_MOMENT3 = 1, ST_OP_MTTKRP_TRI = 2,
               ST_OP_TTM_BLOCKDIAG = 3, ST_OP_SYM_MOMENT4 = 4, ST_OP_MTTKRP_SLICE = 5 } st_op;

/* flags (bit mask) */
#define ST_FLAG_DENSE_CONTROL 1u /* run the same kernel over the dense, unstructured iteration
                                    space (a control for measurements; see each call) */
#define ST_FLAG_TC_TF32       2u /* st_ttm_blockdiag, st_mttkrp_tri, st_sym_moment3, st_sym_moment2 (fp32 input): tensor cores, operands read as TF32 */
#define ST_FLAG_TC_BF16       4u /* st_sym_moment3, st_sym_moment4: tensor cores, operands rounded to bf16 */
#define ST_FLAG_TC_SPLIT      8u /* st_ttm_blockdiag, st_ttm_packed, st_mttkrp_tri, st_mttkrp_slice (and st_sym_moment2 on fp32 input,
                                    see there): tensor cores with
                                    both operands split into two bf16 parts and three of the four partial products
                                    kept: meets the 1e-4 tolerance of the fp32 path, at the speed of the HBM stream
                                    (needs K % 4 == 0, R % 32 == 0, R <= 128, and the split factor, 4*K*R bytes rounded up to
                                    whole chunks of 64 k-values, in shared memory: K*R <= 24576; not with
                                    ST_FLAG_TC_TF32) */

typedef struct {
    int32_t kind;      /* st_kind */
    int32_t reserved;  /* must be 0 */
    int64_t d;         /* structured extent: the matrix is d x d, ST_TET is d x d x d */
    int64_t inner;     /* trailing dense extent carried by every position (>= 1) */
    int64_t kl, ku;    /* ST_BAND: sub- and super-diagonals kept (>= 0); ST_FIXED_ROW / ST_FIXED_COL: kl = the fixed index */
    int64_t nblocks;   /* ST_BLOCKDIAG: number of blocks; d must equal nblocks*bs */
    int64_t bs;        /* ST_BLOCKDIAG: block size */
} st_layout;

/* Number of packed positions times `inner` (elements of the packed array), or -1 for an
 * invalid layout.  Host only. */
int64_t st_packed_elems(const st_layout *layout);

/* Number of elements of the dense counterpart (d*d*inner, d*d*d*inner or d*d*d*d*inner), or -1. */
int64_t st_dense_elems(const st_layout *layout);

/* T_C = T * T_U, stored contiguously (Section 4, "Compressed Tensor"; Section 6,
 * Property 2).  Gathers the positions of the unique set of `dense` into `packed`;
 * positions outside T_U are not read.  A bit copy for any dtype (NaN payloads and
 * -0.0 are preserved).  dense: [d,d,inner] ([d,d,d,inner] for ST_TET); packed:
 * st_packed_elems(layout) elements.  The two arrays must not overlap. */
st_status st_pack(const st_layout *layout, st_dtype dtype, const void *dense, void *packed,
                  void *stream);

/* Reconstruction T = T_C + T_R * T_C (Section 6, Property 5; Section 5.5).  Writes
 * every element of `dense`: positions of T_U from `packed`, the others +0.0
 * (ST_FILL_ZERO: sparsity structure, T_R empty) or through the redundancy map of the
 * symmetric structure (ST_FILL_SYMMETRIC; ST_TRI_UPPER: T(i,j) = T_C(j,i) for j<i,
 * Figure "structures in STUR"; ST_TET: T(i,j,k) = T_C(sorted (i,j,k))).
 * ST_SIMPLEX4 likewise: the sorted 4-tuple, so that the fourth moment is reconstructed once, at
 * the end of a chain).  ST_FILL_SYMMETRIC with any other kind returns ST_ERR_UNSUPPORTED. */
st_status st_unpack(const st_layout *layout, st_dtype dtype, const void *packed, void *dense,
                    st_fill fill, void *stream);

/* Scratch bytes needed by one compute call.  Arguments by op:
 *   ST_OP_SYM_MOMENT2   a=N, b=d, c=st_dtype of X, e unused
 *   ST_OP_SYM_MOMENT3   a=N, b=d (flags select the kernel: they change the size)
 *   ST_OP_SYM_MOMENT4   a=N, b=d (flags as for the call)
 *   ST_OP_MTTKRP_TRI    a=I, b=K, c=R (flags as for the call: they change the size)
 *   ST_OP_MTTKRP_SLICE  a=I, b=J, c=K, e=R (enough for any fixed_i / fixed_j; flags as for the call)
 *   ST_OP_TTM_BLOCKDIAG a=nblocks, b=bs, c=K, e=R
 * Returns 0 for an invalid request (the call itself reports the error).  The current
 * device is queried for its SM count. */
size_t st_workspace_bytes(st_op op, int64_t a, int64_t b, int64_t c, int64_t e, unsigned flags);

/* Second moment over the unique set of the symmetric output (Section 3, M1 = f (x) f
 * summed over samples; Section 5.5, "Vector Self-Outer-Product": y_U = 0<=i<=j<n):
 *     out[p(i,j)] = sum_n X[n,i] * X[n,j]      for 0 <= i <= j < d
 * X: [N, ldx] with ldx >= d, dtype ST_F32 (fp32 FMA path, any d) or ST_BF16 (tensor-core
 * path: bf16 products, fp32 accumulation; needs d % 8 == 0, ldx % 8 == 0).
 * out_packed: d(d+1)/2 floats in ST_TRI_UPPER order.
 * ST_FLAG_TC_TF32 (ST_F32 input only): the tensor cores read the fp32 words of X as TF32 (the 13 low
 * mantissa bits are ignored: both factors of every product are truncated, so sums of positive products come out
 * low by about 1e-3 relative), fp32 accumulation; 5e-3 tolerance; needs d % 4 == 0, ldx % 4 == 0, d <= 4096;
 * about 15 times faster than the fp32 FMA path at d = 1024.
 * ST_FLAG_TC_SPLIT (ST_F32 input only): every x is split into hi = bf16(x) and lo = bf16(x - hi) by a first pass
 * (the workspace holds both parts: 4 bytes per element of X), then hi^T hi + hi^T lo + lo^T hi on the tensor
 * cores with fp32 accumulation: the tolerance of the fp32 path (1e-4) about five times faster; d % 8 == 0,
 * ldx % 4 == 0, d <= 4096, N <= 2^29.
 * ST_FLAG_DENSE_CONTROL: all d*d products are computed (lower-triangle tiles too) and
 * the lower results discarded; the output is the same. */
st_status st_sym_moment2(const void *X, st_dtype xdt, int64_t N, int64_t d, int64_t ldx,
                         float *out_packed, void *ws, size_t ws_bytes, unsigned flags,
                         void *stream);

/* Third moment over the unique set (Section 3, M2 = f (x) vec(f (x) f) summed over
 * samples; its unique elements are i<=j<=k, Section 2 "Tensor Structures"):
 *     out[q(i,j,k)] = sum_n X[n,i] * X[n,j] * X[n,k]   for 0 <= i <= j <= k < d
 * X: fp32 [N, ldx], ldx >= d.  out_packed: d(d+1)(d+2)/6 floats in ST_TET order.  Supported:
 * 1 <= d <= 256 (fastest for d % 8 == 0, d <= 64, ldx % 4 == 0; beyond 64 features the tile table
 * of the call is copied into the workspace first).
 * ST_FLAG_DENSE_CONTROL: all d*d*d products are computed and the results outside the
 * unique set discarded; the output is the same.
 * ST_FLAG_TC_TF32 / ST_FLAG_TC_BF16 (one of them, not with the dense control) select the
 * tensor-core path: with the pair product hoisted out of the k loop (Section 5.5, code
 * motion) the sum is the contraction sum_n P[n,(i,j)] X[n,k] with P = X[n,i] X[n,j]; the
 * kernel makes P on the fly as the left operand of a GEMM over the samples and never issues
 * the tiles with k < j.  1 <= d <= 64, any ldx >= d.  TF32: x and the products
 * rounded to TF32; bf16: x_k and the fp32 products rounded to bf16; fp32 accumulation.
 * Tolerance 5e-3 of sum |terms| (bf16: for N >= 1000; 2^-7 for any N). */
st_status st_sym_moment3(const float *X, int64_t N, int64_t d, int64_t ldx,
                         float *out_packed, void *ws, size_t ws_bytes, unsigned flags,
                         void *stream);

/* Fourth moment over the unique set (Section 3, M3 = vec(f (x) f) (x) vec(f (x) f) summed over
 * samples: the last block of the degree-2 polynomial-regression covariance; its unique elements
 * are the 4-tuples with repetition i<=j<=k<=l, "about 23x" fewer than d^4):
 *     out[s(i,j,k,l)] = sum_n X[n,i] X[n,j] X[n,k] X[n,l]   for 0 <= i <= j <= k <= l < d
 * X: fp32 [N, ldx], ldx >= d, 1 <= d <= 128 (ST_FLAG_TC_BF16: d <= 89).  out_packed: d(d+1)(d+2)(d+3)/24 floats in the
 * lexicographic order of the unique set (slab i holds the tetrahedron (j,k,l) of side d-i).
 * Computed as the second moment of the pair features P[n,(i,j)] = X[n,i] X[n,j], i<=j, which
 * the call materialises in the workspace (N * roundup(d(d+1)/2, 64) elements; query the size
 * with ST_OP_SYM_MOMENT4), followed by a gather of the entries with j <= k.  Default: the 1e-4 tolerance of
 * the fp32 paths -- for d <= 89 every fp32 pair product is stored as hi + lo bf16 parts and the tensor-core
 * triangular tile GEMM adds three partial products (hi hi + hi lo + lo hi) with fp32 accumulation; for larger d
 * an fp32 P and fp32 FMA arithmetic.  ST_FLAG_TC_BF16 stores P rounded to bf16 and runs one pass of the same
 * GEMM (5e-3 tolerance for N >= 1000). */
st_status st_sym_moment4(const float *X, int64_t N, int64_t d, int64_t ldx,
                         float *out_packed, void *ws, size_t ws_bytes, unsigned flags,
                         void *stream);

/* Size of the scratch array built into the library image for st_sym_moment3_static. */
#define ST_STATIC_SCRATCH_BYTES (16u << 20)

/* st_sym_moment3 for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a property of the calling environment, not of the method.)
 *
 * Same operation, same arguments and same result as st_sym_moment3, but without the `ws`
 * pair: the per-slice partial sums go to a 16 MiB array that is part of the library
 * (ST_STATIC_SCRATCH_BYTES; every GPU that loads the library holds it until the process
 * exits).  Meant for code that runs where cudaMalloc is off limits -- inside a framework's
 * hot loop that owns the allocator, in a plug-in that is handed nothing but its input and
 * output buffers, or in a process whose device-memory budget was fixed at start-up.  The
 * call itself allocates and frees nothing, on the device or through any library.
 *
 *   - A request whose partial sums do not fit (st_workspace_bytes(ST_OP_SYM_MOMENT3, N, d)
 *     > ST_STATIC_SCRATCH_BYTES) returns ST_ERR_STATIC_SCRATCH and launches nothing.  All
 *     supported d (<= 64) fit on a GPU with up to 160 SMs.
 *   - The first call on each device looks up the device address of the array (one runtime
 *     query, no allocation); make that first call before any stream capture begins.
 *   - All calls on a device share the one array.  Nothing in it has to be cleared between
 *     calls (each call overwrites every partial sum it later reads), but two calls that
 *     overlap on the GPU -- different streams, or different host threads without ordering --
 *     race on it and give wrong results.  Order them on one stream or with events. */
st_status st_sym_moment3_static(const float *X, int64_t N, int64_t d, int64_t ldx,
                                float *out_packed, unsigned flags, void *stream);

/* MTTKRP (Table 1) on a tensor whose unique set is the "upper half cube" of Table 1,
 * B_U(i,j,k) = (0<=i<I)*(i<=j<I)*(0<=k<K):
 *     A[i,r] = sum_{j>=i} sum_k Bp[p(i,j), k] * C[j,r] * D[k,r]
 * Bp: packed [I(I+1)/2, K] fp32 (ST_TRI_UPPER with inner=K); C: [I,R]; D: [K,R];
 * A: [I,R] fp32 (dense: its unique set is every (i,r)).  Needs K % 4 == 0, R in {8,16,32,64},
 * I <= 32768.  ST_FLAG_TC_TF32 selects the tensor-core path (Bp truncated and D rounded to TF32,
 * fp32 accumulation, the product with C in fp32; 5e-3 tolerance; needs R % 32 == 0, R <= 256).
 * ST_FLAG_TC_SPLIT: tensor cores with split bf16 operands, 1e-4 tolerance (see the flag).
 * ST_FLAG_DENSE_CONTROL: Bp is instead a dense [I,I,K] tensor and all j are visited.
 * The sum over j is taken in a fixed order (per-warp partial sums in the workspace, added by a second
 * kernel): no atomics, every element of A written once, the same bits on every call. */
st_status st_mttkrp_tri(const float *Bp, int64_t I, int64_t K, const float *C, const float *D,
                        int64_t R, float *A, void *ws, size_t ws_bytes, unsigned flags,
                        void *stream);

/* MTTKRP (Table 1) on a tensor that is non-zero in one slice only -- Table 1's "fixed i", "fixed j"
 * and "fixed i,j" structures (the row / column / single-element structures R_r, C_c, H of Figure
 * "matrix structures" applied to the first two modes):
 *     A[i,r] = sum_j sum_k B[i,j,k] * C[j,r] * D[k,r],   B[i,j,k] = 0 unless i = fixed_i and / or j = fixed_j
 * fixed_i, fixed_j: the fixed index, or -1 when that mode is free (at least one is fixed).
 * Bp: the packed slice, fp32: [J, K] (fixed i; row = j), [I, K] (fixed j; row = i), [K] (both).
 * C: [J,R]; D: [K,R]; A: dense [I,R], every element written (with fixed i only row fixed_i is
 * non-zero: A_U(i,r) = (i = fixed_i)).  K % 4 == 0; fp32 path R in {8,16,32,64};
 * ST_FLAG_TC_TF32 as for st_mttkrp_tri (R % 32 == 0, R <= 256, 5e-3 tolerance), ST_FLAG_TC_SPLIT likewise.
 * Workspace: ST_OP_MTTKRP_SLICE.  Fixed-order sum over j as in st_mttkrp_tri. */
st_status st_mttkrp_slice(const float *Bp, int64_t I, int64_t J, int64_t K, int64_t fixed_i,
                          int64_t fixed_j, const float *C, const float *D, int64_t R, float *A,
                          void *ws, size_t ws_bytes, unsigned flags, void *stream);

/* TTM (Table 1) on a tensor that is block-diagonal in its first two modes (a direct sum
 * of nblocks blocks of bs x bs fibres):
 *     Ap[b,i',j',r] = sum_k Bp[b,i',j',k] * U[k,r]
 * The output keeps the structure of the input (A_U(i,j,r) = B_U(i,j,.)).
 * Bp: packed [nblocks*bs*bs, K] fp32; U: [K,R] fp32; Ap: packed [nblocks*bs*bs, R] fp32.
 * Needs K % 4 == 0 and R % 4 == 0.  ST_FLAG_TC_TF32 selects the tensor-core path
 * (Bp truncated and U rounded to TF32, fp32 accumulation; 5e-3 tolerance; needs K % 4 == 0,
 * R % 16 == 0, R <= 256).  ST_FLAG_TC_SPLIT: tensor cores with split bf16 operands, 1e-4 tolerance
 * (see the flag).
 * ST_FLAG_DENSE_CONTROL: Bp is a dense [d,d,K] tensor and Ap a dense [d,d,R] one,
 * d = nblocks*bs; all d*d fibres are multiplied. */
st_status st_ttm_blockdiag(const float *Bp, int64_t nblocks, int64_t bs, int64_t K,
                           const float *U, int64_t R, float *Ap, void *ws, size_t ws_bytes,
                           unsigned flags, void *stream);

/* TTM (Table 1) on a tensor with any supported structure in its first two modes:
 *     Ap[p, r] = sum_k Bp[p, k] * U[k, r]      for every packed position p of the layout
 * `layout` describes B with inner = K: ST_TRI_UPPER is Table 1's "upper half cube" (i <= j),
 * ST_BLOCKDIAG with bs = 1 (or ST_BAND with kl = ku = 0) its "diagonal plane" (i = j), ST_TET a
 * 4-mode tensor with i <= j <= k.  The output has the structure of the input with inner = R
 * (the unique set of the product, projected over k, keeps B's (i,j) part: Section 5.1).
 * Same kernels, flags (ST_FLAG_TC_TF32 or ST_FLAG_TC_SPLIT) and shape limits as st_ttm_blockdiag; the
 * workspace is that of ST_OP_TTM_BLOCKDIAG. */
st_status st_ttm_packed(const st_layout *layout, const float *Bp, const float *U, int64_t R,
                        float *Ap, void *ws, size_t ws_bytes, unsigned flags, void *stream);

/* THP (Table 1), the element-wise product A(i,j,k) = B(i,j,k) * C(i,j,k) of a structured B
 * and a dense C.  The unique set of a product is the intersection of the operands' unique sets
 * (Section 5.1), so A has the structure of B:
 *     Ap[p, k] = Bp[p, k] * C[position of p in the dense tensor, k]
 * `layout` describes B (inner = K); Bp and Ap are packed fp32 arrays of st_packed_elems(layout)
 * elements, C is the dense fp32 tensor [d,d,inner] ([d,d,d,inner] for ST_TET), read only at
 * the positions of the unique set.  Ap may not overlap Bp or C.  ST_BAND slots outside the
 * matrix are written as +0.0. */
st_status st_thp(const st_layout *layout, const float *Bp, const float *C_dense, float *Ap,
                 void *stream);

/* Chained computation in compressed space (Section 5.5: a whole chain of operations runs on T_C
 * and the reconstruction from T_R happens once, at the end).  Two packed fp32 arrays of the SAME
 * layout (n = st_packed_elems) are combined position by position; the result has that layout too:
 *   st_packed_axpby   out = alpha * a + beta * b   (sum of tensors of one structure keeps the
 *                     structure: inference rule for `+` on equal unique sets / redundancy maps,
 *                     Figure "inference rules"; e.g. moments of several batches added up)
 *   st_packed_mul     out = a * b                  (Hadamard product, the UHS example of
 *                     Section 5.3 with both operands already restricted to the unique set)
 * out may alias a or b.  Pointers 16-byte aligned. */
st_status st_packed_axpby(int64_t n, float alpha, const float *a, float beta, const float *b,
                          float *out, void *stream);
st_status st_packed_mul(int64_t n, const float *a, const float *b, float *out, void *stream);

/* Synchronises `stream`, then reads the status word a kernel may have written into the
 * workspace (a bounded wait that ran out, a failed consistency check).  ws may be NULL. */
st_status st_check_status(const void *ws, void *stream);

const char *st_status_string(st_status s);

/* Version of the ABI described in this header. */
int st_abi_version(void);

/* 1 in the debug build of the library (compiled with -DST_BOUNDS_CHECK: every store whose index comes out of the
 * packed-index arithmetic is range-checked on the device, a violation is recorded and the store skipped, and
 * st_check_status -- with or without a workspace -- then returns ST_ERR_DEV_BOUNDS once); 0 in the normal build.
 * The paper has no counterpart. */
int st_bounds_checked_build(void);

/* Debug build only (else ST_ERR_UNSUPPORTED): launches a kernel that hands the range check an index that is out
 * of range by construction -- the check records it and nothing is loaded or stored -- so that the reporting path
 * can be tested: the next st_check_status returns ST_ERR_DEV_BOUNDS, the one after it ST_OK. */
st_status st_bounds_self_test(void *stream);

#ifdef __cplusplus
}
#endif
#endif /* STRUCTTENSOR_H */
