// Entry points that are not tied to one kernel: workspace sizes, status, version.
#include "st_common.cuh"

namespace st {
size_t moment2_workspace(int64_t N, int64_t d, int xdt, unsigned flags);
size_t moment3_workspace(int64_t N, int64_t d, unsigned flags);
size_t moment4_workspace(int64_t N, int64_t d, unsigned flags);
size_t ttm_tf32_tc_workspace(int64_t rows, int64_t K, int64_t R);
size_t ttm_split_workspace(int64_t rows, int64_t K, int64_t R);
size_t mttkrp_workspace(int64_t rows, int64_t I, int64_t K, int64_t R, unsigned flags);
}  // namespace st

#ifdef ST_BOUNDS_CHECK
namespace st {
__device__ unsigned g_st_bounds[2] = {0u, 0u};
// runs the range check on an index that is out of range by construction; nothing is loaded or stored
__global__ void bounds_self_test_kernel()
{
    if (threadIdx.x == 0 && ST_BOUNDS_OK(5, 3, 99)) g_st_bounds[1] = 0xFFFFFFFFu;   // not reached
}
}
#endif

extern "C" {

size_t st_workspace_bytes(st_op op, int64_t a, int64_t b, int64_t c, int64_t e, unsigned flags)
{
    switch (op) {
    case ST_OP_SYM_MOMENT2: return st::moment2_workspace(a, b, (int)c, flags);
    case ST_OP_SYM_MOMENT3: return st::moment3_workspace(a, b, flags);
    case ST_OP_SYM_MOMENT4: return st::moment4_workspace(a, b, flags);
    case ST_OP_MTTKRP_TRI:
        if (a <= 0 || a > (1 << 15)) return 0;
        return st::mttkrp_workspace((flags & ST_FLAG_DENSE_CONTROL) ? a * a : a * (a + 1) / 2, a, b, c, flags);
    case ST_OP_MTTKRP_SLICE: {
        // enough for any choice of the fixed indices: the longest slice, reaching every row of A
        if (a <= 0 || b <= 0) return 0;
        const size_t x = st::mttkrp_workspace(a, a, c, e, flags), y = st::mttkrp_workspace(b, 1, c, e, flags),
                     z = st::mttkrp_workspace(1, 1, c, e, flags);
        if (x == 0 || y == 0 || z == 0) return 0;
        return x > y ? (x > z ? x : z) : (y > z ? y : z);
    }
    case ST_OP_TTM_BLOCKDIAG:
        if (a <= 0 || b <= 0 || c <= 0 || e <= 0) return 0;
        if ((flags & ST_FLAG_TC_TF32) && (flags & ST_FLAG_TC_SPLIT)) return 0;
        if (flags & (ST_FLAG_TC_TF32 | ST_FLAG_TC_SPLIT)) {
            const int64_t d = a * b;
            const int64_t rows = (flags & ST_FLAG_DENSE_CONTROL) ? d * d : a * b * b;
            return (flags & ST_FLAG_TC_TF32) ? st::ttm_tf32_tc_workspace(rows, c, e) : st::ttm_split_workspace(rows, c, e);
        }
        return st::kWsHeaderBytes;
    default: return 0;
    }
}

st_status st_check_status(const void *ws, void *stream)
{
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return ST_ERR_CUDA;
#ifdef ST_BOUNDS_CHECK
    {
        // the range checks of the debug build report here whichever call tripped them; reading clears the record
        unsigned b[2] = {0, 0};
        const unsigned zero[2] = {0, 0};
        if (cudaMemcpyFromSymbol(b, st::g_st_bounds, sizeof(b)) != cudaSuccess) return ST_ERR_CUDA;
        if (b[0] != 0) {
            (void)cudaMemcpyToSymbol(st::g_st_bounds, zero, sizeof(zero));
            return ST_ERR_DEV_BOUNDS;
        }
    }
#endif
    if (!ws) return ST_OK;
    unsigned words[2] = {0, 0};
    if (cudaMemcpy(words, ws, sizeof(words), cudaMemcpyDeviceToHost) != cudaSuccess) return ST_ERR_CUDA;
    if (words[0] == ST_ERR_DEV_TIMEOUT) return ST_ERR_DEV_TIMEOUT;
    if (words[0] == ST_ERR_DEV_BOUNDS) return ST_ERR_DEV_BOUNDS;
    return ST_OK;
}

const char *st_status_string(st_status s)
{
    switch (s) {
    case ST_OK: return "ok";
    case ST_ERR_NULL: return "null pointer";
    case ST_ERR_SHAPE: return "bad shape";
    case ST_ERR_ALIGN: return "misaligned pointer or leading dimension";
    case ST_ERR_DTYPE: return "unsupported element type";
    case ST_ERR_WORKSPACE: return "workspace missing or too small";
    case ST_ERR_UNSUPPORTED: return "request not supported by the kernels";
    case ST_ERR_CUDA: return "CUDA call failed";
    case ST_ERR_DEV_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case ST_ERR_DEV_BOUNDS: return "kernel-side consistency check failed";
    case ST_ERR_STATIC_SCRATCH: return "request needs more scratch than the built-in static array holds";
    default: return "unknown status";
    }
}

int st_abi_version(void) { return 1; }

int st_bounds_checked_build(void)
{
#ifdef ST_BOUNDS_CHECK
    return 1;
#else
    return 0;
#endif
}

st_status st_bounds_self_test(void *stream)
{
#ifdef ST_BOUNDS_CHECK
    st::bounds_self_test_kernel<<<1, 32, 0, (cudaStream_t)stream>>>();
    return cudaGetLastError() == cudaSuccess ? ST_OK : ST_ERR_CUDA;
#else
    (void)stream;
    return ST_ERR_UNSUPPORTED;
#endif
}

}  // extern "C"
