// placeholder
#include "st_common.cuh"
namespace st {
st_status ttm_tf32_tc(const float *, int64_t, int64_t, const float *, int64_t, float *, void *, size_t, cudaStream_t)
{
    return ST_ERR_UNSUPPORTED;
}
size_t ttm_tf32_tc_workspace(int64_t, int64_t, int64_t) { return 0; }
}  // namespace st
