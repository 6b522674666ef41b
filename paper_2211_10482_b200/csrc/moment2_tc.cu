// placeholder
#include "st_common.cuh"
namespace st {
st_status moment2_bf16_tc(const void *, int64_t, int64_t, int64_t, float *, void *, size_t, unsigned, cudaStream_t)
{
    return ST_ERR_UNSUPPORTED;
}
size_t moment2_bf16_tc_workspace(int64_t, int64_t, unsigned) { return 0; }
}  // namespace st
