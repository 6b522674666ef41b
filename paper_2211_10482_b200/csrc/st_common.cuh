// Shared host-side helpers of the library (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include <cstddef>
#include <map>
#include <mutex>
#include <utility>
#include "structtensor.h"

namespace st {

// The first 256 bytes of every workspace: word 0 = device status (st_status written by a
// kernel), word 1 = detail, words 8.. = arrival counters.  Cleared by each call that uses it.
constexpr size_t kWsHeaderBytes = 256;
constexpr int kWsStatusWord = 0;
constexpr int kWsDetailWord = 1;
constexpr int kWsTicketWord = 8;

// Debug build (-DST_BOUNDS_CHECK, relocatable device code): every store whose index comes out of packed-index
// arithmetic is range-checked first; a violation records the site in a device-wide word, the store is skipped
// and st_check_status reports ST_ERR_DEV_BOUNDS.  In the normal build the macro is the constant true.
#ifdef ST_BOUNDS_CHECK
extern __device__ unsigned g_st_bounds[2];          // [0] = number of violations, [1] = site of the last one
__device__ __forceinline__ bool st_bounds_ok(long long idx, long long n, unsigned site)
{
    if (idx >= 0 && idx < n) return true;
    atomicAdd(&g_st_bounds[0], 1u);
    g_st_bounds[1] = site;
    return false;
}
#define ST_BOUNDS_OK(idx, n, site) ::st::st_bounds_ok((long long)(idx), (long long)(n), (site))
#else
#define ST_BOUNDS_OK(idx, n, site) true
#endif
// sites: 1 pack/unpack copy, 2 second-moment reductions, 3 third-moment partial sums, 4 tensor-core third moment,
// 5 MTTKRP partial slots, 6 MTTKRP row sums, 7 fourth-moment gather, 8 TTM rows

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct DeviceInfo {
    int device = -1;
    int sm_count = 0;
    int max_smem_optin = 0;
    bool ok = false;
};

// Properties of the current device (cached per device index).
inline DeviceInfo device_info()
{
    static DeviceInfo cache[64];
    DeviceInfo bad;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return bad;
    if (!cache[dev].ok) {
        DeviceInfo di;
        di.device = dev;
        if (cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return bad;
        if (cudaDeviceGetAttribute(&di.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return bad;
        di.ok = true;
        cache[dev] = di;
    }
    return cache[dev];
}

// SM count used to size grids; 148 (B200) when no device can be queried, so that the
// host-only size queries still answer.
inline int sm_count_or_default()
{
    DeviceInfo di = device_info();
    return di.ok ? di.sm_count : 148;
}

// Raises a kernel's dynamic shared-memory limit once per (kernel, device): the runtime call costs
// tens of microseconds, during which the GPU would idle if it were repeated on every launch.
template <typename Kernel>
inline bool ensure_dynamic_smem(Kernel kernel, size_t bytes)
{
    if (bytes <= 48 * 1024) return true;
    static std::mutex lock;
    static std::map<std::pair<const void *, int>, size_t> done;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> guard(lock);
    size_t &have = done[std::make_pair((const void *)kernel, dev)];
    if (have >= bytes) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    have = bytes;
    return true;
}

inline st_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? ST_OK : ST_ERR_CUDA;
}

}  // namespace st
