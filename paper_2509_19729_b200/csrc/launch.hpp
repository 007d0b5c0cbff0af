// Launch-shape helpers shared by the kernel launchers.
#pragma once
#include <algorithm>
#include <cuda_runtime.h>

#include "plan.hpp"

namespace amoeba {

constexpr int kDefaultCopyPath = 2;  // 1 = vector ld/st, 2 = bulk-copy ring (chosen from measurements)

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;  // bytes of dynamic shared memory one CTA may opt in to
};

// Properties of the current device (two attribute queries; no allocation, no synchronisation).
inline bool device_info(DeviceInfo* out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&out->sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&out->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
        return false;
    return out->sms > 0;
}

struct BulkShape {
    int stages, warps, ctas_per_sm;
};

// Ring depth and warps per CTA for the bulk-copy kernels: as many independent warp rings as fit in shared memory.
inline BulkShape bulk_shape(const DeviceInfo& dev, const Options& opt, int stage_bytes) {
    BulkShape s;
    s.stages = opt.stages ? opt.stages : 4;
    if (s.stages != 2 && s.stages != 3 && s.stages != 4 && s.stages != 6 && s.stages != 8) s.stages = 4;
    s.ctas_per_sm = opt.ctas_per_sm ? opt.ctas_per_sm : 1;
    const int budget = (dev.smem_optin - 1024 * s.ctas_per_sm) / s.ctas_per_sm - 1024;
    while (s.stages > 2 && (int64_t)s.stages * stage_bytes > budget) s.stages = s.stages == 3 ? 2 : s.stages == 4 ? 3 : s.stages == 6 ? 4 : 6;
    s.warps = (int)std::max<int64_t>(1, std::min<int64_t>(16, budget / ((int64_t)s.stages * stage_bytes)));
    return s;
}

}  // namespace amoeba
