// Launch-shape helpers shared by the kernel launchers.
#pragma once
#include <algorithm>
#include <cuda_runtime.h>

#include "copy_engine.cuh"
#include "plan.hpp"

namespace amoeba {

// Defaults, chosen from sweeps over all benchmark configurations on B200: the producer/consumer ring, 8 KiB work
// items, 5 rings of 4 stages per CTA (160 KiB of stages per SM - more in flight lowers DRAM efficiency, less starves
// it), two stores in flight before a slot is handed back, both directions marked evict-first in L2.
struct KernelDefaults {
    int copy_path, stages, lag, warps, hint;
};
constexpr KernelDefaults kKvDefaults{3, 4, 2, 5, 4};
constexpr KernelDefaults kWDefaults{3, 4, 2, 5, 4};
constexpr int kLdstCtasPerSm = 6;  // vector load/store kernels: resident CTAs per SM (and loads in flight per lane)

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;  // bytes of dynamic shared memory one CTA may opt in to
};

// Properties of the current device (attribute queries; no allocation, no synchronisation).
inline bool device_info(DeviceInfo* out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&out->sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&out->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
        return false;
    return out->sms > 0;
}

// Persistent grid size: the default (a multiple of the SM count), or the caller's cap when it leaves SMs to other work.
inline int64_t grid_cap(const KernelOpts& opt, int64_t grid) {
    return opt.max_ctas > 0 ? std::min<int64_t>(grid, opt.max_ctas) : grid;
}

constexpr int kBarrierBytes = 1024;  // head of dynamic shared memory: up to 128 mbarriers

struct BulkShape {
    RingShape ring;
    int path;         // 2 = ring per warp, 3 = producer/consumer pair per ring
    int rings;        // rings per CTA
    int threads;      // CTA size
    int ctas_per_sm;
    size_t smem;
};

// Ring depth, lag and rings per CTA for the bulk-copy kernels: the requested shape, shrunk until it fits the
// shared memory one CTA may use and the barrier area.
inline BulkShape bulk_shape(const DeviceInfo& dev, const KernelOpts& opt, const KernelDefaults& def, int path,
                            int stage_bytes) {
    BulkShape b;
    b.path = path;
    b.ctas_per_sm = opt.ctas_per_sm ? opt.ctas_per_sm : 1;
    int stages = std::min(kMaxStages, std::max(2, opt.stages ? opt.stages : def.stages));
    const int budget = dev.smem_optin / b.ctas_per_sm - kBarrierBytes - (b.ctas_per_sm > 1 ? 1024 : 0);
    while (stages > 2 && (int64_t)stages * stage_bytes > budget) --stages;
    int lag = opt.lag ? opt.lag : (opt.stages ? stages / 2 : def.lag);
    lag = std::max(1, std::min(lag, stages - 1));
    const int bars_per_ring = path == 3 ? 2 * stages : stages;
    int rings = opt.warps ? opt.warps : def.warps;
    rings = (int)std::min<int64_t>(rings, budget / ((int64_t)stages * stage_bytes));
    rings = std::min(rings, kBarrierBytes / 8 / bars_per_ring);
    rings = std::max(1, std::min(rings, path == 3 ? 16 : 32));
    b.rings = rings;
    b.threads = 32 * rings * (path == 3 ? 2 : 1);
    b.ring.stages = stages;
    b.ring.lag = lag;
    b.ring.stage_bytes = stage_bytes;
    const int hint = opt.hint ? opt.hint : (def.hint ? def.hint : 1);
    b.ring.hint = hint - 1;
    b.smem = kBarrierBytes + (size_t)rings * stages * stage_bytes;
    return b;
}

}  // namespace amoeba
