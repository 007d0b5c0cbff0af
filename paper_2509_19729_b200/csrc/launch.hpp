// Launch-shape helpers shared by the kernel launchers.
#pragma once
#include <algorithm>
#include <mutex>
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
// The in-place exchange writes the lines it has just read: no L2 hints there (measured 0.5 - 0.9 % faster).
constexpr KernelDefaults kMergeDefaults{3, 4, 2, 5, 1};
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

// The same, looked up once per device ordinal and remembered (the attributes of a device do not change); sms == 0 if
// the query failed.  Only cudaGetDevice runs per call.
constexpr int kMaxDevices = 64;
inline DeviceInfo cached_device_info() {
    static DeviceInfo cache[kMaxDevices];
    static bool known[kMaxDevices];
    static std::mutex mutex;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DeviceInfo{};
    DeviceInfo d;
    if (dev < 0 || dev >= kMaxDevices) return device_info(&d) ? d : DeviceInfo{};
    std::lock_guard<std::mutex> lock(mutex);
    if (!known[dev]) {
        if (!device_info(&d)) return DeviceInfo{};
        cache[dev] = d;
        known[dev] = true;
    }
    return cache[dev];
}

// Opt a kernel in to `bytes` of dynamic shared memory, once per (device, kernel) and size: the attribute sticks, so
// later launches with the same or a smaller size skip the call.
inline cudaError_t ensure_dynamic_smem(const void* kernel, int bytes) {
    struct Entry {
        int dev;
        const void* kernel;
        int bytes;
    };
    static Entry table[256];
    static int used = 0;
    static std::mutex mutex;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mutex);
    Entry* e = nullptr;
    for (int i = 0; i < used; ++i)
        if (table[i].dev == dev && table[i].kernel == kernel) e = &table[i];
    if (e && e->bytes >= bytes) return cudaSuccess;
    const cudaError_t rc = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (rc != cudaSuccess) return rc;
    if (!e && used < 256) e = &table[used++];
    if (e) *e = Entry{dev, kernel, bytes};
    return cudaSuccess;
}

// Persistent grid size: the default (a multiple of the SM count), or the caller's cap when it leaves SMs to other work.
inline int64_t grid_cap(const KernelOpts& opt, int64_t grid) {
    return opt.max_ctas > 0 ? std::min<int64_t>(grid, opt.max_ctas) : grid;
}

struct BulkShape {
    RingShape ring;
    int path;         // 2 = ring per warp, 3 = producer/consumer pair per ring
    int rings;        // rings per CTA
    int threads;      // CTA size
    int ctas_per_sm;
    size_t smem;
};

// Default shape of the producer/consumer ring against the number of CTAs (= SMs) the copy may use.  With every SM
// copying, DRAM is the limit and the default shape is the most efficient one.  With the grid capped (the copy runs
// beside other kernels), each SM is limited by the bytes it keeps in flight over the DRAM latency: more rings per
// CTA and slots handed back after one store instead of two raise an SM from about 58 to 88 GB/s.  Thresholds and
// shapes from a sweep over 8 ... 148 CTAs on B200.
inline KernelDefaults pair_ring_defaults(KernelDefaults def, int ctas, int sms) {
    if (ctas * 100 <= sms * 54) def.warps = 7, def.lag = 1;
    else if (ctas * 100 <= sms * 70) def.warps = 6, def.lag = 1;
    else if (ctas * 100 <= sms * 90) def.lag = 1;
    return def;
}

// Ring depth, lag and rings per CTA for the bulk-copy kernels: the requested shape, shrunk until it fits the
// shared memory one CTA may use and the barrier area.
inline BulkShape bulk_shape(const DeviceInfo& dev, const KernelOpts& opt, const KernelDefaults& defaults, int path,
                            int stage_bytes) {
    BulkShape b;
    b.path = path;
    b.ctas_per_sm = opt.ctas_per_sm ? opt.ctas_per_sm : 1;
    const int ctas = opt.max_ctas > 0 ? std::min(opt.max_ctas, dev.sms * b.ctas_per_sm) : dev.sms * b.ctas_per_sm;
    const KernelDefaults def = path == 3 && b.ctas_per_sm == 1 ? pair_ring_defaults(defaults, ctas, dev.sms) : defaults;
    int stages = std::min(kMaxStages, std::max(2, opt.stages ? opt.stages : def.stages));
    const int budget = dev.smem_optin / b.ctas_per_sm - kBarrierBytes - (b.ctas_per_sm > 1 ? 1024 : 0);
    while (stages > 2 && (int64_t)stages * stage_bytes > budget) --stages;
    int lag = opt.lag ? opt.lag : (opt.stages ? stages / 2 : def.lag);
    lag = std::max(1, std::min(lag, stages - 1));
    const int bars_per_ring = path == 3 ? 2 * stages : stages;
    int rings = opt.warps ? opt.warps : def.warps;
    rings = (int)std::min<int64_t>(rings, budget / ((int64_t)stages * stage_bytes));
    rings = std::min(rings, kBarrierSlots / bars_per_ring);
    rings = std::max(1, std::min(rings, path == 3 ? 16 : 32));
    b.rings = rings;
    b.threads = 32 * rings * (path == 3 ? 2 : 1);
    b.ring.stages = stages;
    b.ring.lag = lag;
    b.ring.stage_bytes = stage_bytes;
    const int hint = opt.hint ? opt.hint : (def.hint ? def.hint : 1);
    b.ring.hint = hint - 1;
    b.ring.max_polls = opt.wait_tries;
    b.smem = kBarrierBytes + (size_t)rings * stages * stage_bytes;
    return b;
}

}  // namespace amoeba
