// Per-device facts and one-time settings (SM count, kernel attributes that CUDA keeps per device), shared by
// every launcher.  A process may use the library on several GPUs: nothing here is cached across devices.
#pragma once

#include <mutex>

#include <cuda_runtime.h>

namespace mom {

constexpr int MAX_DEVICES = 64;

struct DeviceInfo {
    int sm_count = 0;
    int max_pairs = 0;               // co-resident clusters of the CTA-pair kernel (0: not asked yet)
    bool tc_attr = false;            // dynamic shared-memory limit raised for the tensor-core kernels on this device
    bool pair_attr = false;
    bool inline64_attr = false, inline128_attr = false;
    bool inline_variant_attr[2][2][2] = {}, inline_variant_np[2][2][2] = {};   // per kernel of the one-launch family: [128 columns][A transposed][B transposed]
    int inline_clusters[2][5] = {};  // co-resident clusters of the one-launch tcgen05 kernel, [128-column tiles][log2 cluster size]; 0: not asked, -1: unknown
    bool inline_pair_attr[2] = {false, false};
    int inline_pair_clusters[2] = {0, 0};   // co-resident CTA pairs of the one-launch kernel's pair variant, [128 columns per CTA]
    int mma_clusters16 = 0;          // co-resident clusters of 16 CTAs of the warp-level kernel (0: not asked yet, -1: not available)
    int fused_max_smem[2] = {0, 0};  // largest dynamic shared-memory size set for the fused small-equation kernels
    int batched_max_smem = 0;
};

// Entry of the device that is current on the calling thread (SM count filled in), or nullptr when the
// ordinal is beyond MAX_DEVICES or the runtime call fails.  The entry is only read or changed while the
// caller holds device_info_mutex().
DeviceInfo *current_device_info(int *device = nullptr);
std::mutex &device_info_mutex();

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per device, remembered in `*done`.
template <typename Kernel>
cudaError_t raise_smem_limit_once(Kernel kernel, int bytes, bool DeviceInfo::*done) {
    std::lock_guard<std::mutex> lock(device_info_mutex());
    DeviceInfo *info = current_device_info();
    if (!info) return cudaErrorInvalidDevice;
    if (info->*done) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) info->*done = true;
    return e;
}

// The same for a caller that already holds device_info_mutex().
template <typename Kernel>
cudaError_t raise_smem_limit_locked(Kernel kernel, int bytes, bool *done) {
    if (*done) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) *done = true;
    return e;
}

// SM count of the current device (0 on failure).
int current_sm_count();

}  // namespace mom
