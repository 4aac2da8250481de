#include "device_info.h"

namespace mom {

namespace {
DeviceInfo g_devices[MAX_DEVICES];
std::mutex g_mutex;
}  // namespace

std::mutex &device_info_mutex() { return g_mutex; }

DeviceInfo *current_device_info(int *device) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
    DeviceInfo &info = g_devices[dev];
    if (!info.sm_count && cudaDeviceGetAttribute(&info.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        info.sm_count = 0;
        return nullptr;
    }
    if (device) *device = dev;
    return &info;
}

int current_sm_count() {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo *info = current_device_info();
    return info ? info->sm_count : 0;
}

}  // namespace mom
