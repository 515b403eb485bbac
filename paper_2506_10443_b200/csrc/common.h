// Helpers shared by the C-ABI translation units (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

#include <mutex>

namespace mnnllm {

// Function attributes (shared-memory limits, carve-outs), symbol addresses and occupancy answers
// belong to ONE device: everything the library remembers about them is kept per device ordinal,
// and guarded, since the C ABI may be called from several host threads.
constexpr int kMaxDevices = 64;

// ordinal of the current device, or -1 (no device, or an ordinal beyond kMaxDevices)
inline int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

// One value of T per device.  `with(f)` runs f on the current device's value under the table's lock
// and returns f's cudaError_t (cudaErrorInvalidDevice without a usable current device).
template <typename T>
class PerDevice {
public:
    template <typename F>
    cudaError_t with(F&& f) {
        const int dev = current_device();
        if (dev < 0) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> g(lock_);
        return f(slot_[dev]);
    }

private:
    T slot_[kMaxDevices] = {};
    std::mutex lock_;
};

// 1 when the current device is compute capability 10.x (cached per device).
int device_is_supported();

// SMs of the current device (cached per device); 0 without a usable device.
int device_sm_count();

// Device address of the library's status word on the current device (a __device__ variable of the
// module, resolved once per device); kernels OR a code into it when a bounded wait gives up.
uint32_t* status_word_ptr();

}  // namespace mnnllm
