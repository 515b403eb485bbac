// Helpers shared by the C-ABI translation units (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

namespace mnnllm {

// 1 when the current device is compute capability 10.x (cached per device).
int device_is_supported();

// Device address of the library's status word on the current device (a __device__ variable of the
// module, resolved once per device); kernels OR a code into it when a bounded wait gives up.
uint32_t* status_word_ptr();

}  // namespace mnnllm
