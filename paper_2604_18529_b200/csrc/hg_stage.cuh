// Staging of a step's small host-resident inputs (the query rows and the three range arrays) into the
// device workspace by ONE kernel that reads pinned, device-mapped host memory directly, instead of one
// copy-engine transfer per array.  Each transfer of a few bytes to a few tens of KB costs several
// microseconds of launch and completion latency when issued as its own asynchronous copy; read by the SMs
// they all travel in the same couple of bus round trips.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace hg {

constexpr int STAGE_MAX_SEG = 4;
constexpr int STAGE_THREADS = 256;

struct StageParams {
    const void* src[STAGE_MAX_SEG];     // device-accessible aliases of host buffers
    void* dst[STAGE_MAX_SEG];           // device memory
    uint32_t bytes[STAGE_MAX_SEG];
    int n;
    int32_t* zero;                      // two device words to clear on the way (the work counter of the launch that follows), or NULL
};

// Any number of CTAs; segment s is copied by all of them together, 16 bytes per thread and trip where
// source, destination and length allow it, else 4 or 1.
__global__ void __launch_bounds__(STAGE_THREADS) stage_kernel(const StageParams p) {
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t nt = gridDim.x * blockDim.x;
    if (t == 0 && p.zero) { p.zero[0] = 0; p.zero[1] = 0; }
    for (int s = 0; s < p.n; ++s) {
        const uintptr_t a = reinterpret_cast<uintptr_t>(p.src[s]) | reinterpret_cast<uintptr_t>(p.dst[s]) | p.bytes[s];
        if ((a & 15u) == 0) {
            const uint4* src = static_cast<const uint4*>(p.src[s]);
            uint4* dst = static_cast<uint4*>(p.dst[s]);
            for (uint32_t i = t; i < p.bytes[s] / 16; i += nt) dst[i] = src[i];
        } else if ((a & 3u) == 0) {
            const uint32_t* src = static_cast<const uint32_t*>(p.src[s]);
            uint32_t* dst = static_cast<uint32_t*>(p.dst[s]);
            for (uint32_t i = t; i < p.bytes[s] / 4; i += nt) dst[i] = src[i];
        } else {
            const uint8_t* src = static_cast<const uint8_t*>(p.src[s]);
            uint8_t* dst = static_cast<uint8_t*>(p.dst[s]);
            for (uint32_t i = t; i < p.bytes[s]; i += nt) dst[i] = src[i];
        }
    }
}

}  // namespace hg
