// Plain types shared by the library's host code and its kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace nuna {

constexpr int kMaxRanks = 16;
constexpr int kThreads = 256;            // threads per block, every kernel

// Kernel argument: the rank buffers, by value.
struct RankPtrs {
    const uint4* src[kMaxRanks];
    uint4* dst[kMaxRanks];
};

// Flag-barrier words and the latched device status, in device memory.
struct BarrierWords {
    unsigned int arrive;
    unsigned int epoch;
    unsigned int status;
    unsigned int work[2];     // dynamic work cursors of the fused two-shot's two phases (zero between launches)
    unsigned int pad[3];
};

}  // namespace nuna
