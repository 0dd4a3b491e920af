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
    unsigned int arrive;      // arrivals of the current round (atomics land here)
    unsigned int pad0[31];
    unsigned int epoch;       // bumped by the last arriver; polled by everyone else -- on its own 128-byte
    unsigned int pad1[31];    // line so that the polling loads do not queue behind the arrival atomics
    unsigned int status;
    unsigned int work[2];     // dynamic work cursors of the fused two-shot's two phases (zero between launches)
    unsigned int pad2[29];
};

}  // namespace nuna
