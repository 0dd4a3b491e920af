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

// Kernel argument of the single-kernel chain: the buffer sets its nodes rotate over, by value.
constexpr int kMaxChainSets = 8;
struct ChainSets {
    RankPtrs s[kMaxChainSets];
};

// Control words of the in-kernel synchronisation and the latched device status, in device memory.
struct BarrierWords {
    unsigned int arrive;      // flag barrier: arrivals of the current round (atomics land here)
    unsigned int pad0[31];
    unsigned int epoch;       // flag barrier: bumped by the last arriver; polled by everyone else -- on its own
    unsigned int pad1[31];    // 128-byte line so that the polling loads do not queue behind the arrival atomics
    unsigned int status;      // latched NUNA_ERR_TIMEOUT
    unsigned int pad2;
    unsigned long long ticket;// fused two-shot: launch epoch in the high half, next work-item ticket in the low half
    unsigned int pad3[28];
};
static_assert(sizeof(BarrierWords) == 384, "three 128-byte lines");

}  // namespace nuna
