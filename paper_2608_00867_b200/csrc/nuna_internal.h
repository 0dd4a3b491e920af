// Shared by the library's own translation units (never by the oracle).
#pragma once
#include <cuda_runtime.h>

#include <atomic>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "../../include/nuna.h"
#include "nuna_types.h"

namespace nuna {

constexpr int kMaxDevices = 64;

// Device-resident per-SM work lists of one (nranks, count, co-location) one-shot shape.
struct SmPlan {
    unsigned* base = nullptr;            // one allocation: off | tiles | cursor | present | ctl
    unsigned* off = nullptr;
    unsigned* tiles = nullptr;
    unsigned* cursor = nullptr;
    unsigned* present = nullptr;
    unsigned* ctl = nullptr;
    unsigned total = 0;
    unsigned nonempty = 0;
};

struct Context {
    int device = -1;
    int num_sms = 0;
    size_t l2_bytes = 0;
    BarrierWords* bw = nullptr;          // flag-barrier words + latched status, device memory
    void* scratch = nullptr;             // two-shot shard intermediate
    size_t scratch_bytes = 0;
    void* staging = nullptr;             // device copies of host buffers (nuna_allreduce_host)
    size_t staging_bytes = 0;
    cudaStream_t stream = nullptr;       // private stream of the host-buffer entry point
    unsigned long long timeout_ns = 1000000000ull;
    int blocks_override = 0;             // NUNA_BLOCKS
    int unroll_override = 0;             // NUNA_UNROLL
    int coloc_override = 0;              // NUNA_COLOC: destinations of a tile per block (2, 4, 8)
    size_t auto_min_bytes = 0;           // NUNA_PLACE_AUTO picks the aware kernel from this size per rank
    nuna_topology_t topology = {};       // last probe result (have_topology says whether it is valid)
    bool have_topology = false;
    std::map<std::tuple<int, size_t, int>, SmPlan> sm_plans;
    std::vector<unsigned*> retired_plans; // plans of an earlier topology, freed at shutdown
    std::mutex mutex;
};

extern std::atomic<unsigned long long> g_launches;

int get_context(Context** out);
int ensure_scratch(Context* c, size_t bytes);
int check_args(const void* const* src, void* const* dst, int nranks, size_t src_elems, size_t dst_elems,
               int dtype, unsigned flags, bool device_ptrs);
void plan_oneshot_lists(const nuna_topology_t* topo, int num_sms, int nranks, size_t ntiles, size_t tile_bytes,
                        bool generic, std::vector<std::vector<unsigned>>& lists);
size_t elem_size(int dtype);
int prepare_oneshot(Context* c, int nranks, int dtype, size_t count, unsigned flags);
int launch_oneshot(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream);
int launch_twoshot(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream);
int launch_reduce_scatter(Context* c, const RankPtrs& p, int nranks, int dtype, size_t shard, unsigned flags,
                          cudaStream_t stream);
int launch_allgather(Context* c, const RankPtrs& p, int nranks, size_t shard_bytes, unsigned flags, cudaStream_t stream);

}  // namespace nuna
