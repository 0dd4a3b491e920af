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

// Tuning knobs (nuna_set_option / environment).  Launch paths work on a snapshot taken under the
// context's mutex, so a concurrent nuna_set_option never changes a launch half way through.
struct Options {
    unsigned long long timeout_ns = 1000000000ull;
    int blocks = 0;                      // NUNA_BLOCKS: cap on every grid (0 = none)
    int unroll = 0;                      // NUNA_UNROLL
    int coloc = 0;                       // NUNA_COLOC: destinations of a tile per block (2, 4, 8)
    size_t auto_min_bytes = 0;           // NUNA_PLACE_AUTO picks a placement-aware kernel from this size per rank
    int domains = 0;                     // NUNA_DOMAINS: SM domains the work-list planner deals groups to (0 = what the probe found)
    int stage_vecs = 0;                  // NUNA_STAGE_VECS: vectors per source per tile of the staged one-shot (0 = by size)
    int twoshot_vecs = 0;                // NUNA_TWOSHOT_VECS: vectors per tile of the flag-synchronised two-shot (0 = by size)
    int ag_bulk_vecs = 0;                // NUNA_AG_BULK_VECS: > 0 = allgather through the bulk-copy engine with tiles of that many vectors
    int regs_vecs = 0;                   // NUNA_REGS_VECS: vectors per tile of the register-sharing one-shot (0 = by size)
    int prefetch = 0;                    // NUNA_PREFETCH: 1 = no L2 prefetch ahead of the dependent-launch wait
    int keep_shard = 0;                  // NUNA_KEEP_SHARD: do not discard consumed shard lines from L2 (measurement aid)
};

struct Context {
    int device = -1;
    int num_sms = 0;
    size_t l2_bytes = 0;
    BarrierWords* bw = nullptr;          // flag-barrier words, work cursor, epoch + latched status, device memory
    void* scratch = nullptr;             // two-shot shard intermediate, followed by its per-tile ready flags
    unsigned* flags = nullptr;           // one word per smallest tile of the scratch (inside the same allocation)
    size_t scratch_bytes = 0;
    std::vector<void*> retired_scratch;  // outgrown scratch allocations: captured graphs may still name them
    void* staging = nullptr;             // device copies of host buffers (nuna_allreduce_host)
    size_t staging_bytes = 0;
    cudaStream_t stream = nullptr;       // private stream of the host-buffer entry point
    Options opt;
    nuna_topology_t topology = {};       // last probe result (have_topology says whether it is valid)
    bool have_topology = false;
    std::map<std::tuple<int, size_t, int, int>, SmPlan> sm_plans;   // key: ranks, vectors, co-location, domains
    std::vector<unsigned*> retired_plans; // plans of an earlier topology, freed at shutdown
    std::mutex mutex;                    // guards opt, scratch / flags, topology and plans
    std::mutex host_mutex;               // serialises nuna_allreduce_host (staging buffers, private stream)
};

inline Options snapshot(Context* c)
{
    std::lock_guard<std::mutex> lock(c->mutex);
    return c->opt;
}

extern std::atomic<unsigned long long> g_launches;

int get_context(Context** out);
int ensure_scratch(Context* c, size_t bytes);
int check_args(const void* const* src, void* const* dst, int nranks, size_t src_elems, size_t dst_elems,
               int dtype, unsigned flags, bool device_ptrs);
void plan_oneshot_lists(const nuna_topology_t* topo, int num_sms, int nranks, size_t ntiles, size_t tile_bytes,
                        bool generic, int domains, std::vector<std::vector<unsigned>>& lists);
size_t elem_size(int dtype);
int prepare_oneshot(Context* c, int nranks, int dtype, size_t count, unsigned flags);
int launch_oneshot(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream);
int launch_twoshot(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream);
int launch_twoshot_flags(int num_sms, int blocks_override, const RankPtrs& p, int nranks, int dtype, size_t count,
                         unsigned tv, unsigned min_tv, uint4* scratch, unsigned* tile_flags, BarrierWords* bw,
                         unsigned long long timeout_ns, bool pdl, unsigned debug_bits, cudaStream_t stream);
bool chain_persistent_pays_off(int dtype, size_t count);
int launch_reduce_scatter(Context* c, const RankPtrs& p, int nranks, int dtype, size_t shard, unsigned flags,
                          cudaStream_t stream);
int launch_allgather(Context* c, const RankPtrs& p, int nranks, size_t shard_bytes, unsigned flags, cudaStream_t stream);
int launch_chain_persistent(Context* c, const ChainSets& sets, int nsets, int nnodes, int nranks, int dtype, size_t count,
                            cudaStream_t stream);
bool chain_persistent_supported(const Context* c, int nsets, int nranks, int dtype, size_t count);

}  // namespace nuna
