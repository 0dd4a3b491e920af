// Chain of back-to-back allreduces: one decode step's per-layer collectives, as a CUDA graph of one
// kernel per node or, for small nodes, as a single kernel (k_chain_persistent) that loops over the nodes.
//
// The nodes are captured once from a private stream and replayed with one graph launch, so control
// never returns to the host inside a step.  Node k works on buffer set k mod nsets and may not
// start reading before node k-1 has finished writing: the nodes are ordinary stream-ordered kernel
// launches, optionally with programmatic dependent launch so that a node's launch latency overlaps
// its predecessor's drain (the wait inside the kernel still orders all memory accesses).
#include "nuna_internal.h"

#include <vector>

namespace nuna {

struct Chain {
    cudaGraphExec_t exec = nullptr;      // graph form: one kernel node per allreduce
    bool persistent = false;             // single-kernel form: the fields below
    ChainSets sets = {};
    int nsets = 0, nranks = 0, dtype = 0;
    size_t count = 0;
    Context* ctx = nullptr;
    int device = -1;
    int nnodes = 0;
};

}  // namespace nuna

using namespace nuna;

extern "C" {

int nuna_chain_create(const void* const* src_sets, void* const* dst_sets, int nsets, int nnodes, int nranks,
                      size_t count, int dtype, unsigned flags, int two_shot, void** chain_out)
{
    if (!chain_out || nsets < 1 || nnodes < 1 || nnodes > (1 << 16)) return NUNA_ERR_INVALID_ARG;
    *chain_out = nullptr;
    if (!src_sets || !dst_sets || count == 0) return NUNA_ERR_INVALID_ARG;
    if (nranks < 1) return NUNA_ERR_INVALID_ARG;
    if (nranks > NUNA_MAX_RANKS) return NUNA_ERR_TOO_MANY_RANKS;
    if (!two_shot && (flags & NUNA_TWOSHOT_PUT)) return NUNA_ERR_INVALID_ARG;
    for (int s = 0; s < nsets; ++s) {
        const int st = check_args(src_sets + (size_t)s * nranks, dst_sets + (size_t)s * nranks, nranks, count, count,
                                  dtype, flags, true);
        if (st != NUNA_OK) return st;
    }
    Context* c = nullptr;
    int st = get_context(&c);
    if (st != NUNA_OK) return st;
    if ((flags & NUNA_CHAIN_PERSISTENT) && (flags & NUNA_CHAIN_GRAPH)) return NUNA_ERR_INVALID_ARG;
    const bool can_persist = !two_shot && chain_persistent_supported(c, nsets, nranks, dtype, count);
    if ((flags & NUNA_CHAIN_PERSISTENT) && !can_persist) return NUNA_ERR_INVALID_ARG;
    if (can_persist && !(flags & NUNA_CHAIN_GRAPH) &&
        ((flags & NUNA_CHAIN_PERSISTENT) || chain_persistent_pays_off(dtype, count))) {
        Chain* ch = new Chain();
        ch->persistent = true;
        ch->device = c->device;
        ch->ctx = c;
        ch->nnodes = nnodes;
        ch->nsets = nsets;
        ch->nranks = nranks;
        ch->dtype = dtype;
        ch->count = count;
        for (int s = 0; s < nsets; ++s)
            for (int r = 0; r < nranks; ++r) {
                ch->sets.s[s].src[r] = reinterpret_cast<const uint4*>(src_sets[(size_t)s * nranks + r]);
                ch->sets.s[s].dst[r] = reinterpret_cast<uint4*>(dst_sets[(size_t)s * nranks + r]);
            }
        *chain_out = ch;
        return NUNA_OK;
    }
    flags &= ~(NUNA_CHAIN_PERSISTENT | NUNA_CHAIN_GRAPH);
    if (two_shot && !(flags & NUNA_TWOSHOT_PUT)) {
        std::lock_guard<std::mutex> lock(c->mutex);
        if ((st = ensure_scratch(c, (count * elem_size(dtype) + 15) & ~(size_t)15)) != NUNA_OK) return st;
    }
    if (!two_shot && (st = prepare_oneshot(c, nranks, dtype, count, flags)) != NUNA_OK) return st;
    cudaStream_t cap = nullptr;
    if (cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking) != cudaSuccess) return NUNA_ERR_CUDA;
    cudaGraph_t graph = nullptr;
    st = NUNA_OK;
    if (cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        cudaStreamDestroy(cap);
        return NUNA_ERR_CUDA;
    }
    for (int k = 0; k < nnodes && st == NUNA_OK; ++k) {
        const int s = k % nsets;
        RankPtrs p = {};
        for (int r = 0; r < nranks; ++r) {
            p.src[r] = reinterpret_cast<const uint4*>(src_sets[(size_t)s * nranks + r]);
            p.dst[r] = reinterpret_cast<uint4*>(dst_sets[(size_t)s * nranks + r]);
        }
        st = two_shot ? launch_twoshot(c, p, nranks, dtype, count, flags, cap)
                      : launch_oneshot(c, p, nranks, dtype, count, flags, cap);
    }
    const cudaError_t e = cudaStreamEndCapture(cap, &graph);
    cudaStreamDestroy(cap);
    if (st != NUNA_OK || e != cudaSuccess || !graph) {
        if (graph) cudaGraphDestroy(graph);
        return st != NUNA_OK ? st : NUNA_ERR_CUDA;
    }
    Chain* ch = new Chain();
    ch->device = c->device;
    ch->nnodes = nnodes;
    const cudaError_t ie = cudaGraphInstantiate(&ch->exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ie != cudaSuccess) {
        delete ch;
        return NUNA_ERR_CUDA;
    }
    *chain_out = ch;
    return NUNA_OK;
}

int nuna_chain_launch(void* chain, void* stream)
{
    Chain* ch = static_cast<Chain*>(chain);
    if (!ch) return NUNA_ERR_INVALID_ARG;
    if (ch->persistent)
        return launch_chain_persistent(ch->ctx, ch->sets, ch->nsets, ch->nnodes, ch->nranks, ch->dtype, ch->count,
                                       (cudaStream_t)stream);
    if (!ch->exec) return NUNA_ERR_INVALID_ARG;
    if (cudaGraphLaunch(ch->exec, (cudaStream_t)stream) != cudaSuccess) return NUNA_ERR_CUDA;
    g_launches.fetch_add((unsigned long long)ch->nnodes, std::memory_order_relaxed);
    return NUNA_OK;
}

int nuna_chain_destroy(void* chain)
{
    Chain* ch = static_cast<Chain*>(chain);
    if (!ch) return NUNA_OK;
    if (ch->exec) cudaGraphExecDestroy(ch->exec);
    delete ch;
    return NUNA_OK;
}

}  // extern "C"
