// Host side of the C ABI: argument checks, per-device context, launch configuration.
#include "nuna_internal.h"
#include "nuna_debug.h"
#include "nuna_kernels.cuh"

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <vector>

namespace nuna {

std::atomic<unsigned long long> g_launches{0};
static std::mutex g_ctx_mutex;
static Context* g_ctx[kMaxDevices] = {};

static int static_status_read_and_clear(unsigned* out);     // the allocation-free entry point's status word (end of file)
constexpr unsigned kMinFlagTileVec = 16;                    // smallest two-shot tile (vectors): 256 bytes of shard per flag
constexpr unsigned kStaticTileVec = 128;                    // tile of the allocation-free entry point: 2 KiB of shard per flag

static int env_int(const char* name, int fallback)
{
    const char* s = getenv(name);
    return (s && *s) ? atoi(s) : fallback;
}

int init_barrier_words(Context* c)
{
    return cudaMemset(c->bw, 0, sizeof(BarrierWords)) == cudaSuccess ? NUNA_OK : NUNA_ERR_CUDA;
}

// After a latched timeout the barrier's arrival counter is in an undefined state: zero it and clear the
// status, but keep both epochs moving forward -- the ready flags of earlier launches must never match a
// later launch's epoch.  The device is idle (the caller synchronised).
static int rewind_barrier_words(BarrierWords* dev, const BarrierWords& seen)
{
    BarrierWords h = {};
    h.epoch = seen.epoch + 1u;
    h.ticket = ((seen.ticket >> 32) + 1ull) << 32;
    return cudaMemcpy(dev, &h, sizeof h, cudaMemcpyHostToDevice) == cudaSuccess ? NUNA_OK : NUNA_ERR_CUDA;
}

// Returns the current device's context, creating it on first use (allocates: not capturable).
int get_context(Context** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NUNA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_ctx_mutex);
    if (!g_ctx[dev]) {
        Context* c = new Context();
        c->device = dev;
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { delete c; return NUNA_ERR_CUDA; }
        c->num_sms = prop.multiProcessorCount;
        c->l2_bytes = (size_t)prop.l2CacheSize;
        if (cudaMalloc(&c->bw, sizeof(BarrierWords)) != cudaSuccess) { delete c; return NUNA_ERR_CUDA; }
        if (init_barrier_words(c) != NUNA_OK) { cudaFree(c->bw); delete c; return NUNA_ERR_CUDA; }
        c->opt.timeout_ns = (unsigned long long)env_int("NUNA_TIMEOUT_MS", 1000) * 1000000ull;
        c->opt.blocks = env_int("NUNA_BLOCKS", 0);
        c->opt.unroll = env_int("NUNA_UNROLL", 0);
        c->opt.auto_min_bytes = (size_t)env_int("NUNA_AUTO_MIN_BYTES", 0);
        c->opt.coloc = env_int("NUNA_COLOC", 0);
        c->opt.domains = env_int("NUNA_DOMAINS", 0);
        c->opt.stage_vecs = env_int("NUNA_STAGE_VECS", 0);
        c->opt.twoshot_vecs = env_int("NUNA_TWOSHOT_VECS", 0);
        c->opt.keep_shard = env_int("NUNA_KEEP_SHARD", 0);
        c->opt.ag_bulk_vecs = env_int("NUNA_AG_BULK_VECS", 0);
        c->opt.regs_vecs = env_int("NUNA_REGS_VECS", 0);
        c->opt.prefetch = env_int("NUNA_PREFETCH", 0);
        g_ctx[dev] = c;
    }
    *out = g_ctx[dev];
    return NUNA_OK;
}

// Grows the two-shot scratch (shard intermediate + one ready flag per smallest tile of it).  The caller holds
// c->mutex.  An outgrown allocation is never freed before nuna_shutdown: a CUDA graph captured earlier
// (a chain, or a user's capture of a two-shot call) still carries its address as a kernel argument.
int ensure_scratch(Context* c, size_t bytes)
{
    if (bytes <= c->scratch_bytes && c->scratch) return NUNA_OK;
    const size_t want = (std::max<size_t>(bytes, 4096) + 4095) & ~(size_t)4095;
    const size_t nflags = want / (kMinFlagTileVec * 16) + 1;         // one ready flag per smallest tile
    void* p = nullptr;
    if (cudaMalloc(&p, want + nflags * sizeof(unsigned)) != cudaSuccess) return NUNA_ERR_CUDA;
    // flags start at zero; epochs start at one, so a fresh flag never reads as "ready"
    if (cudaMemset(static_cast<char*>(p) + want, 0, nflags * sizeof(unsigned)) != cudaSuccess) {
        cudaFree(p);
        return NUNA_ERR_CUDA;
    }
    if (c->scratch) c->retired_scratch.push_back(c->scratch);
    c->scratch = p;
    c->flags = reinterpret_cast<unsigned*>(static_cast<char*>(p) + want);
    c->scratch_bytes = want;
    return NUNA_OK;
}

// ---- argument validation -------------------------------------------------------------------

size_t elem_size(int dtype) { return dtype == NUNA_F32 ? 4 : 2; }
static size_t elems_per_vec(int dtype) { return 16 / elem_size(dtype); }

static bool overlaps(const void* a, size_t na, const void* b, size_t nb)
{
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return na && nb && a0 < b0 + nb && b0 < a0 + na;
}

int check_args(const void* const* src, void* const* dst, int nranks, size_t src_elems, size_t dst_elems,
               int dtype, unsigned flags, bool device_ptrs)
{
    if (nranks > NUNA_MAX_RANKS) return NUNA_ERR_TOO_MANY_RANKS;
    if (nranks < 1) return NUNA_ERR_INVALID_ARG;
    if (dtype != NUNA_BF16 && dtype != NUNA_F16 && dtype != NUNA_F32) return NUNA_ERR_UNSUPPORTED_DTYPE;
    if ((flags & ~(NUNA_PLACE_MASK | NUNA_TWOSHOT_PUT | NUNA_HINT_RESIDENT | NUNA_LAUNCH_PDL | NUNA_PLACE_SM_LISTS |
                   NUNA_PLACE_CLUSTER | NUNA_PLACE_STAGED | NUNA_TWOSHOT_SYNC | NUNA_CHAIN_PERSISTENT | NUNA_CHAIN_GRAPH |
                   NUNA_TWOSHOT_SYS_SCOPE | NUNA_PLACE_REGS)) != 0u ||
        (flags & NUNA_PLACE_MASK) == 3u)
        return NUNA_ERR_INVALID_ARG;
    if (src_elems > ((size_t)1 << 40) || dst_elems > ((size_t)1 << 40)) return NUNA_ERR_TOO_LARGE;
    if (src_elems == 0 && dst_elems == 0) return NUNA_OK;
    if (!src || !dst) return NUNA_ERR_INVALID_ARG;
    for (int r = 0; r < nranks; ++r) {
        if (!src[r] || !dst[r]) return NUNA_ERR_INVALID_ARG;
        if (device_ptrs && (((uintptr_t)src[r] | (uintptr_t)dst[r]) & 15u)) return NUNA_ERR_ALIGNMENT;
    }
    const size_t sb = src_elems * elem_size(dtype), db = dst_elems * elem_size(dtype);
    for (int d = 0; d < nranks; ++d) {
        for (int r = 0; r < nranks; ++r)
            if (overlaps(dst[d], db, src[r], sb)) return NUNA_ERR_ALIAS;
        for (int e = d + 1; e < nranks; ++e)
            if (overlaps(dst[d], db, dst[e], db)) return NUNA_ERR_ALIAS;
    }
    return NUNA_OK;
}

// Bits that only nuna_chain_create understands.
static bool has_chain_bits(unsigned flags) { return (flags & (NUNA_CHAIN_PERSISTENT | NUNA_CHAIN_GRAPH)) != 0u; }

static RankPtrs make_ptrs(const void* const* src, void* const* dst, int nranks)
{
    RankPtrs p;
    memset(&p, 0, sizeof p);
    for (int r = 0; r < nranks; ++r) {
        p.src[r] = reinterpret_cast<const uint4*>(src[r]);
        p.dst[r] = reinterpret_cast<uint4*>(dst[r]);
    }
    return p;
}

// ---- launch configuration --------------------------------------------------------------------

// Vectors per thread per item.  One: with one work item per block and N independent 16-byte loads in
// flight per thread, more vectors per thread only mean fewer blocks (measured at 2 and 4 ranks: 64 KiB
// per rank 1.43 us with one vector, 1.64 us with four; no difference at 16 MiB).  NUNA_OPT_UNROLL
// overrides it for experiments.
static int pick_unroll(const Options& o, int nranks)
{
    int u = 1;
    if (o.unroll == 1 || o.unroll == 2 || o.unroll == 4) u = o.unroll;
    while (u > 1 && u * nranks > 16) u >>= 1;
    return u;
}

// Resident blocks per SM of a kernel, looked up once per device (the cache is one slot per device and
// kernel instantiation; racing first calls compute the same value).
template <typename K>
static int occupancy(K kernel, std::atomic<int>* cache /* [kMaxDevices] */)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kThreads, 0) != cudaSuccess || n < 1) n = 1;
        cache[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}
#define NUNA_OCC(kernel) ([&]() { static std::atomic<int> cache_[kMaxDevices]; return occupancy(kernel, cache_); }())

// Grid size: `waves` x (SMs x resident blocks per SM), never more than the work items.  Streaming
// kernels (two-shot put, reduce-scatter, allgather) run one item per block (waves = 0: no cap): leaving
// the balancing to the hardware block scheduler measured 0.99 of the copy peak at 64 MiB per rank
// against 0.90 for a persistent grid-stride loop.  The one-shot wants its N readers of a tile close in
// time so that re-reads hit L2: four waves measured best (0.70 of peak at 64 MiB against 0.63 for one
// wave and 0.62 for an uncapped grid).
static unsigned pick_grid(const Context* c, const Options& o, size_t nitems, int blocks_per_sm, int waves = 1)
{
    size_t cap = waves > 0 ? (size_t)c->num_sms * (size_t)blocks_per_sm * (size_t)waves : ((size_t)1 << 22);
    if (o.blocks > 0) cap = (size_t)o.blocks;
    return (unsigned)std::max<size_t>(1, std::min(nitems, cap));
}

constexpr unsigned kLaunchPlain = 0u, kLaunchCooperative = 1u, kLaunchPdl = 2u;

// Programmatic dependent launch pays off while a kernel is short enough for its launch latency to
// matter.  For the one-shot it was measured to cost a few percent from about 16 MiB of sources (its
// multi-wave grid competes with the successor's early blocks), so it is dropped there; the streaming
// kernels (two-shot put, reduce-scatter, allgather) keep it at every size (4 MiB per rank: 12.6 -> 12.0 us).
static unsigned launch_mode(unsigned flags, size_t total_src_bytes = 0)
{
    return ((flags & NUNA_LAUNCH_PDL) && total_src_bytes <= ((size_t)16 << 20)) ? kLaunchPdl : kLaunchPlain;
}

static thread_local unsigned t_cluster_dim = 0;           // > 0: next launch() uses clusters of this many blocks
static thread_local unsigned t_dyn_smem = 0;              // next launch() requests this much dynamic shared memory

template <typename... Args, typename... Act>
static int launch(void (*kernel)(Args...), unsigned grid, cudaStream_t stream, unsigned mode, Act&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = t_dyn_smem;
    t_dyn_smem = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[3];
    int nattr = 0;
    if (t_cluster_dim > 0) {
        attr[nattr].id = cudaLaunchAttributeClusterDimension;
        attr[nattr].val.clusterDim.x = t_cluster_dim;
        attr[nattr].val.clusterDim.y = 1;
        attr[nattr].val.clusterDim.z = 1;
        ++nattr;
        t_cluster_dim = 0;
    }
    if (mode & kLaunchCooperative) {
        attr[nattr].id = cudaLaunchAttributeCooperative;
        attr[nattr].val.cooperative = 1;
        ++nattr;
    } else if (mode & kLaunchPdl) {
        attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[nattr].val.programmaticStreamSerializationAllowed = 1;
        ++nattr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = nattr;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<Args>(args)...);
    if (e != cudaSuccess) {
        fprintf(stderr, "nuna: kernel launch failed: %s\n", cudaGetErrorString(e));
        return NUNA_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return NUNA_OK;
}

// Compile-time dispatch over the rank count N and the unroll factor U (N * U <= 16 vectors in flight).
template <int V> using IC = std::integral_constant<int, V>;

template <int N, int U, typename F>
static int dispatch_dt(int dtype, F&& f)
{
    switch (dtype) {
        case NUNA_BF16: return f(IC<N>{}, IC<U>{}, IC<kBf16>{});
        case NUNA_F16: return f(IC<N>{}, IC<U>{}, IC<kF16>{});
        case NUNA_F32: return f(IC<N>{}, IC<U>{}, IC<kF32>{});
        default: return NUNA_ERR_UNSUPPORTED_DTYPE;
    }
}

template <int N, typename F>
static int dispatch_u(int u, int dtype, F&& f)
{
    if constexpr (N * 4 <= 16) { if (u == 4) return dispatch_dt<N, 4>(dtype, f); }
    if constexpr (N * 2 <= 16) { if (u >= 2) return dispatch_dt<N, 2>(dtype, f); }
    return dispatch_dt<N, 1>(dtype, f);
}

template <typename F>
static int dispatch(int nranks, int u, int dtype, F&& f)
{
    switch (nranks) {
        case 1: return dispatch_u<1>(u, dtype, f);   case 2: return dispatch_u<2>(u, dtype, f);
        case 3: return dispatch_u<3>(u, dtype, f);   case 4: return dispatch_u<4>(u, dtype, f);
        case 5: return dispatch_u<5>(u, dtype, f);   case 6: return dispatch_u<6>(u, dtype, f);
        case 7: return dispatch_u<7>(u, dtype, f);   case 8: return dispatch_u<8>(u, dtype, f);
        case 9: return dispatch_u<9>(u, dtype, f);   case 10: return dispatch_u<10>(u, dtype, f);
        case 11: return dispatch_u<11>(u, dtype, f); case 12: return dispatch_u<12>(u, dtype, f);
        case 13: return dispatch_u<13>(u, dtype, f); case 14: return dispatch_u<14>(u, dtype, f);
        case 15: return dispatch_u<15>(u, dtype, f); case 16: return dispatch_u<16>(u, dtype, f);
        default: return NUNA_ERR_TOO_MANY_RANKS;
    }
}
#define NUNA_NUD(n_, u_, d_) constexpr int N = decltype(n_)::value; constexpr int U = decltype(u_)::value; \
    constexpr int DT = decltype(d_)::value; (void)U; (void)DT

static size_t ceil_div(size_t a, size_t b) { return (a + b - 1) / b; }

// ---- collectives ---------------------------------------------------------------------------------

// NUNA_PLACE_AUTO picks, per size, the one-shot kernel that was measured fastest on B200, never one that is
// slower than the round-robin baseline.  Measured at 2, 3, 4, 8 and 16 ranks, 8 KiB ... 4 MiB per rank
// (us per graph node, 8 ranks; round-robin | group through L1 | group through registers):
//   dependent launch, cold:      8 KiB 1.60 | 1.16 | 1.26   64 KiB 1.78 | 1.90 | 1.41   512 KiB 3.38 | 3.65 | 2.09   4 MiB 15.6 | 17.2 | 11.8
//   dependent launch, resident:  8 KiB 1.18 | 1.16 | 1.05   64 KiB 1.21 | 1.19 | 1.09   512 KiB 2.99 | 2.48 | 1.64   4 MiB 15.1 | 17.1 | 10.5
//   plain launch, resident:      8 KiB 1.58 | 1.55 | 1.53   64 KiB 1.62 | 1.59 | 1.58   512 KiB 3.41 | 2.88 | 2.15   4 MiB 15.1 | 17.1 | 11.2
//   plain launch, cold:          8 KiB 2.02 | 1.56 | 2.00   64 KiB 2.16 | 2.46 | 2.27   512 KiB 3.78 | 4.24 | 3.29   4 MiB 15.5 | 17.2 | 12.5
// The group that shares its tile through registers wins at every size behind a dependent launch and on
// L2-resident sources; launched plainly on cold sources it wins from 1 MiB of sources in total (2 MiB below 8
// ranks) and the round-robin kernel is kept below that.  The other co-located forms (through L1, through shared
// memory) stay opt-in.
enum class OneShotKernel { RoundRobin, Group, Staged, Regs };

static OneShotKernel auto_kernel(const Context* c, const Options& o, int nranks, size_t bytes, unsigned flags)
{
    (void)c;
    if (nranks < 2) return OneShotKernel::RoundRobin;
    if (bytes < o.auto_min_bytes) return OneShotKernel::RoundRobin;
    if (flags & (NUNA_LAUNCH_PDL | NUNA_HINT_RESIDENT)) return OneShotKernel::Regs;
    const size_t total = bytes * (size_t)nranks;
    const size_t from = nranks >= 8 ? ((size_t)1 << 20) : ((size_t)2 << 20);
    return total >= from ? OneShotKernel::Regs : OneShotKernel::RoundRobin;
}


// ---- per-SM work lists for the one-shot (Algorithm 1 applied to its regular workload) ----------------
//
// Thread blocks = work items (tile, d); item (t, d) touches the N source chunks of tile t and the
// destination chunk (d, t).  Domains and the order of SMs inside a domain come from the probe
// (nearest = lowest mean hit latency).  `domains` = 0 uses what the probe found (one, or the two dies);
// a larger count splits every probed domain into equal latency quantiles (the paper's sweep over the
// number of routing domains, Section 6.5), 1 forces a single domain.  The per-SM budget R_max is
// ceil(groups per domain / SMs of the smallest domain) whole groups, so a small workload fills only the
// nearest SMs, one group each, and a large one spreads evenly.  Up to kGenericPlanTiles tiles the lists
// are produced by the general planner (nuna_plan_placement); beyond that by the closed form it reduces to
// for this workload (tile t -> domain t mod D, SMs of the domain filled in preference order), which the
// host tests check against the general planner.
constexpr size_t kGenericPlanTiles = 1024;

void plan_oneshot_lists(const nuna_topology_t* topo, int num_sms, int nranks, size_t ntiles, size_t tile_bytes,
                        bool generic, int domains, std::vector<std::vector<unsigned>>& lists)
{
    lists.assign((size_t)num_sms, {});
    const bool split = topo && topo->verdict == NUNA_TOPO_NONUNIFORM && topo->num_domains == 2 && domains != 1;
    const int base_domains = split ? 2 : 1;
    std::vector<int> dom(num_sms, 0), rank(num_sms, 0), order(num_sms);
    for (int s = 0; s < num_sms; ++s) {
        order[s] = s;
        if (split && s < NUNA_MAX_SMS) dom[s] = topo->sm_domain[s];
    }
    if (topo && topo->sms_reported > 0)
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
            const float la = a < NUNA_MAX_SMS ? topo->sm_lat_hit[a] : 0.f, lb = b < NUNA_MAX_SMS ? topo->sm_lat_hit[b] : 0.f;
            return la < lb;
        });
    for (int i = 0; i < num_sms; ++i) rank[order[i]] = i;
    // more domains than the probe found: cut each probed domain into `sub` latency quantiles
    int D = base_domains;
    if (domains > base_domains) {
        const int sub = std::max(1, std::min(domains / base_domains, num_sms / base_domains));
        std::vector<int> size(base_domains, 0), seen(base_domains, 0);
        for (int s = 0; s < num_sms; ++s) size[dom[s]]++;
        std::vector<int> fine(num_sms, 0);
        for (int i = 0; i < num_sms; ++i) {                          // in preference order
            const int s = order[i], b = dom[s];
            const int q = std::min(sub - 1, (int)((long long)seen[b]++ * sub / std::max(1, size[b])));
            fine[s] = b * sub + q;
        }
        dom = fine;
        D = base_domains * sub;
    }
    std::vector<int> dsize(D, 0);
    for (int s = 0; s < num_sms; ++s) dsize[dom[s]]++;
    const int smallest = std::max(1, *std::min_element(dsize.begin(), dsize.end()));
    const size_t per_domain = ceil_div(ntiles, (size_t)D);
    const size_t budget = std::max<size_t>(1, ceil_div(per_domain, (size_t)smallest));        // groups per SM
    if (generic) {
        const int N = nranks;
        std::vector<int> tb_gpu(ntiles * N, 0), begin(ntiles * N + 1, 0), chunks;
        chunks.reserve(ntiles * N * (N + 1));
        for (size_t t = 0; t < ntiles; ++t)
            for (int d = 0; d < N; ++d) {
                for (int r = 0; r < N; ++r) chunks.push_back((int)(r * ntiles + t));
                chunks.push_back((int)((N + d) * ntiles + t));
                begin[t * N + d + 1] = (int)chunks.size();
            }
        std::vector<long long> cbytes(2 * (size_t)N * ntiles, (long long)tile_bytes);
        std::vector<int> stack(num_sms, 0), m_compute(ntiles * N, -1);
        nuna_plan_input_t in = {};
        in.num_tbs = (int)(ntiles * N); in.tb_gpu = tb_gpu.data(); in.tb_chunk_begin = begin.data(); in.tb_chunks = chunks.data();
        in.num_chunks = (int)cbytes.size(); in.chunk_bytes = cbytes.data();
        in.num_cus = num_sms; in.cu_domain = dom.data(); in.cu_rank = rank.data();
        in.num_stacks = 1; in.cu_stack = stack.data();
        in.r_max_cu = (long long)(budget * (size_t)N * (size_t)(N + 1) * tile_bytes);
        in.r_max_stack = (long long)1 << 60;
        in.nar_max = D;
        if (nuna_plan_placement(&in, m_compute.data(), nullptr, nullptr, nullptr) == NUNA_OK) {
            for (size_t t = 0; t < ntiles; ++t) lists[(size_t)m_compute[t * N]].push_back((unsigned)t);
            return;
        }
        lists.assign((size_t)num_sms, {});
    }
    // closed form
    std::vector<std::vector<int>> dom_sms(D);
    for (int i = 0; i < num_sms; ++i) dom_sms[dom[order[i]]].push_back(order[i]);
    std::vector<size_t> used(D, 0);
    for (size_t t = 0; t < ntiles; ++t) {
        const int d = (int)(t % (size_t)D);
        size_t slot = used[d]++ / budget;
        if (slot >= dom_sms[d].size()) slot = dom_sms[d].size() - 1;      // cannot happen with the budget above
        lists[(size_t)dom_sms[d][slot]].push_back((unsigned)t);
    }
}

// Looks up (or builds and uploads) the work lists of a shape.  The plan is returned BY VALUE: its device
// tables stay allocated until nuna_shutdown even when a later probe retires the plan, so a copy taken
// under the lock stays usable after the lock is dropped.
static int get_sm_plan(Context* c, int nranks, size_t nvec, int coloc, int domains, cudaStream_t stream, SmPlan* out)
{
    std::lock_guard<std::mutex> lock(c->mutex);
    const auto key = std::make_tuple(nranks, nvec, coloc, domains);
    auto it = c->sm_plans.find(key);
    if (it == c->sm_plans.end()) {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone)
            return NUNA_ERR_CAPTURING;                 // building a plan allocates: make one plain call first
        const size_t lanes = (size_t)(kThreads / coloc);
        const size_t ntiles = ceil_div(nvec, lanes);
        std::vector<std::vector<unsigned>> lists;
        plan_oneshot_lists(c->have_topology ? &c->topology : nullptr, c->num_sms, nranks, ntiles, lanes * 16,
                           ntiles <= kGenericPlanTiles, domains, lists);
        std::vector<unsigned> off((size_t)c->num_sms + 1, 0), tiles;
        tiles.reserve(ntiles);
        for (int s = 0; s < c->num_sms; ++s) {
            tiles.insert(tiles.end(), lists[s].begin(), lists[s].end());
            off[s + 1] = (unsigned)tiles.size();
        }
        SmPlan pl;
        pl.total = (unsigned)tiles.size();
        const size_t words = off.size() + std::max<size_t>(tiles.size(), 1) + 2 * (size_t)c->num_sms + 2;
        unsigned* d = nullptr;
        if (cudaMalloc(&d, words * sizeof(unsigned)) != cudaSuccess) return NUNA_ERR_CUDA;
        std::vector<unsigned> host(words, 0u);
        std::copy(off.begin(), off.end(), host.begin());
        std::copy(tiles.begin(), tiles.end(), host.begin() + off.size());
        const size_t cur0 = off.size() + std::max<size_t>(tiles.size(), 1);
        pl.nonempty = 0;
        for (int s = 0; s < c->num_sms; ++s) pl.nonempty += !lists[s].empty();
        if (cudaMemcpy(d, host.data(), words * sizeof(unsigned), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaFree(d);
            return NUNA_ERR_CUDA;
        }
        pl.base = d;
        pl.off = d;
        pl.tiles = d + off.size();
        pl.cursor = d + cur0;
        pl.present = d + cur0 + c->num_sms;
        pl.ctl = d + cur0 + 2 * (size_t)c->num_sms;
        it = c->sm_plans.emplace(key, pl).first;
    }
    *out = it->second;
    return NUNA_OK;
}

static int coloc_for(const Options& o, int nranks)
{
    int coloc = o.coloc > 0 ? o.coloc : 8;
    while (coloc > 1 && coloc / 2 >= nranks) coloc >>= 1;
    return coloc >= 8 ? 8 : coloc >= 4 ? 4 : 2;
}

// Everything a later launch of this shape would have to allocate (called before stream capture).
int prepare_oneshot(Context* c, int nranks, int dtype, size_t count, unsigned flags)
{
    if ((flags & NUNA_PLACE_MASK) == NUNA_PLACE_AWARE && (flags & NUNA_PLACE_SM_LISTS)) {
        const Options o = snapshot(c);
        SmPlan pl;
        return get_sm_plan(c, nranks, count / elems_per_vec(dtype), coloc_for(o, nranks), o.domains, (cudaStream_t)0, &pl);
    }
    return NUNA_OK;
}

template <int N, int C, int DT>
static int launch_sm_lists(Context* c, const Options& o, const RankPtrs& p, size_t count, unsigned mode, cudaStream_t stream)
{
    auto k = k_oneshot_sm<N, C, DT, false>;
    SmPlan pl;
    const int st = get_sm_plan(c, N, count / Elem<DT>::kElems, C, o.domains, stream, &pl);
    if (st != NUNA_OK) return st;
    SmLists sl;
    sl.off = pl.off; sl.tiles = pl.tiles; sl.cursor = pl.cursor; sl.present = pl.present; sl.ctl = pl.ctl;
    sl.nonempty = pl.nonempty; sl.num_sms = c->num_sms;
    const size_t cap = (size_t)c->num_sms * (size_t)NUNA_OCC(k);
    const unsigned grid = (unsigned)std::min(cap, std::max<size_t>((size_t)c->num_sms, (size_t)pl.total));
    const unsigned blocks_per_sm = (unsigned)std::max<size_t>(1, grid / (size_t)c->num_sms);
    return launch(k, grid, stream, mode, p, count, sl, blocks_per_sm, (unsigned*)nullptr);
}

template <int N, int DT>
static int launch_cluster(const Options& o, const RankPtrs& p, size_t count, unsigned mode, cudaStream_t stream)
{
    auto k = k_oneshot_cluster<N, DT>;
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t ntiles = std::max<size_t>(1, ceil_div(nvec, (size_t)kThreads));
    size_t clusters = std::min<size_t>(ntiles, (size_t)1 << 20);
    if (o.blocks > 0) clusters = std::max<size_t>(1, std::min<size_t>(clusters, (size_t)o.blocks / N));
    t_cluster_dim = N;
    return launch(k, (unsigned)(clusters * N), stream, mode, p, count, ntiles);
}

template <int N, int C, int DT>
static int launch_group(Context* c, const Options& o, const RankPtrs& p, size_t count, unsigned mode, cudaStream_t stream)
{
    auto k = k_oneshot_group<N, C, DT>;
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t ntiles = ceil_div(nvec, (size_t)(kThreads / C));
    const size_t nitems = std::max<size_t>(ntiles * ((N + C - 1) / C), (count % Elem<DT>::kElems) ? (size_t)N : 0);
    const unsigned grid = pick_grid(c, o, nitems, NUNA_OCC(k));
    return launch(k, grid, stream, mode, p, count, ntiles);
}

// Co-located group sharing the tile through registers: one (tile, C destinations) item per block.
// Tile size (vectors per source), measured at 8 ranks, 8 KiB ... 64 MiB per rank, cold and L2-resident:
// one block per SM with tiles of 8 ... 56 vectors while the message is that small (64 blocks of 8 vectors at
// 8 KiB: 1.08 us per L2-resident graph node against 1.38 us with eight full blocks); then four blocks per SM
// with tiles of 56 ... 256 vectors (512 KiB cold behind a dependent launch: 586 blocks of 56 vectors, 2.1 us
// against 2.8 us with 256 full tiles); full tiles beyond.  Tiles never exceed a block's width: contiguous
// chunks of several rows per block were slower from 8 MiB per rank (23.0 against 21.7 us).
// `resident` = blocks of the kernel an SM holds: the blocks must fit in one wave (16 ranks, 3 blocks per SM, 256 KiB
// per rank: 3.46 us with 586 blocks of 56 vectors, 2.42 us with 294 of 112).
static unsigned regs_tile_vecs(const Context* c, const Options& o, size_t nvec, int ksplit, int resident)
{
    if (o.regs_vecs > 0) return (unsigned)std::min(kThreads, std::max(8, o.regs_vecs / 8 * 8));
    const size_t units = nvec * (size_t)ksplit;
    const size_t per_sm = (size_t)std::max(1, std::min(4, resident));
    if (o.blocks > 0 && (size_t)o.blocks < (size_t)c->num_sms * per_sm) {          // a capped grid: as few tiles as blocks, then full tiles
        const size_t capped = ceil_div(ceil_div(units, (size_t)o.blocks), (size_t)8) * 8;
        return (unsigned)std::min<size_t>(kThreads, std::max<size_t>(8, capped));
    }
    const size_t one = ceil_div(ceil_div(units, (size_t)c->num_sms), (size_t)8) * 8;
    if (one <= 56) return (unsigned)std::max<size_t>(8, one);
    const size_t many = ceil_div(ceil_div(units, (size_t)c->num_sms * per_sm), (size_t)8) * 8;
    return (unsigned)std::min<size_t>(kThreads, std::max<size_t>(56, many));
}

template <int N, int C, int DT>
static int launch_regs(Context* c, const Options& o, const RankPtrs& p, size_t count, unsigned flags, unsigned mode, bool may_prefetch,
                       cudaStream_t stream)
{
    auto k = k_oneshot_regs<N, C, DT>;
    constexpr int kSplit = (N + C - 1) / C;
    const size_t nvec = count / Elem<DT>::kElems;
    const unsigned tv = regs_tile_vecs(c, o, nvec, kSplit, NUNA_OCC(k));
    const size_t ntiles = ceil_div(nvec, (size_t)tv);
    const size_t nitems = std::max<size_t>(ntiles * kSplit, (count % Elem<DT>::kElems) ? (size_t)N : 0);
    const unsigned grid = pick_grid(c, o, std::max<size_t>(nitems, 1), NUNA_OCC(k), 0);
    // cold sources behind a dependent launch: fetch into L2 while the predecessor drains
    const bool prefetch = may_prefetch && mode == kLaunchPdl && !(flags & NUNA_HINT_RESIDENT) && o.prefetch != 1;
    return launch(k, grid, stream, mode, p, count, ntiles, tv, ((flags & NUNA_HINT_RESIDENT) ? 0 : 1) | (prefetch ? 2 : 0));
}

// Staged group kernel: one tile per block.  Tile size (vectors per source): large enough that a tile's
// N slices amortise the copy set-up, small enough that a mid-sized message still gives every SM several
// blocks; 32 KiB of shared memory per block at most.
template <int N, int DT>
static int launch_stage(Context* c, const Options& o, const RankPtrs& p, size_t count, unsigned flags, unsigned mode,
                        cudaStream_t stream)
{
    auto k = k_oneshot_stage<N, DT>;
    constexpr unsigned kLanes = kThreads / pow2_at_least(N);
    const size_t nvec = count / Elem<DT>::kElems;
    // measured at 8 ranks (cold): 4 KiB tiles up to 512 KiB per rank, 8 KiB to 4 MiB, 16 KiB to 16 MiB, 32 KiB beyond
    const size_t bytes = count * (size_t)Elem<DT>::kBytes;
    unsigned tile_bytes = bytes <= ((size_t)512 << 10) ? 4096u : bytes <= ((size_t)4 << 20) ? 8192u
                        : bytes <= ((size_t)16 << 20) ? 16384u : 32768u;
    unsigned tv = tile_bytes / 16u / (unsigned)pow2_at_least(N);
    if (o.stage_vecs > 0) tv = (unsigned)o.stage_vecs;
    tv = std::max(kLanes, std::min(tv, 2048u / N)) / kLanes * kLanes;     // a multiple of the row width, <= 32 KiB per tile
    const size_t ntiles = ceil_div(nvec, (size_t)tv);
    const size_t grid = std::max<size_t>(ntiles, (count % Elem<DT>::kElems) ? 1 : 0);
    t_dyn_smem = (unsigned)N * tv * 16u;
    return launch(k, (unsigned)std::max<size_t>(1, grid), stream, mode, p, count, tv,
                  (flags & NUNA_HINT_RESIDENT) ? 0 : 1, &c->bw->status, o.timeout_ns);
}

int launch_oneshot(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream)
{
    const Options o = snapshot(c);
    const size_t bytes = count * elem_size(dtype);                   // per rank
    const size_t epv = elems_per_vec(dtype);
    const unsigned mode = launch_mode(flags, bytes * (size_t)nranks);
    const size_t nvec = count / epv;
    const unsigned place = flags & NUNA_PLACE_MASK;
    OneShotKernel which = OneShotKernel::RoundRobin;
    if (place == NUNA_PLACE_AWARE)
        which = (flags & NUNA_PLACE_REGS) ? OneShotKernel::Regs : (flags & NUNA_PLACE_STAGED) ? OneShotKernel::Staged : OneShotKernel::Group;
    else if (place == NUNA_PLACE_AUTO) which = auto_kernel(c, o, nranks, bytes, flags);
    if (which == OneShotKernel::Regs) {
        const unsigned m = (flags & NUNA_LAUNCH_PDL) ? kLaunchPdl : kLaunchPlain;
        // destinations per thread: all of them, so that a tile crosses the L2 -> SM fabric once (beyond 8 ranks the
        // sixteen-destination form: 9 ranks x 512 KiB 2.25 us against 2.71 in two passes of eight, 16 ranks x 1 MiB
        // 6.39 against 7.35); half of them for large cold messages, where two blocks per tile keep more DRAM loads
        // in flight (8 ranks x 16 MiB cold: 41.8 us with four, 42.0 with eight)
        const int all = nranks > 8 ? 16 : std::min(8, pow2_at_least(nranks));
        const bool large_cold = !(flags & NUNA_HINT_RESIDENT) && bytes >= ((size_t)8 << 20);
        int coloc = o.coloc > 0 ? o.coloc : (large_cold ? std::min(8, std::max(2, pow2_at_least(nranks) / 2)) : all);
        while (coloc > 2 && coloc / 2 >= nranks) coloc >>= 1;
        return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
            constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
            // from 8 MiB per rank the prefetch only adds requests to a saturated memory system
            // (8 ranks, four destinations per thread: 16 MiB 45.5 us with, 41.2 without; 64 MiB 175 against 158)
            if constexpr (N > 8) { if (coloc >= 16) return launch_regs<N, 16, DT>(c, o, p, count, flags, m, !large_cold, stream); }
            if (coloc >= 8) return launch_regs<N, 8, DT>(c, o, p, count, flags, m, !large_cold, stream);
            if (coloc >= 4) return launch_regs<N, 4, DT>(c, o, p, count, flags, m, !large_cold, stream);
            return launch_regs<N, 2, DT>(c, o, p, count, flags, m, !large_cold, stream);
        });
    }
    if (which == OneShotKernel::Staged) {
        return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
            constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
            return launch_stage<N, DT>(c, o, p, count, flags, (flags & NUNA_LAUNCH_PDL) ? kLaunchPdl : kLaunchPlain, stream);
        });
    }
    if (which == OneShotKernel::Group) {
        // co-location factor: C destinations of a tile share a block (C <= N rounded up to a power of two)
        const int coloc = coloc_for(o, nranks);
        if (place == NUNA_PLACE_AWARE && (flags & NUNA_PLACE_CLUSTER) && nranks >= 2 && nranks <= 8) {
            return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
                constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
                if constexpr (N >= 2 && N <= 8) return launch_cluster<N, DT>(o, p, count, mode, stream);
                else return NUNA_ERR_INVALID_ARG;
            });
        }
        if (place == NUNA_PLACE_AWARE && (flags & NUNA_PLACE_SM_LISTS)) {
            return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
                constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
                if (coloc >= 8) return launch_sm_lists<N, 8, DT>(c, o, p, count, mode, stream);
                if (coloc >= 4) return launch_sm_lists<N, 4, DT>(c, o, p, count, mode, stream);
                return launch_sm_lists<N, 2, DT>(c, o, p, count, mode, stream);
            });
        }
        return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
            constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
            if (coloc >= 8) return launch_group<N, 8, DT>(c, o, p, count, mode, stream);
            if (coloc >= 4) return launch_group<N, 4, DT>(c, o, p, count, mode, stream);
            return launch_group<N, 2, DT>(c, o, p, count, mode, stream);
        });
    }
    return dispatch(nranks, pick_unroll(o, nranks), dtype, [&](auto n_, auto u_, auto d_) -> int {
        NUNA_NUD(n_, u_, d_);
        auto k = k_oneshot_rr<N, U, DT>;
        const size_t ntiles = ceil_div(nvec, (size_t)kThreads * U);
        const size_t nitems = std::max<size_t>(ntiles * N, (count % epv) ? (size_t)N : 0);
        // one resident wave while the message is small enough for latency to matter, four beyond
        const unsigned grid = pick_grid(c, o, nitems, NUNA_OCC(k), bytes >= ((size_t)8 << 20) ? 4 : 1);
        return launch(k, grid, stream, mode, p, count, ntiles);
    });
}

// Launches the flag-synchronised two-shot on explicit scratch / flag / control storage (the context's, or
// the fixed arrays of the allocation-free entry point): one block per work item, tiles + lead blocks.
// tv = 0 picks the tile size by message size.  min_tv is the smallest tile the flag array was sized for.
int launch_twoshot_flags(int num_sms, int blocks_override, const RankPtrs& p, int nranks, int dtype, size_t count,
                         unsigned tv, unsigned min_tv, uint4* scratch, unsigned* tile_flags, BarrierWords* bw,
                         unsigned long long timeout_ns, bool pdl, unsigned debug_bits, cudaStream_t stream)
{
    const size_t bytes = count * elem_size(dtype);
    const size_t nvec = count / elems_per_vec(dtype);
    bool mid_sized = false;
    if (tv == 0) {
        // Tile bytes across all N sources, from a sweep at 8 ranks (16 ... 256 vectors per tile at every size):
        // small tiles while the message is small (more blocks, less latency per tile), 32 KiB once there are
        // plenty.  At 8 MiB of sources 16 KiB tiles make 1024 blocks for 592 resident ones and the second
        // wave's consumers wait (10.3 us against 7.6 us with 12 KiB tiles), hence the step back there.
        // Between 16 and 64 MiB of sources 24 KiB tiles with a lead of five blocks per SM are ahead (3 MiB per rank 11.6
        // against 12.3 us, 4 MiB 14.2 against 15.1, 6 MiB 19.1 against 21.3, 7 MiB 21.6 against 24.2; at 8 MiB 27.2
        // against 24.8, hence the upper limit).
        const size_t src_bytes = bytes * (size_t)nranks;
        mid_sized = nranks <= 8 && src_bytes > ((size_t)16 << 20) && src_bytes < ((size_t)64 << 20);   // 16 ranks: no gain
        const unsigned tile_src = src_bytes <= ((size_t)512 << 10) ? 4096u : src_bytes <= ((size_t)1 << 20) ? 8192u
                                : src_bytes <= ((size_t)8 << 20) ? 12288u
                                : src_bytes <= ((size_t)16 << 20) ? 16384u : mid_sized ? 24576u : 32768u;
        tv = tile_src / 16u / (unsigned)nranks;
    }
    tv = std::max(min_tv, std::min(tv, 2048u / (unsigned)nranks));
    tv = std::max(1u, tv / 8u * 8u);
    if (tv < min_tv) tv = min_tv;
    const size_t ntiles = std::max<size_t>(1, ceil_div(nvec, (size_t)tv));
    unsigned lead_max = (unsigned)num_sms * (mid_sized ? 5u : 8u);
    if (blocks_override > 0) lead_max = (unsigned)std::max(1, blocks_override);
    const size_t lead = std::min<size_t>(ntiles, lead_max);
    const unsigned grid = (unsigned)(ntiles + lead);
    return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
        constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
        t_dyn_smem = (unsigned)N * tv * 16u;
        if (bytes * (size_t)nranks >= ((size_t)64 << 20))           // bandwidth-bound: trade registers for resident blocks
            return launch(k_twoshot_flags<N, DT, 6>, grid, stream, pdl ? kLaunchPdl : kLaunchPlain, p, scratch, tile_flags, count,
                          tv, lead_max, bw, timeout_ns, debug_bits);
        return launch(k_twoshot_flags<N, DT, 4>, grid, stream, pdl ? kLaunchPdl : kLaunchPlain, p, scratch, tile_flags, count, tv,
                      lead_max, bw, timeout_ns, debug_bits);
    });
}

// The put form: one tile per block by default; `max_blocks` > 0 makes it a grid-stride loop over that many blocks.
// Whether a two-shot kernel asks L2 for its blocks' first tiles ahead of the dependent-launch wait: cold
// device-memory sources, and a message small enough that the predecessor's drain is a visible share of it.
// Measured with the put form (us, with | without): 8 ranks 2 MiB 6.16 | 6.44, 8 MiB 21.4 | 21.8, 16 MiB 42.1 | 42.1,
// 64 MiB 162.5 | 160.8; 16 ranks 256 KiB 3.25 | 3.46, 1 MiB 6.74 | 6.59, 8 MiB 43.1 | 42.6; 4 ranks 32 MiB 41.3 | 41.7.
static bool prefetch_pays(const Options& o, unsigned flags, int nranks, size_t bytes)
{
    if (!(flags & NUNA_LAUNCH_PDL) || (flags & NUNA_HINT_RESIDENT) || o.prefetch == 1) return false;
    return bytes * (size_t)nranks <= (nranks <= 8 ? (size_t)128 << 20 : (size_t)8 << 20);
}

int launch_twoshot_put(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream,
                       unsigned max_blocks)
{
    const Options o = snapshot(c);
    const unsigned mode = launch_mode(flags);
    const size_t nvec = count / elems_per_vec(dtype);
    return dispatch(nranks, pick_unroll(o, nranks), dtype, [&](auto n_, auto u_, auto d_) -> int {
        NUNA_NUD(n_, u_, d_);
        auto k = k_twoshot_put<N, U, DT>;
        const size_t ntiles = ceil_div(nvec, (size_t)kThreads * U);
        unsigned grid = pick_grid(c, o, std::max<size_t>(ntiles, 1), NUNA_OCC(k), 0);
        if (max_blocks > 0 && o.blocks <= 0) grid = std::min(grid, max_blocks);
        // device-memory sources behind a dependent launch: fetch the first tile into L2 while the predecessor drains
        const bool prefetch = max_blocks == 0 && prefetch_pays(o, flags, nranks, count * elem_size(dtype));
        return launch(k, grid, stream, mode, p, count, ntiles, prefetch ? 1 : 0);
    });
}

int launch_twoshot(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream)
{
    if (flags & NUNA_TWOSHOT_PUT) return launch_twoshot_put(c, p, nranks, dtype, count, flags, stream, 0u);
    const Options o = snapshot(c);
    uint4* scratch;
    unsigned* tile_flags;
    {
        std::lock_guard<std::mutex> lock(c->mutex);
        scratch = reinterpret_cast<uint4*>(c->scratch);
        tile_flags = c->flags;
    }
    return launch_twoshot_flags(c->num_sms, o.blocks, p, nranks, dtype, count, (unsigned)std::max(0, o.twoshot_vecs), kMinFlagTileVec,
                                scratch, tile_flags, c->bw, o.timeout_ns, (flags & NUNA_LAUNCH_PDL) != 0,
                                (o.keep_shard ? 4u : 0u) | ((flags & NUNA_TWOSHOT_SYS_SCOPE) ? 8u : 0u) |
                                    (prefetch_pays(o, flags, nranks, count * elem_size(dtype)) ? 16u : 0u), stream);
}

int launch_reduce_scatter(Context* c, const RankPtrs& p, int nranks, int dtype, size_t shard, unsigned flags,
                          cudaStream_t stream)
{
    const Options o = snapshot(c);
    const size_t epv = elems_per_vec(dtype);
    const unsigned mode = launch_mode(flags);
    if (shard % epv) {
        const unsigned grid = pick_grid(c, o, ceil_div(shard * nranks, kThreads), 8);
        return dispatch(nranks, 1, dtype, [&](auto n_, auto u_, auto d_) -> int {
            NUNA_NUD(n_, u_, d_);
            return launch(k_reduce_scatter_scalar<N, DT>, grid, stream, mode, p, shard);
        });
    }
    const size_t shard_vec = shard / epv;
    return dispatch(nranks, pick_unroll(o, nranks), dtype, [&](auto n_, auto u_, auto d_) -> int {
        NUNA_NUD(n_, u_, d_);
        auto k = k_reduce_scatter<N, U, DT>;
        const size_t tiles = ceil_div(shard_vec, (size_t)kThreads * U);
        const unsigned grid = pick_grid(c, o, tiles * N, NUNA_OCC(k), 0);
        return launch(k, grid, stream, mode, p, shard_vec, tiles);
    });
}

// Allgather and alltoall copy bits: they work on 16-byte vectors when a shard is a whole number of
// them, otherwise on 16-bit units (every element type is a multiple of that).
int launch_allgather(Context* c, const RankPtrs& p, int nranks, size_t shard_bytes, unsigned flags, cudaStream_t stream)
{
    const Options o = snapshot(c);
    const unsigned mode = launch_mode(flags);
    if (shard_bytes % 16) {
        const size_t shard16 = shard_bytes / 2;
        const unsigned grid = pick_grid(c, o, ceil_div(shard16 * nranks, kThreads), 8);
        return launch(k_allgather_scalar, grid, stream, mode, p, nranks, shard16);
    }
    const size_t shard_vec = shard_bytes / 16;
    const size_t out_total = shard_bytes * (size_t)nranks * (size_t)nranks;
    if (o.ag_bulk_vecs == 0 && out_total <= ((size_t)128 << 20)) {
        // register form with small tiles: about four blocks per SM, tiles of 16 ... 256 vectors
        const size_t per = ceil_div(ceil_div(shard_vec * (size_t)nranks, (size_t)c->num_sms * 4), (size_t)8) * 8;
        const unsigned tv = (unsigned)std::min<size_t>(kThreads, std::max<size_t>(16, per));
        const size_t tiles = ceil_div(shard_vec, (size_t)tv);
        const unsigned grid = (unsigned)(tiles * nranks);
        if (o.blocks <= 0 || (size_t)o.blocks >= grid)             // one tile per block: a capped grid takes the looping form below
            return launch(k_allgather_small, grid, stream, mode, p, nranks, shard_vec, tiles, tv,
                          prefetch_pays(o, flags, nranks, shard_vec * 16) ? 1 : 0);
    }
    if (o.ag_bulk_vecs != 1) {
        // Default: the bulk-copy form, one block per (rank, tile); the copy engine moves the tile in once and
        // out N times.  Measured against the register form below: 16 x 64 KiB 4.11 vs 4.99 us, 16 x 8 KiB 2.02
        // vs 3.68 us, 8 x 8 MiB 97.4 vs 102.2 us.  Small tiles (1 KiB) while there are few of them, 2 KiB beyond.
        const size_t out_bytes = shard_bytes * (size_t)nranks * (size_t)nranks;
        unsigned tv = o.ag_bulk_vecs >= 8 ? (unsigned)o.ag_bulk_vecs : (out_bytes <= ((size_t)64 << 20) ? 64u : 128u);
        tv = std::min(2048u, tv) / 8u * 8u;
        const size_t tiles = ceil_div(shard_vec, (size_t)tv);
        if (tiles * (size_t)nranks <= ((size_t)1 << 24)) {
            t_dyn_smem = tv * 16u;
            return launch(k_allgather_bulk, (unsigned)(tiles * nranks), stream, mode, p, nranks, shard_vec, tiles, tv, &c->bw->status,
                          o.timeout_ns, prefetch_pays(o, flags, nranks, shard_vec * 16) ? 1 : 0);
        }
    }
    // One block per (rank, tile) storing to all N destinations.  Splitting a tile's destinations over
    // several blocks (dsplit > 1) was measured slower at every size tried (16 x 64 KiB: 4.4 us with 1,
    // 5.4 us with 8): the stores, not the block count, are the limit.
    constexpr int U = 2;
    const int dsplit = 1;
    auto k = k_allgather<U>;
    const size_t tiles = ceil_div(shard_vec, (size_t)kThreads * U);
    const unsigned grid = pick_grid(c, o, tiles * nranks * dsplit, NUNA_OCC(k), 0);
    return launch(k, grid, stream, mode, p, nranks, shard_vec, tiles, dsplit);
}

int launch_alltoall(Context* c, const RankPtrs& p, int nranks, size_t block_bytes, unsigned flags, cudaStream_t stream)
{
    const Options o = snapshot(c);
    const unsigned mode = launch_mode(flags);
    if (block_bytes % 16) {
        const size_t block16 = block_bytes / 2;
        const unsigned grid = pick_grid(c, o, ceil_div(block16 * nranks * nranks, kThreads), 8);
        return launch(k_alltoall_scalar, grid, stream, mode, p, nranks, block16);
    }
    const size_t block_vec = block_bytes / 16;
    if (o.ag_bulk_vecs != 1) {
        // bulk-copy form (default), as for the allgather; 8 KiB tiles (8 x 8 blocks of 64 KiB: 2.84 us against
        // 3.02 us for the register form and 3.11 us with 2 KiB tiles)
        const unsigned tv = o.ag_bulk_vecs >= 8 ? std::min(2048u, (unsigned)o.ag_bulk_vecs) / 8u * 8u : 512u;
        const size_t tiles = ceil_div(block_vec, (size_t)tv);
        const size_t grid = tiles * (size_t)nranks * (size_t)nranks;
        if (grid <= ((size_t)1 << 24)) {
            t_dyn_smem = tv * 16u;
            return launch(k_alltoall_bulk, (unsigned)grid, stream, mode, p, nranks, block_vec, tiles, tv, &c->bw->status, o.timeout_ns,
                          prefetch_pays(o, flags, nranks, block_vec * 16 * (size_t)nranks) ? 1 : 0);
        }
    }
    constexpr int U = 2;
    auto k = k_alltoall<U>;
    const size_t tiles = ceil_div(block_vec, (size_t)kThreads * U);
    const unsigned grid = pick_grid(c, o, tiles * nranks * nranks, NUNA_OCC(k), 0);
    return launch(k, grid, stream, mode, p, nranks, block_vec, tiles);
}

// ---- single-kernel chain ---------------------------------------------------------------------------------

// One cluster runs the whole chain.  Measured on B200 (160 nodes, 8 ranks): 1.45 us per node at 16 KiB per rank
// against 1.08 us for the graph with dependent launch, 2.5 against 1.15 us at 128 KiB, 12 against 2.4 us at
// 1 MiB: a node still costs two dependent memory round trips (loads; then the stores the cluster barrier has to
// see performed) plus the barrier on sixteen SMs, which is no less than a launch hidden behind its predecessor.
// So the library never picks it by itself (limit 0); NUNA_CHAIN_PERSISTENT runs it on request.
constexpr size_t kChainPersistentMaxBytes = 0;                      // per rank

bool chain_persistent_supported(const Context* c, int nsets, int nranks, int dtype, size_t count)
{
    (void)c;
    return nsets >= 1 && nsets <= kMaxChainSets && nranks >= 1 && count * elem_size(dtype) <= ((size_t)4 << 20);
}

bool chain_persistent_pays_off(int dtype, size_t count) { return count * elem_size(dtype) <= kChainPersistentMaxBytes; }

int launch_chain_persistent(Context* c, const ChainSets& sets, int nsets, int nnodes, int nranks, int dtype, size_t count,
                            cudaStream_t stream)
{
    (void)c;
    // two destinations per thread while that still gives every thread of the cluster an item, all of them beyond
    const bool wide = (count / elems_per_vec(dtype)) * (size_t)((nranks + 1) / 2) > (size_t)16 * kThreads;
    return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
        constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
        constexpr int kAll = pow2_at_least(N) > 8 ? 8 : (pow2_at_least(N) < 2 ? 2 : pow2_at_least(N));
        auto k = wide ? k_chain_persistent<N, kAll, DT> : k_chain_persistent<N, 2, DT>;
        // sixteen blocks per cluster need the non-portable opt-in; fall back to the portable eight
        static std::atomic<int> cluster_size[kMaxDevices];
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
        int cs = cluster_size[dev].load(std::memory_order_relaxed);
        if (cs == 0) {
            cs = 8;
            if (cudaFuncSetAttribute(k_chain_persistent<N, kAll, DT>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
                cudaFuncSetAttribute(k_chain_persistent<N, 2, DT>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(16, 1, 1);
                cfg.blockDim = dim3(kThreads, 1, 1);
                cudaLaunchAttribute at;
                at.id = cudaLaunchAttributeClusterDimension;
                at.val.clusterDim.x = 16; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
                cfg.attrs = &at;
                cfg.numAttrs = 1;
                int nclusters = 0;
                if (cudaOccupancyMaxActiveClusters(&nclusters, k, &cfg) == cudaSuccess && nclusters >= 1) cs = 16;
            }
            cudaGetLastError();
            cluster_size[dev].store(cs, std::memory_order_relaxed);
        }
        t_cluster_dim = (unsigned)cs;
        return launch(k, (unsigned)cs, stream, kLaunchPlain, sets, nsets, nnodes, count);
    });
}

}  // namespace nuna

using namespace nuna;

extern "C" {

int nuna_init(size_t scratch_bytes)
{
    Context* c = nullptr;
    int st = get_context(&c);
    if (st != NUNA_OK) return st;
    std::lock_guard<std::mutex> lock(c->mutex);
    return ensure_scratch(c, scratch_bytes);
}

int nuna_set_option(int option, long long value)
{
    if (value < 0) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    int st = get_context(&c);
    if (st != NUNA_OK) return st;
    std::lock_guard<std::mutex> lock(c->mutex);
    switch (option) {
        case NUNA_OPT_BLOCKS: c->opt.blocks = (int)std::min<long long>(value, 1 << 22); break;
        case NUNA_OPT_UNROLL: c->opt.unroll = (int)value; break;
        case NUNA_OPT_COLOC: c->opt.coloc = (int)value; break;
        case NUNA_OPT_AUTO_MIN_BYTES: c->opt.auto_min_bytes = (size_t)value; break;
        case NUNA_OPT_TIMEOUT_MS: c->opt.timeout_ns = (unsigned long long)(value ? value : 1000) * 1000000ull; break;
        case NUNA_OPT_DOMAINS: c->opt.domains = (int)std::min<long long>(value, NUNA_MAX_SMS); break;
        case NUNA_OPT_STAGE_VECS: c->opt.stage_vecs = (int)std::min<long long>(value, 4096); break;
        case NUNA_OPT_TWOSHOT_VECS: c->opt.twoshot_vecs = (int)std::min<long long>(value, 4096); break;
        case NUNA_OPT_AG_BULK_VECS: c->opt.ag_bulk_vecs = (int)std::min<long long>(value, 2048); break;
        case NUNA_OPT_REGS_VECS: c->opt.regs_vecs = (int)std::min<long long>(value, kThreads); break;
        case NUNA_OPT_PREFETCH: c->opt.prefetch = (int)std::min<long long>(value, 1); break;
        default: return NUNA_ERR_INVALID_ARG;
    }
    return NUNA_OK;
}

int nuna_allreduce_oneshot(const void* const* src, void* const* dst, int nranks, size_t count, int dtype,
                           unsigned flags, void* stream)
{
    if (has_chain_bits(flags)) return NUNA_ERR_INVALID_ARG;
    int st = check_args(src, dst, nranks, count, count, dtype, flags & ~NUNA_TWOSHOT_PUT, true);
    if (st != NUNA_OK || count == 0) return st;
    if (flags & NUNA_TWOSHOT_PUT) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    return launch_oneshot(c, make_ptrs(src, dst, nranks), nranks, dtype, count, flags, (cudaStream_t)stream);
}

int nuna_allreduce_twoshot(const void* const* src, void* const* dst, int nranks, size_t count, int dtype,
                           unsigned flags, void* stream)
{
    if (has_chain_bits(flags)) return NUNA_ERR_INVALID_ARG;
    int st = check_args(src, dst, nranks, count, count, dtype, flags, true);
    if (st != NUNA_OK || count == 0) return st;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    if (!(flags & NUNA_TWOSHOT_PUT)) {
        std::lock_guard<std::mutex> lock(c->mutex);
        const size_t need = (count * elem_size(dtype) + 15) & ~(size_t)15;
        if (need > c->scratch_bytes || !c->scratch) {
            cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
            if (cudaStreamIsCapturing((cudaStream_t)stream, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone)
                return NUNA_ERR_CAPTURING;             // growing the scratch allocates: call nuna_init first
            if ((st = ensure_scratch(c, need)) != NUNA_OK) return st;
        }
    }
    return launch_twoshot(c, make_ptrs(src, dst, nranks), nranks, dtype, count, flags, (cudaStream_t)stream);
}

int nuna_allreduce(const void* const* src, void* const* dst, int nranks, size_t count, int dtype, unsigned flags,
                   void* stream)
{
    // Crossover measured on B200, cold and L2-resident: the one-shot's N-fold re-reads cost more the
    // more ranks there are, so its single step wins up to 1 MiB per rank at 2 ranks, 512 KiB at 4,
    // 128 KiB at 8 and 64 KiB at 16.  Beyond it the put form of the two-shot is the fastest kernel at every
    // size; the flag-synchronised form is used instead when the caller asks for it (NUNA_TWOSHOT_SYNC),
    // from the size where it beats the one-shot (measured per rank count, kSyncFactor x the put crossover).
    const size_t bytes = count * elem_size(dtype);
    size_t limit = nranks <= 2 ? ((size_t)1 << 20) : nranks <= 4 ? ((size_t)512 << 10)
                 : nranks <= 8 ? ((size_t)128 << 10) : ((size_t)64 << 10);
    // with NUNA_PLACE_AUTO the one-shot side is the register-sharing kernel, which stays ahead of the put form up
    // to 8 MiB of sources in total behind a dependent launch (8 ranks, cold: 128 KiB 1.51 vs 1.92 us, 1 MiB 3.33 vs
    // 3.74, 2 MiB 6.44 vs 6.16; 4 ranks: 2 MiB 3.34 vs 3.52, 4 MiB 5.79 vs 5.73) and up to 2 MiB launched plainly
    // (8 ranks: 256 KiB 2.65 vs 2.70, 512 KiB 3.29 vs 3.17; beyond 8 ranks, where it needs two passes over the
    // sources, a quarter of that); 16 ranks behind a dependent launch: 256 KiB 2.33 vs 3.21, 512 KiB 3.52 vs 4.25,
    // 1 MiB 7.3 vs 6.6
    // From 8 MiB per rank at 8 ranks or fewer it is ahead again, with two blocks per tile (8 ranks: 8 MiB 21.3 vs 21.6 us,
    // 16 MiB 41.2 vs 42.1, 64 MiB 157.7 vs 160.8).
    bool oneshot_large = false;
    if ((flags & NUNA_PLACE_MASK) == NUNA_PLACE_AUTO) {
        const size_t total = (flags & NUNA_LAUNCH_PDL) ? (size_t)8 << 20 : (size_t)2 << 20;
        limit = std::max(limit, ((nranks <= 8 || (flags & NUNA_LAUNCH_PDL)) ? total : total / 4) / (size_t)nranks);
        oneshot_large = nranks <= 8 && bytes >= ((size_t)8 << 20) && !(flags & NUNA_HINT_RESIDENT);
    }
    constexpr size_t kSyncFactor = 8;
    const bool sync_form = (flags & NUNA_TWOSHOT_SYNC) && !(flags & NUNA_TWOSHOT_PUT);
    const unsigned base = flags & ~(NUNA_TWOSHOT_SYNC | NUNA_TWOSHOT_PUT | (sync_form ? 0u : NUNA_TWOSHOT_SYS_SCOPE));
    if (nranks <= 1 || bytes <= (sync_form ? limit * kSyncFactor : limit) || (oneshot_large && !sync_form))
        return nuna_allreduce_oneshot(src, dst, nranks, count, dtype, base, stream);
    return nuna_allreduce_twoshot(src, dst, nranks, count, dtype, sync_form ? base : (base | NUNA_TWOSHOT_PUT), stream);
}

int nuna_reduce_scatter(const void* const* src, void* const* dst, int nranks, size_t shard_count, int dtype,
                        unsigned flags, void* stream)
{
    if (has_chain_bits(flags)) return NUNA_ERR_INVALID_ARG;
    if (nranks >= 1 && nranks <= NUNA_MAX_RANKS && shard_count > ((size_t)1 << 40) / (size_t)nranks)
        return NUNA_ERR_TOO_LARGE;
    int st = check_args(src, dst, nranks, shard_count * (size_t)(nranks > 0 ? nranks : 0), shard_count, dtype,
                        flags & ~NUNA_TWOSHOT_PUT, true);
    if (st != NUNA_OK || shard_count == 0) return st;
    if (flags & NUNA_TWOSHOT_PUT) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    return launch_reduce_scatter(c, make_ptrs(src, dst, nranks), nranks, dtype, shard_count, flags, (cudaStream_t)stream);
}

int nuna_allgather(const void* const* src, void* const* dst, int nranks, size_t shard_count, int dtype,
                   unsigned flags, void* stream)
{
    if (has_chain_bits(flags)) return NUNA_ERR_INVALID_ARG;
    if (nranks >= 1 && nranks <= NUNA_MAX_RANKS && shard_count > ((size_t)1 << 40) / (size_t)nranks)
        return NUNA_ERR_TOO_LARGE;
    int st = check_args(src, dst, nranks, shard_count, shard_count * (size_t)(nranks > 0 ? nranks : 0), dtype,
                        flags & ~NUNA_TWOSHOT_PUT, true);
    if (st != NUNA_OK || shard_count == 0) return st;
    if (flags & NUNA_TWOSHOT_PUT) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    return launch_allgather(c, make_ptrs(src, dst, nranks), nranks, shard_count * elem_size(dtype), flags, (cudaStream_t)stream);
}

int nuna_alltoall(const void* const* src, void* const* dst, int nranks, size_t block_count, int dtype,
                  unsigned flags, void* stream)
{
    if (has_chain_bits(flags)) return NUNA_ERR_INVALID_ARG;
    if (nranks >= 1 && nranks <= NUNA_MAX_RANKS && block_count > ((size_t)1 << 40) / (size_t)nranks)
        return NUNA_ERR_TOO_LARGE;
    const size_t per_rank = block_count * (size_t)(nranks > 0 ? nranks : 0);
    int st = check_args(src, dst, nranks, per_rank, per_rank, dtype, flags & ~NUNA_TWOSHOT_PUT, true);
    if (st != NUNA_OK || block_count == 0) return st;
    if (flags & NUNA_TWOSHOT_PUT) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    return launch_alltoall(c, make_ptrs(src, dst, nranks), nranks, block_count * elem_size(dtype), flags, (cudaStream_t)stream);
}

int nuna_allreduce_host(const void* const* src, void* const* dst, int nranks, size_t count, int dtype,
                        unsigned flags, int two_shot)
{
    if (has_chain_bits(flags)) return NUNA_ERR_INVALID_ARG;
    int st = check_args(src, dst, nranks, count, count, dtype, flags, false);
    if (st != NUNA_OK || count == 0) return st;
    if (!two_shot && (flags & NUNA_TWOSHOT_PUT)) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    std::lock_guard<std::mutex> lock(c->host_mutex);       // staging buffers and the private stream: one call at a time
    const size_t bytes = count * elem_size(dtype);
    if (!c->stream && cudaStreamCreateWithFlags(&c->stream, cudaStreamNonBlocking) != cudaSuccess) return NUNA_ERR_CUDA;

    // Page-locked host buffers are visible to the device: the put form of the two-shot reads every source
    // byte once and writes every destination byte once, so it can run directly on them -- one kernel, reads
    // and writes crossing the host link in both directions at once, no staging copies.  (Bringing the sources
    // in by copy engine in 1-16 pipelined chunks while the kernel stores straight into the host destinations
    // was measured slower at every size -- 8 x 512 KiB: 214-690 us against 174 us -- because each of the
    // 8 x chunks asynchronous copies costs about 4 us of host time to enqueue.)
    if (two_shot && (flags & NUNA_TWOSHOT_PUT)) {
        const void* msrc[NUNA_MAX_RANKS];
        void* mdst[NUNA_MAX_RANKS];
        bool mapped = true;
        for (int r = 0; r < nranks && mapped; ++r) {
            cudaPointerAttributes as, ad;
            if (cudaPointerGetAttributes(&as, src[r]) != cudaSuccess || cudaPointerGetAttributes(&ad, dst[r]) != cudaSuccess) {
                cudaGetLastError();
                mapped = false;
                break;
            }
            mapped = as.type == cudaMemoryTypeHost && ad.type == cudaMemoryTypeHost && as.devicePointer && ad.devicePointer &&
                     (((uintptr_t)as.devicePointer | (uintptr_t)ad.devicePointer) & 15u) == 0;
            msrc[r] = as.devicePointer;
            mdst[r] = ad.devicePointer;
        }
        if (mapped) {
            // Few blocks: reads of host memory issued by many SMs at once get less out of the link than the same
            // reads from a few (8 x 512 KiB: 134 us with 24 blocks, 166 us with one block per tile; 8 x 4 MiB: 859
            // against 1084 us; swept over 2-48 blocks and both unroll factors).
            st = launch_twoshot_put(c, make_ptrs(msrc, mdst, nranks), nranks, dtype, count, flags & ~NUNA_LAUNCH_PDL, c->stream, 24u);
            if (st != NUNA_OK) return st;
            return cudaStreamSynchronize(c->stream) == cudaSuccess ? NUNA_OK : NUNA_ERR_CUDA;
        }
    }

    const size_t slot = (bytes + 255) & ~(size_t)255;
    const size_t need = slot * 2 * (size_t)nranks;
    if (need > c->staging_bytes) {
        if (c->staging) cudaFree(c->staging);
        c->staging = nullptr;
        c->staging_bytes = 0;
        if (cudaMalloc(&c->staging, need) != cudaSuccess) return NUNA_ERR_CUDA;
        c->staging_bytes = need;
    }
    if (two_shot && !(flags & NUNA_TWOSHOT_PUT)) {
        std::lock_guard<std::mutex> inner(c->mutex);
        if ((st = ensure_scratch(c, slot)) != NUNA_OK) return st;
    }
    const void* dsrc[NUNA_MAX_RANKS];
    void* ddst[NUNA_MAX_RANKS];
    char* base = static_cast<char*>(c->staging);
    for (int r = 0; r < nranks; ++r) {
        dsrc[r] = base + slot * (size_t)r;
        ddst[r] = base + slot * (size_t)(nranks + r);
        if (cudaMemcpyAsync(const_cast<void*>(dsrc[r]), src[r], bytes, cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
            return NUNA_ERR_CUDA;
    }
    const RankPtrs p = make_ptrs(dsrc, ddst, nranks);
    st = two_shot ? launch_twoshot(c, p, nranks, dtype, count, flags, c->stream)
                  : launch_oneshot(c, p, nranks, dtype, count, flags, c->stream);
    if (st != NUNA_OK) return st;
    for (int d = 0; d < nranks; ++d)
        if (cudaMemcpyAsync(dst[d], ddst[d], bytes, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess)
            return NUNA_ERR_CUDA;
    return cudaStreamSynchronize(c->stream) == cudaSuccess ? NUNA_OK : NUNA_ERR_CUDA;
}

int nuna_device_status(int* out)
{
    if (!out) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    int st = get_context(&c);
    if (st != NUNA_OK) return st;
    if (cudaDeviceSynchronize() != cudaSuccess) return NUNA_ERR_CUDA;
    BarrierWords h;
    if (cudaMemcpy(&h, c->bw, sizeof h, cudaMemcpyDeviceToHost) != cudaSuccess) return NUNA_ERR_CUDA;
    unsigned worst = h.status;
    if (h.status != 0 && (st = rewind_barrier_words(c->bw, h)) != NUNA_OK) return st;
    // the allocation-free entry point keeps its own words in the library's fixed arrays
    unsigned static_status = 0;
    if ((st = static_status_read_and_clear(&static_status)) != NUNA_OK) return st;
    *out = (int)std::max(worst, static_status);
    return NUNA_OK;
}

int nuna_launch_floor(unsigned blocks, unsigned flags, void* stream)
{
    if (blocks == 0 || blocks > (1u << 20) || (flags & ~NUNA_LAUNCH_PDL)) return NUNA_ERR_INVALID_ARG;
    return launch(k_empty, blocks, (cudaStream_t)stream, launch_mode(flags), 0);
}

// See nuna_debug.h.
int nuna_debug_launch_floor(unsigned blocks, unsigned flags, int trigger_first, void* stream)
{
    if (blocks == 0 || blocks > (1u << 20) || (flags & ~NUNA_LAUNCH_PDL)) return NUNA_ERR_INVALID_ARG;
    if (trigger_first) return launch(k_empty_trigger_first, blocks, (cudaStream_t)stream, launch_mode(flags), 0);
    return launch(k_empty, blocks, (cudaStream_t)stream, launch_mode(flags), 0);
}

unsigned long long nuna_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* nuna_status_string(int status)
{
    switch (status) {
        case NUNA_OK: return "ok";
        case NUNA_ERR_INVALID_ARG: return "invalid argument";
        case NUNA_ERR_UNSUPPORTED_DTYPE: return "unsupported dtype";
        case NUNA_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case NUNA_ERR_ALIAS: return "destination overlaps a source or another destination";
        case NUNA_ERR_CUDA: return "CUDA runtime error";
        case NUNA_ERR_TIMEOUT: return "flag barrier timed out";
        case NUNA_ERR_CAPTURING: return "operation would allocate or synchronise during stream capture";
        case NUNA_ERR_TOO_MANY_RANKS: return "more than NUNA_MAX_RANKS ranks";
        case NUNA_ERR_TOO_LARGE: return "size beyond the supported maximum";
        default: return "unknown status";
    }
}

int nuna_shutdown(void)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NUNA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_ctx_mutex);
    Context* c = g_ctx[dev];
    if (!c) return NUNA_OK;
    cudaDeviceSynchronize();
    if (c->bw) cudaFree(c->bw);
    if (c->scratch) cudaFree(c->scratch);
    for (void* d : c->retired_scratch) cudaFree(d);
    if (c->staging) cudaFree(c->staging);
    if (c->stream) cudaStreamDestroy(c->stream);
    for (auto& kv : c->sm_plans) cudaFree(kv.second.base);
    for (unsigned* d : c->retired_plans) cudaFree(d);
    delete c;
    g_ctx[dev] = nullptr;
    return NUNA_OK;
}

/* Test hook: the per-SM work lists planned for a one-shot of `ntiles` tiles under `topo` (NULL = no probe),
 * by the general planner (generic != 0) or the closed form.  off: [num_sms + 1], tiles: [ntiles].          */
int nuna_debug_plan_oneshot(const nuna_topology_t* topo, int num_sms, int nranks, size_t ntiles, size_t tile_bytes,
                            int generic, int domains, unsigned* off, unsigned* tiles)
{
    if (num_sms < 1 || nranks < 1 || nranks > NUNA_MAX_RANKS || !off || !tiles || domains < 0) return NUNA_ERR_INVALID_ARG;
    std::vector<std::vector<unsigned>> lists;
    plan_oneshot_lists(topo, num_sms, nranks, ntiles, tile_bytes, generic != 0, domains, lists);
    size_t n = 0;
    off[0] = 0;
    for (int s = 0; s < num_sms; ++s) {
        for (unsigned t : lists[s]) tiles[n++] = t;
        off[s + 1] = (unsigned)n;
    }
    return n == ntiles ? NUNA_OK : NUNA_ERR_INVALID_ARG;
}

/* Test hook (not part of the public header): every block of a `grid`-block launch arrives at a flag
 * barrier that expects `expected` arrivals and waits at most timeout_ms.  Writes how many blocks
 * passed.  With expected > grid nothing ever completes the barrier, the waits run out, and the
 * status word latches NUNA_ERR_TIMEOUT -- without trapping or hanging the device.                    */
int nuna_debug_barrier_selftest(unsigned grid, unsigned expected, unsigned timeout_ms, unsigned* passed)
{
    Context* c = nullptr;
    int st = get_context(&c);
    if (st != NUNA_OK) return st;
    if (!passed || grid == 0 || grid > (unsigned)c->num_sms || expected == 0) return NUNA_ERR_INVALID_ARG;
    unsigned* d = nullptr;
    if (cudaMalloc(&d, sizeof(unsigned)) != cudaSuccess) return NUNA_ERR_CUDA;
    cudaMemset(d, 0, sizeof(unsigned));
    st = launch(k_barrier_selftest, grid, (cudaStream_t)0, kLaunchCooperative, c->bw, expected,
                (unsigned long long)timeout_ms * 1000000ull, d);
    if (st == NUNA_OK && cudaDeviceSynchronize() != cudaSuccess) st = NUNA_ERR_CUDA;
    if (st == NUNA_OK && cudaMemcpy(passed, d, sizeof(unsigned), cudaMemcpyDeviceToHost) != cudaSuccess) st = NUNA_ERR_CUDA;
    cudaFree(d);
    return st;
}

/* Measurement hook: one launch of the one-shot allreduce (8 ranks, bf16, whole vectors) under a placement --
 * 0 round-robin, 1 co-located groups, 2 per-SM work lists -- with the latency of every work item's first load
 * sampled per warp into hist[NUNA_DEBUG_LAT_BINS] (bins of NUNA_DEBUG_LAT_STEP cycles, added to what hist
 * already holds).  Destinations receive the ordinary result.  Synchronises the device.                   */
int nuna_debug_access_latency(const void* const* src, void* const* dst, size_t count, int placement, unsigned* hist)
{
    constexpr int N = 8;
    int st = check_args(src, dst, N, count, count, NUNA_BF16, 0u, true);
    if (st != NUNA_OK) return st;
    if (!hist || count == 0 || count % 8 != 0 || placement < 0 || placement > 2) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    const Options o = snapshot(c);
    const RankPtrs p = make_ptrs(src, dst, N);
    const size_t nvec = count / 8;
    unsigned* d_hist = nullptr;
    if (cudaMalloc(&d_hist, kLatBins * sizeof(unsigned)) != cudaSuccess) return NUNA_ERR_CUDA;
    cudaMemset(d_hist, 0, kLatBins * sizeof(unsigned));
    if (placement == 0) {
        auto k = k_latency_rr<N, kBf16>;
        const size_t ntiles = ceil_div(nvec, (size_t)kThreads);
        st = launch(k, pick_grid(c, o, ntiles * N, NUNA_OCC(k)), (cudaStream_t)0, kLaunchPlain, p, count, ntiles, d_hist);
    } else if (placement == 1) {
        auto k = k_latency_group<N, 8, kBf16>;
        const size_t ntiles = ceil_div(nvec, (size_t)(kThreads / 8));
        st = launch(k, pick_grid(c, o, ntiles, NUNA_OCC(k)), (cudaStream_t)0, kLaunchPlain, p, count, ntiles, d_hist);
    } else {
        auto k = k_oneshot_sm<N, 8, kBf16, true>;
        SmPlan pl;
        st = get_sm_plan(c, N, nvec, 8, o.domains, (cudaStream_t)0, &pl);
        if (st == NUNA_OK) {
            SmLists sl;
            sl.off = pl.off; sl.tiles = pl.tiles; sl.cursor = pl.cursor; sl.present = pl.present; sl.ctl = pl.ctl;
            sl.nonempty = pl.nonempty; sl.num_sms = c->num_sms;
            const size_t cap = (size_t)c->num_sms * (size_t)NUNA_OCC(k);
            const unsigned grid = (unsigned)std::min(cap, std::max<size_t>((size_t)c->num_sms, (size_t)pl.total));
            st = launch(k, grid, (cudaStream_t)0, kLaunchPlain, p, count, sl,
                        (unsigned)std::max<size_t>(1, grid / (size_t)c->num_sms), d_hist);
        }
    }
    if (st == NUNA_OK && cudaDeviceSynchronize() != cudaSuccess) st = NUNA_ERR_CUDA;
    unsigned h[kLatBins];
    if (st == NUNA_OK && cudaMemcpy(h, d_hist, sizeof h, cudaMemcpyDeviceToHost) != cudaSuccess) st = NUNA_ERR_CUDA;
    if (st == NUNA_OK)
        for (int b = 0; b < kLatBins; ++b) hist[b] += h[b];
    cudaFree(d_hist);
    return st;
}

// See nuna_debug.h.  The same tile size, grid and mode bits as launch_regs<8, 8, bf16>.
int nuna_debug_oneshot_regs_traced(const void* const* src, void* const* dst, size_t count, unsigned flags, unsigned slot,
                                   unsigned long long* trace, unsigned* grid_blocks, void* stream)
{
    constexpr int N = 8;
    int st = check_args(src, dst, N, count, count, NUNA_BF16, flags & (NUNA_LAUNCH_PDL | NUNA_HINT_RESIDENT), true);
    if (st != NUNA_OK) return st;
    if (!trace || count == 0 || (flags & ~(NUNA_LAUNCH_PDL | NUNA_HINT_RESIDENT)) != 0u) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    const Options o = snapshot(c);
    auto k = k_oneshot_regs_timed<N, 8, kBf16>;
    const size_t nvec = count / 8;
    const unsigned tv = regs_tile_vecs(c, o, nvec, 1, NUNA_OCC(k));
    const size_t ntiles = ceil_div(nvec, (size_t)tv);
    const size_t nitems = std::max<size_t>(ntiles, (count % 8) ? (size_t)N : 0);
    const unsigned grid = pick_grid(c, o, std::max<size_t>(nitems, 1), NUNA_OCC(k), 0);
    const unsigned mode = (flags & NUNA_LAUNCH_PDL) ? kLaunchPdl : kLaunchPlain;
    const bool large_cold = !(flags & NUNA_HINT_RESIDENT) && count * 2 >= ((size_t)8 << 20);
    const bool prefetch = !large_cold && mode == kLaunchPdl && !(flags & NUNA_HINT_RESIDENT) && o.prefetch != 1;
    if (grid_blocks) *grid_blocks = grid;
    return launch(k, grid, (cudaStream_t)stream, mode, make_ptrs(src, dst, N), count, ntiles, tv,
                  ((flags & NUNA_HINT_RESIDENT) ? 0 : 1) | (prefetch ? 2 : 0), trace, slot, (unsigned)NUNA_DEBUG_TRACE_BLOCKS);
}

/* Test hook: a flag-synchronised two-shot whose consumers wait for a flag value that nobody publishes
 * (debug_bits = 1): every consumer wait runs out after timeout_ms, the kernel returns, destinations stay
 * unwritten and the status word latches NUNA_ERR_TIMEOUT; nothing traps or hangs.  debug_bits = 0 is the
 * ordinary kernel with an explicit timeout.                                                            */
int nuna_debug_twoshot(const void* const* src, void* const* dst, int nranks, size_t count, int dtype,
                       unsigned timeout_ms, unsigned debug_bits)
{
    int st = check_args(src, dst, nranks, count, count, dtype, 0u, true);
    if (st != NUNA_OK || count == 0) return st;
    if ((debug_bits & ~5u) != 0u) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    uint4* scratch;
    unsigned* tile_flags;
    {
        std::lock_guard<std::mutex> lock(c->mutex);
        if ((st = ensure_scratch(c, (count * elem_size(dtype) + 15) & ~(size_t)15)) != NUNA_OK) return st;
        scratch = reinterpret_cast<uint4*>(c->scratch);
        tile_flags = c->flags;
    }
    return launch_twoshot_flags(c->num_sms, 0, make_ptrs(src, dst, nranks), nranks, dtype, count, 0u, kMinFlagTileVec, scratch,
                                tile_flags, c->bw, (unsigned long long)timeout_ms * 1000000ull, false, debug_bits,
                                (cudaStream_t)0);
}

}  // extern "C"

// ---- two-shot allreduce for callers that cannot allocate ------------------------------------------
//
// Everything the flag-barrier two-shot needs beyond its inputs and outputs -- the shard
// intermediate and the barrier words -- lives in the two file-scope device arrays below, which
// every GPU that loads this library carries from module load to process exit (4 MiB + 384 bytes).
// In host code the names `g_static_shard` and `g_static_barrier` are only stand-ins for the
// symbols, not device addresses; the addresses a kernel can use come from cudaGetSymbolAddress,
// looked up once per device, with that device current, on the entry point's first call there.
namespace nuna {

static __device__ __align__(256) unsigned char g_static_shard[NUNA_STATIC_MAX_COUNT * 2];
static __device__ __align__(256) unsigned int g_static_flags[NUNA_STATIC_MAX_COUNT * 2 / (kStaticTileVec * 16) + 1];   // one per tile
static __device__ __align__(256) BarrierWords g_static_barrier;

struct StaticSetup {
    bool ready = false;
    uint4* shard = nullptr;              // device address of g_static_shard on this device
    unsigned* flags = nullptr;           // device address of g_static_flags
    BarrierWords* barrier = nullptr;     // device address of g_static_barrier
    int num_sms = 0;
};
static StaticSetup g_static_setup[kMaxDevices];
static std::mutex g_static_mutex;

// Once per device: resolve the symbols and zero the control words and ready flags.  No allocation.
static int static_setup(StaticSetup** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NUNA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup& s = g_static_setup[dev];
    if (!s.ready) {
        void* shard = nullptr;
        void* flags = nullptr;
        void* barrier = nullptr;
        if (cudaGetSymbolAddress(&shard, g_static_shard) != cudaSuccess || !shard) return NUNA_ERR_CUDA;
        if (cudaGetSymbolAddress(&flags, g_static_flags) != cudaSuccess || !flags) return NUNA_ERR_CUDA;
        if (cudaGetSymbolAddress(&barrier, g_static_barrier) != cudaSuccess || !barrier) return NUNA_ERR_CUDA;
        if (cudaDeviceGetAttribute(&s.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || s.num_sms < 1)
            return NUNA_ERR_CUDA;
        // epoch, cursor and departure counter start from zero, and no tile may read as ready; the shard
        // needs no clearing (every element is written before it is read)
        if (cudaMemset(barrier, 0, sizeof(BarrierWords)) != cudaSuccess) return NUNA_ERR_CUDA;
        if (cudaMemset(flags, 0, sizeof(g_static_flags)) != cudaSuccess) return NUNA_ERR_CUDA;
        s.shard = static_cast<uint4*>(shard);
        s.flags = static_cast<unsigned*>(flags);
        s.barrier = static_cast<BarrierWords*>(barrier);
        s.ready = true;
    }
    *out = &s;
    return NUNA_OK;
}

// For nuna_device_status: the status latched by the allocation-free entry point on the current device
// (0 if that entry point was never used here).  A latched timeout leaves cursor and departure counter in
// an undefined state, so the control words are zeroed again; the device is idle (the caller synchronised).
static int static_status_read_and_clear(unsigned* out)
{
    *out = 0;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NUNA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup& s = g_static_setup[dev];
    if (!s.ready) return NUNA_OK;
    BarrierWords h;
    if (cudaMemcpy(&h, s.barrier, sizeof h, cudaMemcpyDeviceToHost) != cudaSuccess) return NUNA_ERR_CUDA;
    *out = h.status;
    return h.status != 0 ? rewind_barrier_words(s.barrier, h) : NUNA_OK;
}

}  // namespace nuna

extern "C" int nuna_allreduce_twoshot_static(const void* const* src, void* const* dst, int nranks, size_t count,
                                             int dtype, void* stream)
{
    int st = check_args(src, dst, nranks, count, count, dtype, 0u, true);
    if (st != NUNA_OK || count == 0) return st;
    if (count * elem_size(dtype) > (size_t)NUNA_STATIC_MAX_COUNT * 2) {
        fprintf(stderr, "nuna_allreduce_twoshot_static: %zu bytes per rank exceed the fixed scratch array "
                        "(NUNA_STATIC_MAX_COUNT = %d 16-bit elements, %d bytes); use nuna_allreduce_twoshot for larger "
                        "messages\n", count * elem_size(dtype), (int)NUNA_STATIC_MAX_COUNT, (int)NUNA_STATIC_MAX_COUNT * 2);
        return NUNA_ERR_TOO_LARGE;
    }
    StaticSetup* s = nullptr;
    if ((st = static_setup(&s)) != NUNA_OK) return st;
    // tiles of 4 KiB per source (the fixed flag array has one word per 4 KiB of the shard), fewer vectors for many ranks
    return launch_twoshot_flags(s->num_sms, 0, make_ptrs(src, dst, nranks), nranks, dtype, count, kStaticTileVec, kStaticTileVec,
                                s->shard, s->flags, s->barrier, 1000000000ull, false, 0u, (cudaStream_t)stream);
}
