// Host side of the C ABI: argument checks, per-device context, launch configuration.
#include "nuna_internal.h"
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

static int env_int(const char* name, int fallback)
{
    const char* s = getenv(name);
    return (s && *s) ? atoi(s) : fallback;
}

int init_barrier_words(Context* c)
{
    return cudaMemset(c->bw, 0, sizeof(BarrierWords)) == cudaSuccess ? NUNA_OK : NUNA_ERR_CUDA;
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
        c->timeout_ns = (unsigned long long)env_int("NUNA_TIMEOUT_MS", 1000) * 1000000ull;
        c->blocks_override = env_int("NUNA_BLOCKS", 0);
        c->unroll_override = env_int("NUNA_UNROLL", 0);
        c->auto_min_bytes = (size_t)env_int("NUNA_AUTO_MIN_BYTES", 64 << 10);
        c->coloc_override = env_int("NUNA_COLOC", 0);
        g_ctx[dev] = c;
    }
    *out = g_ctx[dev];
    return NUNA_OK;
}

int ensure_scratch(Context* c, size_t bytes)
{
    if (bytes <= c->scratch_bytes) return NUNA_OK;
    void* p = nullptr;
    const size_t want = (bytes + 255) & ~(size_t)255;
    if (cudaMalloc(&p, want) != cudaSuccess) return NUNA_ERR_CUDA;
    if (c->scratch) cudaFree(c->scratch);
    c->scratch = p;
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
                   NUNA_PLACE_CLUSTER)) != 0u ||
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
static int pick_unroll(const Context* c, int nranks)
{
    int u = 1;
    if (c->unroll_override == 1 || c->unroll_override == 2 || c->unroll_override == 4) u = c->unroll_override;
    while (u > 1 && u * nranks > 16) u >>= 1;
    return u;
}

template <typename K>
static int occupancy(Context* c, K kernel, int* cache)
{
    if (*cache == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kThreads, 0) != cudaSuccess || n < 1) n = 1;
        *cache = n;
    }
    (void)c;
    return *cache;
}

// Grid size: `waves` x (SMs x resident blocks per SM), never more than the work items.  Streaming
// kernels (two-shot put, reduce-scatter, allgather) run one item per block (waves = 0: no cap): leaving
// the balancing to the hardware block scheduler measured 0.99 of the copy peak at 64 MiB per rank
// against 0.90 for a persistent grid-stride loop.  The one-shot wants its N readers of a tile close in
// time so that re-reads hit L2: four waves measured best (0.70 of peak at 64 MiB against 0.63 for one
// wave and 0.62 for an uncapped grid).
static unsigned pick_grid(const Context* c, size_t nitems, int blocks_per_sm, int waves = 1)
{
    size_t cap = waves > 0 ? (size_t)c->num_sms * (size_t)blocks_per_sm * (size_t)waves : ((size_t)1 << 22);
    if (c->blocks_override > 0) cap = (size_t)c->blocks_override;
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

template <typename... Args, typename... Act>
static int launch(void (*kernel)(Args...), unsigned grid, cudaStream_t stream, unsigned mode, Act&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
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

// NUNA_PLACE_AUTO: use the placement-aware kernel only where it is at least as fast as the
// round-robin baseline.  NUNA_AUTO_MIN_BYTES overrides the measured crossover (bytes per rank).
static bool aware_pays_off(const Context* c, int nranks, size_t bytes, unsigned flags)
{
    if (nranks < 2 || !(flags & NUNA_HINT_RESIDENT)) return false;
    // sources and destinations of one call, twice over (the producer's other buffers), must fit in L2
    // for "resident" to be physically possible
    if (4 * bytes * (size_t)nranks > c->l2_bytes) return false;
    return bytes >= c->auto_min_bytes;
}


// ---- per-SM work lists for the one-shot (Algorithm 1 applied to its regular workload) ----------------
//
// Thread blocks = work items (tile, d); item (t, d) touches the N source chunks of tile t and the
// destination chunk (d, t).  Domains and the order of SMs inside a domain come from the probe
// (nearest = lowest mean hit latency).  The per-SM budget R_max is ceil(groups per domain / SMs of
// the smallest domain) whole groups, so a small workload fills only the nearest SMs, one group each,
// and a large one spreads evenly.  Up to kGenericPlanTiles tiles the lists are produced by the
// general planner (nuna_plan_placement); beyond that by the closed form it reduces to for this
// workload (tile t -> domain t mod D, SMs of the domain filled in preference order), which the host
// tests check against the general planner.
constexpr size_t kGenericPlanTiles = 1024;

void plan_oneshot_lists(const nuna_topology_t* topo, int num_sms, int nranks, size_t ntiles, size_t tile_bytes,
                        bool generic, std::vector<std::vector<unsigned>>& lists)
{
    lists.assign((size_t)num_sms, {});
    const bool split = topo && topo->verdict == NUNA_TOPO_NONUNIFORM && topo->num_domains == 2;
    const int D = split ? 2 : 1;
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
    int smallest = num_sms;
    if (split) {
        int n1 = 0;
        for (int s = 0; s < num_sms; ++s) n1 += dom[s];
        smallest = std::max(1, std::min(n1, num_sms - n1));
    }
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

static int get_sm_plan(Context* c, int nranks, size_t nvec, int coloc, cudaStream_t stream, SmPlan** out)
{
    std::lock_guard<std::mutex> lock(c->mutex);
    const auto key = std::make_tuple(nranks, nvec, coloc);
    auto it = c->sm_plans.find(key);
    if (it == c->sm_plans.end()) {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone)
            return NUNA_ERR_CAPTURING;                 // building a plan allocates: make one plain call first
        const size_t lanes = (size_t)(kThreads / coloc);
        const size_t ntiles = ceil_div(nvec, lanes);
        std::vector<std::vector<unsigned>> lists;
        plan_oneshot_lists(c->have_topology ? &c->topology : nullptr, c->num_sms, nranks, ntiles, lanes * 16,
                           ntiles <= kGenericPlanTiles, lists);
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
    *out = &it->second;
    return NUNA_OK;
}

static int coloc_for(const Context* c, int nranks)
{
    int coloc = c->coloc_override > 0 ? c->coloc_override : 8;
    while (coloc > 1 && coloc / 2 >= nranks) coloc >>= 1;
    return coloc >= 8 ? 8 : coloc >= 4 ? 4 : 2;
}

// Everything a later launch of this shape would have to allocate (called before stream capture).
int prepare_oneshot(Context* c, int nranks, int dtype, size_t count, unsigned flags)
{
    if ((flags & NUNA_PLACE_MASK) == NUNA_PLACE_AWARE && (flags & NUNA_PLACE_SM_LISTS)) {
        SmPlan* pl = nullptr;
        return get_sm_plan(c, nranks, count / elems_per_vec(dtype), coloc_for(c, nranks), (cudaStream_t)0, &pl);
    }
    return NUNA_OK;
}

template <int N, int C, int DT>
static int launch_sm_lists(Context* c, const RankPtrs& p, size_t count, unsigned mode, cudaStream_t stream)
{
    static int occ = 0;
    auto k = k_oneshot_sm<N, C, DT>;
    SmPlan* pl = nullptr;
    const int st = get_sm_plan(c, N, count / Elem<DT>::kElems, C, stream, &pl);
    if (st != NUNA_OK) return st;
    SmLists sl;
    sl.off = pl->off; sl.tiles = pl->tiles; sl.cursor = pl->cursor; sl.present = pl->present; sl.ctl = pl->ctl;
    sl.nonempty = pl->nonempty; sl.num_sms = c->num_sms;
    const size_t cap = (size_t)c->num_sms * (size_t)occupancy(c, k, &occ);
    const unsigned grid = (unsigned)std::min(cap, std::max<size_t>((size_t)c->num_sms, (size_t)pl->total));
    const unsigned blocks_per_sm = (unsigned)std::max<size_t>(1, grid / (size_t)c->num_sms);
    return launch(k, grid, stream, mode, p, count, sl, blocks_per_sm);
}

template <int N, int DT>
static int launch_cluster(Context* c, const RankPtrs& p, size_t count, unsigned mode, cudaStream_t stream)
{
    auto k = k_oneshot_cluster<N, DT>;
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t ntiles = std::max<size_t>(1, ceil_div(nvec, (size_t)kThreads));
    size_t clusters = std::min<size_t>(ntiles, (size_t)1 << 20);
    if (c->blocks_override > 0) clusters = std::max<size_t>(1, std::min<size_t>(clusters, (size_t)c->blocks_override / N));
    t_cluster_dim = N;
    return launch(k, (unsigned)(clusters * N), stream, mode, p, count, ntiles);
}

template <int N, int C, int DT>
static int launch_group(Context* c, const RankPtrs& p, size_t count, unsigned mode, cudaStream_t stream)
{
    static int occ = 0;
    auto k = k_oneshot_group<N, C, DT>;
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t ntiles = ceil_div(nvec, (size_t)(kThreads / C));
    const size_t nitems = std::max<size_t>(ntiles * ((N + C - 1) / C), (count % Elem<DT>::kElems) ? (size_t)N : 0);
    const unsigned grid = pick_grid(c, nitems, occupancy(c, k, &occ));
    return launch(k, grid, stream, mode, p, count, ntiles);
}

int launch_oneshot(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream)
{
    const size_t bytes = count * elem_size(dtype);                   // per rank
    const size_t epv = elems_per_vec(dtype);
    const unsigned mode = launch_mode(flags, bytes * (size_t)nranks);
    const size_t nvec = count / epv;
    const unsigned place = flags & NUNA_PLACE_MASK;
    if (place == NUNA_PLACE_AWARE || (place == NUNA_PLACE_AUTO && aware_pays_off(c, nranks, bytes, flags))) {
        // co-location factor: C destinations of a tile share a block (C <= N rounded up to a power of two)
        const int coloc = coloc_for(c, nranks);
        if ((flags & NUNA_PLACE_CLUSTER) && nranks >= 2 && nranks <= 8) {
            return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
                constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
                if constexpr (N >= 2 && N <= 8) return launch_cluster<N, DT>(c, p, count, mode, stream);
                else return NUNA_ERR_INVALID_ARG;
            });
        }
        if (flags & NUNA_PLACE_SM_LISTS) {
            return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
                constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
                if (coloc >= 8) return launch_sm_lists<N, 8, DT>(c, p, count, mode, stream);
                if (coloc >= 4) return launch_sm_lists<N, 4, DT>(c, p, count, mode, stream);
                return launch_sm_lists<N, 2, DT>(c, p, count, mode, stream);
            });
        }
        return dispatch(nranks, 1, dtype, [&](auto n_, auto, auto d_) -> int {
            constexpr int N = decltype(n_)::value, DT = decltype(d_)::value;
            if (coloc >= 8) return launch_group<N, 8, DT>(c, p, count, mode, stream);
            if (coloc >= 4) return launch_group<N, 4, DT>(c, p, count, mode, stream);
            return launch_group<N, 2, DT>(c, p, count, mode, stream);
        });
    }
    return dispatch(nranks, pick_unroll(c, nranks), dtype, [&](auto n_, auto u_, auto d_) -> int {
        NUNA_NUD(n_, u_, d_);
        static int occ = 0;
        auto k = k_oneshot_rr<N, U, DT>;
        const size_t ntiles = ceil_div(nvec, (size_t)kThreads * U);
        const size_t nitems = std::max<size_t>(ntiles * N, (count % epv) ? (size_t)N : 0);
        // one resident wave while the message is small enough for latency to matter, four beyond
        const unsigned grid = pick_grid(c, nitems, occupancy(c, k, &occ), bytes >= ((size_t)8 << 20) ? 4 : 1);
        return launch(k, grid, stream, mode, p, count, ntiles);
    });
}

// Launches the flag-barrier two-shot on explicit scratch / barrier storage (the context's, or the
// fixed arrays of the allocation-free entry point).
static int launch_twoshot_fused(int num_sms, int blocks_override, const RankPtrs& p, int nranks, int dtype, size_t count,
                                int u, uint4* scratch, BarrierWords* bw, unsigned long long timeout_ns,
                                cudaStream_t stream)
{
    // chunk = ceil(count / N) rounded up to whole vectors
    const size_t chunk_vec = ceil_div(ceil_div(count, (size_t)nranks), elems_per_vec(dtype));
    return dispatch(nranks, u, dtype, [&](auto n_, auto u_, auto d_) -> int {
        NUNA_NUD(n_, u_, d_);
        static int occ = 0;
        auto k = k_twoshot_fused<N, U, DT>;
        const size_t tiles_per_chunk = ceil_div(chunk_vec, (size_t)kThreads * U);
        // every block must be resident for the flag barrier: never more than the device holds at once
        size_t cap = (size_t)num_sms * (size_t)occupancy(nullptr, k, &occ);
        if (blocks_override > 0) cap = std::min<size_t>(cap, (size_t)blocks_override);
        const unsigned grid = (unsigned)std::max<size_t>(1, std::min(tiles_per_chunk * N, cap));
        return launch(k, grid, stream, kLaunchCooperative, p, scratch, count, chunk_vec, bw, timeout_ns);
    });
}

int launch_twoshot(Context* c, const RankPtrs& p, int nranks, int dtype, size_t count, unsigned flags, cudaStream_t stream)
{
    const size_t epv = elems_per_vec(dtype);
    const unsigned mode = launch_mode(flags);
    const size_t nvec = count / epv;
    if (flags & NUNA_TWOSHOT_PUT) {
        return dispatch(nranks, pick_unroll(c, nranks), dtype, [&](auto n_, auto u_, auto d_) -> int {
            NUNA_NUD(n_, u_, d_);
            static int occ = 0;
            auto k = k_twoshot_put<N, U, DT>;
            const size_t ntiles = ceil_div(nvec, (size_t)kThreads * U);
            const unsigned grid = pick_grid(c, std::max<size_t>(ntiles, 1), occupancy(c, k, &occ), 0);
            return launch(k, grid, stream, mode, p, count, ntiles);
        });
    }
    return launch_twoshot_fused(c->num_sms, c->blocks_override, p, nranks, dtype, count, pick_unroll(c, nranks),
                                reinterpret_cast<uint4*>(c->scratch), c->bw, c->timeout_ns, stream);
}

int launch_reduce_scatter(Context* c, const RankPtrs& p, int nranks, int dtype, size_t shard, unsigned flags,
                          cudaStream_t stream)
{
    const size_t epv = elems_per_vec(dtype);
    const unsigned mode = launch_mode(flags);
    if (shard % epv) {
        const unsigned grid = pick_grid(c, ceil_div(shard * nranks, kThreads), 8);
        return dispatch(nranks, 1, dtype, [&](auto n_, auto u_, auto d_) -> int {
            NUNA_NUD(n_, u_, d_);
            return launch(k_reduce_scatter_scalar<N, DT>, grid, stream, mode, p, shard);
        });
    }
    const size_t shard_vec = shard / epv;
    return dispatch(nranks, pick_unroll(c, nranks), dtype, [&](auto n_, auto u_, auto d_) -> int {
        NUNA_NUD(n_, u_, d_);
        static int occ = 0;
        auto k = k_reduce_scatter<N, U, DT>;
        const size_t tiles = ceil_div(shard_vec, (size_t)kThreads * U);
        const unsigned grid = pick_grid(c, tiles * N, occupancy(c, k, &occ), 0);
        return launch(k, grid, stream, mode, p, shard_vec, tiles);
    });
}

// Allgather and alltoall copy bits: they work on 16-byte vectors when a shard is a whole number of
// them, otherwise on 16-bit units (every element type is a multiple of that).
int launch_allgather(Context* c, const RankPtrs& p, int nranks, size_t shard_bytes, unsigned flags, cudaStream_t stream)
{
    const unsigned mode = launch_mode(flags);
    if (shard_bytes % 16) {
        const size_t shard16 = shard_bytes / 2;
        const unsigned grid = pick_grid(c, ceil_div(shard16 * nranks, kThreads), 8);
        return launch(k_allgather_scalar, grid, stream, mode, p, nranks, shard16);
    }
    const size_t shard_vec = shard_bytes / 16;
    static int occ = 0;
    // One block per (rank, tile) storing to all N destinations.  Splitting a tile's destinations over
    // several blocks (dsplit > 1) was measured slower at every size tried (16 x 64 KiB: 4.4 us with 1,
    // 5.4 us with 8): the stores, not the block count, are the limit.
    constexpr int U = 2;
    const int dsplit = 1;
    auto k = k_allgather<U>;
    const size_t tiles = ceil_div(shard_vec, (size_t)kThreads * U);
    const unsigned grid = pick_grid(c, tiles * nranks * dsplit, occupancy(c, k, &occ), 0);
    return launch(k, grid, stream, mode, p, nranks, shard_vec, tiles, dsplit);
}

int launch_alltoall(Context* c, const RankPtrs& p, int nranks, size_t block_bytes, unsigned flags, cudaStream_t stream)
{
    const unsigned mode = launch_mode(flags);
    if (block_bytes % 16) {
        const size_t block16 = block_bytes / 2;
        const unsigned grid = pick_grid(c, ceil_div(block16 * nranks * nranks, kThreads), 8);
        return launch(k_alltoall_scalar, grid, stream, mode, p, nranks, block16);
    }
    const size_t block_vec = block_bytes / 16;
    static int occ = 0;
    constexpr int U = 2;
    auto k = k_alltoall<U>;
    const size_t tiles = ceil_div(block_vec, (size_t)kThreads * U);
    const unsigned grid = pick_grid(c, tiles * nranks * nranks, occupancy(c, k, &occ), 0);
    return launch(k, grid, stream, mode, p, nranks, block_vec, tiles);
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
        case NUNA_OPT_BLOCKS: c->blocks_override = (int)std::min<long long>(value, 1 << 22); break;
        case NUNA_OPT_UNROLL: c->unroll_override = (int)value; break;
        case NUNA_OPT_COLOC: c->coloc_override = (int)value; break;
        case NUNA_OPT_AUTO_MIN_BYTES: c->auto_min_bytes = value ? (size_t)value : ((size_t)64 << 10); break;
        case NUNA_OPT_TIMEOUT_MS: c->timeout_ns = (unsigned long long)(value ? value : 1000) * 1000000ull; break;
        default: return NUNA_ERR_INVALID_ARG;
    }
    return NUNA_OK;
}

int nuna_allreduce_oneshot(const void* const* src, void* const* dst, int nranks, size_t count, int dtype,
                           unsigned flags, void* stream)
{
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
    int st = check_args(src, dst, nranks, count, count, dtype, flags, true);
    if (st != NUNA_OK || count == 0) return st;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    if (!(flags & NUNA_TWOSHOT_PUT)) {
        std::lock_guard<std::mutex> lock(c->mutex);
        const size_t need = (count * elem_size(dtype) + 15) & ~(size_t)15;
        if (need > c->scratch_bytes) {
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
    // Crossover measured on B200, cold and L2-resident, with dependent launch: the one-shot's N-fold
    // re-reads cost more the more ranks there are, so it wins up to 1 MiB per rank at 2 ranks,
    // 512 KiB at 4, 128 KiB at 8 and 64 KiB at 16.
    const size_t bytes = count * elem_size(dtype);
    const size_t limit = nranks <= 2 ? ((size_t)1 << 20) : nranks <= 4 ? ((size_t)512 << 10)
                       : nranks <= 8 ? ((size_t)128 << 10) : ((size_t)64 << 10);
    if (nranks <= 1 || bytes <= limit)
        return nuna_allreduce_oneshot(src, dst, nranks, count, dtype, flags & ~NUNA_TWOSHOT_PUT, stream);
    return nuna_allreduce_twoshot(src, dst, nranks, count, dtype, flags, stream);
}

int nuna_reduce_scatter(const void* const* src, void* const* dst, int nranks, size_t shard_count, int dtype,
                        unsigned flags, void* stream)
{
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
    int st = check_args(src, dst, nranks, count, count, dtype, flags, false);
    if (st != NUNA_OK || count == 0) return st;
    if (!two_shot && (flags & NUNA_TWOSHOT_PUT)) return NUNA_ERR_INVALID_ARG;
    Context* c = nullptr;
    if ((st = get_context(&c)) != NUNA_OK) return st;
    std::lock_guard<std::mutex> lock(c->mutex);
    const size_t bytes = count * elem_size(dtype);
    if (!c->stream && cudaStreamCreateWithFlags(&c->stream, cudaStreamNonBlocking) != cudaSuccess) return NUNA_ERR_CUDA;

    // Page-locked host buffers are visible to the device: the put form of the two-shot reads every source
    // byte once and writes every destination byte once, so it can run directly on them -- one kernel, reads
    // and writes crossing the host link in both directions at once, no staging copies.
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
            st = launch_twoshot(c, make_ptrs(msrc, mdst, nranks), nranks, dtype, count, flags & ~NUNA_LAUNCH_PDL, c->stream);
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
    if (two_shot && !(flags & NUNA_TWOSHOT_PUT) && (st = ensure_scratch(c, slot)) != NUNA_OK) return st;
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
    *out = (int)h.status;
    if (h.status != 0) return init_barrier_words(c);
    return NUNA_OK;
}

int nuna_launch_floor(unsigned blocks, unsigned flags, void* stream)
{
    if (blocks == 0 || blocks > (1u << 20) || (flags & ~NUNA_LAUNCH_PDL)) return NUNA_ERR_INVALID_ARG;
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
                            int generic, unsigned* off, unsigned* tiles)
{
    if (num_sms < 1 || nranks < 1 || nranks > NUNA_MAX_RANKS || !off || !tiles) return NUNA_ERR_INVALID_ARG;
    std::vector<std::vector<unsigned>> lists;
    plan_oneshot_lists(topo, num_sms, nranks, ntiles, tile_bytes, generic != 0, lists);
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
static __device__ __align__(256) BarrierWords g_static_barrier;

struct StaticSetup {
    bool ready = false;
    uint4* shard = nullptr;              // device address of g_static_shard on this device
    BarrierWords* barrier = nullptr;     // device address of g_static_barrier on this device
    int num_sms = 0;
};
static StaticSetup g_static_setup[kMaxDevices];
static std::mutex g_static_mutex;

// Once per device: resolve the two symbols and zero the barrier words.  No allocation.
static int static_setup(StaticSetup** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NUNA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup& s = g_static_setup[dev];
    if (!s.ready) {
        void* shard = nullptr;
        void* barrier = nullptr;
        if (cudaGetSymbolAddress(&shard, g_static_shard) != cudaSuccess || !shard) return NUNA_ERR_CUDA;
        if (cudaGetSymbolAddress(&barrier, g_static_barrier) != cudaSuccess || !barrier) return NUNA_ERR_CUDA;
        if (cudaDeviceGetAttribute(&s.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || s.num_sms < 1)
            return NUNA_ERR_CUDA;
        // the barrier counts arrivals from zero; the shard needs no clearing (written before it is read)
        if (cudaMemset(barrier, 0, sizeof(BarrierWords)) != cudaSuccess) return NUNA_ERR_CUDA;
        s.shard = static_cast<uint4*>(shard);
        s.barrier = static_cast<BarrierWords*>(barrier);
        s.ready = true;
    }
    *out = &s;
    return NUNA_OK;
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
    const int u = 1;
    return launch_twoshot_fused(s->num_sms, 0, make_ptrs(src, dst, nranks), nranks, dtype, count, u, s->shard, s->barrier,
                                1000000000ull, (cudaStream_t)stream);
}
