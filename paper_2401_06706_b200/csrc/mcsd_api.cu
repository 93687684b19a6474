// Host side of libmcsd.so: argument validation, tree plan, launch configuration
// and the extern "C" entry points declared in mcsd.h.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <initializer_list>
#include <mutex>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "mcsd_device.cuh"

namespace mcsd {
namespace {

thread_local int g_last_launches = 0;

// Tuning and test overrides (mcsd_set_option).  Initial values come from the environment
// variables of the same names, read once when the library is loaded.
int env_int(const char *name, int fallback)
{
    const char *v = std::getenv(name);
    return (v && *v) ? std::atoi(v) : fallback;
}
struct Options {
    int v[MCSD_OPT_COUNT];
    Options()
    {
        for (int &x : v) x = 0;
        v[MCSD_OPT_CLUSTER] = env_int("MCSD_CLUSTER", 0);
        v[MCSD_OPT_EPT] = env_int("MCSD_EPT", 0);
        v[MCSD_OPT_DIRECT] = env_int("MCSD_DIRECT", 0);
        v[MCSD_OPT_SAMPLE_AHEAD] = env_int("MCSD_SAMPLE_AHEAD", 100);
        v[MCSD_OPT_WAIT_POLLS] = 0;
        v[MCSD_OPT_TEST_EXTRA_TX] = 0;
        v[MCSD_OPT_PDL] = env_int("MCSD_PDL", 1);
        v[MCSD_OPT_SPLIT] = env_int("MCSD_SPLIT", 0);
        v[MCSD_OPT_TRACE] = env_int("MCSD_TRACE", 0);
        v[MCSD_OPT_WALK_CLUSTER] = env_int("MCSD_WALK_CLUSTER", 0);
    }
};
Options g_opt;

// MCSD_OPT_TRACE: bit 0, one line per call of a verification entry point on stderr (what was asked for,
// how the node stage was laid out, the return code); bit 1, an NVTX range around the call, for timelines.
// Host side only; the kernels are not touched.
struct TraceNote {
    int cluster = 0, ept = 0, threads = 0, direct = 0, split = 0;
    long long clusters = 0, stream_ctas = 0;
};
thread_local TraceNote g_note;
struct Trace {
    const char *name;
    const mcsd_desc *d;
    float T;
    int mode, bits;
    Trace(const char *n, const mcsd_desc *desc, float temperature, int replacement_mode)
        : name(n), d(desc), T(temperature), mode(replacement_mode), bits(g_opt.v[MCSD_OPT_TRACE])
    {
        if (bits & 2) nvtxRangePushA(name);
        if (bits & 1) g_note = TraceNote();
    }
    int done(int rc)
    {
        if (bits & 2) nvtxRangePop();
        if (bits & 1) {
            if (d)
                std::fprintf(stderr, "[mcsd] %s batch=%d nodes=%d internal=%d vocab=%d dtype=%d T=%g mode=%d -> rc=%d launches=%d",
                             name, d->batch, d->n_nodes, d->n_internal, d->vocab, d->dtype, static_cast<double>(T), mode, rc,
                             rc == MCSD_OK ? g_last_launches : 0);
            else
                std::fprintf(stderr, "[mcsd] %s desc=NULL -> rc=%d", name, rc);
            if (rc == MCSD_OK && g_note.threads)
                std::fprintf(stderr, " node stage: cluster=%d x %d threads, %d elements/thread%s, %lld clusters%s",
                             g_note.cluster, g_note.threads, g_note.ept, g_note.direct ? ", element loads" : "",
                             g_note.clusters, g_note.split ? ", split launch" : "");
            if (rc == MCSD_OK && g_note.split) std::fprintf(stderr, " (%lld streaming CTAs)", g_note.stream_ctas);
            std::fprintf(stderr, "\n");
        }
        return rc;
    }
};

struct TreePlan {
    int gamma = 0;
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
};

// Checks the layout contract (level order, contiguous children, internal nodes
// first) and fills the per-node child ranges.  Returns MCSD_OK or an error code.
int plan_tree(const int32_t *parent, int n_nodes, int n_internal, TreePlan *plan)
{
    if (!parent) return MCSD_ERR_NULL;
    if (n_nodes < 1) return MCSD_ERR_SHAPE;
    if (n_nodes > MCSD_MAX_NODES) return MCSD_ERR_UNSUPPORTED;
    if (parent[0] != -1) return MCSD_ERR_TREE;
    std::vector<int> depth(n_nodes, 0);
    std::memset(plan->child_first, 0, sizeof(plan->child_first));
    std::memset(plan->child_count, 0, sizeof(plan->child_count));
    int gamma = 0;
    for (int n = 1; n < n_nodes; ++n) {
        const int p = parent[n];
        if (p < 0 || p >= n) return MCSD_ERR_TREE;
        if (p < parent[n - 1]) return MCSD_ERR_TREE;  // level order <=> parents never decrease
        if (plan->child_count[p] == 0) plan->child_first[p] = static_cast<uint16_t>(n);
        if (plan->child_count[p] >= MCSD_MAX_CHILDREN) return MCSD_ERR_UNSUPPORTED;
        ++plan->child_count[p];
        depth[n] = depth[p] + 1;
        if (depth[n] > gamma) gamma = depth[n];
    }
    if (n_internal >= 0) {
        for (int n = 0; n < n_nodes; ++n)
            if ((plan->child_count[n] > 0) != (n < n_internal)) return MCSD_ERR_TREE;
    }
    plan->gamma = gamma;
    return MCSD_OK;
}

// The tree a host thread verified last is almost always the tree it verifies next: its plan is
// kept and found again by comparing the parent array (at most 2 KB).
struct CachedPlan {
    int n_nodes = 0, n_internal = -2;
    int32_t parent[MCSD_MAX_NODES];
    TreePlan plan;
};
thread_local CachedPlan g_plan_cache;

int plan_tree_cached(const int32_t *parent, int n_nodes, int n_internal, TreePlan *plan)
{
    if (!parent) return MCSD_ERR_NULL;
    CachedPlan &cp = g_plan_cache;
    if (n_nodes >= 1 && n_nodes <= MCSD_MAX_NODES && cp.n_nodes == n_nodes && cp.n_internal == n_internal &&
        std::memcmp(cp.parent, parent, sizeof(int32_t) * n_nodes) == 0) {
        *plan = cp.plan;
        return MCSD_OK;
    }
    const int rc = plan_tree(parent, n_nodes, n_internal, plan);
    if (rc == MCSD_OK) {
        cp.n_nodes = n_nodes;
        cp.n_internal = n_internal;
        std::memcpy(cp.parent, parent, sizeof(int32_t) * n_nodes);
        cp.plan = *plan;
    }
    return rc;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// MCSD_OPT_TIME_KERNELS: CUDA events around every kernel the verification entry points launch, on
// the stream they are launched on; mcsd_last_kernel_times reads the last call's.  Slots: 0 cluster
// (or argmax / naive) kernel, 1 streaming kernel, 2 single-test kernel, 3 walk kernel.
constexpr int kTimeSlots = 4;
struct KernelTimers {
    cudaEvent_t ev[kTimeSlots][2] = {};
    bool used[kTimeSlots] = {};
    bool created = false;
    int device = -1;   // the device the events belong to
};
thread_local KernelTimers g_timers;

inline void reset_timers_used()
{
    for (bool &u : g_timers.used) u = false;
}
struct ScopedTimer {
    int slot;
    cudaStream_t stream;
    bool on;
    ScopedTimer(int s, cudaStream_t st) : slot(s), stream(st), on(g_opt.v[MCSD_OPT_TIME_KERNELS] != 0)
    {
        if (!on) return;
        int dev = 0;
        cudaGetDevice(&dev);
        if (g_timers.created && g_timers.device != dev) {   // the thread moved to another device
            for (auto &pair : g_timers.ev)
                for (auto &e : pair) cudaEventDestroy(e);
            g_timers.created = false;
            reset_timers_used();
        }
        if (!g_timers.created) {
            for (auto &pair : g_timers.ev)
                for (auto &e : pair) cudaEventCreate(&e);
            g_timers.created = true;
            g_timers.device = dev;
        }
        cudaEventRecord(g_timers.ev[slot][0], stream);
    }
    ~ScopedTimer()
    {
        if (!on) return;
        cudaEventRecord(g_timers.ev[slot][1], stream);
        g_timers.used[slot] = true;
    }
};
void reset_timers() { reset_timers_used(); }

// Checked build: the address ranges the kernels of the next launches on `stream` may read.  An
// empty list switches the checks off (kernels whose inputs are not registered).
struct Range { const void *p; size_t bytes; };
#ifdef MCSD_DEBUG_BOUNDS
int debug_register(cudaStream_t stream, std::initializer_list<Range> ranges)
{
    DebugRanges r = {};
    for (const Range &x : ranges) {
        if (!x.p || x.bytes == 0 || r.n >= 12) continue;
        // (MCSD_OPT_TEST_SHRINK_RANGES: a test of the checker itself registers less than is there)
        const size_t cut = static_cast<size_t>(g_opt.v[MCSD_OPT_TEST_SHRINK_RANGES]);
        r.lo[r.n] = reinterpret_cast<unsigned long long>(x.p);
        r.hi[r.n] = r.lo[r.n] + (x.bytes > cut ? x.bytes - cut : 0);
        ++r.n;
    }
    return cudaMemcpyToSymbolAsync(g_dbg_ranges, &r, sizeof(r), 0, cudaMemcpyHostToDevice, stream) == cudaSuccess
               ? MCSD_OK : MCSD_ERR_CUDA;
}
#else
inline int debug_register(cudaStream_t, std::initializer_list<Range>) { return MCSD_OK; }
#endif

struct Workspace {
    int32_t *node_accept;
    int32_t *node_bonus;
    NodeStats *stats;
    float2 *leaf_part;
    float4 *single_part;
    int32_t *status;
    int32_t *path[2];
    size_t bytes;
};

Workspace carve(void *base, long long n_items, long long n_leaf_items, int batch)
{
    const long long n_internal_items = n_items - n_leaf_items;
    Workspace w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        unsigned char *p = base ? static_cast<unsigned char *>(base) + off : nullptr;
        off += align_up(bytes, 256);
        return p;
    };
    w.node_accept = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * n_items));
    w.node_bonus = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * n_items));
    w.stats = reinterpret_cast<NodeStats *>(take(sizeof(NodeStats) * n_items));
    w.leaf_part = reinterpret_cast<float2 *>(take(sizeof(float2) * kLeafEntries * n_leaf_items));
    w.single_part = reinterpret_cast<float4 *>(take(sizeof(float4) * kLeafEntries * n_internal_items));
    w.status = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * (batch > 0 ? batch : 1)));
    w.path[0] = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * (batch > 0 ? batch : 1)));
    w.path[1] = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * (batch > 0 ? batch : 1)));
    w.bytes = off;
    return w;
}

int check_desc(const mcsd_desc *d)
{
    if (!d) return MCSD_ERR_NULL;
    if (d->reserved != 0) return MCSD_ERR_SHAPE;
    if (d->batch < 0 || d->n_nodes < 1 || d->vocab < 1 || d->n_internal < 0 ||
        d->n_internal > d->n_nodes)
        return MCSD_ERR_SHAPE;
    if (d->n_nodes > MCSD_MAX_NODES || d->vocab > MCSD_MAX_VOCAB) return MCSD_ERR_UNSUPPORTED;
    if (static_cast<long long>(d->batch) * d->n_nodes > 0x7fffffffLL) return MCSD_ERR_UNSUPPORTED;
    if (d->dtype != MCSD_DTYPE_F32 && d->dtype != MCSD_DTYPE_BF16 && d->dtype != MCSD_DTYPE_F16)
        return MCSD_ERR_DTYPE;
    if (d->ld_target < d->vocab) return MCSD_ERR_STRIDE;
    return MCSD_OK;
}

int check_workspace(const mcsd_desc *d)
{
    const Workspace need = carve(nullptr, static_cast<long long>(d->batch) * d->n_nodes,
                                 static_cast<long long>(d->batch) * (d->n_nodes - d->n_internal), d->batch);
    if (!d->workspace) return MCSD_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d->workspace) % 256 != 0) return MCSD_ERR_WORKSPACE;
    if (d->workspace_bytes < need.bytes) return MCSD_ERR_WORKSPACE;
    return MCSD_OK;
}

int elem_bytes(int dtype) { return dtype == MCSD_DTYPE_F32 ? 4 : 2; }

bool rows_aligned16(const void *base, long long ld, int dtype)
{
    return reinterpret_cast<uintptr_t>(base) % 16 == 0 && (ld * elem_bytes(dtype)) % 16 == 0;
}

// ---- node-kernel variants ---------------------------------------------------
using NodeKernel = void (*)(const NodeParams);
constexpr int kEptChoices[3] = {16, 32, 64};

template <int DT, bool DIRECT, bool PATH>
NodeKernel pick_ept(int ept)
{
    switch (ept) {
    case 16: return node_kernel<DT, 16, DIRECT, PATH>;
    case 32: return node_kernel<DT, 32, DIRECT, PATH>;
    default: return node_kernel<DT, 64, DIRECT, PATH>;
    }
}
template <int DT>
NodeKernel pick_flags(int ept, bool direct, bool path)
{
    if (direct) return path ? pick_ept<DT, true, true>(ept) : pick_ept<DT, true, false>(ept);
    return path ? pick_ept<DT, false, true>(ept) : pick_ept<DT, false, false>(ept);
}
NodeKernel pick_node_kernel(int dtype, int ept, bool direct, bool path)
{
    switch (dtype) {
    case MCSD_DTYPE_F32: return pick_flags<MCSD_DTYPE_F32>(ept, direct, path);
    case MCSD_DTYPE_BF16: return pick_flags<MCSD_DTYPE_BF16>(ept, direct, path);
    default: return pick_flags<MCSD_DTYPE_F16>(ept, direct, path);
    }
}

struct NodeConfig {
    int cluster, ept, slice, threads;
    bool direct;
};

// Smallest (cluster size x elements per thread) that holds one vocabulary row,
// larger per-thread share first so that fewer CTAs have to agree per node.
// The options MCSD_OPT_CLUSTER / MCSD_OPT_EPT / MCSD_OPT_DIRECT override the choice (tuning and tests).
int choose_config(int vocab, int dtype, bool aligned, NodeConfig *cfg)
{
    const int vec = 16 / elem_bytes(dtype);
    int best_c = 0, best_e = 0;
    long long best_cap = -1;
    const int force_c = g_opt.v[MCSD_OPT_CLUSTER], force_e = g_opt.v[MCSD_OPT_EPT];
    for (int c = 1; c <= kMaxCluster; ++c) {
        if (force_c && c != force_c) continue;
        for (int ei = 2; ei >= 0; --ei) {
            const int e = kEptChoices[ei];
            if (force_e && e != force_e) continue;
            const long long cap = static_cast<long long>(c) * kNodeThreads * e;
            if (cap < vocab) continue;
            if (best_cap < 0 || cap < best_cap) { best_cap = cap; best_c = c; best_e = e; }
        }
    }
    if (best_cap < 0) return MCSD_ERR_UNSUPPORTED;
    cfg->cluster = best_c;
    cfg->ept = best_e;
    // every CTA but the last owns a full slice, so that only the last one has ragged warps
    cfg->slice = kNodeThreads * best_e;
    cfg->threads = kNodeThreads;
    (void)vec;
    cfg->direct = !aligned || g_opt.v[MCSD_OPT_DIRECT] != 0;
    return MCSD_OK;
}

// Clusters that can be resident at once, cached per (device, kernel, cluster size).
struct OccKey { int dev; NodeKernel fn; int cluster; int clusters; };
std::mutex g_occ_mutex;
std::vector<OccKey> g_occ;

int resident_clusters(NodeKernel fn, int cluster, size_t smem, cudaStream_t stream, int threads = kNodeThreads)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    {
        std::lock_guard<std::mutex> lock(g_occ_mutex);
        for (const OccKey &k : g_occ)
            if (k.dev == dev && k.fn == fn && k.cluster == cluster) return k.clusters;
    }
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return -1;
    // shared-memory carveout: what the CTAs the register budget admits need (dynamic +
    // static + 1 KB the system reserves per CTA), the rest stays L1
    int n_sm = 0, smem_sm = 0;
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
    cudaFuncAttributes fa = {};
    if (cudaFuncGetAttributes(&fa, fn) == cudaSuccess && smem_sm > 0 && fa.numRegs > 0) {
        int by_regs = 65536 / (fa.numRegs * threads);
        if (by_regs < 1) by_regs = 1;
        const size_t per_cta = smem + fa.sharedSizeBytes + 1024;
        size_t want = per_cta * static_cast<size_t>(by_regs);
        if (want > static_cast<size_t>(smem_sm)) want = static_cast<size_t>(smem_sm);
        int pct = static_cast<int>((want * 100 + smem_sm - 1) / smem_sm);
        if (pct > 100) pct = 100;
        cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, pct);
    }
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(static_cast<unsigned>(cluster * n_sm * 8));
    lc.blockDim = dim3(static_cast<unsigned>(threads));
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, fn, &lc) != cudaSuccess || clusters < 1) {
        cudaGetLastError();
        return -1;
    }
    std::lock_guard<std::mutex> lock(g_occ_mutex);
    g_occ.push_back({dev, fn, cluster, clusters});
    return clusters;
}

struct Call {
    const mcsd_desc *d;
    TreePlan plan;
    Workspace ws;
    int32_t *node_accept, *node_bonus, *status;
    cudaStream_t stream;
};

int prepare(const mcsd_desc *d, const int32_t *parent, Call *c)
{
    int rc = check_desc(d);
    if (rc != MCSD_OK) return rc;
    rc = plan_tree_cached(parent, d->n_nodes, d->n_internal, &c->plan);
    if (rc != MCSD_OK) return rc;
    rc = check_workspace(d);
    if (rc != MCSD_OK) return rc;
    c->d = d;
    c->ws = carve(d->workspace, static_cast<long long>(d->batch) * d->n_nodes,
                  static_cast<long long>(d->batch) * (d->n_nodes - d->n_internal), d->batch);
    c->node_accept = d->node_accept ? d->node_accept : c->ws.node_accept;
    c->node_bonus = d->node_bonus ? d->node_bonus : c->ws.node_bonus;
    c->status = d->out_status ? d->out_status : c->ws.status;
    c->stream = static_cast<cudaStream_t>(d->stream);
    if (g_opt.v[MCSD_OPT_TIME_KERNELS]) reset_timers();
    return MCSD_OK;
}

int check_common(const mcsd_desc *d, const void *target, const void *draft, const int32_t *cand,
                 const float *unif, float T, int mode, bool need_unif, bool naive_ok = false)
{
    if (!target || !cand) return MCSD_ERR_NULL;
    if (!(T >= 0.f) || std::isinf(T)) return MCSD_ERR_TEMPERATURE;
    if (mode != MCSD_MODE_WITH_REPLACEMENT && mode != MCSD_MODE_WITHOUT_REPLACEMENT &&
        !(naive_ok && mode == MCSD_MODE_NAIVE))
        return MCSD_ERR_MODE;
    if (T > 0.f) {
        if (need_unif && !unif) return MCSD_ERR_NULL;
        if (d->n_internal > 0 && mode != MCSD_MODE_NAIVE) {
            if (!draft) return MCSD_ERR_NULL;
            if (d->ld_draft < d->vocab) return MCSD_ERR_STRIDE;
        }
    }
    return MCSD_OK;
}

// level < 0: the all-node form (every node of every tree is an item).  level >= 0: path
// mode, the items are the sequences.  At temperature > 0 ONE launch (level 0) walks every
// sequence from the root to the node where its walk stops; at temperature 0 there is one
// launch per level and each sequence works on the node its walk stands on at that level
// (path arrays in the workspace, swapped level by level).
int launch_nodes(const Call &c, const void *target, const void *draft, const int32_t *cand,
                 const float *unif, float T, int mode, int level = -1)
{
    const mcsd_desc *d = c.d;
    const bool path = level >= 0;
    const long long n_items = path ? d->batch : static_cast<long long>(d->batch) * d->n_nodes;
    if (n_items == 0) return MCSD_OK;
    const int32_t *path_cur = path ? c.ws.path[level & 1] : nullptr;
    int32_t *path_next = path ? c.ws.path[(level + 1) & 1] : nullptr;
    // (the status words need no clearing: the walk stage writes them)
    if (level == 0 && T == 0.f &&
        cudaMemsetAsync(c.ws.path[0], 0, sizeof(int32_t) * d->batch, c.stream) != cudaSuccess)
        return MCSD_ERR_CUDA;  // every walk starts at the root

    {
        const size_t es = static_cast<size_t>(d->dtype == MCSD_DTYPE_F32 ? 4 : 2);
        const size_t n_all = static_cast<size_t>(d->batch) * d->n_nodes;
        if (debug_register(c.stream, {{target, n_all * d->ld_target * es},
                                      {T > 0.f ? draft : nullptr, static_cast<size_t>(d->batch) * d->n_internal * d->ld_draft * es},
                                      {cand, n_all * 4}, {unif, n_all * 8}, {d->workspace, d->workspace_bytes},
                                      {d->node_accept, n_all * 4}, {d->node_bonus, n_all * 4}}) != MCSD_OK)
            return MCSD_ERR_CUDA;
    }
    if (T == 0.f) {
        ArgmaxParams p = {};
        p.target = target; p.cand = cand;
        p.node_accept = c.node_accept; p.node_bonus = c.node_bonus; p.node_ratio = d->node_ratio;
        p.ld_t = d->ld_target;
        p.n_nodes = d->n_nodes; p.n_internal = d->n_internal; p.V = d->vocab;
        p.n_rows = static_cast<int32_t>(n_items);
        p.vector_ok = rows_aligned16(target, d->ld_target, d->dtype) ? 1 : 0;
        p.path_cur = path_cur; p.path_next = path_next;
        std::memcpy(p.child_first, c.plan.child_first, sizeof(p.child_first));
        std::memcpy(p.child_count, c.plan.child_count, sizeof(p.child_count));
        int dev = 0, n_sm = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
        const long long cap = static_cast<long long>(n_sm) * 8;   // 8 resident CTAs of 256 threads per SM
        const unsigned grid = static_cast<unsigned>(n_items < cap ? n_items : cap);
        ScopedTimer timer(0, c.stream);
        switch (d->dtype) {
        case MCSD_DTYPE_F32: argmax_kernel<MCSD_DTYPE_F32><<<grid, kThreads, 0, c.stream>>>(p); break;
        case MCSD_DTYPE_BF16: argmax_kernel<MCSD_DTYPE_BF16><<<grid, kThreads, 0, c.stream>>>(p); break;
        default: argmax_kernel<MCSD_DTYPE_F16><<<grid, kThreads, 0, c.stream>>>(p); break;
        }
        if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
        g_last_launches += 1;
        return MCSD_OK;
    }

    const bool aligned = rows_aligned16(target, d->ld_target, d->dtype) &&
        (d->n_internal == 0 || rows_aligned16(draft, d->ld_draft, d->dtype));
    NodeConfig cfg;
    int rc = choose_config(d->vocab, d->dtype, aligned, &cfg);
    if (rc != MCSD_OK) return rc;
    NodeKernel fn = pick_node_kernel(d->dtype, cfg.ept, cfg.direct, path);
    const size_t smem = node_smem_bytes(elem_bytes(d->dtype), cfg.ept, cfg.direct);
    const int resident = resident_clusters(fn, cfg.cluster, smem, c.stream, cfg.threads);
    if (resident < 1) return MCSD_ERR_CUDA;
    // Large launches of the all-node form: the cluster kernel takes only the nodes with two or more
    // children; the rows of all others are streamed for their statistics by a kernel of its own and
    // the single test of the nodes with one child is made from those (MCSD_OPT_SPLIT: 1 never, 2 always).
    int n_stream = 0, n_keep = 0, n_single = 0;
    uint16_t stream_nodes[MCSD_MAX_NODES], keep_nodes[MCSD_MAX_NODES];
    for (int n = 0; n < d->n_nodes; ++n) {
        const int k = n < d->n_internal ? c.plan.child_count[n] : 0;
        if (k >= 2) keep_nodes[n_keep++] = static_cast<uint16_t>(n);
        else stream_nodes[n_stream++] = static_cast<uint16_t>(n);
        n_single += k == 1;
    }
    // (measured: a tree without such nodes, a chain, always gains; otherwise the split pays with 2-byte
    // logits from about fourteen items per resident cluster on, and with 4-byte logits, where the cluster
    // kernel is close to the memory bandwidth anyway, only on launches that run for hundreds of
    // microseconds back to back)
    const int split_opt = g_opt.v[MCSD_OPT_SPLIT];
    const long long split_from = n_keep == 0 ? 0 : (d->dtype == MCSD_DTYPE_F32 ? 96LL : 14LL) * resident;
    const bool split = !path && n_stream > 0 && split_opt != 1 && (split_opt == 2 || n_items >= split_from);
    const int n_list = split ? n_keep : d->n_nodes;
    const long long n_cluster_items = path ? n_items : static_cast<long long>(d->batch) * n_list;
    const long long n_clusters = n_cluster_items < resident ? n_cluster_items : resident;

    NodeParams p = {};
    p.target = target; p.draft = draft; p.cand = cand; p.unif = unif;
    p.node_accept = c.node_accept; p.node_ratio = d->node_ratio;
    p.stats = c.ws.stats; p.leaf_part = c.ws.leaf_part; p.single_part = c.ws.single_part;
    p.ld_t = d->ld_target; p.ld_d = d->ld_draft;
    p.wait_polls = g_opt.v[MCSD_OPT_WAIT_POLLS] > 0 ? static_cast<uint32_t>(g_opt.v[MCSD_OPT_WAIT_POLLS]) : kWaitPolls;
    p.test_extra_tx = static_cast<uint32_t>(g_opt.v[MCSD_OPT_TEST_EXTRA_TX]) & ~15u;
    p.B = d->batch; p.n_nodes = d->n_nodes; p.n_internal = d->n_internal; p.V = d->vocab;
    p.slice = cfg.slice;
    p.n_items = static_cast<int32_t>(n_cluster_items);
    p.n_list = path ? 1 : n_list;
    p.step_b = static_cast<int32_t>(path ? n_clusters : (n_list ? n_clusters / n_list : 0));
    p.step_n = static_cast<int32_t>(path ? 0 : (n_list ? n_clusters % n_list : 0));
    for (int i = 0; i < d->n_nodes; ++i) p.item_node[i] = static_cast<uint16_t>(split ? (i < n_keep ? keep_nodes[i] : 0) : i);
    p.mode = mode;
    const double scale_d = 1.4426950408889634 / static_cast<double>(T);
    p.scale = static_cast<float>(scale_d);
    p.scale_lo = static_cast<float>(scale_d - static_cast<double>(p.scale));
    std::memcpy(p.child_first, c.plan.child_first, sizeof(p.child_first));
    std::memcpy(p.child_count, c.plan.child_count, sizeof(p.child_count));

    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(static_cast<unsigned>(n_clusters * cfg.cluster));
    lc.blockDim = dim3(static_cast<unsigned>(cfg.threads));
    lc.dynamicSmemBytes = smem;
    lc.stream = c.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cfg.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (g_opt.v[MCSD_OPT_TRACE] & 1) {
        g_note.cluster = cfg.cluster; g_note.ept = cfg.ept; g_note.threads = cfg.threads; g_note.direct = cfg.direct;
        g_note.split = split; g_note.clusters = n_clusters;
    }
    if (n_clusters > 0) {
        ScopedTimer timer(0, c.stream);
        if (cudaLaunchKernelEx(&lc, fn, p) != cudaSuccess) {
            cudaGetLastError();
            return MCSD_ERR_CUDA;
        }
        g_last_launches += 1;
    }
    if (split) {
        StreamParams sp = {};
        sp.target = target; sp.draft = draft;
        sp.leaf_part = c.ws.leaf_part; sp.single_part = c.ws.single_part; sp.node_accept = c.node_accept;
        sp.ld_t = d->ld_target; sp.ld_d = d->ld_draft;
        sp.B = d->batch; sp.n_nodes = d->n_nodes; sp.n_internal = d->n_internal; sp.V = d->vocab;
        sp.n_entries = cfg.cluster * (cfg.threads / 32);   // every entry the walk and decide stages read, empty runs included
        sp.n_list = n_stream;
        sp.vector_ok = cfg.direct ? 0 : 1;
        sp.scale = p.scale;
        for (int i = 0; i < n_stream; ++i) sp.item_node[i] = stream_nodes[i];
        int dev = 0, n_sm = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
        const long long warps = static_cast<long long>(d->batch) * n_stream * sp.n_entries;
        long long ctas = (warps + 3) / 4;
        if (ctas > static_cast<long long>(n_sm) * 64) ctas = static_cast<long long>(n_sm) * 64;
        const unsigned grid = static_cast<unsigned>(ctas);
        g_note.stream_ctas = ctas;
        ScopedTimer timer(1, c.stream);
        switch (d->dtype * 100 + cfg.ept) {
        case MCSD_DTYPE_F32 * 100 + 16: stream_stats_kernel<MCSD_DTYPE_F32, 16><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        case MCSD_DTYPE_F32 * 100 + 32: stream_stats_kernel<MCSD_DTYPE_F32, 32><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        case MCSD_DTYPE_F32 * 100 + 64: stream_stats_kernel<MCSD_DTYPE_F32, 64><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        case MCSD_DTYPE_BF16 * 100 + 16: stream_stats_kernel<MCSD_DTYPE_BF16, 16><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        case MCSD_DTYPE_BF16 * 100 + 32: stream_stats_kernel<MCSD_DTYPE_BF16, 32><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        case MCSD_DTYPE_BF16 * 100 + 64: stream_stats_kernel<MCSD_DTYPE_BF16, 64><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        case MCSD_DTYPE_F16 * 100 + 16: stream_stats_kernel<MCSD_DTYPE_F16, 16><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        case MCSD_DTYPE_F16 * 100 + 32: stream_stats_kernel<MCSD_DTYPE_F16, 32><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        default: stream_stats_kernel<MCSD_DTYPE_F16, 64><<<grid, kNodeThreads, 0, c.stream>>>(sp); break;
        }
        if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
        g_last_launches += 1;
    }
    // ... and the one test of every node with exactly one child is made from those statistics
    if (split && n_single > 0) {
        SingleParams sp = {};
        sp.target = target; sp.draft = draft; sp.cand = cand; sp.unif = unif;
        sp.single_part = c.ws.single_part; sp.node_accept = c.node_accept; sp.node_ratio = d->node_ratio;
        sp.stats = c.ws.stats;
        sp.ld_t = d->ld_target; sp.ld_d = d->ld_draft;
        sp.B = d->batch; sp.n_nodes = d->n_nodes; sp.n_internal = d->n_internal; sp.V = d->vocab;
        sp.n_entries = cfg.cluster * (cfg.threads / 32);
        sp.mode = mode;
        sp.pdl = g_opt.v[MCSD_OPT_PDL] ? 1 : 0;
        sp.scale = p.scale; sp.scale_lo = p.scale_lo;
        std::memcpy(sp.child_first, c.plan.child_first, sizeof(sp.child_first));
        std::memcpy(sp.child_count, c.plan.child_count, sizeof(sp.child_count));
        using SingleKernel = void (*)(const SingleParams);
        SingleKernel sk = d->dtype == MCSD_DTYPE_F32 ? single_decide_kernel<MCSD_DTYPE_F32>
                        : d->dtype == MCSD_DTYPE_BF16 ? single_decide_kernel<MCSD_DTYPE_BF16>
                                                      : single_decide_kernel<MCSD_DTYPE_F16>;
        int dev = 0, n_sm = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
        const long long warps = static_cast<long long>(d->batch) * d->n_internal;
        long long ctas = (warps + 3) / 4;
        if (ctas > static_cast<long long>(n_sm) * 16) ctas = static_cast<long long>(n_sm) * 16;
        cudaLaunchConfig_t sc = {};
        sc.gridDim = dim3(static_cast<unsigned>(ctas));
        sc.blockDim = dim3(kNodeThreads);
        sc.stream = c.stream;
        cudaLaunchAttribute sa[1];
        sa[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        sa[0].val.programmaticStreamSerializationAllowed = 1;
        sc.attrs = sa;
        sc.numAttrs = sp.pdl ? 1 : 0;
        ScopedTimer timer(2, c.stream);
        if (cudaLaunchKernelEx(&sc, sk, sp) != cudaSuccess) {
            cudaGetLastError();
            return MCSD_ERR_CUDA;
        }
        g_last_launches += 1;
    }
    return MCSD_OK;
}

// Naive sampling: one kernel walks every tree level by level (nothing else is launched).
int launch_naive(const Call &c, const void *target, const int32_t *cand, const float *unif, float T,
                 int32_t *out_accept_len, int32_t *out_tokens, float *out_residual)
{
    const mcsd_desc *d = c.d;
    if (d->batch == 0) return MCSD_OK;
    {
        const size_t es = static_cast<size_t>(d->dtype == MCSD_DTYPE_F32 ? 4 : 2);
        const size_t n_all = static_cast<size_t>(d->batch) * d->n_nodes;
        if (debug_register(c.stream, {{target, n_all * d->ld_target * es}, {cand, n_all * 4}, {unif, n_all * 8}}) != MCSD_OK)
            return MCSD_ERR_CUDA;
    }
    NaiveParams p = {};
    p.target = target; p.cand = cand; p.unif = unif;
    p.node_accept = c.node_accept;
    p.out_accept_len = out_accept_len; p.out_tokens = out_tokens; p.out_residual = out_residual;
    p.out_path_nodes = d->out_path_nodes;
    p.status = c.status;
    p.ld_t = d->ld_target;
    p.n_nodes = d->n_nodes; p.n_internal = d->n_internal; p.V = d->vocab; p.gamma = c.plan.gamma;
    p.vector_ok = rows_aligned16(target, d->ld_target, d->dtype) ? 1 : 0;
    p.scale = static_cast<float>(1.4426950408889634 / static_cast<double>(T));
    std::memcpy(p.child_first, c.plan.child_first, sizeof(p.child_first));
    std::memcpy(p.child_count, c.plan.child_count, sizeof(p.child_count));
    const unsigned grid = static_cast<unsigned>(d->batch);
    switch (d->dtype) {
    case MCSD_DTYPE_F32: naive_kernel<MCSD_DTYPE_F32><<<grid, kWalkThreads, 0, c.stream>>>(p); break;
    case MCSD_DTYPE_BF16: naive_kernel<MCSD_DTYPE_BF16><<<grid, kWalkThreads, 0, c.stream>>>(p); break;
    default: naive_kernel<MCSD_DTYPE_F16><<<grid, kWalkThreads, 0, c.stream>>>(p); break;
    }
    if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
    g_last_launches += 1;
    return MCSD_OK;
}

// Batches up to this size take the clustered walk kernel, the smallest ones its form without a register
// budget (measured on 148 SMs: one wave of 8-CTA clusters holds 18 sequences at 2 CTAs per SM; at 64
// sequences the clustered form is no faster with a vocabulary of 32000 and slower with 50272).
constexpr int kWalkClusterFewBatch = 18;
constexpr int kWalkClusterMaxBatch = 37;

int launch_walk(const Call &c, const void *target, const void *draft, const int32_t *cand,
                const float *unif, float T, int32_t *out_accept_len, int32_t *out_tokens, float *out_residual,
                bool all_nodes_allowed = true)
{
    const mcsd_desc *d = c.d;
    if (d->batch == 0) return MCSD_OK;
    {
        const size_t es = static_cast<size_t>(d->dtype == MCSD_DTYPE_F32 ? 4 : 2);
        const size_t n_all = static_cast<size_t>(d->batch) * d->n_nodes;
        if (debug_register(c.stream, {{target, n_all * d->ld_target * es},
                                      {T > 0.f ? draft : nullptr, static_cast<size_t>(d->batch) * d->n_internal * d->ld_draft * es},
                                      {cand, n_all * 4}, {unif, n_all * 8}, {d->workspace, d->workspace_bytes},
                                      {d->node_accept, n_all * 4}, {d->node_bonus, n_all * 4}}) != MCSD_OK)
            return MCSD_ERR_CUDA;
    }
    WalkParams p = {};
    p.target = target; p.draft = draft; p.cand = cand; p.unif = unif;
    p.node_accept = c.node_accept; p.node_bonus = c.node_bonus;
    p.stats = c.ws.stats; p.leaf_part = c.ws.leaf_part; p.status = c.status;
    p.out_accept_len = out_accept_len; p.out_tokens = out_tokens; p.out_residual = out_residual;
    p.out_path_nodes = d->out_path_nodes;
    p.node_residual = d->node_residual;
    p.ld_t = d->ld_target; p.ld_d = d->ld_draft;
    p.n_nodes = d->n_nodes; p.n_internal = d->n_internal; p.V = d->vocab; p.gamma = c.plan.gamma;
    p.scale = T > 0.f ? static_cast<float>(1.4426950408889634 / static_cast<double>(T)) : 0.f;
    const bool aligned = rows_aligned16(target, d->ld_target, d->dtype) &&
        (T == 0.f || d->n_internal == 0 || rows_aligned16(draft, d->ld_draft, d->dtype));
    p.vector_ok = aligned ? 1 : 0;
    if (T > 0.f) {
        // the leaf statistics were left one entry per warp of the node kernel's cluster
        const bool node_aligned = rows_aligned16(target, d->ld_target, d->dtype) &&
            (d->n_internal == 0 || rows_aligned16(draft, d->ld_draft, d->dtype));
        NodeConfig cfg;
        const int rc = choose_config(d->vocab, d->dtype, node_aligned, &cfg);
        if (rc != MCSD_OK) return rc;
        p.n_entries = cfg.cluster * (cfg.threads / 32);
    }
    // The walk stage may be set up on the GPU while the node stage still runs (programmatic
    // dependent launch): its CTAs wait for the node stage's results at their first instruction.
    p.pdl = g_opt.v[MCSD_OPT_PDL] ? 1 : 0;
    using WalkKernel = void (*)(const WalkParams);
    WalkKernel fn;
    int threads;
    // 512 threads (two CTAs per SM) when the vocabulary allows it and there are more CTAs than SMs;
    // a small batch takes 1024 threads per sequence: half the work per thread, shorter chains
    int n_sm = 148;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    }
    const bool want_all_early = all_nodes_allowed && ((T > 0.f && d->node_bonus) || d->node_residual);
    // a small batch: a cluster of eight CTAs of 128 threads per sequence, so that eight SMs share its
    // exponentials (MCSD_OPT_WALK_CLUSTER: 1 never, 2 always)
    const int wc_opt = g_opt.v[MCSD_OPT_WALK_CLUSTER];
    int walk_cluster = 1;
    if (wc_opt == 2 || (wc_opt == 0 && !want_all_early && d->batch <= kWalkClusterMaxBatch)) {
        walk_cluster = 8;
        threads = 128;
        if (d->batch <= kWalkClusterFewBatch)
            fn = d->dtype == MCSD_DTYPE_F32 ? walk_kernel<MCSD_DTYPE_F32, 128, 8, 1>
               : d->dtype == MCSD_DTYPE_BF16 ? walk_kernel<MCSD_DTYPE_BF16, 128, 8, 1> : walk_kernel<MCSD_DTYPE_F16, 128, 8, 1>;
        else
            fn = d->dtype == MCSD_DTYPE_F32 ? walk_kernel<MCSD_DTYPE_F32, 128, 8, 4>
               : d->dtype == MCSD_DTYPE_BF16 ? walk_kernel<MCSD_DTYPE_BF16, 128, 8, 4> : walk_kernel<MCSD_DTYPE_F16, 128, 8, 4>;
    } else if (d->vocab <= MCSD_MAX_VOCAB / 2 && (d->batch > n_sm || want_all_early)) {
        threads = 512;
        fn = d->dtype == MCSD_DTYPE_F32 ? walk_kernel<MCSD_DTYPE_F32, 512>
           : d->dtype == MCSD_DTYPE_BF16 ? walk_kernel<MCSD_DTYPE_BF16, 512> : walk_kernel<MCSD_DTYPE_F16, 512>;
    } else {
        threads = 1024;
        fn = d->dtype == MCSD_DTYPE_F32 ? walk_kernel<MCSD_DTYPE_F32, 1024>
           : d->dtype == MCSD_DTYPE_BF16 ? walk_kernel<MCSD_DTYPE_BF16, 1024> : walk_kernel<MCSD_DTYPE_F16, 1024>;
    }
    // all-nodes pass first (only when per-node endpoint tokens or distributions were asked for;
    // at temperature 0 the tokens are there already), then the walks
    const bool want_all = all_nodes_allowed && ((T > 0.f && d->node_bonus) || d->node_residual);
    for (int all = want_all ? 1 : 0; all >= 0; --all) {
        p.all_nodes = all;
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(static_cast<unsigned>((all ? static_cast<long long>(d->batch) * d->n_nodes : d->batch) * walk_cluster));
        lc.blockDim = dim3(static_cast<unsigned>(threads));
        lc.stream = c.stream;
        cudaLaunchAttribute attr[2];
        int n_attr = 0;
        if (p.pdl) {
            attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
            ++n_attr;
        }
        if (walk_cluster > 1) {
            attr[n_attr].id = cudaLaunchAttributeClusterDimension;
            attr[n_attr].val.clusterDim.x = static_cast<unsigned>(walk_cluster);
            attr[n_attr].val.clusterDim.y = 1;
            attr[n_attr].val.clusterDim.z = 1;
            ++n_attr;
        }
        lc.attrs = attr;
        lc.numAttrs = static_cast<unsigned>(n_attr);
        ScopedTimer timer(3, c.stream);
        cudaError_t err = cudaLaunchKernelEx(&lc, fn, p);
        if (err != cudaSuccess && walk_cluster > 1) {
            // a device (or partition of one) that cannot place clusters of eight: the one-CTA form does the same
            cudaGetLastError();
            WalkKernel one = d->dtype == MCSD_DTYPE_F32 ? walk_kernel<MCSD_DTYPE_F32, 1024>
                           : d->dtype == MCSD_DTYPE_BF16 ? walk_kernel<MCSD_DTYPE_BF16, 1024> : walk_kernel<MCSD_DTYPE_F16, 1024>;
            lc.gridDim = dim3(static_cast<unsigned>(all ? static_cast<long long>(d->batch) * d->n_nodes : d->batch));
            lc.blockDim = dim3(1024);
            lc.numAttrs = p.pdl ? 1 : 0;   // (the attribute of the dependent launch comes first)
            err = cudaLaunchKernelEx(&lc, one, p);
        }
        if (err != cudaSuccess) {
            cudaGetLastError();
            return MCSD_ERR_CUDA;
        }
        g_last_launches += 1;
    }
    return MCSD_OK;
}

}  // namespace
}  // namespace mcsd

using namespace mcsd;

extern "C" {

int mcsd_version(void) { return MCSD_VERSION; }

const char *mcsd_status_string(int code)
{
    switch (code) {
    case MCSD_OK: return "ok";
    case MCSD_ERR_NULL: return "a required pointer is NULL";
    case MCSD_ERR_SHAPE: return "batch, n_nodes, n_internal or vocab out of range";
    case MCSD_ERR_DTYPE: return "unknown logit dtype";
    case MCSD_ERR_MODE: return "unknown replacement mode";
    case MCSD_ERR_TEMPERATURE: return "temperature is negative, NaN or infinite";
    case MCSD_ERR_TREE: return "tree_parent breaks the layout contract";
    case MCSD_ERR_STRIDE: return "row stride smaller than vocab";
    case MCSD_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MCSD_ERR_CUDA: return "a CUDA runtime call or kernel launch failed";
    case MCSD_ERR_UNSUPPORTED: return "size beyond the library limits";
    case MCSD_ERR_STATIC_LIMIT: return "scratch need exceeds the built-in array of mcsd_verify_static; use mcsd_verify";
    default: return "unknown code";
    }
}

size_t mcsd_workspace_bytes(const mcsd_desc *desc)
{
    if (check_desc(desc) != MCSD_OK) return 0;
    return carve(nullptr, static_cast<long long>(desc->batch) * desc->n_nodes,
                 static_cast<long long>(desc->batch) * (desc->n_nodes - desc->n_internal), desc->batch).bytes;
}

int mcsd_tree_depth(const int32_t *tree_parent, int32_t n_nodes)
{
    TreePlan plan;
    const int rc = plan_tree(tree_parent, n_nodes, -1, &plan);
    return rc == MCSD_OK ? plan.gamma : rc;
}

int mcsd_last_launch_count(void) { return g_last_launches; }

long long mcsd_debug_bounds_hits(int reset)
{
#ifdef MCSD_DEBUG_BOUNDS
    unsigned long long hits = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return MCSD_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&hits, g_dbg_hits, sizeof(hits)) != cudaSuccess) return MCSD_ERR_CUDA;
    if (reset) {
        const unsigned long long zero = 0;
        if (cudaMemcpyToSymbol(g_dbg_hits, &zero, sizeof(zero)) != cudaSuccess) return MCSD_ERR_CUDA;
    }
    return static_cast<long long>(hits);
#else
    (void)reset;
    return -1;
#endif
}

int mcsd_last_kernel_times(float *ms, int32_t n)
{
    if (!ms || n < 0) return MCSD_ERR_NULL;
    int filled = 0;
    for (int s = 0; s < kTimeSlots && s < n; ++s) {
        ms[s] = -1.f;
        if (g_timers.created && g_timers.used[s]) {
            if (cudaEventSynchronize(g_timers.ev[s][1]) != cudaSuccess ||
                cudaEventElapsedTime(&ms[s], g_timers.ev[s][0], g_timers.ev[s][1]) != cudaSuccess) {
                cudaGetLastError();
                return MCSD_ERR_CUDA;
            }
            ++filled;
        }
    }
    return filled;
}

int mcsd_set_option(int option, int value)
{
    if (option < 0 || option >= MCSD_OPT_COUNT) return MCSD_ERR_SHAPE;
    if (value < 0) return MCSD_ERR_SHAPE;
    g_opt.v[option] = value;
    return MCSD_OK;
}

int mcsd_get_option(int option)
{
    if (option < 0 || option >= MCSD_OPT_COUNT) return MCSD_ERR_SHAPE;
    return g_opt.v[option];
}

static int mcsd_verify_nodes_impl(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                      const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                      float temperature, int replacement_mode)
{
    Call c;
    int rc = prepare(desc, tree_parent, &c);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0) return MCSD_OK;
    rc = check_common(desc, target_logits, draft_logits, cand_tokens, uniforms, temperature,
                      replacement_mode, true);
    if (rc != MCSD_OK) return rc;
    return launch_nodes(c, target_logits, draft_logits, cand_tokens, uniforms, temperature, replacement_mode);
}

int mcsd_verify_nodes(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                      const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                      float temperature, int replacement_mode)
{
    Trace trace("mcsd_verify_nodes", desc, temperature, replacement_mode);
    return trace.done(mcsd_verify_nodes_impl(desc, target_logits, draft_logits, tree_parent, cand_tokens, uniforms, temperature, replacement_mode));
}

static int mcsd_verify_walk_impl(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int32_t *out_accept_len, int32_t *out_tokens, float *out_residual)
{
    Call c;
    int rc = prepare(desc, tree_parent, &c);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0) return MCSD_OK;
    rc = check_common(desc, target_logits, draft_logits, cand_tokens, uniforms, temperature,
                      MCSD_MODE_WITH_REPLACEMENT, true);
    if (rc != MCSD_OK) return rc;
    if (!out_accept_len || !out_tokens) return MCSD_ERR_NULL;
    return launch_walk(c, target_logits, draft_logits, cand_tokens, uniforms, temperature, out_accept_len,
                       out_tokens, out_residual);
}

int mcsd_verify_walk(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int32_t *out_accept_len, int32_t *out_tokens, float *out_residual)
{
    Trace trace("mcsd_verify_walk", desc, temperature, 0);
    return trace.done(mcsd_verify_walk_impl(desc, target_logits, draft_logits, tree_parent, cand_tokens, uniforms, temperature, out_accept_len, out_tokens, out_residual));
}

static int mcsd_verify_impl(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                float temperature, int replacement_mode, int32_t *out_accept_len,
                int32_t *out_tokens, float *out_residual)
{
    Call c;
    int rc = prepare(desc, tree_parent, &c);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0) return MCSD_OK;
    rc = check_common(desc, target_logits, draft_logits, cand_tokens, uniforms, temperature,
                      replacement_mode, true, true);
    if (rc != MCSD_OK) return rc;
    if (!out_accept_len || !out_tokens) return MCSD_ERR_NULL;
    if (replacement_mode == MCSD_MODE_NAIVE) {
        // at temperature 0 the draw is the target argmax: the ordinary argmax rule
        if (temperature > 0.f)
            return launch_naive(c, target_logits, cand_tokens, uniforms, temperature, out_accept_len, out_tokens,
                                out_residual);
        replacement_mode = MCSD_MODE_WITH_REPLACEMENT;
    }
    rc = launch_nodes(c, target_logits, draft_logits, cand_tokens, uniforms, temperature, replacement_mode);
    if (rc != MCSD_OK) return rc;
    return launch_walk(c, target_logits, draft_logits, cand_tokens, uniforms, temperature, out_accept_len,
                       out_tokens, out_residual);
}

int mcsd_verify(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                float temperature, int replacement_mode, int32_t *out_accept_len,
                int32_t *out_tokens, float *out_residual)
{
    Trace trace("mcsd_verify", desc, temperature, replacement_mode);
    return trace.done(mcsd_verify_impl(desc, target_logits, draft_logits, tree_parent, cand_tokens, uniforms, temperature, replacement_mode, out_accept_len, out_tokens, out_residual));
}

static int mcsd_verify_path_impl(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int replacement_mode, int32_t *out_accept_len,
                     int32_t *out_tokens, float *out_residual)
{
    Call c;
    int rc = prepare(desc, tree_parent, &c);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0) return MCSD_OK;
    rc = check_common(desc, target_logits, draft_logits, cand_tokens, uniforms, temperature,
                      replacement_mode, true, true);
    if (rc != MCSD_OK) return rc;
    if (!out_accept_len || !out_tokens) return MCSD_ERR_NULL;
    if (replacement_mode == MCSD_MODE_NAIVE) {
        // at temperature 0 the draw is the target argmax: the ordinary argmax rule
        if (temperature > 0.f)
            return launch_naive(c, target_logits, cand_tokens, uniforms, temperature, out_accept_len, out_tokens,
                                out_residual);
        replacement_mode = MCSD_MODE_WITH_REPLACEMENT;
    }
    // temperature > 0: one launch, every cluster walks its sequences from the root.  Temperature
    // 0: one launch per level of the tree; level l evaluates, for every sequence, the node its
    // walk stands on after l accepted tokens (nothing for walks that have ended)
    const int n_levels = temperature > 0.f ? 1 : c.plan.gamma + 1;
    for (int level = 0; level < n_levels; ++level) {
        rc = launch_nodes(c, target_logits, draft_logits, cand_tokens, uniforms, temperature, replacement_mode, level);
        if (rc != MCSD_OK) return rc;
    }
    return launch_walk(c, target_logits, draft_logits, cand_tokens, uniforms, temperature, out_accept_len,
                       out_tokens, out_residual, false);
}

int mcsd_verify_path(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int replacement_mode, int32_t *out_accept_len,
                     int32_t *out_tokens, float *out_residual)
{
    Trace trace("mcsd_verify_path", desc, temperature, replacement_mode);
    return trace.done(mcsd_verify_path_impl(desc, target_logits, draft_logits, tree_parent, cand_tokens, uniforms, temperature, replacement_mode, out_accept_len, out_tokens, out_residual));
}

static int mcsd_sample_candidates_impl(const mcsd_desc *desc, const void *draft_logits, const int32_t *tree_parent,
                           const float *uniforms_draw, float temperature, int replacement_mode,
                           int32_t node_begin, int32_t node_end, int32_t *cand_tokens)
{
    int rc = check_desc(desc);
    if (rc != MCSD_OK) return rc;
    TreePlan plan;
    rc = plan_tree(tree_parent, desc->n_nodes, desc->n_internal, &plan);
    if (rc != MCSD_OK) return rc;
    if (!(temperature >= 0.f) || std::isinf(temperature)) return MCSD_ERR_TEMPERATURE;
    if (replacement_mode != MCSD_MODE_WITH_REPLACEMENT && replacement_mode != MCSD_MODE_WITHOUT_REPLACEMENT)
        return MCSD_ERR_MODE;
    if (node_begin < 0 || node_end > desc->n_internal || node_begin > node_end) return MCSD_ERR_SHAPE;
    g_last_launches = 0;
    const long long n_ctas = static_cast<long long>(desc->batch) * (node_end - node_begin);
    if (n_ctas == 0) return MCSD_OK;
    if (!draft_logits || !cand_tokens || (temperature > 0.f && !uniforms_draw)) return MCSD_ERR_NULL;
    if (desc->ld_draft < desc->vocab) return MCSD_ERR_STRIDE;
    if (n_ctas > 0x7fffffffLL) return MCSD_ERR_UNSUPPORTED;
    {
        const size_t es = static_cast<size_t>(desc->dtype == MCSD_DTYPE_F32 ? 4 : 2);
        if (debug_register(static_cast<cudaStream_t>(desc->stream),
                           {{draft_logits, static_cast<size_t>(desc->batch) * desc->n_internal * desc->ld_draft * es},
                            {uniforms_draw, static_cast<size_t>(desc->batch) * desc->n_nodes * 4}}) != MCSD_OK)
            return MCSD_ERR_CUDA;
    }
    SampleParams p = {};
    p.draft = draft_logits; p.unif_draw = uniforms_draw; p.cand = cand_tokens; p.status = desc->out_status;
    p.ld_d = desc->ld_draft;
    p.n_nodes = desc->n_nodes; p.n_internal = desc->n_internal; p.V = desc->vocab;
    p.node_begin = node_begin; p.n_range = node_end - node_begin;
    p.mode = replacement_mode;
    p.vector_ok = rows_aligned16(draft_logits, desc->ld_draft, desc->dtype) ? 1 : 0;
    p.scale = temperature > 0.f ? static_cast<float>(1.4426950408889634 / static_cast<double>(temperature)) : 0.f;
    std::memcpy(p.child_first, plan.child_first, sizeof(p.child_first));
    std::memcpy(p.child_count, plan.child_count, sizeof(p.child_count));
    cudaStream_t stream = static_cast<cudaStream_t>(desc->stream);
    const unsigned grid = static_cast<unsigned>(n_ctas);
    // A vocabulary of at most half the maximum fits the per-warp step budget of smaller CTAs, of
    // which several are resident per SM: 512 threads (two) with 4-byte logits, 256 (four) with 2-byte
    const bool small = desc->vocab <= MCSD_MAX_VOCAB / 2;
    const int threads = !small ? 1024 : (desc->dtype == MCSD_DTYPE_F32 ? 512 : 256);
    {
        // CTAs resident at once: how far ahead in the grid the kernel asks rows into L2
        int dev = 0, n_sm = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MCSD_ERR_CUDA;
        p.prefetch_ahead = n_sm * (1024 / threads);
        // (MCSD_OPT_SAMPLE_AHEAD: percent of that distance, for tuning)
        p.prefetch_ahead = static_cast<int>(static_cast<long long>(p.prefetch_ahead) * g_opt.v[MCSD_OPT_SAMPLE_AHEAD] / 100);
    }
    if (!small) {
        switch (desc->dtype) {
        case MCSD_DTYPE_F32: sample_kernel<MCSD_DTYPE_F32, 1024><<<grid, 1024, 0, stream>>>(p); break;
        case MCSD_DTYPE_BF16: sample_kernel<MCSD_DTYPE_BF16, 1024><<<grid, 1024, 0, stream>>>(p); break;
        default: sample_kernel<MCSD_DTYPE_F16, 1024><<<grid, 1024, 0, stream>>>(p); break;
        }
    } else {
        switch (desc->dtype) {
        case MCSD_DTYPE_F32: sample_kernel<MCSD_DTYPE_F32, 512><<<grid, 512, 0, stream>>>(p); break;
        case MCSD_DTYPE_BF16: sample_kernel<MCSD_DTYPE_BF16, 256><<<grid, 256, 0, stream>>>(p); break;
        default: sample_kernel<MCSD_DTYPE_F16, 256><<<grid, 256, 0, stream>>>(p); break;
        }
    }
    if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
    g_last_launches = 1;
    return MCSD_OK;
}

int mcsd_sample_candidates(const mcsd_desc *desc, const void *draft_logits, const int32_t *tree_parent,
                           const float *uniforms_draw, float temperature, int replacement_mode,
                           int32_t node_begin, int32_t node_end, int32_t *cand_tokens)
{
    Trace trace("mcsd_sample_candidates", desc, temperature, replacement_mode);
    return trace.done(mcsd_sample_candidates_impl(desc, draft_logits, tree_parent, uniforms_draw, temperature, replacement_mode, node_begin, node_end, cand_tokens));
}

int mcsd_tree_attention_layout(const int32_t *tree_parent, int32_t n_nodes, int32_t prefix_len,
                               uint8_t *mask, int32_t *position_ids, void *stream)
{
    TreePlan plan;
    const int rc = plan_tree(tree_parent, n_nodes, -1, &plan);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (!mask && !position_ids) return MCSD_OK;
    if (debug_register(static_cast<cudaStream_t>(stream), {}) != MCSD_OK) return MCSD_ERR_CUDA;
    LayoutParams p = {};
    p.mask = mask; p.position_ids = position_ids; p.n_nodes = n_nodes; p.prefix_len = prefix_len;
    for (int n = 0; n < n_nodes; ++n) p.parent[n] = static_cast<int16_t>(tree_parent[n]);
    layout_kernel<<<static_cast<unsigned>(n_nodes), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
    g_last_launches = 1;
    return MCSD_OK;
}

int mcsd_gather_accepted_kv(void *cache, int64_t n_slabs, int64_t slab_stride, int32_t batch,
                            int64_t seq_stride, int64_t pos_stride, int64_t row_bytes,
                            int64_t n_positions, const int32_t *prefix_len, const int32_t *path_nodes,
                            const int32_t *accept_len, int32_t gamma, void *stream)
{
    if (n_slabs < 0 || batch < 0 || row_bytes < 0 || gamma < 0 || slab_stride < 0 || seq_stride < 0 || n_positions < 0)
        return MCSD_ERR_SHAPE;
    if (pos_stride < row_bytes) return MCSD_ERR_STRIDE;
    g_last_launches = 0;
    const long long n_items = static_cast<long long>(n_slabs) * batch;
    if (n_items == 0 || row_bytes == 0 || gamma == 0) return MCSD_OK;
    if (!cache || !prefix_len || !path_nodes || !accept_len) return MCSD_ERR_NULL;
    // widest unit that divides the base address, the strides and the row length
    const unsigned long long all = reinterpret_cast<uintptr_t>(cache) | static_cast<unsigned long long>(slab_stride) |
        static_cast<unsigned long long>(seq_stride) | static_cast<unsigned long long>(pos_stride) |
        static_cast<unsigned long long>(row_bytes);
    int unit = 16;
    while (unit > 1 && (all & static_cast<unsigned long long>(unit - 1))) unit >>= 1;
    if (row_bytes / unit > 0x7fffffffLL) return MCSD_ERR_UNSUPPORTED;
    if (debug_register(static_cast<cudaStream_t>(stream), {}) != MCSD_OK) return MCSD_ERR_CUDA;
    GatherParams p = {};
    p.cache = static_cast<unsigned char *>(cache);
    p.slab_stride = slab_stride; p.seq_stride = seq_stride; p.pos_stride = pos_stride;
    p.n_items = n_items; p.n_positions = n_positions; p.batch = batch; p.gamma = gamma;
    p.row_units = static_cast<int32_t>(row_bytes / unit);
    p.prefix_len = prefix_len; p.path_nodes = path_nodes; p.accept_len = accept_len;
    int dev = 0, n_sm = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    const long long cap = static_cast<long long>(n_sm) * 8;
    const unsigned grid = static_cast<unsigned>(n_items < cap ? n_items : cap);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (unit) {
    case 16: gather_kernel<uint4><<<grid, kThreads, 0, st>>>(p); break;
    case 8: gather_kernel<uint2><<<grid, kThreads, 0, st>>>(p); break;
    case 4: gather_kernel<uint32_t><<<grid, kThreads, 0, st>>>(p); break;
    case 2: gather_kernel<uint16_t><<<grid, kThreads, 0, st>>>(p); break;
    default: gather_kernel<uint8_t><<<grid, kThreads, 0, st>>>(p); break;
    }
    if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
    g_last_launches = 1;
    return MCSD_OK;
}

// ---- verification with the vocabulary split over several devices ------------------------
namespace {

struct ShardLayout {
    int ept, run, n_entries, eps_max, entry_begin, eps, col_begin, n_cols;
};

// Runs are those of the node kernel for this vocabulary and dtype (32 * elements per thread);
// shard s owns the entries [s * eps_max, (s + 1) * eps_max) that exist.
int shard_layout(int vocab, int dtype, int n_shards, int shard, ShardLayout *L)
{
    if (n_shards < 1 || n_shards > 32 || shard < 0 || shard >= n_shards) return MCSD_ERR_SHAPE;
    NodeConfig cfg;
    const int rc = choose_config(vocab, dtype, true, &cfg);
    if (rc != MCSD_OK) return rc;
    L->ept = cfg.ept;
    L->run = 32 * cfg.ept;
    L->n_entries = (vocab + L->run - 1) / L->run;
    L->eps_max = (L->n_entries + n_shards - 1) / n_shards;
    L->entry_begin = shard * L->eps_max;
    int e_end = L->entry_begin + L->eps_max;
    if (e_end > L->n_entries) e_end = L->n_entries;
    L->eps = e_end > L->entry_begin ? e_end - L->entry_begin : 0;
    L->col_begin = L->entry_begin * L->run < vocab ? L->entry_begin * L->run : vocab;
    int col_end = e_end * L->run;
    if (col_end > vocab) col_end = vocab;
    L->n_cols = col_end > L->col_begin ? col_end - L->col_begin : 0;
    return MCSD_OK;
}

struct ShardWorkspace {
    float4 *act;
    float2 *req;
    float *s_hist;
    int32_t *node_accept;
    NodeStats *stats;
    int32_t *retry;
    size_t bytes;
};

ShardWorkspace carve_shard(void *base, long long n_items, int batch)
{
    ShardWorkspace w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        unsigned char *p = base ? static_cast<unsigned char *>(base) + off : nullptr;
        off += align_up(bytes, 256);
        return p;
    };
    w.act = reinterpret_cast<float4 *>(take(sizeof(float4) * n_items));
    w.req = reinterpret_cast<float2 *>(take(sizeof(float2) * n_items));
    w.s_hist = reinterpret_cast<float *>(take(sizeof(float) * MCSD_MAX_CHILDREN * n_items));
    w.node_accept = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * n_items));
    w.stats = reinterpret_cast<NodeStats *>(take(sizeof(NodeStats) * n_items));
    w.retry = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * (batch > 0 ? batch : 1)));
    w.bytes = off;
    return w;
}

int check_shard_desc(const mcsd_shard_desc *d, ShardLayout *L)
{
    if (!d) return MCSD_ERR_NULL;
    if (d->reserved != 0) return MCSD_ERR_SHAPE;
    if (d->batch < 0 || d->n_nodes < 1 || d->vocab < 1 || d->n_internal < 0 || d->n_internal > d->n_nodes)
        return MCSD_ERR_SHAPE;
    if (d->n_nodes > MCSD_MAX_NODES || d->vocab > MCSD_MAX_VOCAB) return MCSD_ERR_UNSUPPORTED;
    if (static_cast<long long>(d->batch) * d->n_nodes > 0x7fffffffLL) return MCSD_ERR_UNSUPPORTED;
    if (d->dtype != MCSD_DTYPE_F32 && d->dtype != MCSD_DTYPE_BF16 && d->dtype != MCSD_DTYPE_F16) return MCSD_ERR_DTYPE;
    const int rc = shard_layout(d->vocab, d->dtype, d->n_shards, d->shard, L);
    if (rc != MCSD_OK) return rc;
    if (d->ld_target < L->n_cols || (d->n_internal > 0 && d->ld_draft < L->n_cols)) return MCSD_ERR_STRIDE;
    return MCSD_OK;
}

int fill_shard_params(const mcsd_shard_desc *d, const int32_t *parent, float T, int mode, ShardParams *p, TreePlan *plan,
                      ShardLayout *L)
{
    int rc = check_shard_desc(d, L);
    if (rc != MCSD_OK) return rc;
    rc = plan_tree_cached(parent, d->n_nodes, d->n_internal, plan);
    if (rc != MCSD_OK) return rc;
    if (!(T > 0.f) || std::isinf(T)) return T == 0.f ? MCSD_ERR_UNSUPPORTED : MCSD_ERR_TEMPERATURE;
    if (mode != MCSD_MODE_WITH_REPLACEMENT && mode != MCSD_MODE_WITHOUT_REPLACEMENT) return MCSD_ERR_MODE;
    const long long n_items = static_cast<long long>(d->batch) * d->n_nodes;
    const ShardWorkspace need = carve_shard(nullptr, n_items, d->batch);
    if (!d->workspace || reinterpret_cast<uintptr_t>(d->workspace) % 256 != 0 || d->workspace_bytes < need.bytes)
        return MCSD_ERR_WORKSPACE;
    const ShardWorkspace ws = carve_shard(d->workspace, n_items, d->batch);
    if (debug_register(static_cast<cudaStream_t>(d->stream), {}) != MCSD_OK) return MCSD_ERR_CUDA;
    *p = ShardParams();
    p->ld_t = d->ld_target; p->ld_d = d->ld_draft;
    p->B = d->batch; p->n_nodes = d->n_nodes; p->n_internal = d->n_internal; p->V = d->vocab;
    p->col_begin = L->col_begin; p->n_cols = L->n_cols; p->eps = L->eps; p->entry_begin = L->entry_begin;
    p->n_entries = L->n_entries; p->eps_max = L->eps_max; p->n_shards = d->n_shards; p->mode = mode;
    p->gamma = plan->gamma;
    const double scale_d = 1.4426950408889634 / static_cast<double>(T);
    p->scale = static_cast<float>(scale_d);
    p->scale_lo = static_cast<float>(scale_d - static_cast<double>(p->scale));
    p->act = ws.act; p->req = ws.req; p->s_hist = ws.s_hist; p->stats = ws.stats;
    p->node_accept = d->node_accept ? d->node_accept : ws.node_accept;
    p->retry = ws.retry;
    p->node_ratio = d->node_ratio;
    std::memcpy(p->child_first, plan->child_first, sizeof(p->child_first));
    std::memcpy(p->child_count, plan->child_count, sizeof(p->child_count));
    for (int n = 0; n < d->n_nodes; ++n) p->parent[n] = static_cast<int16_t>(parent[n]);
    return MCSD_OK;
}

unsigned shard_grid(long long warps)
{
    int dev = 0, n_sm = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    long long ctas = (warps + 3) / 4;
    const long long cap = static_cast<long long>(n_sm) * 16;
    if (ctas > cap) ctas = cap;
    return static_cast<unsigned>(ctas < 1 ? 1 : ctas);
}

#define MCSD_SHARD_LAUNCH(kernel, dtype, ept, grid, stream, params)                                             \
    do {                                                                                                        \
        switch ((dtype) * 100 + (ept)) {                                                                        \
        case MCSD_DTYPE_F32 * 100 + 16: kernel<MCSD_DTYPE_F32, 16><<<grid, kShardThreads, 0, stream>>>(params); break;   \
        case MCSD_DTYPE_F32 * 100 + 32: kernel<MCSD_DTYPE_F32, 32><<<grid, kShardThreads, 0, stream>>>(params); break;   \
        case MCSD_DTYPE_F32 * 100 + 64: kernel<MCSD_DTYPE_F32, 64><<<grid, kShardThreads, 0, stream>>>(params); break;   \
        case MCSD_DTYPE_BF16 * 100 + 16: kernel<MCSD_DTYPE_BF16, 16><<<grid, kShardThreads, 0, stream>>>(params); break; \
        case MCSD_DTYPE_BF16 * 100 + 32: kernel<MCSD_DTYPE_BF16, 32><<<grid, kShardThreads, 0, stream>>>(params); break; \
        case MCSD_DTYPE_BF16 * 100 + 64: kernel<MCSD_DTYPE_BF16, 64><<<grid, kShardThreads, 0, stream>>>(params); break; \
        case MCSD_DTYPE_F16 * 100 + 16: kernel<MCSD_DTYPE_F16, 16><<<grid, kShardThreads, 0, stream>>>(params); break;   \
        case MCSD_DTYPE_F16 * 100 + 32: kernel<MCSD_DTYPE_F16, 32><<<grid, kShardThreads, 0, stream>>>(params); break;   \
        default: kernel<MCSD_DTYPE_F16, 64><<<grid, kShardThreads, 0, stream>>>(params); break;                          \
        }                                                                                                       \
    } while (0)

}  // namespace

int mcsd_shard_columns(int32_t vocab, int32_t dtype, int32_t n_shards, int32_t shard, int32_t *col_begin,
                       int32_t *n_cols, int32_t *entries_per_shard)
{
    if (vocab < 1 || vocab > MCSD_MAX_VOCAB) return MCSD_ERR_SHAPE;
    if (dtype != MCSD_DTYPE_F32 && dtype != MCSD_DTYPE_BF16 && dtype != MCSD_DTYPE_F16) return MCSD_ERR_DTYPE;
    ShardLayout L;
    const int rc = shard_layout(vocab, dtype, n_shards, shard, &L);
    if (rc != MCSD_OK) return rc;
    if (col_begin) *col_begin = L.col_begin;
    if (n_cols) *n_cols = L.n_cols;
    if (entries_per_shard) *entries_per_shard = L.eps_max;
    return MCSD_OK;
}

size_t mcsd_shard_workspace_bytes(const mcsd_shard_desc *desc)
{
    ShardLayout L;
    if (check_shard_desc(desc, &L) != MCSD_OK) return 0;
    return carve_shard(nullptr, static_cast<long long>(desc->batch) * desc->n_nodes, desc->batch).bytes;
}

int mcsd_shard_rounds(const int32_t *tree_parent, int32_t n_nodes)
{
    TreePlan plan;
    const int rc = plan_tree(tree_parent, n_nodes, -1, &plan);
    if (rc != MCSD_OK) return rc;
    int k_max = 0;
    for (int n = 0; n < n_nodes; ++n) k_max = plan.child_count[n] > k_max ? plan.child_count[n] : k_max;
    return k_max > 1 ? k_max - 1 : 0;
}

int mcsd_shard_partials(const mcsd_shard_desc *desc, const void *target_slice, const void *draft_slice,
                        const int32_t *tree_parent, const int32_t *cand_tokens, float temperature, int32_t round,
                        void *part_out, void *cand_logits_out)
{
    ShardParams p;
    TreePlan plan;
    ShardLayout L;
    int rc = fill_shard_params(desc, tree_parent, temperature, MCSD_MODE_WITH_REPLACEMENT, &p, &plan, &L);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0) return MCSD_OK;
    if (!part_out || !cand_tokens || (round == 0 && !cand_logits_out)) return MCSD_ERR_NULL;
    if (L.n_cols > 0 && (!target_slice || (desc->n_internal > 0 && !draft_slice))) return MCSD_ERR_NULL;
    if (round < 0 || round >= MCSD_MAX_CHILDREN) return MCSD_ERR_SHAPE;
    p.target = target_slice; p.draft = draft_slice; p.cand = cand_tokens; p.round = round;
    p.part_out = static_cast<float4 *>(part_out);
    p.cval_out = static_cast<float2 *>(cand_logits_out);
    p.vector_ok = (rows_aligned16(target_slice, desc->ld_target, desc->dtype) &&
                   (desc->n_internal == 0 || rows_aligned16(draft_slice, desc->ld_draft, desc->dtype))) ? 1 : 0;
    cudaStream_t st = static_cast<cudaStream_t>(desc->stream);
    const long long n_items = static_cast<long long>(desc->batch) * desc->n_nodes;
    if (L.eps > 0) {
        const unsigned grid = shard_grid(n_items * L.eps);
        MCSD_SHARD_LAUNCH(shard_partials_kernel, desc->dtype, L.ept, grid, st, p);
        if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
        g_last_launches += 1;
    }
    if (round == 0) {
        const unsigned grid = static_cast<unsigned>((n_items + 255) / 256 < 2048 ? (n_items + 255) / 256 : 2048);
        switch (desc->dtype) {
        case MCSD_DTYPE_F32: shard_candidates_kernel<MCSD_DTYPE_F32><<<grid, 256, 0, st>>>(p); break;
        case MCSD_DTYPE_BF16: shard_candidates_kernel<MCSD_DTYPE_BF16><<<grid, 256, 0, st>>>(p); break;
        default: shard_candidates_kernel<MCSD_DTYPE_F16><<<grid, 256, 0, st>>>(p); break;
        }
        if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
        g_last_launches += 1;
    }
    return MCSD_OK;
}

int mcsd_shard_decide(const mcsd_shard_desc *desc, const int32_t *tree_parent, const int32_t *cand_tokens,
                      const float *uniforms, float temperature, int replacement_mode, int32_t round,
                      const void *part_all, const void *cand_logits_all)
{
    ShardParams p;
    TreePlan plan;
    ShardLayout L;
    int rc = fill_shard_params(desc, tree_parent, temperature, replacement_mode, &p, &plan, &L);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0 || desc->n_internal == 0) return MCSD_OK;
    if (!part_all || !cand_logits_all || !cand_tokens || !uniforms) return MCSD_ERR_NULL;
    if (round < 0 || round >= MCSD_MAX_CHILDREN) return MCSD_ERR_SHAPE;
    p.cand = cand_tokens; p.unif = uniforms; p.round = round;
    p.part_all = static_cast<const float4 *>(part_all);
    p.cval_all = static_cast<const float2 *>(cand_logits_all);
    const unsigned grid = shard_grid(static_cast<long long>(desc->batch) * desc->n_internal);
    shard_decide_kernel<<<grid, kShardThreads, 0, static_cast<cudaStream_t>(desc->stream)>>>(p);
    if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
    g_last_launches = 1;
    return MCSD_OK;
}

int mcsd_shard_endpoint(const mcsd_shard_desc *desc, const void *target_slice, const void *draft_slice,
                        const int32_t *tree_parent, float temperature, int32_t attempt, const void *stats_all,
                        void *totals_out, float *out_residual_slice)
{
    ShardParams p;
    TreePlan plan;
    ShardLayout L;
    int rc = fill_shard_params(desc, tree_parent, temperature, MCSD_MODE_WITH_REPLACEMENT, &p, &plan, &L);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0 || L.eps == 0) return MCSD_OK;
    if (!target_slice || (desc->n_internal > 0 && !draft_slice) || !stats_all || !totals_out) return MCSD_ERR_NULL;
    if (attempt != 0 && attempt != 1) return MCSD_ERR_SHAPE;
    p.target = target_slice; p.draft = draft_slice; p.attempt = attempt;
    p.stats_all = static_cast<const float4 *>(stats_all);
    p.tot_out = static_cast<double *>(totals_out);
    p.out_residual = out_residual_slice;
    const unsigned grid = shard_grid(static_cast<long long>(desc->batch) * L.eps);
    cudaStream_t st = static_cast<cudaStream_t>(desc->stream);
    MCSD_SHARD_LAUNCH(shard_endpoint_kernel, desc->dtype, L.ept, grid, st, p);
    if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
    g_last_launches = 1;
    return MCSD_OK;
}

int mcsd_shard_finish(const mcsd_shard_desc *desc, const void *target_slice, const void *draft_slice,
                      const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                      float temperature, int32_t attempt, const void *stats_all, const void *totals_all,
                      int32_t *out_accept_len, int32_t *out_tokens, int32_t *out_status, int32_t *out_path_nodes,
                      int32_t *endpoint_part, float *out_residual_slice)
{
    ShardParams p;
    TreePlan plan;
    ShardLayout L;
    int rc = fill_shard_params(desc, tree_parent, temperature, MCSD_MODE_WITH_REPLACEMENT, &p, &plan, &L);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0) return MCSD_OK;
    if (!stats_all || !totals_all || !cand_tokens || !uniforms || !out_accept_len || !out_tokens || !out_status ||
        !endpoint_part)
        return MCSD_ERR_NULL;
    if (L.n_cols > 0 && (!target_slice || (desc->n_internal > 0 && !draft_slice))) return MCSD_ERR_NULL;
    if (attempt != 0 && attempt != 1) return MCSD_ERR_SHAPE;
    p.target = target_slice; p.draft = draft_slice; p.cand = cand_tokens; p.unif = uniforms; p.attempt = attempt;
    p.stats_all = static_cast<const float4 *>(stats_all);
    p.tot_all = static_cast<const double *>(totals_all);
    p.out_accept_len = out_accept_len; p.out_tokens = out_tokens; p.out_status = out_status;
    p.out_path_nodes = out_path_nodes; p.endpoint_part = endpoint_part;
    p.out_residual = out_residual_slice;
    const unsigned grid = shard_grid(desc->batch);
    cudaStream_t st = static_cast<cudaStream_t>(desc->stream);
    MCSD_SHARD_LAUNCH(shard_finish_kernel, desc->dtype, L.ept, grid, st, p);
    if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
    g_last_launches = 1;
    return MCSD_OK;
}

int mcsd_shard_commit(const mcsd_shard_desc *desc, const int32_t *tree_parent, const int32_t *endpoint_all,
                      const int32_t *accept_len, int32_t *out_tokens)
{
    ShardLayout L;
    int rc = check_shard_desc(desc, &L);
    if (rc != MCSD_OK) return rc;
    TreePlan plan;
    rc = plan_tree_cached(tree_parent, desc->n_nodes, desc->n_internal, &plan);
    if (rc != MCSD_OK) return rc;
    g_last_launches = 0;
    if (desc->batch == 0) return MCSD_OK;
    if (!endpoint_all || !accept_len || !out_tokens) return MCSD_ERR_NULL;
    shard_commit_kernel<<<(desc->batch + 255) / 256, 256, 0, static_cast<cudaStream_t>(desc->stream)>>>(
        endpoint_all, accept_len, out_tokens, desc->batch, plan.gamma);
    if (cudaGetLastError() != cudaSuccess) return MCSD_ERR_CUDA;
    g_last_launches = 1;
    return MCSD_OK;
}

// ---- mcsd_verify_static: the scratch memory is an array built into the library --------
// In host code the name below is only a handle for the runtime; the address kernels can
// use comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_static_workspace[MCSD_STATIC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices] = {};

// Device address of the built-in array on the current device, or nullptr on failure.
void *static_workspace()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        g_static_ptr[dev] = ptr;
    }
    return g_static_ptr[dev];
}
}  // namespace

static int mcsd_verify_static_impl(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                       const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                       float temperature, int replacement_mode, int32_t *out_accept_len,
                       int32_t *out_tokens, float *out_residual)
{
    const int rc = check_desc(desc);
    if (rc != MCSD_OK) return rc;
    if (mcsd_workspace_bytes(desc) > MCSD_STATIC_WORKSPACE_BYTES) return MCSD_ERR_STATIC_LIMIT;
    void *ws = static_workspace();
    if (!ws) return MCSD_ERR_CUDA;
    mcsd_desc with_scratch = *desc;
    with_scratch.workspace = ws;
    with_scratch.workspace_bytes = MCSD_STATIC_WORKSPACE_BYTES;
    // the status words are cleared by the node stage itself; everything else in the
    // array is written before it is read
    return mcsd_verify_impl(&with_scratch, target_logits, draft_logits, tree_parent, cand_tokens, uniforms,
                       temperature, replacement_mode, out_accept_len, out_tokens, out_residual);
}

int mcsd_verify_static(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                       const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                       float temperature, int replacement_mode, int32_t *out_accept_len,
                       int32_t *out_tokens, float *out_residual)
{
    Trace trace("mcsd_verify_static", desc, temperature, replacement_mode);
    return trace.done(mcsd_verify_static_impl(desc, target_logits, draft_logits, tree_parent, cand_tokens, uniforms, temperature, replacement_mode, out_accept_len, out_tokens, out_residual));
}

// ---- mcsd_verify_host: device staging buffers kept between calls ------------------------
namespace {
struct HostSlot {
    cudaStream_t stream = nullptr;
    unsigned char *buf = nullptr;   // one allocation, carved per call
    size_t bytes = 0;
};
struct HostStaging {
    HostSlot slot[2];
};
std::mutex g_host_mutex;
HostStaging g_host[kMaxDevices];

void release_staging(HostStaging &hs)
{
    for (HostSlot &sl : hs.slot) {
        if (sl.buf) cudaFree(sl.buf);
        if (sl.stream) cudaStreamDestroy(sl.stream);
        sl = HostSlot();
    }
}
}  // namespace

int mcsd_release_host_staging(void)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MCSD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_host_mutex);
    release_staging(g_host[dev]);
    return MCSD_OK;
}

static int mcsd_verify_host_impl(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int replacement_mode, int32_t *out_accept_len,
                     int32_t *out_tokens, float *out_residual, int32_t *out_status)
{
    int rc = check_desc(desc);
    if (rc != MCSD_OK) return rc;
    TreePlan plan;
    rc = plan_tree_cached(tree_parent, desc->n_nodes, desc->n_internal, &plan);
    if (rc != MCSD_OK) return rc;
    rc = check_common(desc, target_logits, draft_logits, cand_tokens, uniforms, temperature,
                      replacement_mode, true, true);
    if (rc != MCSD_OK) return rc;
    if (!out_accept_len || !out_tokens) return MCSD_ERR_NULL;
    const int B = desc->batch;
    if (B == 0) return MCSD_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MCSD_ERR_CUDA;

    const size_t es = elem_bytes(desc->dtype);
    const bool use_draft = temperature > 0.f && desc->n_internal > 0 && replacement_mode != MCSD_MODE_NAIVE;
    const size_t t_seq = static_cast<size_t>(desc->n_nodes) * desc->ld_target * es;
    const size_t d_seq = use_draft ? static_cast<size_t>(desc->n_internal) * desc->ld_draft * es : 0;
    const size_t c_seq = sizeof(int32_t) * desc->n_nodes, u_seq = sizeof(float) * 2 * desc->n_nodes;
    const size_t tok_seq = sizeof(int32_t) * (plan.gamma + 1), res_seq = sizeof(float) * desc->vocab;
    // sequences per slice: about 256 MiB of logits, at least 1, at most ceil(B/2) so that
    // two slices exist to overlap whenever B > 1
    size_t per = (size_t(256) << 20) / (t_seq + d_seq ? t_seq + d_seq : 1);
    if (per < 1) per = 1;
    if (per > static_cast<size_t>((B + 1) / 2)) per = static_cast<size_t>((B + 1) / 2);
    const int chunk = static_cast<int>(per);

    mcsd_desc cd = *desc;
    cd.batch = chunk;
    cd.node_accept = nullptr; cd.node_bonus = nullptr; cd.node_ratio = nullptr; cd.out_path_nodes = nullptr;
    cd.node_residual = nullptr;
    const size_t ws_bytes = mcsd_workspace_bytes(&cd);
    // layout of one slot's staging buffer
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes, 256); return o; };
    const size_t o_t = take(t_seq * chunk), o_d = take(d_seq * chunk), o_c = take(c_seq * chunk),
                 o_u = take(u_seq * chunk), o_len = take(sizeof(int32_t) * chunk), o_tok = take(tok_seq * chunk),
                 o_st = take(sizeof(int32_t) * chunk), o_res = take(out_residual ? res_seq * chunk : 0),
                 o_ws = take(ws_bytes);
    const size_t need = off;

    // one call at a time per device uses the staging buffers
    std::lock_guard<std::mutex> lock(g_host_mutex);
    HostStaging &hs = g_host[dev];
    bool ok = true;
    auto chk = [&](cudaError_t e) { if (e != cudaSuccess) ok = false; return e == cudaSuccess; };
    for (HostSlot &sl : hs.slot) {
        if (!sl.stream) chk(cudaStreamCreateWithFlags(&sl.stream, cudaStreamNonBlocking));
        if (ok && sl.bytes < need) {
            if (sl.buf) cudaFree(sl.buf);
            sl.buf = nullptr;
            sl.bytes = 0;
            if (chk(cudaMalloc(&sl.buf, need))) sl.bytes = need;
        }
    }
    int launches = 0;
    for (int b0 = 0, i = 0; b0 < B && ok && rc == MCSD_OK; b0 += chunk, ++i) {
        HostSlot &sl = hs.slot[i & 1];
        const int nb = (B - b0 < chunk) ? B - b0 : chunk;
        unsigned char *base = sl.buf;
        const unsigned char *ht = static_cast<const unsigned char *>(target_logits) + t_seq * b0;
        chk(cudaMemcpyAsync(base + o_t, ht, t_seq * nb, cudaMemcpyHostToDevice, sl.stream));
        if (use_draft) {
            const unsigned char *hd = static_cast<const unsigned char *>(draft_logits) + d_seq * b0;
            chk(cudaMemcpyAsync(base + o_d, hd, d_seq * nb, cudaMemcpyHostToDevice, sl.stream));
        }
        chk(cudaMemcpyAsync(base + o_c, cand_tokens + static_cast<size_t>(b0) * desc->n_nodes, c_seq * nb,
                            cudaMemcpyHostToDevice, sl.stream));
        if (uniforms)
            chk(cudaMemcpyAsync(base + o_u, uniforms + static_cast<size_t>(b0) * 2 * desc->n_nodes, u_seq * nb,
                                cudaMemcpyHostToDevice, sl.stream));
        if (!ok) break;
        cd.batch = nb;
        cd.stream = sl.stream;
        cd.workspace = base + o_ws;
        cd.workspace_bytes = ws_bytes;
        cd.out_status = reinterpret_cast<int32_t *>(base + o_st);
        rc = mcsd_verify_impl(&cd, base + o_t, use_draft ? base + o_d : nullptr, tree_parent,
                         reinterpret_cast<const int32_t *>(base + o_c),
                         uniforms ? reinterpret_cast<const float *>(base + o_u) : nullptr, temperature,
                         replacement_mode, reinterpret_cast<int32_t *>(base + o_len),
                         reinterpret_cast<int32_t *>(base + o_tok),
                         out_residual ? reinterpret_cast<float *>(base + o_res) : nullptr);
        if (rc != MCSD_OK) break;   // nothing of this slice is copied back
        launches += g_last_launches;
        chk(cudaMemcpyAsync(out_accept_len + b0, base + o_len, sizeof(int32_t) * nb, cudaMemcpyDeviceToHost, sl.stream));
        chk(cudaMemcpyAsync(out_tokens + static_cast<size_t>(b0) * (plan.gamma + 1), base + o_tok, tok_seq * nb,
                            cudaMemcpyDeviceToHost, sl.stream));
        if (out_residual)
            chk(cudaMemcpyAsync(out_residual + static_cast<size_t>(b0) * desc->vocab, base + o_res, res_seq * nb,
                                cudaMemcpyDeviceToHost, sl.stream));
        if (out_status)
            chk(cudaMemcpyAsync(out_status + b0, base + o_st, sizeof(int32_t) * nb, cudaMemcpyDeviceToHost, sl.stream));
    }
    for (HostSlot &sl : hs.slot)
        if (sl.stream) chk(cudaStreamSynchronize(sl.stream));
    g_last_launches = launches;
    if (rc != MCSD_OK) return rc;
    if (!ok) { cudaGetLastError(); return MCSD_ERR_CUDA; }
    return MCSD_OK;
}

int mcsd_verify_host(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int replacement_mode, int32_t *out_accept_len,
                     int32_t *out_tokens, float *out_residual, int32_t *out_status)
{
    Trace trace("mcsd_verify_host", desc, temperature, replacement_mode);
    return trace.done(mcsd_verify_host_impl(desc, target_logits, draft_logits, tree_parent, cand_tokens, uniforms, temperature, replacement_mode, out_accept_len, out_tokens, out_residual, out_status));
}

}  // extern "C"
