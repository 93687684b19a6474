// Device code of the MCSD verification library (sm_100a).
//
// Three kernels:
//   node_kernel      T > 0.  One thread-block cluster per tree node.  Each CTA of the
//                    cluster owns a contiguous slice of the vocabulary, brings its
//                    slice of the target row (and of the draft row for a node that
//                    has children) into shared memory with one bulk async copy (TMA,
//                    no multicast), moves it into registers, and from then on the two
//                    distributions stay in registers while the k candidates of the
//                    node are tested in order (Algorithm 1 / Algorithm 2).  Each logit
//                    row is read from HBM exactly once.
//   argmax_kernel    T == 0.  One CTA per target row; argmax with lowest index on ties
//                    and the "candidate equals argmax" test (Section 4.4).
//   walk_kernel      One row of CTAs per sequence: follows the accepted children from
//                    the root (Section 3), writes the accepted tokens and the endpoint
//                    token, and rebuilds the residual distribution of the stopping node.
//
// How the rejection loop avoids rewriting the residual.  After n rejections the
// unnormalised residual of Algorithm 1/2 is  P_n(x) = max(p(x) - c_n q(x), 0)  with
// c_0 = 0 and c_{n+1} = c_n + S_n / W_n, where S_n = sum_x P_n(x), and W_n = 1 for
// Algorithm 1 or 1 - (original draft mass of the tokens rejected so far) for
// Algorithm 2 (p and q are the ORIGINAL softmax outputs).  This follows from
// p_{n+1} ~ max(p_n - q_n, 0) by induction and holds for every rejection that can
// occur with r in (0,1).  The test of candidate n+1 is r <= [P_n(x~)/S_n]/[q(x~)/W_n].
// So one rejection costs one scalar-parameter reduction over the register-resident
// p and q, and nothing is written back.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mcsd.h"

namespace mcsd {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxCluster = 8;
// Polls of a bounded wait before it gives up (each poll can itself block for a
// hardware-defined time slice, so this is seconds, far beyond any legitimate wait).
constexpr uint32_t kWaitPolls = 1u << 22;

struct __align__(16) NodeStats {
    float r_t, r_d;  // references of the sums: fl(row maximum * scale), log2 units
    float z_t, z_d;  // sum_x exp2(l * scale - r)
    float c, s;      // final c_n and S_n of the node (0 and 1 for a leaf)
    int32_t pad0, pad1;
};

struct NodeParams {
    const void *target;
    const void *draft;
    const int32_t *cand;
    const float *unif;
    int32_t *node_accept;
    int32_t *node_bonus;
    float *node_ratio;  // may be null
    NodeStats *stats;
    int32_t *status;  // [B]
    long long ld_t, ld_d;
    int32_t B, n_nodes, n_internal, V;
    int32_t slice;   // vocabulary elements owned by one CTA of the cluster
    int32_t n_items; // B * n_nodes
    int32_t mode;
    float scale;     // log2(e) / T
    double scale_d;  // the same in double, for the candidates' own probabilities
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
};

// ------------------------------------------------------------------ element types
template <int DT> struct Elem;
template <> struct Elem<MCSD_DTYPE_F32> {
    static constexpr int kBytes = 4, kVec = 4;
    static __device__ __forceinline__ void unpack(const uint4 &r, float *o) {
        o[0] = __uint_as_float(r.x); o[1] = __uint_as_float(r.y);
        o[2] = __uint_as_float(r.z); o[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ float load(const void *base, long long i) {
        return __ldg(reinterpret_cast<const float *>(base) + i);
    }
};
template <> struct Elem<MCSD_DTYPE_BF16> {
    static constexpr int kBytes = 2, kVec = 8;
    static __device__ __forceinline__ void unpack(const uint4 &r, float *o) {
        o[0] = __uint_as_float(r.x << 16); o[1] = __uint_as_float(r.x & 0xffff0000u);
        o[2] = __uint_as_float(r.y << 16); o[3] = __uint_as_float(r.y & 0xffff0000u);
        o[4] = __uint_as_float(r.z << 16); o[5] = __uint_as_float(r.z & 0xffff0000u);
        o[6] = __uint_as_float(r.w << 16); o[7] = __uint_as_float(r.w & 0xffff0000u);
    }
    static __device__ __forceinline__ float load(const void *base, long long i) {
        unsigned short h = __ldg(reinterpret_cast<const unsigned short *>(base) + i);
        return __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
};
template <> struct Elem<MCSD_DTYPE_F16> {
    static constexpr int kBytes = 2, kVec = 8;
    static __device__ __forceinline__ void unpack(const uint4 &r, float *o) {
        const __half2 *h = reinterpret_cast<const __half2 *>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __half22float2(h[i]);
            o[2 * i] = f.x; o[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ float load(const void *base, long long i) {
        return __half2float(__ldg(reinterpret_cast<const __half *>(base) + i));
    }
};

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded waits: false when the poll budget ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitPolls; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitPolls; ++i)
        if (mbar_try_wait_cluster(bar, parity)) return true;
    return false;
}
// One bulk async copy global -> this CTA's shared memory (TMA, no multicast);
// completion is signalled on an mbarrier of this CTA as a byte count.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f4(uint32_t addr, float4 v) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};"
                 ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_scan_incl(float v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        float t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}
__device__ __forceinline__ double shfl_d(double v, int src) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_sync(0xffffffffu, lo, src);
    hi = __shfl_sync(0xffffffffu, hi, src);
    return __hiloint2double(hi, lo);
}
// Factor that moves a partial sum taken relative to reference r (log2 units) to the
// reference R >= r; an empty partial sum has r = -inf and factor 0.
__device__ __forceinline__ float rebase(float r, float R) {
    return (r == -INFINITY) ? 0.f : ex2f(r - R);
}

// Shared state of the cluster-wide exchange: every CTA owns two slots of one float4
// per cluster rank and one mbarrier per slot.  In round r every CTA stores its value
// into slot r&1 of every CTA (its own included) and arrives on that CTA's barrier;
// a CTA that has seen `cluster size` arrivals holds all values of the round.  A slot
// is rewritten two rounds later, which a peer can only reach after this CTA has
// arrived for the round in between, i.e. after it finished reading (release/acquire
// at cluster scope orders the accesses).
struct Exchange {
    float4 slot[2][kMaxCluster];
    unsigned long long bar[2];
};

// ------------------------------------------------------------------ node kernel
// Warp totals of N values per lane in N-1 + (5 - log2 N) shuffles instead of 5 N: each
// halving step pairs lanes and splits the value indices between them.  On return
// every lane holds in `out` the warp total of value index `idx` (the return value),
// idx being fixed by lane bits 4, 3, 2 (N = 8), bits 4, 3 (N = 4) or bit 4 (N = 2).
template <int HALF>
__device__ __forceinline__ void halve_step(float *w, int lane, int off, int &idx)
{
    const bool hi = (lane & off) != 0;
#pragma unroll
    for (int j = 0; j < HALF; ++j) {
        const float send = hi ? w[j] : w[j + HALF];
        const float keep = hi ? w[j + HALF] : w[j];
        w[j] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
    idx += hi ? HALF : 0;
}
template <int N>
__device__ __forceinline__ int warp_multi_sum(const float (&v)[N], int lane, float &out)
{
    static_assert(N == 1 || N == 2 || N == 4 || N == 8, "unsupported count");
    float w[N];
#pragma unroll
    for (int j = 0; j < N; ++j) w[j] = v[j];
    int idx = 0;
    if constexpr (N >= 2) halve_step<N / 2>(w, lane, 16, idx);
    else w[0] += __shfl_xor_sync(0xffffffffu, w[0], 16);
    if constexpr (N >= 4) halve_step<N / 4>(w, lane, 8, idx);
    else w[0] += __shfl_xor_sync(0xffffffffu, w[0], 8);
    if constexpr (N >= 8) halve_step<N / 8>(w, lane, 4, idx);
    else w[0] += __shfl_xor_sync(0xffffffffu, w[0], 4);
    w[0] += __shfl_xor_sync(0xffffffffu, w[0], 2);
    w[0] += __shfl_xor_sync(0xffffffffu, w[0], 1);
    out = w[0];
    return idx;
}

// DT: element type; EPT: vocabulary elements per thread per row; DIRECT: read the
// rows with plain scalar loads (any alignment) instead of bulk copies.
template <int DT, int EPT, bool DIRECT>
__global__ void __launch_bounds__(kThreads, (EPT >= 32 ? 2 : (EPT >= 16 ? 3 : 4)))
node_kernel(const __grid_constant__ NodeParams P)
{
    using E = Elem<DT>;
    constexpr int VEC = E::kVec;
    constexpr int NVEC = EPT / VEC;
    constexpr int kRowBytes = kThreads * EPT * E::kBytes;
    static_assert(EPT % VEC == 0, "EPT must be a whole number of 16-byte vectors");

    extern __shared__ __align__(128) unsigned char stage[];  // [2][kRowBytes]: target slice, draft slice
    __shared__ Exchange xch;
    __shared__ __align__(8) unsigned long long full_bar;
    __shared__ float4 red[kWarps];
    __shared__ float wsum[NVEC * kWarps];
    __shared__ double s_px[MCSD_MAX_CHILDREN], s_qx[MCSD_MAX_CHILDREN];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t crank = cluster_ctarank(), csize = cluster_nctarank();
    const int cluster_id = blockIdx.x / csize, n_clusters = gridDim.x / csize;
    const float scale = P.scale;

    const uint32_t full_addr = smem_u32(&full_bar);
    const uint32_t xbar_addr[2] = {smem_u32(&xch.bar[0]), smem_u32(&xch.bar[1])};
    const uint32_t stage_addr = smem_u32(stage);

    // this CTA's slice of the vocabulary
    const int v_begin = static_cast<int>(crank) * P.slice;
    int n_mine = P.V - v_begin;
    n_mine = n_mine < 0 ? 0 : (n_mine > P.slice ? P.slice : n_mine);
    const int n_full_vec = n_mine / VEC;  // vectors that lie wholly inside the slice
    const uint32_t row_bytes = (static_cast<uint32_t>(n_mine) * E::kBytes + 15u) & ~15u;

    if (tid == 0) {
        mbar_init(full_addr, 1);
        mbar_init(xbar_addr[0], csize);
        mbar_init(xbar_addr[1], csize);
        fence_mbar_init();
    }
    __syncthreads();
    cluster_sync_all();  // every CTA's barriers exist before anyone arrives remotely

    uint32_t full_parity = 0, round = 0;
    int poisoned = 0;

    auto issue = [&](int item) {
        const int b = item / P.n_nodes, n = item - b * P.n_nodes;
        const bool internal = n < P.n_internal;
        const uint32_t total = row_bytes * (internal ? 2u : 1u);
        mbar_arrive_expect_tx(full_addr, total);
        if (row_bytes) {
            const unsigned char *t = reinterpret_cast<const unsigned char *>(P.target) +
                (static_cast<long long>(item) * P.ld_t + v_begin) * E::kBytes;
            bulk_load(stage_addr, t, row_bytes, full_addr);
            if (internal) {
                const unsigned char *d = reinterpret_cast<const unsigned char *>(P.draft) +
                    ((static_cast<long long>(b) * P.n_internal + n) * P.ld_d + v_begin) * E::kBytes;
                bulk_load(stage_addr + kRowBytes, d, row_bytes, full_addr);
            }
        }
    };

    // Cluster-wide exchange of one float4 per CTA; `mine` must be valid in lanes
    // 0..csize-1 of warp 0.  Returns the slot holding all CTAs' values.
    auto exchange = [&](float4 mine) -> const float4 * {
        const uint32_t s = round & 1u;
        if (warp == 0 && lane < static_cast<int>(csize)) {
            const uint32_t dst = map_to_rank(smem_u32(&xch.slot[s][crank]), lane);
            st_cluster_f4(dst, mine);
            mbar_arrive_remote(map_to_rank(xbar_addr[s], lane));
        }
        if (!mbar_wait_cluster(xbar_addr[s], (round >> 1) & 1u)) poisoned = 1;
        ++round;
        return xch.slot[s];
    };

    // Candidate data is fetched ahead of use so that no DRAM latency sits on the
    // per-node critical path: lane i of every warp holds candidate i of the node.
    //   tokens (token id, acceptance uniform) two nodes ahead,
    //   the candidate's own two logits one node ahead (they need the token id).
    auto fetch_tokens = [&](int item, int &xt, float &u) {
        xt = -1; u = 2.f;
        if (item < P.n_items) {
            const int b = item / P.n_nodes, n = item - b * P.n_nodes;
            const int k = n < P.n_internal ? P.child_count[n] : 0;
            if (lane < k) {
                const long long ci = static_cast<long long>(b) * P.n_nodes + P.child_first[n] + lane;
                xt = __ldg(P.cand + ci);
                u = __ldg(P.unif + 2 * ci);
            }
        }
    };
    auto fetch_logits = [&](int item, int xt, float &tl, float &dl) {
        tl = 0.f; dl = 0.f;
        if (item < P.n_items && xt >= 0 && xt < P.V) {
            const int b = item / P.n_nodes, n = item - b * P.n_nodes;
            tl = E::load(P.target, static_cast<long long>(item) * P.ld_t + xt);
            dl = E::load(P.draft, (static_cast<long long>(b) * P.n_internal + n) * P.ld_d + xt);
        }
    };

    int item = cluster_id;
    if (!DIRECT && tid == 0 && item < P.n_items) issue(item);
    int xt, xt_n1, xt_n2;
    float u_acc, u_n1, u_n2, tl, dl, tl_n1, dl_n1;
    fetch_tokens(item, xt, u_acc);
    fetch_tokens(item + n_clusters, xt_n1, u_n1);
    fetch_logits(item, xt, tl, dl);

    for (; item < P.n_items; item += n_clusters) {
        const int b = item / P.n_nodes, n = item - b * P.n_nodes;
        const bool internal = n < P.n_internal;
        const int k = internal ? P.child_count[n] : 0;
        const int first = P.child_first[n];
        const long long node_idx = item;  // b * n_nodes + n
        int status_bits = 0;

        fetch_logits(item + n_clusters, xt_n1, tl_n1, dl_n1);
        fetch_tokens(item + 2 * n_clusters, xt_n2, u_n2);
        const float u_end = __ldg(P.unif + 2 * node_idx + 1);

        // ---- bring the slice into registers: tv = target, dv = draft
        float tv[EPT], dv[EPT];
        if (!DIRECT) {
            if (!mbar_wait(full_addr, full_parity)) poisoned = 1;
            full_parity ^= 1u;
#pragma unroll
            for (int j = 0; j < NVEC; ++j) {
                const int vec = j * kThreads + tid;
                uint4 raw = *reinterpret_cast<const uint4 *>(stage + vec * 16);
                E::unpack(raw, &tv[j * VEC]);
                if (internal) {
                    raw = *reinterpret_cast<const uint4 *>(stage + kRowBytes + vec * 16);
                    E::unpack(raw, &dv[j * VEC]);
                }
                if (vec >= n_full_vec) {  // ragged or empty vector: only at the slice end
                    const int rem = n_mine - vec * VEC;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        if (e >= rem) { tv[j * VEC + e] = -INFINITY; dv[j * VEC + e] = -INFINITY; }
                    }
                }
            }
            __syncthreads();  // stage fully consumed: refill it with the next node of this cluster
            if (tid == 0 && item + n_clusters < P.n_items) issue(item + n_clusters);
        } else {
            const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) +
                node_idx * P.ld_t * E::kBytes;
            const unsigned char *d_row = reinterpret_cast<const unsigned char *>(P.draft) +
                (static_cast<long long>(b) * P.n_internal + n) * P.ld_d * E::kBytes;
#pragma unroll
            for (int j = 0; j < NVEC; ++j) {
                const int base = (j * kThreads + tid) * VEC;
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    const bool ok = base + e < n_mine;
                    tv[j * VEC + e] = ok ? E::load(t_row, v_begin + base + e) : -INFINITY;
                    if (internal) dv[j * VEC + e] = ok ? E::load(d_row, v_begin + base + e) : -INFINITY;
                }
            }
        }

        // ---- softmax statistics, one cluster-wide round for both rows.  Each thread
        // exponentiates relative to its own maximum (reference r = max * scale, in
        // log2 units); the factor to the global reference and the normaliser are
        // applied as per-thread scalars afterwards, never per element.
        float vs[NVEC];  // per-vector weight sums of this thread, in the thread's own units
        float mt = -INFINITY, md = -INFINITY;
#pragma unroll
        for (int e = 0; e < EPT; ++e) mt = fmaxf(mt, tv[e]);
        // rt / rd: this thread's references (-inf when it holds no finite element)
        const float rt = (mt == -INFINITY) ? -INFINITY : mt * scale;
        const float rt0 = (mt == -INFINITY) ? 0.f : rt;
        float zt = 0.f, zd = 0.f, rd = -INFINITY;
#pragma unroll
        for (int j = 0; j < NVEC; ++j) {
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                const float x = ex2f(fmaf(tv[j * VEC + e], scale, -rt0));
                tv[j * VEC + e] = x;
                s += x;
            }
            vs[j] = s;
            zt += s;
        }
        if (internal) {
#pragma unroll
            for (int e = 0; e < EPT; ++e) md = fmaxf(md, dv[e]);
            rd = (md == -INFINITY) ? -INFINITY : md * scale;
            const float rd0 = (md == -INFINITY) ? 0.f : rd;
#pragma unroll
            for (int e = 0; e < EPT; ++e) {
                const float x = ex2f(fmaf(dv[e], scale, -rd0));
                dv[e] = x;
                zd += x;
            }
        }
        {
            const float Rt = warp_max(rt), Rd = warp_max(rd);
            const float st = warp_sum(zt * rebase(rt, Rt));
            const float sd = warp_sum(zd * rebase(rd, Rd));
            if (lane == 0) red[warp] = make_float4(Rt, st, Rd, sd);
        }
        __syncthreads();
        float4 cta = make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
        if (warp == 0) {
            if (lane < kWarps) cta = red[lane];
            const float Rt = warp_max(cta.x), Rd = warp_max(cta.z);
            cta.y = warp_sum(cta.y * rebase(cta.x, Rt));
            cta.w = warp_sum(cta.w * rebase(cta.z, Rd));
            cta.x = Rt; cta.z = Rd;
        }
        const float4 *slot = exchange(cta);  // per CTA: (ref_t, z_t, ref_d, z_d)
        float R_t = -INFINITY, R_d = -INFINITY;  // global references: fl(row maximum * scale)
#pragma unroll
        for (uint32_t r = 0; r < kMaxCluster; ++r)
            if (r < csize) { R_t = fmaxf(R_t, slot[r].x); R_d = fmaxf(R_d, slot[r].z); }
        float Z_t = 0.f, Z_d = 0.f;
#pragma unroll
        for (uint32_t r = 0; r < kMaxCluster; ++r)
            if (r < csize) {
                Z_t += slot[r].y * rebase(slot[r].x, R_t);
                Z_d += slot[r].w * rebase(slot[r].z, R_d);
            }
        const bool t_ok = Z_t > 0.f && Z_t < INFINITY;            // false for an all -inf or NaN row
        const bool d_ok = internal && Z_d > 0.f && Z_d < INFINITY;
        if (!t_ok) status_bits |= MCSD_STATUS_NO_MASS;
        // p(x) = tv * a, q(x) = dv * bq for this thread's elements
        const float a = t_ok ? rebase(rt, R_t) / Z_t : 0.f;
        const float bq = d_ok ? rebase(rd, R_d) / Z_d : 0.f;
        const float b_over_a = a > 0.f ? bq / a : 0.f;
        bool leaf_masses = true;  // slot holds softmax statistics (true) or residual partial sums

        // ---- probabilities of the candidates themselves, once per CTA, in double
        if (k > 0) {
            if (warp == 0 && lane < k) {
                const bool ok = xt >= 0 && xt < P.V;
                s_px[lane] = (ok && t_ok) ? exp2(static_cast<double>(tl) * P.scale_d - static_cast<double>(R_t)) /
                                                static_cast<double>(Z_t) : 0.0;
                s_qx[lane] = (ok && d_ok) ? exp2(static_cast<double>(dl) * P.scale_d - static_cast<double>(R_d)) /
                                                static_cast<double>(Z_d) : 0.0;
            }
            __syncthreads();
        }

        // ---- the rejection loop (Algorithm 1 / Algorithm 2), identical in every thread
        double c = 0.0, S = 1.0, W = 1.0;
        float kappa = 0.f;  // c * bq / a: the residual weight of an element is max(tv - kappa dv, 0) * a
        int accepted = -1;
        for (int i = 0; i < k; ++i) {
            const int xi = __shfl_sync(0xffffffffu, xt, i);
            const float ui = __shfl_sync(0xffffffffu, u_acc, i);
            const double pxi = s_px[i], qxi = s_qx[i];
            const bool valid = xi >= 0 && xi < P.V;
            if (!valid) status_bits |= MCSD_STATUS_BAD_TOKEN;
            // Algorithm 2: a token rejected earlier at this node has draft probability 0 now
            const bool dup = P.mode == 1 &&
                (__ballot_sync(0xffffffffu, lane < i && xt == xi) != 0u);
            const bool zero_q = !valid || dup || !(qxi > 0.0) || !(W > 0.0);
            double Pn = pxi - c * qxi;
            Pn = Pn > 0.0 ? Pn : 0.0;
            // r <= [P_n(x~)/S_n] / [q(x~)/W_n], written without the divisions (all factors > 0)
            const bool accept = !zero_q && static_cast<double>(ui) * S * qxi <= Pn * W;
            if (P.node_ratio && crank == 0 && tid == 0)
                P.node_ratio[static_cast<long long>(b) * P.n_nodes + first + i] =
                    zero_q ? -1.f : static_cast<float>((Pn / S) / (qxi / W));
            if (accept) { accepted = first + i; break; }
            // rejected: p := norm(max(0, p - q)); Algorithm 2 also removes x~ from q
            double c_try = c;
            if (W > 0.0) c_try = (P.mode == 1) ? c + S / W : c + S;
            if (P.mode == 1 && !zero_q) { W -= qxi; if (!(W > 0.0)) W = 0.0; }
            for (int attempt = 0; attempt < 2; ++attempt) {
                kappa = static_cast<float>(c_try) * b_over_a;
                float part = 0.f;
#pragma unroll
                for (int j = 0; j < NVEC; ++j) {
                    float s = 0.f;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) s += fmaxf(fmaf(-kappa, dv[j * VEC + e], tv[j * VEC + e]), 0.f);
                    vs[j] = s;
                    part += s;
                }
                part = warp_sum(part * a);
                if (lane == 0) red[warp].x = part;
                __syncthreads();
                float cta_part = 0.f;
                if (warp == 0) cta_part = warp_sum(lane < kWarps ? red[lane].x : 0.f);
                slot = exchange(make_float4(cta_part, 0.f, 0.f, 0.f));
                leaf_masses = false;
                float S_new = 0.f;
#pragma unroll
                for (uint32_t r = 0; r < kMaxCluster; ++r)
                    if (r < csize) S_new += slot[r].x;
                if (S_new > 0.f) {
                    if (attempt == 0) { c = c_try; S = static_cast<double>(S_new); }
                    break;
                }
                // zero residual mass: keep the previous residual (recompute its sums once)
                status_bits |= MCSD_STATUS_DEGENERATE;
                c_try = c;
            }
        }

        // ---- endpoint token of a node that can end the walk: inverse CDF in token
        // order over w(x) = max(p - c q, 0); only the CTA whose slice holds the
        // quantile searches, the others go on to their next node.  vs[] holds this
        // thread's per-vector sums of w / a.
        int bonus = -1;
        bool bonus_mine = false;
        if (accepted < 0) {
            const float inv_zt = t_ok ? 1.f / Z_t : 0.f;
            float total = 0.f;
#pragma unroll
            for (uint32_t r = 0; r < kMaxCluster; ++r)
                if (r < csize)
                    total += leaf_masses ? slot[r].y * rebase(slot[r].x, R_t) * inv_zt : slot[r].x;
            const float target = u_end * total;
            int owner = -1, last_pos = -1;
            float cum = 0.f, before = 0.f, last_before = 0.f;
#pragma unroll
            for (uint32_t r = 0; r < kMaxCluster; ++r) {
                if (r < csize) {
                    const float m = leaf_masses ? slot[r].y * rebase(slot[r].x, R_t) * inv_zt : slot[r].x;
                    if (m > 0.f) {
                        last_pos = r; last_before = cum;
                        if (owner < 0 && cum + m > target) { owner = r; before = cum; }
                    }
                    cum += m;
                }
            }
            if (owner < 0) { owner = last_pos; before = last_before; }  // rounding pushed the quantile past the end
            if (owner < 0 || !(total > 0.f)) {
                status_bits |= MCSD_STATUS_NO_MASS;
                bonus_mine = crank == 0;
            } else if (owner == static_cast<int>(crank)) {
                bonus_mine = true;
                float tgt = target - before;  // quantile inside this CTA's slice
                float wv[NVEC];
#pragma unroll
                for (int j = 0; j < NVEC; ++j) wv[j] = vs[j] * a;
                float wtot;
                const int wj = warp_multi_sum<NVEC>(wv, lane, wtot);
                if ((lane & 3) == 0) wsum[wj * kWarps + warp] = wtot;  // lanes sharing an index write the same total
                __syncthreads();
                // level 1: (chunk j, warp) in token order
                constexpr int kEntries = NVEC * kWarps;
                int pick = -1, last_e = -1;
                float run = 0.f, pick_before = 0.f, last_b = 0.f;
#pragma unroll
                for (int base = 0; base < kEntries; base += 32) {
                    const int idx = base + lane;
                    const float w = idx < kEntries ? wsum[idx] : 0.f;
                    const float inc = warp_scan_incl(w, lane) + run;
                    const unsigned hit = __ballot_sync(0xffffffffu, w > 0.f && inc > tgt);
                    const unsigned pos = __ballot_sync(0xffffffffu, w > 0.f);
                    if (pick < 0 && hit) {
                        const int l = __ffs(hit) - 1;
                        pick = base + l;
                        pick_before = __shfl_sync(0xffffffffu, inc, l) - __shfl_sync(0xffffffffu, w, l);
                    }
                    if (pos) {
                        const int l = 31 - __clz(pos);
                        last_e = base + l;
                        last_b = __shfl_sync(0xffffffffu, inc, l) - __shfl_sync(0xffffffffu, w, l);
                    }
                    run = __shfl_sync(0xffffffffu, inc, 31);
                }
                if (pick < 0) { pick = last_e; pick_before = last_b; }  // clamp to the last entry with mass
                if (pick >= 0) {
                    const int pj = pick / kWarps, pw = pick - pj * kWarps;
                    if (warp == pw) {
                        tgt -= pick_before;
                        float v = wv[0];
#pragma unroll
                        for (int j = 1; j < NVEC; ++j) v = (pj == j) ? wv[j] : v;
                        const float inc = warp_scan_incl(v, lane);
                        const unsigned hit = __ballot_sync(0xffffffffu, v > 0.f && inc > tgt);
                        const unsigned pos = __ballot_sync(0xffffffffu, v > 0.f);
                        const int l = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : -1);
                        if (l >= 0 && lane == l) {
                            const float rem = tgt - (inc - v);
                            float acc = 0.f;
                            int pe = -1, last = -1;
#pragma unroll
                            for (int j = 0; j < NVEC; ++j) {
                                if (j == pj) {
#pragma unroll
                                    for (int e = 0; e < VEC; ++e) {
                                        const float w = (internal ? fmaxf(fmaf(-kappa, dv[j * VEC + e], tv[j * VEC + e]), 0.f)
                                                                  : tv[j * VEC + e]) * a;
                                        if (w > 0.f) {
                                            acc += w;
                                            last = e;
                                            if (pe < 0 && acc > rem) pe = e;
                                        }
                                    }
                                }
                            }
                            if (pe < 0) pe = last;
                            bonus = v_begin + (pj * kThreads + warp * 32 + lane) * VEC + pe;
                            P.node_bonus[node_idx] = bonus;
                        }
                    }
                } else if (tid == 0) {
                    P.node_bonus[node_idx] = -1;
                    status_bits |= MCSD_STATUS_NO_MASS;
                }
            }
        }

        // ---- per-node results
        if (crank == 0 && tid == 0) {
            P.node_accept[node_idx] = accepted;
            if (accepted >= 0 || (bonus_mine && bonus < 0 && (status_bits & MCSD_STATUS_NO_MASS)))
                P.node_bonus[node_idx] = -1;
            NodeStats st;
            st.r_t = R_t; st.r_d = R_d;
            st.z_t = Z_t; st.z_d = Z_d;
            st.c = static_cast<float>(c); st.s = static_cast<float>(S);
            st.pad0 = 0; st.pad1 = 0;
            P.stats[node_idx] = st;
        }
        if (poisoned) status_bits |= MCSD_STATUS_TIMEOUT;
        status_bits = __reduce_or_sync(0xffffffffu, status_bits);
        if (status_bits && lane == 0) atomicOr(P.status + b, status_bits);

        // rotate the candidate pipeline
        xt = xt_n1; u_acc = u_n1; tl = tl_n1; dl = dl_n1;
        xt_n1 = xt_n2; u_n1 = u_n2;
    }

    // no CTA may leave while a peer can still write into its shared memory
    cluster_sync_all();
}

// ------------------------------------------------------------------ argmax kernel (T == 0)
struct ArgmaxParams {
    const void *target;
    const int32_t *cand;
    int32_t *node_accept;
    int32_t *node_bonus;
    float *node_ratio;  // may be null
    long long ld_t;
    int32_t n_nodes, n_internal, V, n_rows;
    int32_t vector_ok;  // rows are 16-byte aligned
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
};

template <int DT>
__global__ void __launch_bounds__(kThreads)
argmax_kernel(const __grid_constant__ ArgmaxParams P)
{
    using E = Elem<DT>;
    constexpr int VEC = E::kVec;
    __shared__ float s_val[kWarps];
    __shared__ int s_idx[kWarps];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int row = blockIdx.x; row < P.n_rows; row += gridDim.x) {
        const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) +
            static_cast<long long>(row) * P.ld_t * E::kBytes;
        float best = -INFINITY;
        int best_i = 0x7fffffff;
        // strict '>' keeps the lowest index inside a thread (indices ascend); NaN never wins
        if (P.vector_ok) {
            const int n_vec = P.V / VEC;
            const uint4 *src = reinterpret_cast<const uint4 *>(t_row);
            int v = tid;
            for (; v + 3 * kThreads < n_vec; v += 4 * kThreads) {
                uint4 r[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) r[u] = __ldg(src + v + u * kThreads);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float f[VEC];
                    E::unpack(r[u], f);
#pragma unroll
                    for (int e = 0; e < VEC; ++e)
                        if (f[e] > best) { best = f[e]; best_i = (v + u * kThreads) * VEC + e; }
                }
            }
            for (; v < n_vec; v += kThreads) {
                float f[VEC];
                E::unpack(__ldg(src + v), f);
#pragma unroll
                for (int e = 0; e < VEC; ++e)
                    if (f[e] > best) { best = f[e]; best_i = v * VEC + e; }
            }
            for (int x = n_vec * VEC + tid; x < P.V; x += kThreads) {
                const float f = E::load(t_row, x);
                if (f > best) { best = f; best_i = x; }
            }
        } else {
            for (int x = tid; x < P.V; x += kThreads) {
                const float f = E::load(t_row, x);
                if (f > best) { best = f; best_i = x; }
            }
        }
        // combine: larger value wins, equal values -> lower index
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
            if (ov > best || (ov == best && oi < best_i)) { best = ov; best_i = oi; }
        }
        if (lane == 0) { s_val[warp] = best; s_idx[warp] = best_i; }
        __syncthreads();
        if (warp == 0) {
            best = lane < kWarps ? s_val[lane] : -INFINITY;
            best_i = lane < kWarps ? s_idx[lane] : 0x7fffffff;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best, o);
                const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
                if (ov > best || (ov == best && oi < best_i)) { best = ov; best_i = oi; }
            }
            // a row with no finite-or-inf maximum (all NaN / all -inf) falls back to token 0
            const int a = best_i == 0x7fffffff ? 0 : best_i;
            const int b = row / P.n_nodes, n = row - b * P.n_nodes;
            const int k = n < P.n_internal ? P.child_count[n] : 0;
            const int first = P.child_first[n];
            int tok = -2;
            if (lane < k) tok = __ldg(P.cand + static_cast<long long>(b) * P.n_nodes + first + lane);
            const unsigned match = __ballot_sync(0xffffffffu, lane < k && tok == a);
            const int acc = match ? first + __ffs(match) - 1 : -1;
            if (P.node_ratio && lane < k && (acc < 0 || first + lane <= acc))
                P.node_ratio[static_cast<long long>(b) * P.n_nodes + first + lane] = (tok == a) ? 1.f : 0.f;
            if (lane == 0) {
                P.node_accept[row] = acc;
                P.node_bonus[row] = acc >= 0 ? -1 : a;
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ walk + terminal residual
struct WalkParams {
    const void *target;
    const void *draft;
    const int32_t *cand;
    const int32_t *node_accept;
    const int32_t *node_bonus;
    const NodeStats *stats;
    int32_t *out_accept_len;
    int32_t *out_tokens;
    float *out_residual;  // may be null
    long long ld_t, ld_d;
    int32_t n_nodes, n_internal, V, gamma;
    float scale;  // log2(e)/T, or 0 for the argmax rule
};

// grid = (ceil(V / (kThreads*4)), B).  Every CTA of a row repeats the (at most gamma
// hop) walk; the first one writes the tokens.
template <int DT>
__global__ void __launch_bounds__(kThreads)
walk_kernel(const __grid_constant__ WalkParams P)
{
    using E = Elem<DT>;
    __shared__ int s_term;
    const int b = blockIdx.y;
    const long long nb = static_cast<long long>(b) * P.n_nodes;
    if (threadIdx.x == 0) {
        int n = 0, len = 0;
        int32_t *tok = P.out_tokens + static_cast<long long>(b) * (P.gamma + 1);
        const bool writer = blockIdx.x == 0;
        // bounded by the depth of the tree even if node_accept were corrupt
        for (int hop = 0; hop < P.gamma; ++hop) {
            const int nx = P.node_accept[nb + n];
            if (nx <= n || nx >= P.n_nodes) break;
            n = nx;
            if (writer) tok[len] = P.cand[nb + n];
            ++len;
        }
        if (writer) {
            tok[len] = P.node_bonus[nb + n];
            for (int i = len + 1; i <= P.gamma; ++i) tok[i] = -1;
            P.out_accept_len[b] = len;
        }
        s_term = n;
    }
    __syncthreads();
    if (!P.out_residual) return;
    const int n = s_term;
    float *out = P.out_residual + static_cast<long long>(b) * P.V;
    const int x0 = (blockIdx.x * kThreads + threadIdx.x) * 4;
    if (x0 >= P.V) return;
    if (P.scale == 0.f) {
        const int a = P.node_bonus[nb + n];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (x0 + e < P.V) out[x0 + e] = (x0 + e == a) ? 1.f : 0.f;
        return;
    }
    const NodeStats st = P.stats[nb + n];
    const bool internal = n < P.n_internal;
    const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) +
        (nb + n) * P.ld_t * E::kBytes;
    const unsigned char *d_row = reinterpret_cast<const unsigned char *>(P.draft) +
        (static_cast<long long>(b) * P.n_internal + n) * P.ld_d * E::kBytes;
    const float r_t = st.r_t == -INFINITY ? 0.f : st.r_t;
    const float r_d = st.r_d == -INFINITY ? 0.f : st.r_d;
    const float inv_zt = st.z_t > 0.f ? 1.f / st.z_t : 0.f;
    const float cq = (internal && st.z_d > 0.f) ? st.c / st.z_d : 0.f;
    const float inv_s = st.s > 0.f ? 1.f / st.s : 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int x = x0 + e;
        if (x < P.V) {
            float w = ex2f(fmaf(E::load(t_row, x), P.scale, -r_t)) * inv_zt;
            if (internal && cq > 0.f) w = fmaxf(fmaf(-cq, ex2f(fmaf(E::load(d_row, x), P.scale, -r_d)), w), 0.f);
            out[x] = w * inv_s;
        }
    }
}

}  // namespace mcsd
