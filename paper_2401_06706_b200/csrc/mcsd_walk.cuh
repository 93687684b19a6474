// walk_kernel: the walk of Section 3 over the per-node decisions, the endpoint token and the
// residual distribution of the stopping node.
#pragma once

#include "mcsd_common.cuh"

namespace mcsd {

struct WalkParams {
    const void *target;
    const void *draft;
    const int32_t *cand;
    const float *unif;           // may be null at temperature 0
    const int32_t *node_accept;
    int32_t *node_bonus;         // T == 0: read (argmax of every node); T > 0: written in all-nodes mode
    const NodeStats *stats;
    const float2 *leaf_part;
    int32_t *out_accept_len;
    int32_t *out_tokens;
    float *out_residual;  // may be null
    float *node_residual; // [B][n_nodes][V], may be null: where the all-nodes pass leaves each node's distribution
    int32_t *out_path_nodes;  // may be null
    int32_t *status;      // [B]
    long long ld_t, ld_d;
    int32_t n_nodes, n_internal, V, gamma;
    int32_t n_entries;    // per-warp statistics entries a leaf row has (cluster size * warps per CTA)
    int32_t all_nodes;    // 0: one CTA per sequence, walk then endpoint of the stopping node;
                          // 1: one CTA per (sequence, node), endpoint of every node into node_bonus
    int32_t vector_ok;    // logit rows are 16-byte aligned
    float scale;          // log2(e)/T, or 0 for the argmax rule
};

constexpr int kWalkThreads = 1024;
constexpr int kWalkWarps = kWalkThreads / 32;

// One CTA per sequence.  Thread 0 follows the accepted children from the root (Section 3)
// and writes the accepted tokens.  Then the whole CTA forms the distribution the endpoint
// token of the stopping node is drawn from, w(x) = max(p(x) - c q(x), 0) / S with the
// statistics the node kernel left (p alone for a leaf), writes it to out_residual, and
// draws the token by inverse CDF in token order with that node's second uniform:
// warp totals of contiguous runs -> the run holding the quantile -> that warp walks its
// run again, 128 elements at a time.
// NT threads per CTA: 512 (two CTAs per SM) when the vocabulary is at most half the maximum,
// else 1024; a warp's run is at most MCSD_MAX_VOCAB / 32 elements either way.
template <int DT, int NT>
__global__ void __launch_bounds__(NT, NT == 512 ? 2 : 1)
walk_kernel(const __grid_constant__ WalkParams P)
{
    using E = Elem<DT>;
    constexpr int GV = E::kVec;
    __shared__ int s_term, s_len;
    __shared__ int32_t s_acc[MCSD_MAX_NODES], s_tok[MCSD_MAX_NODES];
    constexpr int kW = NT / 32;  // warps
    __shared__ float s_wtot[32];
    __shared__ float s_leaf[2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int b, n;
    if (P.all_nodes) {
        b = blockIdx.x / P.n_nodes;
        n = blockIdx.x - b * P.n_nodes;
    } else {
        b = blockIdx.x;
        n = 0;
    }
    const long long nb = static_cast<long long>(b) * P.n_nodes;
    int32_t *tok = P.out_tokens + static_cast<long long>(b) * (P.gamma + 1);
    int len = 0;
    if (!P.all_nodes) {
        // the tree's decisions and tokens come into shared memory with one parallel load, so
        // that the walk itself is not a chain of dependent global loads
        for (int i = tid; i < P.n_nodes; i += NT) {
            s_acc[i] = P.node_accept[nb + i];
            s_tok[i] = P.cand[nb + i];
        }
        __syncthreads();
        if (tid == 0) {
            // bounded by the depth of the tree even if node_accept were corrupt
            for (int hop = 0; hop < P.gamma; ++hop) {
                const int nx = s_acc[n];
                if (nx <= n || nx >= P.n_nodes) break;
                n = nx;
                tok[len] = s_tok[n];
                if (P.out_path_nodes) P.out_path_nodes[static_cast<long long>(b) * (P.gamma + 1) + len] = n;
                ++len;
            }
            for (int i = len + 1; i <= P.gamma; ++i) tok[i] = -1;
            if (P.out_path_nodes)
                for (int i = len; i <= P.gamma; ++i) P.out_path_nodes[static_cast<long long>(b) * (P.gamma + 1) + i] = -1;
            P.out_accept_len[b] = len;
            s_term = n;
            s_len = len;
        }
        __syncthreads();
        n = s_term;
        len = s_len;
    } else if (P.node_accept[nb + n] >= 0) {
        if (tid == 0) P.node_bonus[nb + n] = -1;  // a walk never stops here
        return;
    }
    float *out = P.all_nodes ? (P.node_residual ? P.node_residual + (nb + n) * P.V : nullptr)
                             : (P.out_residual ? P.out_residual + static_cast<long long>(b) * P.V : nullptr);

    if (P.scale == 0.f) {
        // argmax rule: the endpoint is the target argmax of the stopping node, the
        // distribution is one-hot (all-nodes mode has nothing to add here)
        const int a = P.node_bonus[nb + n];
        if (tid == 0 && !P.all_nodes) tok[len] = a;
        if (out)
            for (int x = tid; x < P.V; x += NT) out[x] = (x == a) ? 1.f : 0.f;
        return;
    }

    // ---- statistics of the stopping node
    const bool internal = n < P.n_internal;
    float r_t, z_t, r_d = 0.f, z_d = 0.f, c = 0.f, S = 1.f;
    if (internal) {
        const NodeStats st = P.stats[nb + n];
        r_t = st.r_t; r_d = st.r_d; z_t = st.z_t; z_d = st.z_d; c = st.c; S = st.s;
    } else {
        if (warp == 0) {
            float2 e = make_float2(-INFINITY, 0.f);
            if (lane < P.n_entries)
                e = P.leaf_part[(static_cast<long long>(b) * (P.n_nodes - P.n_internal) + (n - P.n_internal)) * 32 + lane];
            const float R = warp_max(e.x);
            const float Z = warp_sum(e.y * exp2i(e.x - R));
            if (lane == 0) { s_leaf[0] = R; s_leaf[1] = Z; }
        }
        __syncthreads();
        r_t = s_leaf[0]; z_t = s_leaf[1];
    }
    const bool t_ok = z_t > 0.f && z_t < INFINITY;
    const float r_t0 = r_t == -INFINITY ? 0.f : r_t, r_d0 = r_d == -INFINITY ? 0.f : r_d;
    const float inv_zt = t_ok ? 1.f / z_t : 0.f;
    const float cq = (internal && z_d > 0.f && z_d < INFINITY) ? c / z_d : 0.f;
    const float inv_s = S > 0.f ? 1.f / S : 0.f;
    const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) + (nb + n) * P.ld_t * E::kBytes;
    const unsigned char *d_row = reinterpret_cast<const unsigned char *>(P.draft) +
        (static_cast<long long>(b) * P.n_internal + n) * P.ld_d * E::kBytes;

    // weights of the GV elements starting at x0 (0 past the end of the vocabulary)
    auto weights = [&](int x0, float *w) {
        float t[GV], d[GV];
        if (P.vector_ok && x0 + GV <= P.V) {
            E::unpack(__ldg(reinterpret_cast<const uint4 *>(t_row + static_cast<size_t>(x0) * E::kBytes)), t);
            if (cq > 0.f) E::unpack(__ldg(reinterpret_cast<const uint4 *>(d_row + static_cast<size_t>(x0) * E::kBytes)), d);
        } else {
#pragma unroll
            for (int e = 0; e < GV; ++e) {
                t[e] = x0 + e < P.V ? E::load(t_row, x0 + e) : -INFINITY;
                d[e] = (cq > 0.f && x0 + e < P.V) ? E::load(d_row, x0 + e) : -INFINITY;
            }
        }
#pragma unroll
        for (int e = 0; e < GV; ++e) {
            float v = ex2f(fmaf(t[e], P.scale, -r_t0)) * inv_zt;
            if (cq > 0.f) v = fmaxf(fmaf(-cq, ex2f(fmaf(d[e], P.scale, -r_d0)), v), 0.f);
            w[e] = v;
        }
    };

    // contiguous runs: warp w owns [w * run, (w + 1) * run), walked 32 * GV elements at a time
    constexpr int kStep = 32 * GV;
    const int run = ((P.V + kW - 1) / kW + kStep - 1) / kStep * kStep;
    const int x_lo = warp * run;
    int x_hi = x_lo + run;
    x_hi = x_hi > P.V ? P.V : x_hi;

    // pass 1: the distribution itself, the mass of every run, and per lane the mass of its
    // group in every step of the run (kept for the search below)
    constexpr int kMaxSteps = MCSD_MAX_VOCAB / 32 / kStep;
    float g[kMaxSteps];
    float mass = 0.f;
#pragma unroll
    for (int st = 0; st < kMaxSteps; ++st) {
        g[st] = 0.f;
        const int x0 = x_lo + st * kStep + lane * GV;
        if (x0 < x_hi) {
            float w[GV];
            weights(x0, w);
#pragma unroll
            for (int e = 0; e < GV; ++e) {
                g[st] += w[e];
                if (out && x0 + e < P.V) out[x0 + e] = w[e] * inv_s;
            }
            mass += g[st];
        }
    }
    mass = warp_sum(mass);
    if (lane == 0) s_wtot[warp] = mass;
    __syncthreads();

    // the run that holds the quantile (every warp finds the same one)
    const float u_end = P.unif[2 * (nb + n) + 1];
    const float m = lane < kW ? s_wtot[lane] : 0.f;
    const float total = warp_sum(m);
    const float target = u_end * total;
    const float inc = warp_scan_incl(m, lane);
    const unsigned hit = __ballot_sync(0xffffffffu, m > 0.f && inc > target);
    const unsigned pos = __ballot_sync(0xffffffffu, m > 0.f);
    // (rounding may push the quantile past the end: clamp to the last run with mass)
    const int pick = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : -1);
    int32_t *dst = P.all_nodes ? P.node_bonus + nb + n : tok + len;
    if (pick < 0 || !(total > 0.f)) {
        if (tid == 0) {
            *dst = -1;
            atomicOr(P.status + b, MCSD_STATUS_NO_MASS);
        }
        return;
    }
    if (warp != pick) return;

    // the step of the run that holds the quantile, from the step totals; then the lane and
    // the element inside that step (its weights are formed once more)
    const float tgt = target - __shfl_sync(0xffffffffu, inc - m, pick);
    float tj;
    warp_multi_sum<kMaxSteps>(g, lane, tj);  // lane st * (32 / kMaxSteps) holds the total of step st
    int ps = -1, last_s = -1;
    float runsum = 0.f, ps_before = 0.f;
#pragma unroll
    for (int st = 0; st < kMaxSteps; ++st) {
        const float ms = __shfl_sync(0xffffffffu, tj, st * (32 / kMaxSteps));
        if (ms > 0.f) {
            last_s = st;
            if (ps < 0 && runsum + ms > tgt) { ps = st; ps_before = runsum; }
        }
        runsum += ms;
    }
    // rounding may leave the quantile past the run's own sum: take its last element with mass
    float t2 = tgt - ps_before;
    if (ps < 0) { ps = last_s; t2 = INFINITY; }
    int found = -1;
    if (ps >= 0) {
        float gs = g[0];
#pragma unroll
        for (int st = 1; st < kMaxSteps; ++st) gs = (ps == st) ? g[st] : gs;
        const float gi = warp_scan_incl(gs, lane);
        const unsigned h2 = __ballot_sync(0xffffffffu, gs > 0.f && gi > t2);
        const unsigned p2 = __ballot_sync(0xffffffffu, gs > 0.f);
        if (p2) {
            const int l = h2 ? __ffs(h2) - 1 : 31 - __clz(p2);
            int pe = -1, last = -1;
            if (lane == l) {
                float w[GV];
                weights(x_lo + ps * kStep + lane * GV, w);
                const float rem = t2 - (gi - gs);
                float acc = 0.f;
#pragma unroll
                for (int e = 0; e < GV; ++e) {
                    if (w[e] > 0.f) {
                        acc += w[e];
                        last = e;
                        if (pe < 0 && acc > rem) pe = e;
                    }
                }
                if (pe < 0) pe = last;
            }
            found = __shfl_sync(0xffffffffu, pe < 0 ? -1 : x_lo + ps * kStep + lane * GV + pe, l);
        }
    }
    if (lane == 0) {
        *dst = found;
        if (found < 0) atomicOr(P.status + b, MCSD_STATUS_NO_MASS);
    }
}

}  // namespace mcsd
