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
    int32_t *status;      // [B], written (not accumulated) by the walk of each sequence
    long long ld_t, ld_d;
    int32_t n_nodes, n_internal, V, gamma;
    int32_t n_entries;    // per-warp statistics entries a leaf row has (cluster size * warps per CTA)
    int32_t all_nodes;    // 0: one CTA per sequence, walk then endpoint of the stopping node;
                          // 1: one CTA per (sequence, node), endpoint of every node into node_bonus
    int32_t vector_ok;    // logit rows are 16-byte aligned
    int32_t pdl;          // launched with programmatic stream serialisation: wait for the node stage first
    float scale;          // log2(e)/T, or 0 for the argmax rule
};

constexpr int kWalkThreads = 1024;
constexpr int kWalkWarps = kWalkThreads / 32;

// One CTA per sequence.  Thread 0 follows the accepted children from the root (Section 3),
// writes the accepted tokens and gathers the status bits the node stage left at the nodes of
// the walk (out_status describes the walk, i.e. the nodes the sequential procedure of
// Section 3 evaluates).  Then the whole CTA forms the distribution the endpoint token of the
// stopping node is drawn from, w(x) = max(p(x) - c q(x), 0) / S with the statistics the node
// kernel left (p alone for a leaf).  S, the residual sum that follows the node's last
// rejection, is formed here: a first sweep over the two rows gives the group sums and S and
// leaves the unnormalised weights in out_residual, which a second sweep scales.  If S is
// zero the residual before the last rejection is the one that is kept (status DEGENERATE).
// The token is drawn by inverse CDF in token order with that node's second uniform: totals of
// contiguous runs (one per warp) -> the run holding the quantile -> that warp finds the step,
// the lane and the element from the group sums it kept (the helpers of mcsd_common.cuh).
// NT threads per CTA: 512 (two CTAs per SM) when the vocabulary is at most half the maximum,
// else 1024; a warp's run is at most MCSD_MAX_VOCAB / 32 elements either way.
// CL > 1 (small batches, which leave most SMs idle): a thread-block cluster of CL CTAs works on one
// sequence, so that its 2 V exponentials are spread over CL SMs instead of queueing at the special-
// function unit of one (at batch 1 that queue alone is 2 us per sweep).  The CL * NT / 32 warps of the
// cluster own the runs exactly as the warps of one large CTA would (the results are the same bit for
// bit); every warp sends its run's total into the shared memory of all CTAs, one cluster barrier, and
// every CTA goes on alone.  The walk itself is followed by every CTA; CTA 0 writes it.
// MB: CTAs per SM the register budget is held to.  The clustered form exists with 1 (the compiler then has
// all row loads of a sweep in flight: the fastest form for a handful of sequences) and with 4 (128
// registers: 74 clusters resident at once, for batches up to that).
template <int DT, int NT, int CL = 1, int MB = (NT == 512 ? 2 : 1)>
__global__ void __launch_bounds__(NT, MB)
walk_kernel(const __grid_constant__ WalkParams P)
{
    using E = Elem<DT>;
    static_assert(CL * NT <= 1024, "the cluster's warps are the at most 32 runs of the search");
    constexpr int GV = E::kVec;
    __shared__ int s_term, s_len, s_stat;
    __shared__ int32_t s_acc[MCSD_MAX_NODES], s_tok[MCSD_MAX_NODES];
    // what the node stage left at every node with children, and every node's endpoint uniform: loaded
    // up front in parallel, so that nothing the walk decides has to wait for another trip to memory
    __shared__ NodeStats s_stats[MCSD_MAX_NODES];
    __shared__ float s_uend[MCSD_MAX_NODES];
    constexpr int kW = CL * NT / 32;  // warps (of the whole cluster)
    __shared__ double s_wtot[32];
    __shared__ float s_leaf[2];
    const int crank = CL > 1 ? static_cast<int>(cluster_ctarank()) : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = crank * (NT / 32) + (tid >> 5);   // warp: index in the cluster
    const bool writer = crank == 0;   // the CTA that writes what all CTAs of the cluster compute alike
    const int unit = CL > 1 ? static_cast<int>(blockIdx.x) / CL : static_cast<int>(blockIdx.x);
    int b, n;
    if (P.all_nodes) {
        b = unit / P.n_nodes;
        n = unit - b * P.n_nodes;
    } else {
        b = unit;
        n = 0;
    }
    const long long nb = static_cast<long long>(b) * P.n_nodes;
    int32_t *tok = P.out_tokens + static_cast<long long>(b) * (P.gamma + 1);
    int len = 0;
    if (!P.all_nodes) {
        // the tree's decisions and tokens come into shared memory with one parallel load, so
        // that the walk itself is not a chain of dependent global loads
        // (the caller's inputs first: they do not depend on the node stage, whose results must be
        // complete and visible before anything of them is read)
        for (int i = tid; i < P.n_nodes; i += NT) {
            s_tok[i] = P.cand[nb + i];
            if (P.scale != 0.f) s_uend[i] = P.unif[2 * (nb + i) + 1];
        }
        if (P.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int i = tid; i < P.n_nodes; i += NT) {
            s_acc[i] = P.node_accept[nb + i];
            if (P.scale != 0.f && i < P.n_internal) s_stats[i] = P.stats[nb + i];
        }
        __syncthreads();
        if (tid == 0) {
            int st = 0;
            // bounded by the depth of the tree even if node_accept were corrupt
            for (int hop = 0; hop < P.gamma; ++hop) {
                if (P.scale != 0.f && n < P.n_internal) st |= s_stats[n].status;
                const int nx = s_acc[n];
                if (nx <= n || nx >= P.n_nodes) break;
                n = nx;
                if (writer) {
                    tok[len] = s_tok[n];
                    if (P.out_path_nodes) P.out_path_nodes[static_cast<long long>(b) * (P.gamma + 1) + len] = n;
                }
                ++len;
            }
            if (P.scale != 0.f && n < P.n_internal) st |= s_stats[n].status;
            if (writer) {
                for (int i = len + 1; i <= P.gamma; ++i) tok[i] = -1;
                if (P.out_path_nodes)
                    for (int i = len; i <= P.gamma; ++i) P.out_path_nodes[static_cast<long long>(b) * (P.gamma + 1) + i] = -1;
                P.out_accept_len[b] = len;
            }
            s_term = n;
            s_len = len;
            s_stat = st;
        }
        __syncthreads();
        n = s_term;
        len = s_len;
    } else {
        if (P.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
        if (P.node_accept[nb + n] >= 0) {
            if (tid == 0 && writer) P.node_bonus[nb + n] = -1;  // a walk never stops here
            return;
        }
    }
    float *out = P.all_nodes ? (P.node_residual ? P.node_residual + (nb + n) * P.V : nullptr)
                             : (P.out_residual ? P.out_residual + static_cast<long long>(b) * P.V : nullptr);
    // what thread `tid == 0` or lane 0 of the deciding warp writes at the end of a walk
    auto finish = [&](int token, int extra_bits) {
        if (P.all_nodes) {
            P.node_bonus[nb + n] = token;
        } else {
            tok[len] = token;
            P.status[b] = s_stat | extra_bits;
        }
    };

    if (P.scale == 0.f) {
        // argmax rule: the endpoint is the target argmax of the stopping node, the
        // distribution is one-hot (all-nodes mode has nothing to add here)
        const int a = P.node_bonus[nb + n];
        if (tid == 0 && writer && !P.all_nodes) finish(a, 0);
        if (out)
            for (int x = crank * NT + tid; x < P.V; x += CL * NT) out[x] = (x == a) ? 1.f : 0.f;
        return;
    }

    // ---- statistics of the stopping node
    const bool internal = n < P.n_internal;
    float r_t, z_t, r_d = 0.f, z_d = 0.f, c = 0.f, c_prev = 0.f;
    if (internal) {
        const NodeStats st = P.all_nodes ? P.stats[nb + n] : s_stats[n];
        r_t = st.r_t; r_d = st.r_d; z_t = st.z_t; z_d = st.z_d; c = st.c; c_prev = st.c_prev;
    } else {
        if ((tid >> 5) == 0) {
            const float2 *part = P.leaf_part +
                (static_cast<long long>(b) * (P.n_nodes - P.n_internal) + (n - P.n_internal)) * kLeafEntries;
            float2 e = make_float2(-INFINITY, 0.f);
            if (lane < P.n_entries) e = part[lane];
            const float R = warp_max(e.x);
            const float Z = warp_sum(e.y * exp2i(e.x - R));
            if (lane == 0) { s_leaf[0] = R; s_leaf[1] = Z; }
        }
        __syncthreads();
        r_t = s_leaf[0]; z_t = s_leaf[1];
    }
    const bool t_ok = z_t > 0.f && z_t < INFINITY;
    const bool d_ok = internal && z_d > 0.f && z_d < INFINITY;
    const float r_t0 = r_t == -INFINITY ? 0.f : r_t, r_d0 = r_d == -INFINITY ? 0.f : r_d;
    // p(x) = et(x) / Z_t and q(x) = ed(x) / Z_d with et, ed the exponentials against the rows'
    // references: max(p - c q, 0) = max(et - kappa ed, 0) / Z_t, kappa = c Z_t / Z_d
    // (the form the node kernel sums, so that equal rows cancel exactly here as they do there)
    const float dq = (t_ok && d_ok) ? z_t / z_d : 0.f;
    const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) + (nb + n) * P.ld_t * E::kBytes;
    const unsigned char *d_row = reinterpret_cast<const unsigned char *>(P.draft) +
        (static_cast<long long>(b) * P.n_internal + n) * P.ld_d * E::kBytes;

    // contiguous runs: warp w owns [w * run, (w + 1) * run), walked 32 * GV elements at a time
    constexpr int kStep = 32 * GV;
    constexpr int kMaxSteps = MCSD_MAX_VOCAB / 32 / kStep;
    const int run = ((P.V + kW - 1) / kW + kStep - 1) / kStep * kStep;
    const int x_lo = warp * run;
    int x_hi = x_lo + run;
    x_hi = x_hi > P.V ? P.V : x_hi;

    // whole 16-byte stores where the row of `out` allows it
    const bool out_vec = out && (reinterpret_cast<uintptr_t>(out) % 16 == 0);
    float kappa = fminf(c * dq, 3.0e38f);
    int extra_bits = 0;
    float g[kMaxSteps];
    double tgt = 0.0;
    int pick = -1;
    // weights of the GV elements starting at x0 (0 past the end of the vocabulary), times Z_t
    auto weights = [&](int x0, float *w) {
        float t[GV], d[GV];
        if (P.vector_ok && x0 + GV <= P.V) {
            E::unpack(ldg_v4(t_row + static_cast<size_t>(x0) * E::kBytes), t);
            if (kappa > 0.f) E::unpack(ldg_v4(d_row + static_cast<size_t>(x0) * E::kBytes), d);
        } else {
#pragma unroll
            for (int e = 0; e < GV; ++e) {
                t[e] = x0 + e < P.V ? E::load(t_row, x0 + e) : -INFINITY;
                d[e] = (kappa > 0.f && x0 + e < P.V) ? E::load(d_row, x0 + e) : -INFINITY;
            }
        }
#pragma unroll
        for (int e = 0; e < GV; ++e) {
            float v = t_ok ? ex2f(fmaf(t[e], P.scale, -r_t0)) : 0.f;
            if (kappa > 0.f) v = fmaxf(fmaf(-kappa, ex2f(fmaf(d[e], P.scale, -r_d0)), v), 0.f);
            w[e] = v;
        }
    };
    const float u_end = P.all_nodes ? P.unif[2 * (nb + n) + 1] : s_uend[n];
    // at most two attempts: the residual after the last rejection and, if that one has no mass,
    // the one before it
#pragma unroll 1
    for (int attempt = 0; attempt < 2; ++attempt) {
        // sweep 1: unnormalised weights (left in `out`), per lane the mass of its group in every
        // step of the run (kept for the search below), per warp the mass of its run
#pragma unroll
        for (int st = 0; st < kMaxSteps; ++st) {
            g[st] = 0.f;
            const int x0 = x_lo + st * kStep + lane * GV;
            if (x0 < x_hi) {
                float w[GV];
                weights(x0, w);
#pragma unroll
                for (int e = 0; e < GV; ++e) g[st] += w[e];
                if (out_vec && x0 + GV <= P.V) {
#pragma unroll
                    for (int e = 0; e < GV; e += 4)
                        *reinterpret_cast<float4 *>(out + x0 + e) = make_float4(w[e], w[e + 1], w[e + 2], w[e + 3]);
                } else if (out) {
#pragma unroll
                    for (int e = 0; e < GV; ++e)
                        if (x0 + e < P.V) out[x0 + e] = w[e];
                }
            }
        }
        const double mass = run_total<kMaxSteps>(g);
        if constexpr (CL > 1) {
            // (second attempt: every CTA has read the totals of the first before they are overwritten)
            if (attempt) cluster_sync_all();
            if (lane < CL) {
                const uint32_t dst = map_to_rank(smem_u32(&s_wtot[warp]), static_cast<uint32_t>(lane));
                asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(dst), "d"(mass) : "memory");
            }
            cluster_sync_all();   // release / acquire: the totals of all CTAs are in this CTA's shared memory
        } else {
            __syncthreads();   // (second attempt: everybody has read the totals of the first)
            if (lane == 0) s_wtot[warp] = mass;
            __syncthreads();
        }
        // the run that holds the quantile (every warp finds the same one)
        pick = pick_run(lane < kW ? s_wtot[lane] : 0.0, u_end, lane, tgt);
        if (pick >= 0 || !internal) break;
        // a node with children whose residual has no mass: the update that led to it is void
        extra_bits |= MCSD_STATUS_DEGENERATE;
        if (attempt == 1 || !(c != c_prev)) break;
        kappa = fminf(c_prev * dq, 3.0e38f);
    }
    if (pick < 0) {
        if (tid == 0 && writer) finish(-1, extra_bits | MCSD_STATUS_NO_MASS);
        return;   // (`out` keeps the unnormalised weights: zeros or NaN, there is no distribution)
    }
    // sweep 2: every thread scales what it wrote by 1 / S
    if (out) {
        double tot = lane < kW ? s_wtot[lane] : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
        const float inv_s = static_cast<float>(1.0 / tot);
#pragma unroll 1
        for (int st = 0; st < kMaxSteps; ++st) {
            const int x0 = x_lo + st * kStep + lane * GV;
            if (x0 < x_hi) {
                if (out_vec && x0 + GV <= P.V) {
#pragma unroll
                    for (int e = 0; e < GV; e += 4) {
                        float4 v = *reinterpret_cast<float4 *>(out + x0 + e);
                        v.x *= inv_s; v.y *= inv_s; v.z *= inv_s; v.w *= inv_s;
                        *reinterpret_cast<float4 *>(out + x0 + e) = v;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < GV; ++e)
                        if (x0 + e < P.V) out[x0 + e] *= inv_s;
                }
            }
        }
    }
    if (warp != pick) return;

    // the step of the run and the lane that hold the quantile, then the element inside that
    // lane's group (its weights are formed once more)
    int ps, l, found = -1;
    float rem;
    const float tj = step_totals<kMaxSteps>(g, lane);
    if (search_run<kMaxSteps>(g, tj, tgt, lane, ps, l, rem)) {
        int pe = -1;
        if (lane == l) {
            float w[GV];
            weights(x_lo + ps * kStep + lane * GV, w);
            pe = pick_element<GV>(w, rem);
        }
        found = __shfl_sync(0xffffffffu, pe < 0 ? -1 : x_lo + ps * kStep + lane * GV + pe, l);
    }
    if (lane == 0) finish(found, extra_bits | (found < 0 ? MCSD_STATUS_NO_MASS : 0));
}

}  // namespace mcsd
