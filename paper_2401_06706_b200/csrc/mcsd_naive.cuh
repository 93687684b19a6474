// naive_kernel: the sample-and-match baseline of the ablation (Section 4.5), one CTA per sequence.
#pragma once

#include "mcsd_common.cuh"

namespace mcsd {

struct NaiveParams {
    const void *target;
    const int32_t *cand;
    const float *unif;
    int32_t *node_accept;   // written for the visited nodes
    int32_t *out_accept_len;
    int32_t *out_tokens;
    float *out_residual;    // may be null
    int32_t *out_path_nodes;  // may be null
    int32_t *status;
    long long ld_t;
    int32_t n_nodes, n_internal, V, gamma;
    int32_t vector_ok;
    float scale;            // log2(e)/T
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
};

// Multi-candidate naive sampling, the baseline that Section 4.5 and Appendix C compare
// with: at the node the walk stands on, draw x from the target distribution (inverse CDF
// with the node's second uniform); if a child carries x move to the first such child,
// otherwise x is the endpoint token.  The draws depend on one another level by level and
// only visited nodes matter, so one CTA per sequence walks its tree: per level one target
// row is read (maximum, then weights with run / step / lane sums kept for the search).
template <int DT>
__global__ void __launch_bounds__(kWalkThreads)
naive_kernel(const __grid_constant__ NaiveParams P)
{
    using E = Elem<DT>;
    constexpr int GV = E::kVec;
    constexpr int kStep = 32 * GV;
    constexpr int kMaxSteps = MCSD_MAX_VOCAB / kWalkWarps / kStep;
    __shared__ double s_wtot[kWalkWarps];
    __shared__ float s_red[kWalkWarps];
    __shared__ int s_pick, s_next;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const long long nb = static_cast<long long>(b) * P.n_nodes;
    int32_t *tok = P.out_tokens + static_cast<long long>(b) * (P.gamma + 1);
    const int run = ((P.V + kWalkWarps - 1) / kWalkWarps + kStep - 1) / kStep * kStep;
    const int x_lo = warp * run;
    int x_hi = x_lo + run;
    x_hi = x_hi > P.V ? P.V : x_hi;

    int n = 0, len = 0, x = -1;
    float ref0 = 0.f, total = 0.f;
    const unsigned char *row = nullptr;
    auto load_group = [&](int x0, float *v) {
        if (P.vector_ok && x0 + GV <= P.V) {
            E::unpack(ldg_v4(row + static_cast<size_t>(x0) * E::kBytes), v);
        } else {
#pragma unroll
            for (int e = 0; e < GV; ++e) v[e] = x0 + e < P.V ? E::load(row, x0 + e) : -INFINITY;
        }
    };
    auto weights = [&](int x0, float *w) {
        float v[GV];
        load_group(x0, v);
#pragma unroll
        for (int e = 0; e < GV; ++e) w[e] = ex2f(fmaf(v[e], P.scale, -ref0));
    };
    for (int hop = 0; hop <= P.gamma; ++hop) {  // bounded by the depth of the tree
        row = reinterpret_cast<const unsigned char *>(P.target) + (nb + n) * P.ld_t * E::kBytes;
        // reference of the row, then weights and their partial sums
        float mx = -INFINITY;
        for (int x0 = x_lo + lane * GV; x0 < x_hi; x0 += kStep) {
            float v[GV];
            load_group(x0, v);
#pragma unroll
            for (int e = 0; e < GV; ++e) mx = fmaxf(mx, v[e]);
        }
        mx = warp_max(mx);
        if (lane == 0) s_red[warp] = mx;
        __syncthreads();
        const float ref = int_ref(warp_max(s_red[lane]) * P.scale);
        ref0 = ref == -INFINITY ? 0.f : ref;
        float g[kMaxSteps];
#pragma unroll
        for (int st = 0; st < kMaxSteps; ++st) {
            g[st] = 0.f;
            const int x0 = x_lo + st * kStep + lane * GV;
            if (x0 < x_hi) {
                float w[GV];
                weights(x0, w);
#pragma unroll
                for (int e = 0; e < GV; ++e) g[st] += w[e];
            }
        }
        const double mass = run_total<kMaxSteps>(g);
        if (lane == 0) s_wtot[warp] = mass;
        if (tid == 0) s_pick = -1;
        __syncthreads();
        // the draw: run, step, lane, element
        const float u = P.unif[2 * (nb + n) + 1];
        double tgt = 0.0;
        const double m = s_wtot[lane];
        const int pick = pick_run(m, u, lane, tgt);
        {
            double t = m;   // the row's mass, for the distribution written at the end
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            total = static_cast<float>(t);
        }
        if (pick >= 0 && warp == pick) {
            int ps, l;
            float rem;
            const float tj = step_totals<kMaxSteps>(g, lane);
            if (search_run<kMaxSteps>(g, tj, tgt, lane, ps, l, rem) && lane == l) {
                const int x0 = x_lo + ps * kStep + lane * GV;
                float w[GV];
                weights(x0, w);
                const int pe = pick_element<GV>(w, rem);
                if (pe >= 0) s_pick = x0 + pe;
            }
        }
        __syncthreads();
        x = s_pick;
        // does a child carry x?
        if (warp == 0) {
            const int k = (x >= 0 && n < P.n_internal) ? P.child_count[n] : 0;
            const int first = P.child_first[n];
            int t = -2;
            if (lane < k) t = P.cand[nb + first + lane];
            const unsigned match = __ballot_sync(0xffffffffu, lane < k && t == x);
            if (lane == 0) {
                s_next = match ? first + __ffs(match) - 1 : -1;
                P.node_accept[nb + n] = s_next;
            }
        }
        __syncthreads();
        const int nx = s_next;
        if (nx <= n || nx >= P.n_nodes) break;
        if (tid == 0) {
            tok[len] = x;
            if (P.out_path_nodes) P.out_path_nodes[static_cast<long long>(b) * (P.gamma + 1) + len] = nx;
        }
        ++len;
        n = nx;
    }
    if (tid == 0) {
        tok[len] = x;
        for (int i = len + 1; i <= P.gamma; ++i) tok[i] = -1;
        if (P.out_path_nodes)
            for (int i = len; i <= P.gamma; ++i) P.out_path_nodes[static_cast<long long>(b) * (P.gamma + 1) + i] = -1;
        P.out_accept_len[b] = len;
        P.status[b] = x < 0 ? MCSD_STATUS_NO_MASS : 0;   // written, not accumulated: nothing clears it beforehand
    }
    if (P.out_residual) {
        // the distribution the endpoint token was drawn from: the stopping node's p
        float *out = P.out_residual + static_cast<long long>(b) * P.V;
        const float inv = total > 0.f ? 1.f / total : 0.f;
        for (int x0 = x_lo + lane * GV; x0 < x_hi; x0 += kStep) {
            float w[GV];
            weights(x0, w);
#pragma unroll
            for (int e = 0; e < GV; ++e)
                if (x0 + e < P.V) out[x0 + e] = w[e] * inv;
        }
    }
}

}  // namespace mcsd
