// argmax_kernel (T == 0): the greedy rule of Section 4.5, one CTA per target row.
#pragma once

#include "mcsd_common.cuh"

namespace mcsd {

struct ArgmaxParams {
    const void *target;
    const int32_t *cand;
    int32_t *node_accept;
    int32_t *node_bonus;
    float *node_ratio;  // may be null
    long long ld_t;
    int32_t n_nodes, n_internal, V, n_rows;
    int32_t vector_ok;  // rows are 16-byte aligned
    // path mode, as in NodeParams: n_rows = sequences, item b works on node path_cur[b]
    const int32_t *path_cur;
    int32_t *path_next;
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
    for (int item = blockIdx.x; item < P.n_rows; item += gridDim.x) {
        int row = item;
        if (P.path_cur) {
            const int pn = __ldg(P.path_cur + item);
            if (pn < 0) {  // this walk ended at an earlier level
                if (tid == 0) P.path_next[item] = -1;
                continue;
            }
            row = item * P.n_nodes + pn;
        }
        const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) +
            static_cast<long long>(row) * P.ld_t * E::kBytes;
        float best = -INFINITY;
        int best_i = 0x7fffffff;
        // strict '>' keeps the lowest index inside a thread (indices ascend); NaN never wins
        if (P.vector_ok) {
            const int n_vec = P.V / VEC;
            const uint4 *src = reinterpret_cast<const uint4 *>(t_row);
            // eight predicated loads in flight per thread, the ragged end of the row included:
            // where the predicate is off the vector is -inf, which never wins
            for (int v = tid; v < n_vec; v += 8 * kThreads) {
                uint4 r[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    r[u] = ld_v4_if(src + v + u * kThreads, v + u * kThreads < n_vec, E::kNegInfWord);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float f[VEC];
                    E::unpack(r[u], f);
#pragma unroll
                    for (int e = 0; e < VEC; ++e)
                        if (f[e] > best) { best = f[e]; best_i = (v + u * kThreads) * VEC + e; }
                }
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
                if (P.path_next) P.path_next[item] = acc;
            }
        }
        __syncthreads();
    }
}

}  // namespace mcsd
