// Verification with the vocabulary split over several devices (a tensor-parallel LM head that
// leaves the logits column-split, as the two-GPU setup of Section 4.1 would): every shard holds
// columns [col_begin, col_begin + n_cols) of both logit tensors.
//
// The node kernel already splits a row over the warps of a thread-block cluster and combines one
// float4 per warp through shared memory.  Here the same per-warp values ("entries", one per run of
// 32 * EPT columns) are written to global memory instead, the caller gathers the entries of all
// shards with a collective of its own, and a small kernel takes the decisions of Algorithm 1 /
// Algorithm 2 from the gathered entries, exactly as the cluster's leader warp does.  Rounds are
// level-synchronous: round 0 the softmax statistics of every node, then one round per rejection
// that is followed by another test.  Nothing stays on chip between rounds, so a later round reads
// the rows of the nodes that need it again.  Because runs, lanes and the order of every sum are
// those of the node kernel, the decisions are the same bit for bit.
#pragma once

#include "mcsd_common.cuh"

namespace mcsd {

struct ShardParams {
    const void *target;      // this shard's columns: [B][n_nodes][ld_t]
    const void *draft;       // [B][n_internal][ld_d]
    const int32_t *cand;     // [B][n_nodes] (replicated on every shard)
    const float *unif;       // [B][n_nodes][2] (replicated)
    long long ld_t, ld_d;
    int32_t B, n_nodes, n_internal, V;
    int32_t col_begin, n_cols;   // global column range of this shard
    int32_t eps;                 // entries (runs) of this shard
    int32_t entry_begin;         // global index of this shard's first entry
    int32_t n_entries;           // entries of the whole vocabulary (<= 32)
    int32_t n_shards, mode, round, gamma;
    int32_t vector_ok;
    float scale, scale_lo;
    // per node, replicated on every shard (written by the decide kernel)
    float4 *act;             // [B*n_nodes] (R_t, R_d, 1/Z_t, Z_t/Z_d)
    float2 *req;             // [B*n_nodes] (more, c_try)
    float *s_hist;           // [B*n_nodes][MCSD_MAX_CHILDREN] residual sums of the rounds so far
    int32_t *node_accept;    // [B*n_nodes]
    float *node_ratio;       // may be null
    NodeStats *stats;        // [B*n_nodes]
    // exchanged buffers
    float4 *part_out;        // this shard's entries of the round: [B*n_nodes][eps_max]
    float2 *cval_out;        // this shard's candidate logits: [B*n_nodes] (t, d), 0 where the token is elsewhere
    const float4 *part_all;  // gathered entries of this round: [n_shards][B*n_nodes][eps_max]
    const float4 *stats_all; // gathered entries of round 0 (kept by the caller for the endpoint stage)
    const float2 *cval_all;  // gathered: [n_shards][B*n_nodes]
    int32_t eps_max;         // entries per shard in the gathered layout (the largest shard's)
    // endpoint stage
    double *tot_out;         // [B][eps_max] mass of every run of the stopping node's residual
    const double *tot_all;   // gathered: [n_shards][B][eps_max]
    float *out_residual;     // this shard's columns: [B][n_cols], may be null
    int32_t *out_accept_len, *out_tokens, *out_status, *out_path_nodes;
    int32_t *endpoint_part;  // [B] endpoint token if it lies in this shard, else -1
    int32_t *retry;          // [B] 1: the residual after the last rejection had no mass, use the one before
    int32_t attempt;         // 0 / 1 (see retry)
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
    int16_t parent[MCSD_MAX_NODES];
};

constexpr int kShardThreads = 128;

// One run of one row -> registers, exponentiated against the run's own integer reference, in the
// element-to-lane mapping and summation order of the node kernel: lane l owns the 16-byte groups
// j * 32 + l of the run.  row: first column of the run; n_valid: columns of the run that exist.
template <int DT, int EPT>
__device__ __forceinline__ void run_exponentials(const unsigned char *row, int n_valid, bool vector_ok, float scale, int lane,
                                                 f32x2 (&v)[EPT / 2], float &ref, float &z)
{
    using E = Elem<DT>;
    constexpr int GV = E::kVec, NG = EPT / GV;
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        const int x = (j * 32 + lane) * GV;
        float f[GV];
        if (vector_ok && x + GV <= n_valid) {
            E::unpack(ldg_v4(row + static_cast<size_t>(x) * E::kBytes), f);
        } else {
#pragma unroll
            for (int e = 0; e < GV; ++e) f[e] = (x + e < n_valid) ? E::load(row, x + e) : -INFINITY;
        }
#pragma unroll
        for (int e = 0; e < GV; e += 2) v[(j * GV + e) / 2] = pack2(f[e], f[e + 1]);
    }
    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
    for (int p = 0; p < EPT / 2; p += 2) {
        m0 = max3(m0, v[p].x, v[p].y);
        m1 = max3(m1, v[p + 1].x, v[p + 1].y);
    }
    ref = int_ref(warp_max(fmaxf(m0, m1)) * scale);
    const float r0 = (ref == -INFINITY) ? 0.f : ref;
    const f32x2 scale2 = pack2(scale, scale), nref2 = pack2(-r0, -r0);
    f32x2 z0 = pack2(0.f, 0.f), z1 = z0;
#pragma unroll
    for (int p = 0; p < EPT / 2; p += 2) {
        const f32x2 x01 = fma2(v[p], scale2, nref2), x23 = fma2(v[p + 1], scale2, nref2);
        v[p] = pack2(ex2f(x01.x), ex2f(x01.y));
        v[p + 1] = pack2(ex2f(x23.x), ex2f(x23.y));
        z0 = add2(z0, v[p]);
        z1 = add2(z1, v[p + 1]);
    }
    const f32x2 zz = add2(z0, z1);
    z = zz.x + zz.y;
}

// Round 0: softmax statistics of every run of every row of this shard, one warp per (node, run).
// Round r >= 1: the residual sum of every run of the nodes that asked for one.
template <int DT, int EPT>
__global__ void __launch_bounds__(kShardThreads)
shard_partials_kernel(const __grid_constant__ ShardParams P)
{
    using E = Elem<DT>;
    constexpr int RUN = 32 * EPT;
    const int lane = threadIdx.x & 31;
    const long long n_items = static_cast<long long>(P.B) * P.n_nodes * P.eps;
    const long long warp_id = (static_cast<long long>(blockIdx.x) * kShardThreads + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * kShardThreads) >> 5;
    for (long long item = warp_id; item < n_items; item += n_warps) {
        const long long node_idx = item / P.eps;
        const int e = static_cast<int>(item - node_idx * P.eps);
        const int b = static_cast<int>(node_idx / P.n_nodes), n = static_cast<int>(node_idx - static_cast<long long>(b) * P.n_nodes);
        const bool internal = n < P.n_internal;
        if (P.round > 0 && (!internal || P.req[node_idx].x == 0.f)) continue;
        int n_valid = P.n_cols - e * RUN;
        n_valid = n_valid > RUN ? RUN : n_valid;
        const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) +
            (node_idx * P.ld_t + static_cast<long long>(e) * RUN) * E::kBytes;
        f32x2 tv[EPT / 2];
        float rt, zt;
        run_exponentials<DT, EPT>(t_row, n_valid, P.vector_ok != 0, P.scale, lane, tv, rt, zt);
        if (!internal) {
            const float st = warp_sum(zt);
            if (lane == 0) P.part_out[node_idx * P.eps_max + e] = make_float4(rt, st, -INFINITY, 0.f);
            continue;
        }
        const unsigned char *d_row = reinterpret_cast<const unsigned char *>(P.draft) +
            ((static_cast<long long>(b) * P.n_internal + n) * P.ld_d + static_cast<long long>(e) * RUN) * E::kBytes;
        f32x2 dv[EPT / 2];
        float rd, zd;
        run_exponentials<DT, EPT>(d_row, n_valid, P.vector_ok != 0, P.scale, lane, dv, rd, zd);
        if (P.round == 0) {
            const float st = warp_sum(zt), sd = warp_sum(zd);
            if (lane == 0) P.part_out[node_idx * P.eps_max + e] = make_float4(rt, st, rd, sd);
            continue;
        }
        // the residual sum max(p - c q, 0) of this run for the c the decide kernel asked for
        const float4 st4 = P.act[node_idx];
        const float c_f = P.req[node_idx].y;
        const float a = exp2i(rt - st4.x) * st4.z;
        float b_over_a = 0.f;
        if (a > 0.f && st4.w > 0.f && rd != -INFINITY) b_over_a = exp2i((rd - st4.y) - (rt - st4.x)) * st4.w;
        const float kappa = fminf(c_f * b_over_a, 3.0e38f);
        const f32x2 nk2 = pack2(-kappa, -kappa);
        f32x2 s0 = pack2(0.f, 0.f), s1 = s0;
#pragma unroll
        for (int p = 0; p < EPT / 2; p += 2) {
            const f32x2 x01 = fma2(dv[p], nk2, tv[p]);
            const f32x2 x23 = fma2(dv[p + 1], nk2, tv[p + 1]);
            s0 = add2(s0, pack2(fmaxf(x01.x, 0.f), fmaxf(x01.y, 0.f)));
            s1 = add2(s1, pack2(fmaxf(x23.x, 0.f), fmaxf(x23.y, 0.f)));
        }
        const f32x2 t = add2(s0, s1);
        const float part = warp_sum((t.x + t.y) * a);
        if (lane == 0) P.part_out[node_idx * P.eps_max + e] = make_float4(part, 0.f, 0.f, 0.f);
    }
}

// The candidates' own logits: the shard that holds column x of a candidate token writes the pair
// (target logit, draft logit) of the PARENT's rows, every other shard writes zeros, so that the sum
// over shards is the pair itself.
template <int DT>
__global__ void shard_candidates_kernel(const __grid_constant__ ShardParams P)
{
    using E = Elem<DT>;
    const long long total = static_cast<long long>(P.B) * P.n_nodes;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int b = static_cast<int>(i / P.n_nodes), n = static_cast<int>(i - static_cast<long long>(b) * P.n_nodes);
        float2 v = make_float2(0.f, 0.f);
        if (n > 0) {
            const int x = P.cand[i], p = P.parent[n];
            if (x >= P.col_begin && x < P.col_begin + P.n_cols && x < P.V) {
                const int xl = x - P.col_begin;
                v.x = E::load(reinterpret_cast<const unsigned char *>(P.target) +
                              (static_cast<long long>(b) * P.n_nodes + p) * P.ld_t * E::kBytes, xl);
                v.y = E::load(reinterpret_cast<const unsigned char *>(P.draft) +
                              (static_cast<long long>(b) * P.n_internal + p) * P.ld_d * E::kBytes, xl);
            }
        }
        P.cval_out[i] = v;
    }
}

// Decisions from the gathered entries, one warp per node with children; every shard runs this
// on the same inputs and obtains the same results.  The warp replays the node's tests from the
// first candidate with the residual sums gathered so far; when it needs a sum it does not have
// yet it asks for it (req = (1, c)) and the next round supplies it.
__global__ void __launch_bounds__(kShardThreads)
shard_decide_kernel(const __grid_constant__ ShardParams P)
{
    const int lane = threadIdx.x & 31;
    const long long n_int_items = static_cast<long long>(P.B) * P.n_internal;
    const long long warp_id = (static_cast<long long>(blockIdx.x) * kShardThreads + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * kShardThreads) >> 5;
    const long long n_all = static_cast<long long>(P.B) * P.n_nodes;
    for (long long item = warp_id; item < n_int_items; item += n_warps) {
        const int b = static_cast<int>(item / P.n_internal), n = static_cast<int>(item - static_cast<long long>(b) * P.n_internal);
        const long long node_idx = static_cast<long long>(b) * P.n_nodes + n;
        if (P.round > 0 && P.req[node_idx].x == 0.f) continue;   // decided in an earlier round
        const int k = P.child_count[n], first = P.child_first[n];
        // entry `lane` of the round, in vocabulary order (shard-major)
        auto entry = [&](float4 identity) -> float4 {
            if (lane >= P.n_entries) return identity;
            int s = 0, i = lane;
            // shards hold eps_max entries each, the last one possibly fewer
            s = lane / P.eps_max;
            i = lane - s * P.eps_max;
            return P.part_all[(static_cast<long long>(s) * n_all + node_idx) * P.eps_max + i];
        };
        if (P.round > 0) {
            const float4 ent = entry(make_float4(0.f, 0.f, 0.f, 0.f));
            const float S_new = warp_sum(ent.x);
            if (lane == 0) P.s_hist[node_idx * MCSD_MAX_CHILDREN + (P.round - 1)] = S_new;
            __syncwarp();
        }
        int status_bits = 0;
        // ---- statistics (formed again in every round from the entries of round 0, which the caller keeps)
        float R_t, R_d, Z_t, Z_d;
        {
            float4 ent;
            if (P.round == 0) {
                ent = entry(make_float4(-INFINITY, 0.f, -INFINITY, 0.f));
                R_t = warp_max(ent.x); R_d = warp_max(ent.z);
                Z_t = warp_sum(ent.y * exp2i(ent.x - R_t));
                Z_d = warp_sum(ent.w * exp2i(ent.z - R_d));
                if (lane == 0) *reinterpret_cast<float4 *>(&P.stats[node_idx]) = make_float4(R_t, R_d, Z_t, Z_d);
            } else {
                const float4 st = *reinterpret_cast<const float4 *>(&P.stats[node_idx]);
                R_t = st.x; R_d = st.y; Z_t = st.z; Z_d = st.w;
            }
        }
        const bool t_ok = Z_t > 0.f && Z_t < INFINITY, d_ok = Z_d > 0.f && Z_d < INFINITY;
        if (!t_ok || !d_ok) status_bits |= MCSD_STATUS_DEGENERATE;
        double K = static_cast<double>(Z_t) * static_cast<double>(Z_d), Wk = K;
        double px = 0.0, qx = 0.0;
        int my_tok = -1;
        float u_acc = 2.f;
        if (lane < k) {
            const long long ci = static_cast<long long>(b) * P.n_nodes + first + lane;
            my_tok = P.cand[ci];
            u_acc = fminf(P.unif[2 * ci], 1.f);
            if (my_tok >= 0 && my_tok < P.V && t_ok && d_ok) {
                float2 lv = make_float2(0.f, 0.f);
                for (int s = 0; s < P.n_shards; ++s) {
                    const float2 x = P.cval_all[static_cast<long long>(s) * n_all + ci];
                    lv.x += x.x; lv.y += x.y;
                }
                int int_t, int_d;
                const float frac_t = split_exp2(lv.x, P.scale, P.scale_lo, int_t);
                const float frac_d = split_exp2(lv.y, P.scale, P.scale_lo, int_d);
                px = static_cast<double>(frac_t) * exp2i_d(int_t - static_cast<int>(R_t)) * static_cast<double>(Z_d);
                qx = static_cast<double>(frac_d) * exp2i_d(int_d - static_cast<int>(R_d)) * static_cast<double>(Z_t);
            }
        }
        // ---- the tests, replayed from the first candidate
        double c = 0.0, S = 1.0, c_try = 0.0;
        float c_prev = 0.f;
        int accepted = -1, used = 0, more = 0;
        for (int i = 0; i < k; ++i) {
            const int xi = __shfl_sync(0xffffffffu, my_tok, i);
            const double ui = static_cast<double>(__shfl_sync(0xffffffffu, u_acc, i));
            const double pxi = __shfl_sync(0xffffffffu, px, i), qxi = __shfl_sync(0xffffffffu, qx, i);
            const bool valid = xi >= 0 && xi < P.V;
            if (!valid) status_bits |= MCSD_STATUS_BAD_TOKEN;
            const bool dup = P.mode == 1 && (__ballot_sync(0xffffffffu, lane < i && my_tok == xi) != 0u);
            const bool zero_q = !valid || dup || !(qxi > 0.0) || !(Wk > 0.0);
            double Pn = pxi - c * qxi;
            Pn = Pn > 0.0 ? Pn : 0.0;
            const bool accept = !zero_q && ui * S * qxi * K <= Pn * Wk;
            if (P.node_ratio && lane == 0)
                P.node_ratio[static_cast<long long>(b) * P.n_nodes + first + i] =
                    zero_q ? -1.f : static_cast<float>((Pn / S) / (qxi * K / Wk));
            if (accept) { accepted = first + i; break; }
            c_try = c;
            if (Wk > 0.0) c_try = (P.mode == 1) ? c + S * K / Wk : c + S;
            if (P.mode == 1 && !zero_q) { Wk -= qxi; if (!(Wk > 0.0)) Wk = 0.0; }
            if (i + 1 >= k) { c_prev = static_cast<float>(c); c = c_try; break; }
            // the residual sum that follows this rejection: known from an earlier round, or asked for now
            if (used >= P.round) { more = 1; break; }
            const float S_new = P.s_hist[node_idx * MCSD_MAX_CHILDREN + used];
            ++used;
            // (the sum was formed for static_cast<float>(c_try), as the node kernel does)
            if (S_new > 0.f) { c = c_try; S = static_cast<double>(S_new); }
            else status_bits |= MCSD_STATUS_DEGENERATE;
        }
        if (lane == 0) {
            P.req[node_idx] = make_float2(more ? 1.f : 0.f, static_cast<float>(c_try));
            if (P.round == 0)
                P.act[node_idx] = make_float4(R_t, R_d, t_ok ? 1.f / Z_t : 0.f, (t_ok && d_ok) ? Z_t / Z_d : 0.f);
            if (!more) {
                P.node_accept[node_idx] = accepted;
                reinterpret_cast<float4 *>(&P.stats[node_idx])[1] =
                    make_float4(static_cast<float>(c), c_prev, __int_as_float(status_bits), 0.f);
            }
        }
    }
}

// Endpoint stage, first half: one warp per (sequence, run of this shard).  The warp follows the
// walk of its sequence (node_accept is the same on every shard), forms the unnormalised residual
// of the stopping node on its run, leaves it in out_residual and writes the run's mass.
template <int DT, int EPT>
__global__ void __launch_bounds__(kShardThreads)
shard_endpoint_kernel(const __grid_constant__ ShardParams P)
{
    using E = Elem<DT>;
    constexpr int GV = E::kVec, RUN = 32 * EPT, kStep = 32 * GV, S = RUN / kStep;
    const int lane = threadIdx.x & 31;
    const long long n_items = static_cast<long long>(P.B) * P.eps;
    const long long warp_id = (static_cast<long long>(blockIdx.x) * kShardThreads + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * kShardThreads) >> 5;
    for (long long item = warp_id; item < n_items; item += n_warps) {
        const int b = static_cast<int>(item / P.eps), e = static_cast<int>(item - static_cast<long long>(b) * P.eps);
        if (P.attempt == 1 && P.retry[b] == 0) continue;
        const long long nb = static_cast<long long>(b) * P.n_nodes;
        int n = 0;
        for (int hop = 0; hop < P.gamma; ++hop) {
            const int nx = P.node_accept[nb + n];
            if (nx <= n || nx >= P.n_nodes) break;
            n = nx;
        }
        const bool internal = n < P.n_internal;
        // statistics of the stopping node: kept by the decide kernel (node with children), or formed
        // from the entries of round 0 (leaf)
        float r_t, z_t, r_d = 0.f, z_d = 0.f, c = 0.f;
        if (internal) {
            const NodeStats st = P.stats[nb + n];
            r_t = st.r_t; r_d = st.r_d; z_t = st.z_t; z_d = st.z_d; c = P.attempt ? st.c_prev : st.c;
        } else {
            float4 ent = make_float4(-INFINITY, 0.f, 0.f, 0.f);
            if (lane < P.n_entries) {
                const int s = lane / P.eps_max, i = lane - s * P.eps_max;
                ent = P.stats_all[(static_cast<long long>(s) * P.B * P.n_nodes + nb + n) * P.eps_max + i];
            }
            r_t = warp_max(ent.x);
            z_t = warp_sum(ent.y * exp2i(ent.x - r_t));
        }
        const bool t_ok = z_t > 0.f && z_t < INFINITY, d_ok = internal && z_d > 0.f && z_d < INFINITY;
        const float r_t0 = r_t == -INFINITY ? 0.f : r_t, r_d0 = r_d == -INFINITY ? 0.f : r_d;
        const float kappa = fminf(c * ((t_ok && d_ok) ? z_t / z_d : 0.f), 3.0e38f);
        const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) +
            ((nb + n) * P.ld_t + static_cast<long long>(e) * RUN) * E::kBytes;
        const unsigned char *d_row = reinterpret_cast<const unsigned char *>(P.draft) +
            ((static_cast<long long>(b) * P.n_internal + n) * P.ld_d + static_cast<long long>(e) * RUN) * E::kBytes;
        int n_valid = P.n_cols - e * RUN;
        n_valid = n_valid > RUN ? RUN : n_valid;
        float *out = P.out_residual ? P.out_residual + static_cast<long long>(b) * P.n_cols + static_cast<long long>(e) * RUN : nullptr;
        float g[S];
#pragma unroll
        for (int st = 0; st < S; ++st) {
            g[st] = 0.f;
            const int x0 = st * kStep + lane * GV;
            if (x0 < n_valid) {
#pragma unroll
                for (int el = 0; el < GV; ++el) {
                    float w = 0.f;
                    if (x0 + el < n_valid) {
                        w = t_ok ? ex2f(fmaf(E::load(t_row, x0 + el), P.scale, -r_t0)) : 0.f;
                        if (kappa > 0.f) w = fmaxf(fmaf(-kappa, ex2f(fmaf(E::load(d_row, x0 + el), P.scale, -r_d0)), w), 0.f);
                        if (out) out[x0 + el] = w;
                    }
                    g[st] += w;
                }
            }
        }
        const double mass = run_total<S>(g);
        if (lane == 0) P.tot_out[static_cast<long long>(b) * P.eps_max + e] = mass;
    }
}

// Endpoint stage, second half: one warp per sequence, on every shard.  Writes the walk's outputs
// (the same on every shard), finds the run that holds the quantile from the gathered masses and, if
// that run belongs to this shard, the token inside it; scales this shard's part of the residual.
template <int DT, int EPT>
__global__ void __launch_bounds__(kShardThreads)
shard_finish_kernel(const __grid_constant__ ShardParams P)
{
    using E = Elem<DT>;
    constexpr int GV = E::kVec, RUN = 32 * EPT, kStep = 32 * GV, S = RUN / kStep;
    const int lane = threadIdx.x & 31;
    const long long warp_id = (static_cast<long long>(blockIdx.x) * kShardThreads + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * kShardThreads) >> 5;
    for (long long bb = warp_id; bb < P.B; bb += n_warps) {
        const int b = static_cast<int>(bb);
        if (P.attempt == 1 && P.retry[b] == 0) continue;
        const long long nb = static_cast<long long>(b) * P.n_nodes;
        int32_t *tok = P.out_tokens + static_cast<long long>(b) * (P.gamma + 1);
        int n = 0, len = 0, st_bits = 0;
        for (int hop = 0; hop < P.gamma; ++hop) {
            if (n < P.n_internal) st_bits |= P.stats[nb + n].status;
            const int nx = P.node_accept[nb + n];
            if (nx <= n || nx >= P.n_nodes) break;
            n = nx;
            if (lane == 0) {
                tok[len] = P.cand[nb + n];
                if (P.out_path_nodes) P.out_path_nodes[static_cast<long long>(b) * (P.gamma + 1) + len] = n;
            }
            ++len;
        }
        if (n < P.n_internal) st_bits |= P.stats[nb + n].status;
        const bool internal = n < P.n_internal;
        if (lane == 0) {
            for (int i = len + 1; i <= P.gamma; ++i) tok[i] = -1;
            if (P.out_path_nodes)
                for (int i = len; i <= P.gamma; ++i) P.out_path_nodes[static_cast<long long>(b) * (P.gamma + 1) + i] = -1;
            P.out_accept_len[b] = len;
        }
        // the run that holds the quantile
        double m = 0.0;
        if (lane < P.n_entries) {
            const int s = lane / P.eps_max, i = lane - s * P.eps_max;
            m = P.tot_all[(static_cast<long long>(s) * P.B + b) * P.eps_max + i];
        }
        double tgt = 0.0, total = m;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
        const float u_end = P.unif[2 * (nb + n) + 1];
        const int pick = pick_run(m, u_end, lane, tgt);
        if (pick < 0) {
            NodeStats stn = {};
            if (internal) stn = P.stats[nb + n];
            const bool again = P.attempt == 0 && internal && stn.c != stn.c_prev;
            if (lane == 0) {
                P.retry[b] = again ? 1 : 0;
                P.endpoint_part[b] = -1;
                tok[len] = -1;
                P.out_status[b] = st_bits | (internal ? MCSD_STATUS_DEGENERATE : 0) | (again ? 0 : MCSD_STATUS_NO_MASS);
            }
            continue;
        }
        if (lane == 0) {
            if (P.attempt == 0) P.retry[b] = 0;
            P.out_status[b] = st_bits | (P.attempt ? MCSD_STATUS_DEGENERATE : 0);
        }
        // scale this shard's part of the distribution
        if (P.out_residual) {
            const float inv = static_cast<float>(1.0 / total);
            float *out = P.out_residual + static_cast<long long>(b) * P.n_cols;
            for (int x = lane; x < P.n_cols; x += 32) out[x] *= inv;
        }
        int found = -1;
        const int e = pick - P.entry_begin;
        if (e >= 0 && e < P.eps) {
            // the quantile lies in a run of this shard: its group sums once more, then step, lane, element
            float r_t, z_t, r_d = 0.f, z_d = 0.f, c = 0.f;
            if (internal) {
                const NodeStats stn = P.stats[nb + n];
                r_t = stn.r_t; r_d = stn.r_d; z_t = stn.z_t; z_d = stn.z_d; c = P.attempt ? stn.c_prev : stn.c;
            } else {
                float4 ent = make_float4(-INFINITY, 0.f, 0.f, 0.f);
                if (lane < P.n_entries) {
                    const int s = lane / P.eps_max, i = lane - s * P.eps_max;
                    ent = P.stats_all[(static_cast<long long>(s) * P.B * P.n_nodes + nb + n) * P.eps_max + i];
                }
                r_t = warp_max(ent.x);
                z_t = warp_sum(ent.y * exp2i(ent.x - r_t));
            }
            const bool t_ok = z_t > 0.f && z_t < INFINITY, d_ok = internal && z_d > 0.f && z_d < INFINITY;
            const float r_t0 = r_t == -INFINITY ? 0.f : r_t, r_d0 = r_d == -INFINITY ? 0.f : r_d;
            const float kappa = fminf(c * ((t_ok && d_ok) ? z_t / z_d : 0.f), 3.0e38f);
            const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) +
                ((nb + n) * P.ld_t + static_cast<long long>(e) * RUN) * E::kBytes;
            const unsigned char *d_row = reinterpret_cast<const unsigned char *>(P.draft) +
                ((static_cast<long long>(b) * P.n_internal + n) * P.ld_d + static_cast<long long>(e) * RUN) * E::kBytes;
            int n_valid = P.n_cols - e * RUN;
            n_valid = n_valid > RUN ? RUN : n_valid;
            auto weights = [&](int x0, float *w) {
#pragma unroll
                for (int el = 0; el < GV; ++el) {
                    float v = 0.f;
                    if (x0 + el < n_valid) {
                        v = t_ok ? ex2f(fmaf(E::load(t_row, x0 + el), P.scale, -r_t0)) : 0.f;
                        if (kappa > 0.f) v = fmaxf(fmaf(-kappa, ex2f(fmaf(E::load(d_row, x0 + el), P.scale, -r_d0)), v), 0.f);
                    }
                    w[el] = v;
                }
            };
            float g[S];
#pragma unroll
            for (int st = 0; st < S; ++st) {
                g[st] = 0.f;
                const int x0 = st * kStep + lane * GV;
                if (x0 < n_valid) {
                    float w[GV];
                    weights(x0, w);
#pragma unroll
                    for (int el = 0; el < GV; ++el) g[st] += w[el];
                }
            }
            const float tj = step_totals<S>(g, lane);
            int ps, l;
            float rem;
            if (search_run<S>(g, tj, tgt, lane, ps, l, rem)) {
                int pe = -1;
                if (lane == l) {
                    float w[GV];
                    weights(ps * kStep + lane * GV, w);
                    pe = pick_element<GV>(w, rem);
                }
                found = __shfl_sync(0xffffffffu, pe < 0 ? -1 : P.col_begin + e * RUN + ps * kStep + lane * GV + pe, l);
            }
        }
        if (lane == 0) P.endpoint_part[b] = found;   // -1 on the shards that do not hold the run
    }
}

// After the caller has reduced endpoint_part over the shards (maximum): the endpoint token goes
// behind the accepted tokens of every sequence.
__global__ void shard_commit_kernel(const int32_t *endpoint, const int32_t *accept_len, int32_t *tokens, int32_t B, int32_t gamma)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) {
        const int len = accept_len[b];
        if (len >= 0 && len <= gamma) tokens[static_cast<long long>(b) * (gamma + 1) + len] = endpoint[b];
    }
}

}  // namespace mcsd
