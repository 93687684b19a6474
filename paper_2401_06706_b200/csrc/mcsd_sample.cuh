// sample_kernel: the k candidate draws of a node from the draft distribution, with
// replacement or without (Eq. 1), top-k at temperature 0.
#pragma once

#include "mcsd_common.cuh"

namespace mcsd {

struct SampleParams {
    const void *draft;
    const float *unif_draw;  // [B][n_nodes] the uniform that draws the token of each draft node
    int32_t *cand;           // [B][n_nodes]
    int32_t *status;         // [B] or null
    long long ld_d;
    int32_t n_nodes, n_internal, V;
    int32_t node_begin, n_range;  // nodes node_begin .. node_begin + n_range - 1 of every tree
    int32_t mode;
    int32_t vector_ok;
    int32_t prefetch_ahead;       // CTAs resident at once: the row of the CTA that far ahead is asked into L2
    float scale;                  // log2(e)/T, or 0 for top-k
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
};

// One CTA per (sequence, node with children): draws the tokens of the node's k children from
// softmax(draft row / T) by inverse CDF in token order with one supplied uniform each
// (Section 3.2).  With replacement the k draws are independent; without (Eq. 1) every
// drawn token is taken out of the distribution before the next draw, which here means
// subtracting its weight from the partial sums of its lane, its warp's run and the
// element scan.  The row is read once, from L2: the CTA that held this CTA's place before asked
// for the row while it computed.  There is no separate pass for the row's maximum: every
// thread exponentiates its groups batch by batch against the batch's own integer reference and
// moves the sums to the row's reference afterwards (an exact power of two);
// temperature 0 takes the k largest logits instead (lowest index first on ties).
// NT threads per CTA: 1024 when the vocabulary exceeds half the maximum, else as many independent
// chains per SM as 16 steps per warp allow: 512 (two CTAs per SM) with 4-byte logits, 256 (four
// CTAs per SM) with 2-byte logits.
template <int DT, int NT>
__global__ void __launch_bounds__(NT, NT == 512 ? 2 : (NT == 256 ? 4 : 1))
sample_kernel(const __grid_constant__ SampleParams P)
{
    using E = Elem<DT>;
    constexpr int GV = E::kVec;
    constexpr int kStep = 32 * GV;
    constexpr int kW = NT / 32;  // warps
    // steps of a warp's run: CTAs of 1024 threads cover the largest vocabulary, smaller ones half of it
    constexpr int kMaxSteps = (NT == 1024 ? MCSD_MAX_VOCAB : MCSD_MAX_VOCAB / 2) / kW / kStep;
    static_assert(kMaxSteps <= 16, "the per-lane group sums are kept in registers");
    __shared__ double s_wtot[32];
    __shared__ float s_red[32];
    __shared__ int s_redi[32];
    __shared__ int32_t s_rem_tok[MCSD_MAX_CHILDREN];
    __shared__ int s_pick, s_run;
    __shared__ double s_tgt;
    __shared__ int s_runs[MCSD_MAX_CHILDREN];
    __shared__ double s_tgts[MCSD_MAX_CHILDREN];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / P.n_range, n = P.node_begin + (blockIdx.x - b * P.n_range);
    const int k = P.child_count[n], first = P.child_first[n];
    if (k == 0) return;
    int32_t *out = P.cand + static_cast<long long>(b) * P.n_nodes + first;
    const unsigned char *row = reinterpret_cast<const unsigned char *>(P.draft) +
        (static_cast<long long>(b) * P.n_internal + n) * P.ld_d * E::kBytes;
    auto load_group = [&](int x0, float *v) {   // GV logits from x0 on, -inf past the vocabulary
        if (P.vector_ok && x0 + GV <= P.V) {
            E::unpack(ldg_v4(row + static_cast<size_t>(x0) * E::kBytes), v);
        } else {
#pragma unroll
            for (int e = 0; e < GV; ++e) v[e] = x0 + e < P.V ? E::load(row, x0 + e) : -INFINITY;
        }
    };
    // Branch-free variant for unrolled loops (their loads are then in flight together): on
    // 16-byte aligned rows a group that starts past the vocabulary reads the row's last group
    // instead, i.e. values that are in the row anyway.  That leaves a maximum unchanged; a sum
    // must drop those groups (x0 >= V).  The padding an incomplete last group brings along is
    // masked to -inf.
    const bool tail_mask = P.V % GV != 0;
    const int x_last = (P.V - 1) / GV * GV;
    auto load_group_clamped = [&](int x0, float *v) {
        if (P.vector_ok) {
            const int xc = x0 < x_last ? x0 : x_last;
            E::unpack(ldg_v4(row + static_cast<size_t>(xc) * E::kBytes), v);
            if (tail_mask) {
#pragma unroll
                for (int e = 0; e < GV; ++e) v[e] = xc + e < P.V ? v[e] : -INFINITY;
            }
        } else {
#pragma unroll
            for (int e = 0; e < GV; ++e) v[e] = x0 + e < P.V ? E::load(row, x0 + e) : -INFINITY;
        }
    };
    // The same, left packed (2-byte types only): 4 registers for 8 elements while the load is in flight.
    [[maybe_unused]] auto load_raw_clamped = [&](int x0) -> uint4 {
        uint4 r = make_uint4(0u, 0u, 0u, 0u);
        if constexpr (E::kBytes == 2) {
            float v[GV];
            if (P.vector_ok) {
                const int xc = x0 < x_last ? x0 : x_last;
                r = ldg_v4(row + static_cast<size_t>(xc) * E::kBytes);
                if (!(tail_mask && xc == x_last)) return r;
                E::unpack(r, v);   // the row's last, incomplete group: its padding becomes -inf
#pragma unroll
                for (int e = 0; e < GV; ++e) v[e] = xc + e < P.V ? v[e] : -INFINITY;
            } else {
#pragma unroll
                for (int e = 0; e < GV; ++e) v[e] = x0 + e < P.V ? E::load(row, x0 + e) : -INFINITY;
            }
            r.x = E::to_bits(v[0]) | (E::to_bits(v[1]) << 16);
            r.y = E::to_bits(v[2]) | (E::to_bits(v[3]) << 16);
            r.z = E::to_bits(v[4]) | (E::to_bits(v[5]) << 16);
            r.w = E::to_bits(v[6]) | (E::to_bits(v[7]) << 16);
        }
        return r;
    };
    // The CTA that takes this one's place when it has finished is about `prefetch_ahead` blocks
    // further on: its row is asked into L2 now, so that HBM streams while this CTA computes and
    // that CTA's two passes both read from L2.
    auto prefetch_later_row = [&]() {
        if (P.vector_ok && tid == 0) {
            const long long nb = static_cast<long long>(blockIdx.x) + P.prefetch_ahead;
            if (nb < static_cast<long long>(gridDim.x)) {
                const int b2 = static_cast<int>(nb / P.n_range), n2 = P.node_begin + static_cast<int>(nb - static_cast<long long>(b2) * P.n_range);
                const unsigned char *r2 = reinterpret_cast<const unsigned char *>(P.draft) +
                    (static_cast<long long>(b2) * P.n_internal + n2) * P.ld_d * E::kBytes;
                const uint32_t bytes = (static_cast<uint32_t>(P.V) * E::kBytes) & ~15u;
                if (bytes) bulk_prefetch_l2(r2, bytes);
            }
        }
    };
    const int run = ((P.V + kW - 1) / kW + kStep - 1) / kStep * kStep;
    const int x_lo = warp * run;
    int x_hi = x_lo + run;
    x_hi = x_hi > P.V ? P.V : x_hi;

    if (P.scale == 0.f) {
        prefetch_later_row();
        // ---- top-k.  One pass leaves in every thread the best of its own elements (largest
        // logit, lowest index among equals).  Each pick is the block-wide best of those; then only
        // the thread that held it needs a new best, which its warp finds together (lane j takes
        // the thread's j-th group) among the elements after the pick in the order (logit
        // descending, index ascending).
        float best = -INFINITY;
        int best_i = 0x7fffffff;
        {
            // (2-byte groups stay packed until they are looked at, so eight loads in flight cost the
            // registers of four unpacked 4-byte groups)
            constexpr int kAhead = E::kBytes == 2 ? 8 : 4;
            constexpr int UT = kAhead < kMaxSteps ? kAhead : kMaxSteps;
            constexpr int VW = E::kBytes == 2 ? 1 : GV;
#pragma unroll 1
            for (int s0 = 0; s0 < kMaxSteps; s0 += UT) {
                if (x_lo + s0 * kStep >= x_hi) break;
                float v[UT][VW];
                [[maybe_unused]] uint4 raw[E::kBytes == 2 ? UT : 1];
#pragma unroll
                for (int u = 0; u < UT; ++u) {
                    if constexpr (E::kBytes == 2) raw[u] = load_raw_clamped(x_lo + (s0 + u) * kStep + lane * GV);
                    else load_group_clamped(x_lo + (s0 + u) * kStep + lane * GV, v[u]);
                }
#pragma unroll
                for (int u = 0; u < UT; ++u) {
                    const int x0 = x_lo + (s0 + u) * kStep + lane * GV;
                    if (x0 < x_hi) {   // (a group read in place of one past the run is not this thread's)
                        float f[GV];
                        if constexpr (E::kBytes == 2) {
                            E::unpack(raw[u], f);
                        } else {
#pragma unroll
                            for (int e = 0; e < GV; ++e) f[e] = v[u][e];
                        }
#pragma unroll
                        for (int e = 0; e < GV; ++e)
                            if (f[e] > best) { best = f[e]; best_i = x0 + e; }   // ascending index: ties keep the lowest
                    }
                }
            }
        }
        auto better = [](float av, int ai, float bv, int bi) { return av > bv || (av == bv && ai < bi); };
        for (int i = 0; i < k; ++i) {
            float wv = best;
            int wi = best_i;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, wv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, wi, o);
                if (better(ov, oi, wv, wi)) { wv = ov; wi = oi; }
            }
            if (lane == 0) { s_red[warp] = wv; s_redi[warp] = wi; }
            __syncthreads();
            wv = lane < kW ? s_red[lane] : -INFINITY;
            wi = lane < kW ? s_redi[lane] : 0x7fffffff;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, wv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, wi, o);
                if (better(ov, oi, wv, wi)) { wv = ov; wi = oi; }
            }
            const float pv = wv;
            const int pi = wi == 0x7fffffff ? -1 : wi;
            if (tid == 0) out[i] = pi;
            // the holder of the pick (one thread of one warp) gets its next best
            const unsigned own = __ballot_sync(0xffffffffu, pi >= 0 && best_i == pi);
            if (own && i + 1 < k) {
                const int src = __ffs(own) - 1;
                float nv = -INFINITY;
                int ni = 0x7fffffff;
                const int x0 = x_lo + lane * kStep + src * GV;   // lane = step of the holder's run
                if (lane < kMaxSteps && x0 < x_hi) {
                    float v[GV];
                    load_group(x0, v);
#pragma unroll
                    for (int e = 0; e < GV; ++e) {
                        const int x = x0 + e;
                        const bool after = v[e] < pv || (v[e] == pv && x > pi);
                        if (x < P.V && after && v[e] > nv) { nv = v[e]; ni = x; }
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, nv, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, ni, o);
                    if (better(ov, oi, nv, ni)) { nv = ov; ni = oi; }
                }
                if (lane == src) { best = nv; best_i = ni; }
            }
            __syncthreads();
        }
        return;
    }

    // ---- unnormalised weights in ONE pass over the row: per lane the sum of its group in every
    // step, per warp its run.  A thread takes its groups in batches of U (that many 16-byte
    // loads in flight; more cost registers the two resident CTAs do not have) and
    // exponentiates each batch against the batch's own integer reference ceil(max * scale); once
    // the row's reference is known every batch is moved to it by an exact power of two.
    // Eight loads in flight either way: 4-byte groups are held unpacked (4 registers each), 2-byte
    // groups as they were loaded (4 registers for 8 elements; their maximum is taken on the packed
    // words and they are unpacked one at a time for the exponentials).
    constexpr int kBatch = 8;
    constexpr int U = kBatch < kMaxSteps ? kBatch : kMaxSteps;
    constexpr int NB = kMaxSteps / U;
    static_assert(kMaxSteps % U == 0, "whole batches");
    float g[kMaxSteps];
    float rb[NB];   // reference of each batch (-inf: nothing there)
    if constexpr (E::kBytes == 2) {
#pragma unroll
        for (int bi = 0; bi < NB; ++bi) {
            uint4 raw[U];
#pragma unroll
            for (int u = 0; u < U; ++u) raw[u] = load_raw_clamped(x_lo + (bi * U + u) * kStep + lane * GV);
            // (groups read in place of groups past the end are row elements too: they can only
            // raise the batch's reference towards the row's, never beyond it)
            typename E::MaxAcc acc = E::max_init();
#pragma unroll
            for (int u = 0; u < U; ++u) E::max_step(acc, raw[u]);
            rb[bi] = int_ref(E::max_final(acc) * P.scale);
            const float r0 = rb[bi] == -INFINITY ? 0.f : rb[bi];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int x0 = x_lo + (bi * U + u) * kStep + lane * GV;
                float v[GV];
                E::unpack(raw[u], v);
                float gs = 0.f;
#pragma unroll
                for (int e = 0; e < GV; ++e) gs += ex2f(fmaf(v[e], P.scale, -r0));
                g[bi * U + u] = x0 < x_hi ? gs : 0.f;   // a group past this warp's run (or the vocabulary) has no weight
            }
        }
    } else {
#pragma unroll
        for (int bi = 0; bi < NB; ++bi) {
            float v[U][GV];
#pragma unroll
            for (int u = 0; u < U; ++u) load_group_clamped(x_lo + (bi * U + u) * kStep + lane * GV, v[u]);
            float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int e = 0; e < GV; e += 4) {
                    m0 = max3(m0, v[u][e], v[u][e + 1]);
                    m1 = max3(m1, v[u][e + 2], v[u][e + 3]);
                }
            rb[bi] = int_ref(fmaxf(m0, m1) * P.scale);
            const float r0 = rb[bi] == -INFINITY ? 0.f : rb[bi];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int x0 = x_lo + (bi * U + u) * kStep + lane * GV;
                float gs = 0.f;
#pragma unroll
                for (int e = 0; e < GV; ++e) gs += ex2f(fmaf(v[u][e], P.scale, -r0));
                g[bi * U + u] = x0 < x_hi ? gs : 0.f;
            }
        }
    }
    prefetch_later_row();
    // reference of the row
    float rmax = rb[0];
#pragma unroll
    for (int bi = 1; bi < NB; ++bi) rmax = fmaxf(rmax, rb[bi]);
    rmax = warp_max(rmax);
    if (lane == 0) s_red[warp] = rmax;
    __syncthreads();
    const float ref = warp_max(lane < kW ? s_red[lane] : -INFINITY);
    float fb[NB];   // 2^(batch reference - row reference)
#pragma unroll
    for (int bi = 0; bi < NB; ++bi) {
        fb[bi] = exp2i(rb[bi] - ref);
#pragma unroll
        for (int u = 0; u < U; ++u) g[bi * U + u] *= fb[bi];
    }
    // the weights of one group again, bit for bit as they went into g (st: the group's step)
    auto weights = [&](int x0, int st, float *w) {
        float v[GV];
        load_group(x0, v);
        float r = rb[0], f = fb[0];
#pragma unroll
        for (int bi = 1; bi < NB; ++bi) {
            r = (st / U == bi) ? rb[bi] : r;
            f = (st / U == bi) ? fb[bi] : f;
        }
        const float r0 = r == -INFINITY ? 0.f : r;
#pragma unroll
        for (int e = 0; e < GV; ++e) w[e] = ex2f(fmaf(v[e], P.scale, -r0)) * f;
    };
    {
        const double run_mass = run_total<kMaxSteps>(g);
        if (lane == 0) s_wtot[warp] = run_mass;
    }
    __syncthreads();

    if (P.mode != 1) {
        // Independent draws (the candidates of Algorithm 1): warp 0 finds the run of every draw, the CTA
        // meets once, and every warp serves the draws that fell into its run.
        if (warp == 0) {
            const double m = lane < kW ? s_wtot[lane] : 0.0;
            for (int i = 0; i < k; ++i) {
                const float u = P.unif_draw[static_cast<long long>(b) * P.n_nodes + first + i];
                double t = 0.0;
                const int r = pick_run(m, u, lane, t);
                if (lane == 0) { s_runs[i] = r; s_tgts[i] = t; }
            }
        }
        __syncthreads();
        float tj = 0.f;
        bool have_tj = false;
        for (int i = 0; i < k; ++i) {
            const int pick = s_runs[i];
            if (pick < 0) {
                if (tid == 0) {
                    out[i] = -1;
                    if (P.status) atomicOr(P.status + b, MCSD_STATUS_NO_MASS);
                }
                continue;
            }
            if (pick != warp) continue;
            if (!have_tj) { tj = step_totals<kMaxSteps>(g, lane); have_tj = true; }
            int ps, l, found = -1;
            float rem;
            if (search_run<kMaxSteps>(g, tj, s_tgts[i], lane, ps, l, rem)) {
                int pe = -1;
                if (lane == l) {
                    float w[GV];
                    weights(x_lo + ps * kStep + lane * GV, ps, w);
                    pe = pick_element<GV>(w, rem);
                }
                found = __shfl_sync(0xffffffffu, pe < 0 ? -1 : x_lo + ps * kStep + lane * GV + pe, l);
            }
            if (lane == 0) {
                out[i] = found;
                if (found < 0 && P.status) atomicOr(P.status + b, MCSD_STATUS_NO_MASS);
            }
        }
        return;
    }

    // Without replacement (Eq. 1) every draw changes the distribution of the next: one draw at a time.
    int n_rem = 0;  // tokens taken out so far (Eq. 1); the same in every thread
    for (int i = 0; i < k; ++i) {
        // warp 0 finds the run that holds the quantile ...
        if (warp == 0) {
            const float u = P.unif_draw[static_cast<long long>(b) * P.n_nodes + first + i];
            double t = 0.0;
            const int r = pick_run(lane < kW ? s_wtot[lane] : 0.0, u, lane, t);
            if (lane == 0) { s_run = r; s_tgt = t; }
        }
        __syncthreads();
        const int pick = s_run;
        // ... and the warp that owns that run finds the step, the lane and the element
        if (pick >= 0 && warp == pick) {
            const double tgt = s_tgt;
            const float tj = step_totals<kMaxSteps>(g, lane);
            int ps, l, found = -1;
            float rem;
            if (search_run<kMaxSteps>(g, tj, tgt, lane, ps, l, rem)) {
                int pe = -1;
                if (lane == l) {
                    const int x0 = x_lo + ps * kStep + lane * GV;
                    float w[GV];
                    weights(x0, ps, w);
                    // tokens drawn before (Eq. 1) have left the distribution
                    for (int j = 0; j < n_rem; ++j) {
                        const int gone = s_rem_tok[j] - x0;
#pragma unroll
                        for (int e = 0; e < GV; ++e) w[e] = (gone == e) ? 0.f : w[e];
                    }
                    pe = pick_element<GV>(w, rem);
                    if (pe >= 0 && P.mode == 1) {
                        // ... and so does this one: the group's sum is formed again from the
                        // tokens that remain (subtracting would lose everything when the drawn
                        // token dominated the group)
                        float rest = 0.f;
#pragma unroll
                        for (int e = 0; e < GV; ++e) rest += (e == pe) ? 0.f : w[e];
#pragma unroll
                        for (int st = 0; st < kMaxSteps; ++st)
                            if (st == ps) g[st] = rest;
                    }
                }
                found = __shfl_sync(0xffffffffu, pe < 0 ? -1 : x_lo + ps * kStep + lane * GV + pe, l);
                // ... and the run's total, from the lanes' current group sums (only warp 0 reads the
                // totals, and not before the barrier below)
                if (P.mode == 1 && found >= 0) {
                    const double left = run_total<kMaxSteps>(g);
                    if (lane == 0) s_wtot[warp] = left;
                }
            }
            if (lane == 0) {
                s_pick = found;
                out[i] = found;
                if (found < 0 && P.status) atomicOr(P.status + b, MCSD_STATUS_NO_MASS);
                if (P.mode == 1) s_rem_tok[n_rem] = found;
            }
        } else if (pick < 0 && tid == 0) {
            s_pick = -1;
            out[i] = -1;
            if (P.status) atomicOr(P.status + b, MCSD_STATUS_NO_MASS);
            if (P.mode == 1) s_rem_tok[n_rem] = -1;
        }
        __syncthreads();
        if (P.mode == 1 && s_pick >= 0) ++n_rem;
    }
}

}  // namespace mcsd
