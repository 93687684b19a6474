// node_kernel (T > 0): Algorithm 1 / Algorithm 2 at every node of every tree, one
// thread-block cluster per (sequence, node) item with the two logit rows held on chip.
#pragma once

#include "mcsd_common.cuh"

namespace mcsd {

// Shared state of the cluster-wide exchange: two buffers of one float4 per (cluster
// rank, warp) and one mbarrier per buffer.  In round r every warp of every CTA sends its
// value into buffer r&1 of every CTA of the cluster (its own included) with asynchronous
// stores that report their bytes to that CTA's barrier; the CTA armed the barrier with
// the byte count of a whole round, so when its phase completes all values of the round
// are there, in vocabulary order (rank-major, then warp).  One warp per CTA watches the
// barrier (bounded, with back-off), the others wait for it at a CTA barrier, so nobody
// spins on the issue slots the working CTAs need.  A buffer is rewritten two rounds
// later, which a peer can only reach after all warps of this CTA have sent the round in
// between, i.e. after they finished reading.
struct Exchange {
    float4 slot[2][kMaxCluster * 4];
    unsigned long long bar[2];
};

// What the leader warp of a CTA tells the other warps at the end of an exchange round.
struct Action {
    float4 stats;  // (row reference of p, of q, 1 / Z_t, Z_t / Z_d); written in the statistics round only
    float c_try;   // c of the residual sum to form next
    int more;      // 1: form that sum and run another round; 0: the node is decided
    int accepted;  // path mode, with more == 0: the accepted child of the node, or -1
    int poisoned;  // the leader's wait for this round expired: from here on the CTA's results are void
};

// Candidate data of the next items, fetched ahead of use by warp 0 so that no DRAM
// latency sits on the per-node critical path: lane i handles candidate i.
//   token id and acceptance uniform   two items ahead  (ring of 3)
//   the candidate's own two logits    one item ahead   (ring of 2; they need the token)
struct CandRing {
    int32_t tok[3][MCSD_MAX_CHILDREN];
    float u[3][MCSD_MAX_CHILDREN];
    uint32_t tl[2][MCSD_MAX_CHILDREN];  // aligned 32-bit word holding the target logit
    uint32_t dl[2][MCSD_MAX_CHILDREN];  // same for the draft logit
};

// Threads of one node-kernel CTA.  Few threads with many elements each: the per-thread
// bookkeeping (about 60 registers) is paid once per 64 elements, so that four CTAs
// with a 64-element target slice per thread fit the register file without spilling.
constexpr int kNodeThreads = 128;
constexpr int kNodeWarps = kNodeThreads / 32;
// Resident CTAs per SM the register budget is held to (128 / 96 / 80 registers).
constexpr int node_min_blocks(int ept) { return ept >= 64 ? 4 : (ept >= 32 ? 5 : 6); }
// Dynamic shared memory of one CTA: the exponentiated draft slice (float) and, for
// 2-byte logits on the bulk-copy path, the zone the raw draft slice lands in.
constexpr size_t node_smem_bytes(int elem_bytes, int ept, bool direct) {
    return static_cast<size_t>(kNodeThreads) * ept * 4 +
           ((!direct && elem_bytes == 2) ? static_cast<size_t>(kNodeThreads) * ept * 2 : 0);
}

// DT: element type; EPT: vocabulary elements per thread per row; DIRECT: read the
// rows with plain scalar loads (any alignment) instead of vector loads and bulk copies;
// PATH: the items are the sequences; a cluster walks each of its sequences from the root,
// evaluating only the nodes the walk visits (see NodeParams).
//
// Ownership inside a CTA: the slice is cut into 16-byte groups of GV elements; thread
// (warp w, lane l) owns groups (w * NG + j) * 32 + l, j < NG, so that one warp-wide
// access is contiguous and a warp's elements are one contiguous run of the vocabulary.
// Groups past the end of the slice hold -inf (probability 0).
//
// Every decision of the rejection loop is taken by every warp of the cluster from
// bit-identical inputs, so all CTAs of a cluster execute the same number of exchange
// rounds (the byte counts the exchange barriers are armed with rely on it).
//
// Which nodes need this kernel at all: those with two or more children, whose rows must stay on
// chip for the residual sums.  A leaf tests nothing; a node with one child needs no residual (the
// sum after a node's last rejection is formed by the walk stage, and only where a walk stops).
// Large launches of the all-node form therefore give this kernel only the nodes with two or more
// children (NodeParams::item_node) and leave the others to stream_stats_kernel and
// single_decide_kernel below; small launches, where a further kernel launch costs more than it
// saves, and the path form take every node through this kernel.
template <int DT, int EPT, bool DIRECT, bool PATH>
__global__ void __launch_bounds__(kNodeThreads, node_min_blocks(EPT))
node_kernel(const __grid_constant__ NodeParams P)
{
    using E = Elem<DT>;
    constexpr int NT = kNodeThreads, NW = kNodeWarps;
    constexpr int GV = E::kVec;
    constexpr int NG = EPT / GV;
    constexpr int H = GV / 4;  // float4 per group once exponentiated
    constexpr bool kRawZone = !DIRECT && E::kBytes == 2;
    // L2 prefetch of the cluster's next item: with 2-byte logits the kernel is bound by the
    // SMs and the prefetch takes DRAM latency off the per-node chain (measured +20 %); with
    // 4-byte logits it is bound by HBM and the extra request stream only costs (-1 %, and
    // -30 % on leaf-only trees), so it is left out there
    constexpr bool kPrefetch = !DIRECT && !PATH && E::kBytes == 2;
    static_assert(EPT % GV == 0, "EPT must be a whole number of 16-byte groups");
    static_assert(NW == 4, "the exchange buffers hold four warps per CTA");
    // warp 0 leads the exchange rounds and takes the decisions; the look-ahead requests for the
    // next items are another warp's job so that they do not lengthen the leader's path
    constexpr int kFetchWarp = 1;

    extern __shared__ __align__(128) unsigned char dyn[];
    float4 *qbuf = reinterpret_cast<float4 *>(dyn);  // exponentiated draft slice, thread-private slots
    uint4 *qraw = reinterpret_cast<uint4 *>(dyn + static_cast<size_t>(NT) * EPT * 4);
    __shared__ Exchange xch;
    __shared__ __align__(8) unsigned long long full_bar;
    __shared__ CandRing ring;
    __shared__ Action act[2];
    // the leader's view of the node's candidates (candidate i: its p and q times K, its uniform), kept
    // in shared memory rather than in registers that every warp of the kernel would have to set aside
    __shared__ double s_px[MCSD_MAX_CHILDREN], s_qx[MCSD_MAX_CHILDREN];
    __shared__ float s_u[MCSD_MAX_CHILDREN];

    const int tid = threadIdx.x, lane = tid & 31;
    // (broadcast from lane 0 so that the compiler knows the warp index is warp-uniform)
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const uint32_t crank = __clusterRelativeBlockRank(), csize = __clusterSizeInBlocks();
    const int cluster_id = blockIdx.x / csize;
    const int n_entries = static_cast<int>(csize) * NW;  // values per exchange round (<= 32)
    const float scale = P.scale;
    const uint32_t full_addr = smem_u32(&full_bar);
    // barrier of exchange buffer s (computed, not looked up: an array indexed at run time would
    // live in local memory)
    const uint32_t xbar_base = smem_u32(&xch.bar[0]);
    auto xbar_addr = [&](uint32_t s) -> uint32_t { return xbar_base + s * 8u; };

    // this CTA's slice of the vocabulary and this warp's run of it
    const int v_begin = static_cast<int>(crank) * P.slice;
    int n_mine = P.V - v_begin;
    n_mine = n_mine < 0 ? 0 : (n_mine > P.slice ? P.slice : n_mine);
    const int n_full_groups = n_mine / GV;            // whole 16-byte groups
    const int g0 = warp * (NG * 32) + lane;           // this thread's group of chunk 0
    // every group of this warp is a whole group: the common case takes unpredicated loads
    const bool warp_full = !DIRECT && (warp + 1) * (NG * 32) <= n_full_groups;
    // bytes of the slice that are whole groups: what one bulk copy / prefetch moves
    const uint32_t bulk_bytes = DIRECT ? 0u : static_cast<uint32_t>(n_full_groups) * 16u;

    // slot of (chunk j, quarter h) in qbuf: for 4-byte logits it is the group's own place in
    // the slice, so that the bulk copy lands the raw values where the exponentiated ones go
    auto qslot = [&](int j, int h) -> int {
        return E::kBytes == 4 ? g0 + j * 32 : (j * H + h) * NT + tid;
    };

    // the walk stage may be set up while this kernel runs; it waits for this kernel's results itself
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        mbar_init(full_addr, 1);
        mbar_init(xbar_addr(0), 1);
        mbar_init(xbar_addr(1), 1);
        fence_mbar_init();
    }
    __syncthreads();
    cluster_sync_all();  // every CTA's barriers exist before anyone stores into a peer

    uint32_t full_parity = 0, round = 0;
    int poisoned = 0;

    auto t_slice = [&](long long item) -> const unsigned char * {
        return reinterpret_cast<const unsigned char *>(P.target) + (item * P.ld_t + v_begin) * E::kBytes;
    };
    auto d_slice = [&](int b, int n) -> const unsigned char * {
        return reinterpret_cast<const unsigned char *>(P.draft) +
            ((static_cast<long long>(b) * P.n_internal + n) * P.ld_d + v_begin) * E::kBytes;
    };

    // One exchange round.  send: `mine` is this warp's value (the same in all lanes);
    // whatever is placed between send and wait overlaps the round's latency.  wait:
    // returns entry `lane` of the round (rank-major, then warp), the given identity for
    // lanes beyond the entry count.
    auto exchange_send = [&](float4 mine) {
        const uint32_t s = round & 1u;
        // (once a wait has expired nothing is armed or sent any more: the barriers' phases no
        // longer follow the rounds)
        if (poisoned) return;
        if (tid == 0) mbar_arrive_expect_tx(xbar_addr(s), static_cast<uint32_t>(n_entries) * 16u + P.test_extra_tx);
        if (lane < static_cast<int>(csize)) {
            const uint32_t dst = map_to_rank(smem_u32(&xch.slot[s][crank * NW + warp]), lane);
            st_async_f4(dst, mine, map_to_rank(xbar_addr(s), lane));
        }
    };
    // leader (warp 0) only: waits for the round and returns entry `lane`
    auto exchange_leader_wait = [&](float4 identity) -> float4 {
        const uint32_t s = round & 1u;
        // once a wait has expired the results are void and later rounds do not wait again
        if (!poisoned && !mbar_wait(xbar_addr(s), (round >> 1) & 1u, P.wait_polls)) poisoned = 1;
        return lane < n_entries ? xch.slot[s][lane] : identity;
    };
    // all warps: ends the round (the other warps have been waiting here for the leader)
    auto exchange_release = [&]() {
        __syncthreads();
        poisoned |= act[round & 1u].poisoned;
        ++round;
    };

    // (sequence, position in the node list) of the items this cluster visits: the current one
    // and the two after it, advanced by the precomputed quotient and remainder of the stride
    auto advance = [&](int &b, int &i) {
        b += P.step_b;
        i += P.step_n;
        if (i >= P.n_list) { i -= P.n_list; ++b; }
    };

    // ---- candidate pipeline (the fetch warp only) -------------------------------------------
    auto fetch_tokens = [&](int b, int n, int slot3) {
        if (b < P.B) {
            const int k = n < P.n_internal ? P.child_count[n] : 0;
            if (lane < k) {
                const long long ci = static_cast<long long>(b) * P.n_nodes + P.child_first[n] + lane;
                cp_async4(&ring.tok[slot3][lane], P.cand + ci);
                cp_async4(&ring.u[slot3][lane], P.unif + 2 * ci);
            }
        }
    };
    // needs the item's tokens to have arrived (cp_async_wait_all by this thread)
    auto fetch_logits = [&](int b, int n, int slot3, int slot2) {
        if (b < P.B) {
            const int k = n < P.n_internal ? P.child_count[n] : 0;
            if (lane < k) {
                const int xt = ring.tok[slot3][lane];
                if (xt >= 0 && xt < P.V) {
                    const unsigned char *t = reinterpret_cast<const unsigned char *>(P.target) +
                        ((static_cast<long long>(b) * P.n_nodes + n) * P.ld_t + xt) * E::kBytes;
                    const unsigned char *d = reinterpret_cast<const unsigned char *>(P.draft) +
                        ((static_cast<long long>(b) * P.n_internal + n) * P.ld_d + xt) * E::kBytes;
                    if (!DIRECT) {  // rows are 16-byte aligned: the enclosing word lies inside the row
                        cp_async4(&ring.tl[slot2][lane], reinterpret_cast<const void *>(reinterpret_cast<uintptr_t>(t) & ~uintptr_t(3)));
                        cp_async4(&ring.dl[slot2][lane], reinterpret_cast<const void *>(reinterpret_cast<uintptr_t>(d) & ~uintptr_t(3)));
                    } else {        // any alignment: plain loads of exactly the element, kept as float
                        ring.tl[slot2][lane] = __float_as_uint(E::load(t, 0));
                        ring.dl[slot2][lane] = __float_as_uint(E::load(d, 0));
                    }
                }
            }
        }
    };

    int b = cluster_id / P.n_list, ipos = cluster_id - b * P.n_list;  // current item: sequence, list position
    int n = P.item_node[ipos];
    if (PATH) { b = cluster_id; n = 0; }  // every walk starts at the root
    uint32_t it = 0;  // iteration count of this cluster
    bool prev_internal = false;
    if (!PATH && warp == kFetchWarp) {
        fetch_tokens(b, n, 0);
        cp_async_wait_all();
        __syncwarp();
        fetch_logits(b, n, 0, 0);
        int b1 = b, i1 = ipos;           // (the items that follow are found again from the current one when needed)
        advance(b1, i1);
        fetch_tokens(b1, P.item_node[i1], 1);
    }
    if (kPrefetch && tid == 0 && b < P.B && bulk_bytes) {
        bulk_prefetch_l2(t_slice(static_cast<long long>(b) * P.n_nodes + n), bulk_bytes);
        if (n < P.n_internal) bulk_prefetch_l2(d_slice(b, n), bulk_bytes);
    }

    for (; b < P.B; ++it) {
        const bool internal = n < P.n_internal;
        const int k = internal ? P.child_count[n] : 0;
        const int first = P.child_first[n];
        const long long node_idx = static_cast<long long>(b) * P.n_nodes + n;
        const int s3 = it % 3u, s2 = it & 1u;
        int status_bits = 0;

        // this item's candidate data has landed (it was requested one item ago) ...
        if (!PATH && warp == kFetchWarp) cp_async_wait_all();
        // ... and, around an item with children, all warps meet: they are done with the
        // previous item (its draft buffer and ring entries may be overwritten) and they
        // see this item's ring entries.  A run of leaves needs no meeting at all.
        if (internal || prev_internal) {
            if (!DIRECT) fence_proxy_async();
            __syncthreads();
        }
        prev_internal = internal;
        // path mode: the next node is only known once this one is decided, so nothing is fetched
        // ahead; the leader warp asks for this node's candidate data now and picks it up when it
        // needs it, behind the row work and the exchange
        if (PATH && warp == 0 && internal) fetch_tokens(b, n, s3);

        const unsigned char *t_row = t_slice(node_idx);
        const unsigned char *d_row = d_slice(b, n);
        const bool q_bulk = internal && bulk_bytes != 0;
        if (tid == 0 && q_bulk && !poisoned) {  // (after an expired wait nothing more is copied)
            mbar_arrive_expect_tx(full_addr, bulk_bytes);
            bulk_load(smem_u32(kRawZone ? static_cast<const void *>(qraw) : static_cast<const void *>(qbuf)),
                      d_row, bulk_bytes, full_addr);
        }
        // look-ahead duties of the fetch warp: L2 prefetch of the next item's slices, candidate
        // data of the next two items
        auto look_ahead = [&]() {
            if (!PATH && warp == kFetchWarp) {
                int b1 = b, i1 = ipos;
                advance(b1, i1);
                const int n1 = P.item_node[i1];
                if (kPrefetch && lane == 0 && b1 < P.B && bulk_bytes) {
                    bulk_prefetch_l2(t_slice(static_cast<long long>(b1) * P.n_nodes + n1), bulk_bytes);
                    if (n1 < P.n_internal) bulk_prefetch_l2(d_slice(b1, n1), bulk_bytes);
                }
                fetch_logits(b1, n1, (it + 1) % 3u, s2 ^ 1);
                int b2 = b1, i2 = i1;
                advance(b2, i2);
                fetch_tokens(b2, P.item_node[i2], (it + 2) % 3u);
            }
        };
        auto next_item = [&]() {
            advance(b, ipos);
            n = P.item_node[ipos];
        };

        // ---- target slice -> registers, as packed pairs
        f32x2 tv[EPT / 2];
        if (warp_full) {
            // every group of this warp is a whole group inside the slice
#pragma unroll
            for (int j = 0; j < NG; ++j) {
                float f[GV];
                E::unpack(ld_stream_v4(t_row + static_cast<size_t>(g0 + j * 32) * 16), f);
#pragma unroll
                for (int e = 0; e < GV; e += 2) tv[(j * GV + e) / 2] = pack2(f[e], f[e + 1]);
            }
        } else if constexpr (DIRECT) {
#pragma unroll
            for (int j = 0; j < NG; ++j) {
                const int g = g0 + j * 32;
                float f[GV];
#pragma unroll
                for (int e = 0; e < GV; ++e) f[e] = (g * GV + e < n_mine) ? E::load(t_row, g * GV + e) : -INFINITY;
#pragma unroll
                for (int e = 0; e < GV; e += 2) tv[(j * GV + e) / 2] = pack2(f[e], f[e + 1]);
            }
        } else {
            // a warp at the ragged end of the vocabulary: predicated vector loads of the groups
            // that hold data (no branch between them, so their latencies overlap as in the
            // common case), -inf where there is none ...
            const int n_groups = (n_mine + GV - 1) / GV;
#pragma unroll
            for (int j = 0; j < NG; ++j) {
                const int g = g0 + j * 32;
                float f[GV];
                E::unpack(ld_stream_v4_if(t_row + static_cast<size_t>(g) * 16, g < n_groups, E::kNegInfWord), f);
#pragma unroll
                for (int e = 0; e < GV; e += 2) tv[(j * GV + e) / 2] = pack2(f[e], f[e + 1]);
            }
            // ... and where the vocabulary is no multiple of the vector width, the last group's
            // elements past the end (padding of the 16-byte aligned row) are set to -inf
            if (n_groups != n_full_groups) {
#pragma unroll
                for (int j = 0; j < NG; ++j) {
                    if (g0 + j * 32 == n_full_groups) {
#pragma unroll
                        for (int e = 0; e < GV; e += 2) {
                            const int x = n_full_groups * GV + e;
                            f32x2 &v = tv[(j * GV + e) / 2];
                            v = pack2(x < n_mine ? v.x : -INFINITY, x + 1 < n_mine ? v.y : -INFINITY);
                        }
                    }
                }
            }
        }
        // Each warp exponentiates relative to its own integer reference; the factor to the
        // row's reference and the normaliser are applied as per-warp scalars later.
        float rt, zt;
        {
            float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
            for (int p = 0; p < EPT / 2; p += 2) {
                m0 = max3(m0, tv[p].x, tv[p].y);
                m1 = max3(m1, tv[p + 1].x, tv[p + 1].y);
            }
            rt = int_ref(warp_max(fmaxf(m0, m1)) * scale);  // one reference per warp
            const float rt0 = (rt == -INFINITY) ? 0.f : rt;
            const f32x2 scale2 = pack2(scale, scale), nref2 = pack2(-rt0, -rt0);
            f32x2 z0 = pack2(0.f, 0.f), z1 = z0;
#pragma unroll
            for (int p = 0; p < EPT / 2; p += 2) {
                const f32x2 x01 = fma2(tv[p], scale2, nref2), x23 = fma2(tv[p + 1], scale2, nref2);
                tv[p] = pack2(ex2f(x01.x), ex2f(x01.y));
                tv[p + 1] = pack2(ex2f(x23.x), ex2f(x23.y));
                z0 = add2(z0, tv[p]);
                z1 = add2(z1, tv[p + 1]);
            }
            const f32x2 z = add2(z0, z1);
            zt = z.x + z.y;
        }

        if (!internal) {
            // A leaf decides nothing.  Its softmax statistics are only needed if a walk ends
            // here, so each warp leaves the partial statistics of its run in global memory
            // (the walk kernel combines them) and goes on: no exchange, no barrier.
            const float st = warp_sum(zt);
            if (lane == 0)
                P.leaf_part[(static_cast<long long>(b) * (P.n_nodes - P.n_internal) + (n - P.n_internal)) * kLeafEntries +
                            crank * NW + warp] = make_float2(rt, st);
            if (crank == 0 && tid == 0) P.node_accept[node_idx] = -1;
            if (PATH) {  // the walk ends at this leaf: on to the cluster's next sequence
                b += P.step_b;
                n = 0;
            } else {
                look_ahead();
                next_item();
            }
            continue;
        }

        // ---- draft slice: exponentiated in shared memory, in the slots of its owner
        float zd = 0.f, rd = -INFINITY;
        {
            if (DIRECT) {
                // the owner copies its raw elements into its slots, as float
#pragma unroll
                for (int j = 0; j < NG; ++j) {
                    const int g = g0 + j * 32;
                    float f[GV];
#pragma unroll
                    for (int e = 0; e < GV; ++e) f[e] = (g * GV + e < n_mine) ? E::load(d_row, g * GV + e) : -INFINITY;
#pragma unroll
                    for (int h = 0; h < H; ++h)
                        qbuf[qslot(j, h)] = make_float4(f[4 * h], f[4 * h + 1], f[4 * h + 2], f[4 * h + 3]);
                }
            } else {
                if (q_bulk && !poisoned) {
                    if (!mbar_wait(full_addr, full_parity)) poisoned = 1;
                    full_parity ^= 1u;
                }
                if (!warp_full) {
                    // groups the bulk copy did not bring: -inf past the data, and the ragged
                    // last group of the slice element by element (the slots are this thread's own)
#pragma unroll
                    for (int j = 0; j < NG; ++j) {
                        const int g = g0 + j * 32;
                        if (g >= n_full_groups) {
                            float f[GV];
#pragma unroll
                            for (int e = 0; e < GV; ++e) f[e] = -INFINITY;
                            if (g * GV < n_mine) {  // the ragged last group of the slice
#pragma unroll
                                for (int e = 0; e < GV; ++e) f[e] = (g * GV + e < n_mine) ? E::load(d_row, g * GV + e) : -INFINITY;
                            }
                            if constexpr (kRawZone) {
                                uint4 r;
                                r.x = E::to_bits(f[0]) | (E::to_bits(f[1]) << 16);
                                r.y = E::to_bits(f[2]) | (E::to_bits(f[3]) << 16);
                                r.z = E::to_bits(f[4]) | (E::to_bits(f[5]) << 16);
                                r.w = E::to_bits(f[6]) | (E::to_bits(f[7]) << 16);
                                qraw[g] = r;
                            } else {
                                qbuf[g] = make_float4(f[0], f[1], f[2], f[3]);
                            }
                        }
                    }
                }
            }
            auto read_q_raw = [&](int j, float *r) {
                if constexpr (kRawZone) {
                    E::unpack(qraw[g0 + j * 32], r);
                } else {
#pragma unroll
                    for (int h = 0; h < H; ++h) {
                        const float4 v = qbuf[qslot(j, h)];
                        r[4 * h] = v.x; r[4 * h + 1] = v.y; r[4 * h + 2] = v.z; r[4 * h + 3] = v.w;
                    }
                }
            };
            float md;
            if constexpr (kRawZone || E::kBytes == 4) {
                // maximum over the raw vectors as they lie in shared memory (packed for 2-byte types)
                typename E::MaxAcc acc = E::max_init();
#pragma unroll
                for (int j = 0; j < NG; ++j)
                    E::max_step(acc, kRawZone ? qraw[g0 + j * 32] : *reinterpret_cast<const uint4 *>(&qbuf[qslot(j, 0)]));
                md = E::max_final(acc);
            } else {
                float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
                for (int j = 0; j < NG; ++j) {
                    float r[GV];
                    read_q_raw(j, r);
#pragma unroll
                    for (int e = 0; e < GV; e += 4) {
                        m0 = max3(m0, r[e], r[e + 1]);
                        m1 = max3(m1, r[e + 2], r[e + 3]);
                    }
                }
                md = fmaxf(m0, m1);
            }
            rd = int_ref(warp_max(md) * scale);
            const float rd0 = (rd == -INFINITY) ? 0.f : rd;
            const f32x2 scale2 = pack2(scale, scale), nref2 = pack2(-rd0, -rd0);
            f32x2 z0 = pack2(0.f, 0.f), z1 = z0;
#pragma unroll
            for (int j = 0; j < NG; ++j) {
                float r[GV];
                read_q_raw(j, r);
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    const f32x2 x01 = fma2(pack2(r[4 * h], r[4 * h + 1]), scale2, nref2);
                    const f32x2 x23 = fma2(pack2(r[4 * h + 2], r[4 * h + 3]), scale2, nref2);
                    const float4 ev = make_float4(ex2f(x01.x), ex2f(x01.y), ex2f(x23.x), ex2f(x23.y));
                    qbuf[qslot(j, h)] = ev;
                    z0 = add2(z0, pack2(ev.x, ev.y));
                    z1 = add2(z1, pack2(ev.z, ev.w));
                }
            }
            const f32x2 z = add2(z0, z1);
            zd = z.x + z.y;
        }

        // ---- softmax statistics of both rows: one exchange round
        exchange_send(make_float4(rt, warp_sum(zt), rd, warp_sum(zd)));  // per warp: (ref_t, z_t, ref_d, z_d)
        look_ahead();  // in the shadow of the exchange

        // From here on warp 0 of every CTA is the leader: it alone combines the exchanged
        // values, evaluates the acceptance tests (Algorithm 1 / Algorithm 2) and tells the
        // other warps through `act` what to do next; they only stream and reduce.  The
        // leaders of a cluster work from bit-identical inputs and decide identically.
        //
        // leader state of the rejection loop, in units where W' = W * K, K = Z_t * Z_d:
        double c = 0.0, S = 1.0, Wk = 0.0, K = 0.0, c_try = 0.0;
        float c_prev = 0.f;  // c before the last rejection
        int cand_i = 0, accepted = -1;
        // tests candidates from cand_i on until one is accepted (returns 0), all are rejected
        // (returns 0) or one is rejected and its residual sum is needed (returns 1, c_try set).
        // The sum after the LAST rejection is not needed here (nothing is tested against that
        // residual): c moves on, the walk kernel forms the sum if a walk stops at this node.
        auto leader_decide = [&]() -> int {
            while (cand_i < k) {
                const int i = cand_i;
                const int xi = ring.tok[s3][i];
                const double ui = static_cast<double>(s_u[i]);
                const double pxi = s_px[i], qxi = s_qx[i];
                const bool valid = xi >= 0 && xi < P.V;
                if (!valid) status_bits |= MCSD_STATUS_BAD_TOKEN;
                // Algorithm 2: a token rejected earlier at this node has draft probability 0 now
                const bool dup = P.mode == 1 &&
                    (__ballot_sync(0xffffffffu, lane < i && ring.tok[s3][lane] == xi) != 0u);
                const bool zero_q = !valid || dup || !(qxi > 0.0) || !(Wk > 0.0);
                double Pn = pxi - c * qxi;
                Pn = Pn > 0.0 ? Pn : 0.0;
                // r <= [P_n(x~)/S_n] / [q(x~)/W_n] without divisions (all factors > 0)
                const bool accept = !zero_q && ui * S * qxi * K <= Pn * Wk;
                if (P.node_ratio && crank == 0 && lane == 0)
                    P.node_ratio[static_cast<long long>(b) * P.n_nodes + first + i] =
                        zero_q ? -1.f : static_cast<float>((Pn / S) / (qxi * K / Wk));
                if (accept) { accepted = first + i; return 0; }
                // rejected: p := norm(max(0, p - q)); Algorithm 2 also removes x~ from q
                c_try = c;
                if (Wk > 0.0) c_try = (P.mode == 1) ? c + S * K / Wk : c + S;
                if (P.mode == 1 && !zero_q) { Wk -= qxi; if (!(Wk > 0.0)) Wk = 0.0; }
                if (i + 1 >= k) { c_prev = static_cast<float>(c); c = c_try; cand_i = k; return 0; }
                return 1;
            }
            return 0;
        };

        if (warp == 0) {
            if (PATH) {  // tokens and uniforms have landed by now; then the candidates' own logits
                cp_async_wait_all();
                __syncwarp();
                fetch_logits(b, n, s3, s2);
                cp_async_wait_all();
                __syncwarp();
            }
            // while the round is in flight: 2^(scaled logit) of the candidates' own logits as
            // 2^int * frac (lane i = candidate i)
            float frac_t = 0.f, frac_d = 0.f;
            int int_t = 0, int_d = 0;
            bool cand_ok = false;
            if (lane < k) {
                const int my_tok = ring.tok[s3][lane];
                s_u[lane] = fminf(ring.u[s3][lane], 1.f);  // supplied in place of r ~ U(0,1): not below 1 (NaN too) counts as 1
                cand_ok = my_tok >= 0 && my_tok < P.V;
                if (cand_ok) {
                    const uint32_t wt = ring.tl[s2][lane], wd = ring.dl[s2][lane];
                    frac_t = split_exp2(DIRECT ? __uint_as_float(wt) : E::from_word(wt, my_tok), scale, P.scale_lo, int_t);
                    frac_d = split_exp2(DIRECT ? __uint_as_float(wd) : E::from_word(wd, my_tok), scale, P.scale_lo, int_d);
                }
            }
            const float4 ent = exchange_leader_wait(make_float4(-INFINITY, 0.f, -INFINITY, 0.f));
            // row references ceil(row maximum * scale) and normalisers
            const float R_t = warp_max(ent.x), R_d = warp_max(ent.z);
            const float Z_t = warp_sum(ent.y * exp2i(ent.x - R_t));
            const float Z_d = warp_sum(ent.w * exp2i(ent.z - R_d));
            const bool t_ok = Z_t > 0.f && Z_t < INFINITY;  // false for an all -inf or NaN row
            const bool d_ok = Z_d > 0.f && Z_d < INFINITY;
            // (a target row without mass: nothing can be accepted and a walk that stops here finds no
            // token; a draft row without mass: nothing to test against, every candidate is rejected and
            // p is kept; both count as a residual update that found no mass)
            if (!t_ok || !d_ok) status_bits |= MCSD_STATUS_DEGENERATE;
            // candidates' probabilities, both multiplied by K so that no division is needed:
            // px' = 2^(l_t*scale - R_t) * Z_d, qx' = 2^(l_d*scale - R_d) * Z_t
            K = static_cast<double>(Z_t) * static_cast<double>(Z_d);
            Wk = K;
            if (lane < k) {
                const bool ok = cand_ok && t_ok && d_ok;
                s_px[lane] = ok ? static_cast<double>(frac_t) * exp2i_d(int_t - static_cast<int>(R_t)) * static_cast<double>(Z_d) : 0.0;
                s_qx[lane] = ok ? static_cast<double>(frac_d) * exp2i_d(int_d - static_cast<int>(R_d)) * static_cast<double>(Z_t) : 0.0;
            }
            __syncwarp();
            const int more = leader_decide();
            if (lane == 0) {
                act[round & 1u].stats = make_float4(R_t, R_d, t_ok ? 1.f / Z_t : 0.f, (t_ok && d_ok) ? Z_t / Z_d : 0.f);
                act[round & 1u].c_try = static_cast<float>(c_try);
                act[round & 1u].more = more;
                act[round & 1u].poisoned = poisoned;
                if (PATH) act[round & 1u].accepted = accepted;
                if (crank == 0) *reinterpret_cast<float4 *>(&P.stats[node_idx]) = make_float4(R_t, R_d, Z_t, Z_d);
            }
        }
        exchange_release();  // CTA barrier: the leader's verdict is visible to all warps
        const float4 st4 = act[(round - 1u) & 1u].stats;
        int more = act[(round - 1u) & 1u].more;
        float c_next = act[(round - 1u) & 1u].c_try;
        // p(x) = tv * a, q(x) = dv * bq for this warp's elements
        const float a = exp2i(rt - st4.x) * st4.z;
        float b_over_a = 0.f;  // bq / a
        if (a > 0.f && st4.w > 0.f && rd != -INFINITY) b_over_a = exp2i((rd - st4.y) - (rt - st4.x)) * st4.w;

        // residual mass of this warp's run for a given c
        auto residual_pass = [&](float c_f) -> float {
            const float kappa = fminf(c_f * b_over_a, 3.0e38f);
            const f32x2 nk2 = pack2(-kappa, -kappa);
            f32x2 s0 = pack2(0.f, 0.f), s1 = s0;
#pragma unroll
            for (int j = 0; j < NG; ++j) {
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    const float4 d = qbuf[qslot(j, h)];
                    const int o = (j * GV + 4 * h) / 2;
                    const f32x2 x01 = fma2(pack2(d.x, d.y), nk2, tv[o]);
                    const f32x2 x23 = fma2(pack2(d.z, d.w), nk2, tv[o + 1]);
                    s0 = add2(s0, pack2(fmaxf(x01.x, 0.f), fmaxf(x01.y, 0.f)));
                    s1 = add2(s1, pack2(fmaxf(x23.x, 0.f), fmaxf(x23.y, 0.f)));
                }
            }
            const f32x2 t = add2(s0, s1);
            return warp_sum((t.x + t.y) * a);
        };

        // ---- one round per rejection: all warps reduce, the leader decides what comes next
#pragma unroll 1
        while (more) {
            exchange_send(make_float4(residual_pass(c_next), 0.f, 0.f, 0.f));
            if (warp == 0) {
                const float4 ent = exchange_leader_wait(make_float4(0.f, 0.f, 0.f, 0.f));
                const float S_new = warp_sum(ent.x);
                // zero residual mass: the previous residual, i.e. (c, S), is kept
                if (S_new > 0.f) { c = c_try; S = static_cast<double>(S_new); }
                else status_bits |= MCSD_STATUS_DEGENERATE;
                ++cand_i;
                const int next = leader_decide();
                if (lane == 0) {
                    act[round & 1u].c_try = static_cast<float>(c_try);
                    act[round & 1u].more = next;
                    act[round & 1u].poisoned = poisoned;
                    if (PATH) act[round & 1u].accepted = accepted;
                }
            }
            exchange_release();
            more = act[(round - 1u) & 1u].more;
            c_next = act[(round - 1u) & 1u].c_try;
        }

        // ---- per-node results (the endpoint token is drawn by the walk kernel, and only
        // for the node where a walk stops)
        if (warp == 0) {
            if (poisoned) status_bits |= MCSD_STATUS_TIMEOUT;
            status_bits = __reduce_or_sync(0xffffffffu, status_bits);
            if (crank == 0 && lane == 0) {
                P.node_accept[node_idx] = accepted;
                reinterpret_cast<float4 *>(&P.stats[node_idx])[1] =
                    make_float4(static_cast<float>(c), c_prev, __int_as_float(status_bits), 0.f);
            }
        }
        if (PATH) {
            // the walk goes on at the accepted child, or ends here
            const int acc = act[(round - 1u) & 1u].accepted;
            if (acc >= 0) n = acc;
            else { b += P.step_b; n = 0; }
        } else {
            next_item();
        }
    }

    if (warp == kFetchWarp) cp_async_wait_all();
    // After an expired wait the rounds were no longer waited for: give stores that peers issued
    // before they noticed time to land (they take about a microsecond) before anybody leaves.
    if (poisoned) __nanosleep(20000);
    // no CTA may leave while a peer can still write into its shared memory
    cluster_sync_all();
}

// Large launches of the all-node form: the rows of the nodes that need no exchange (leaves: the
// target row; nodes with one child: both rows) are only streamed for their statistics, and a
// kernel that keeps nothing on chip does that with many more warps per SM and therefore far more
// loads in flight than the cluster kernel can afford.  One warp per (sequence, node, run); runs,
// lanes and the order of every sum are those of node_kernel, so the statistics are the same bit
// for bit and go to the same places (leaf_part, single_part).
struct StreamParams {
    const void *target;
    const void *draft;
    float2 *leaf_part;
    float4 *single_part;
    int32_t *node_accept;   // -1 is written for every leaf
    long long ld_t, ld_d;
    int32_t B, n_nodes, n_internal, V, n_entries, n_list, vector_ok;
    float scale;
    uint16_t item_node[MCSD_MAX_NODES];   // leaves and nodes with one child, ascending
};

template <int DT, int EPT>
__device__ __forceinline__ void stream_run(const unsigned char *row, int n_valid, bool vector_ok, float scale, int lane,
                                           float &ref, float &z)
{
    using E = Elem<DT>;
    constexpr int GV = E::kVec, NG = EPT / GV;
    uint4 raw[NG];
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        const int x = (j * 32 + lane) * GV;
        if (vector_ok && x + GV <= n_valid) {
            raw[j] = ld_stream_v4(row + static_cast<size_t>(x) * E::kBytes);
        } else {
            // the ragged end (or rows without 16-byte alignment): element loads, -inf past the end,
            // repacked so that both cases continue alike
            float f[GV];
#pragma unroll
            for (int e = 0; e < GV; ++e) f[e] = (x + e < n_valid) ? E::load(row, x + e) : -INFINITY;
            if constexpr (E::kBytes == 4) {
                raw[j] = make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
            } else {
                raw[j].x = E::to_bits(f[0]) | (E::to_bits(f[1]) << 16);
                raw[j].y = E::to_bits(f[2]) | (E::to_bits(f[3]) << 16);
                raw[j].z = E::to_bits(f[4]) | (E::to_bits(f[5]) << 16);
                raw[j].w = E::to_bits(f[6]) | (E::to_bits(f[7]) << 16);
            }
        }
    }
    typename E::MaxAcc acc = E::max_init();
#pragma unroll
    for (int j = 0; j < NG; ++j) E::max_step(acc, raw[j]);
    ref = int_ref(warp_max(E::max_final(acc)) * scale);
    const float r0 = (ref == -INFINITY) ? 0.f : ref;
    // four running sums, by element index modulo 4 in the thread's own order: what the packed
    // accumulators of node_kernel hold
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        float f[GV];
        E::unpack(raw[j], f);
#pragma unroll
        for (int e = 0; e < GV; e += 4) {
            a0 += ex2f(fmaf(f[e], scale, -r0));
            a1 += ex2f(fmaf(f[e + 1], scale, -r0));
            a2 += ex2f(fmaf(f[e + 2], scale, -r0));
            a3 += ex2f(fmaf(f[e + 3], scale, -r0));
        }
    }
    z = (a0 + a2) + (a1 + a3);
}

template <int DT, int EPT>
__global__ void __launch_bounds__(kNodeThreads, Elem<DT>::kBytes == 2 ? 8 : 4)
stream_stats_kernel(const __grid_constant__ StreamParams P)
{
    using E = Elem<DT>;
    constexpr int RUN = 32 * EPT;
    const int lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long n_items = static_cast<long long>(P.B) * P.n_list * P.n_entries;
    const long long warp_id = (static_cast<long long>(blockIdx.x) * kNodeThreads + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * kNodeThreads) >> 5;
    for (long long item = warp_id; item < n_items; item += n_warps) {
        const long long bi = item / P.n_entries;
        const int e = static_cast<int>(item - bi * P.n_entries);
        const int b = static_cast<int>(bi / P.n_list), n = P.item_node[bi - static_cast<long long>(b) * P.n_list];
        int n_valid = P.V - e * RUN;    // (a run past the end of the vocabulary holds nothing: statistics (-inf, 0))
        n_valid = n_valid > RUN ? RUN : (n_valid < 0 ? 0 : n_valid);
        const long long node_idx = static_cast<long long>(b) * P.n_nodes + n;
        const unsigned char *t_row = reinterpret_cast<const unsigned char *>(P.target) +
            (node_idx * P.ld_t + static_cast<long long>(e) * RUN) * E::kBytes;
        float rt, zt;
        stream_run<DT, EPT>(t_row, n_valid, P.vector_ok != 0, P.scale, lane, rt, zt);
        const float st = warp_sum(zt);
        if (n >= P.n_internal) {
            if (lane == 0) {
                P.leaf_part[(static_cast<long long>(b) * (P.n_nodes - P.n_internal) + (n - P.n_internal)) * kLeafEntries + e] =
                    make_float2(rt, st);
                if (e == 0) P.node_accept[node_idx] = -1;
            }
            continue;
        }
        const unsigned char *d_row = reinterpret_cast<const unsigned char *>(P.draft) +
            ((static_cast<long long>(b) * P.n_internal + n) * P.ld_d + static_cast<long long>(e) * RUN) * E::kBytes;
        float rd, zd;
        stream_run<DT, EPT>(d_row, n_valid, P.vector_ok != 0, P.scale, lane, rd, zd);
        const float sd = warp_sum(zd);
        if (lane == 0)
            P.single_part[(static_cast<long long>(b) * P.n_internal + n) * kLeafEntries + e] = make_float4(rt, st, rd, sd);
    }
}

// The one test of every node that has exactly one child (all-node form), from the per-run
// statistics the node kernel left: one warp per node.  The arithmetic is the leader warp's.
struct SingleParams {
    const void *target;
    const void *draft;
    const int32_t *cand;
    const float *unif;
    const float4 *single_part;
    int32_t *node_accept;
    float *node_ratio;   // may be null
    NodeStats *stats;
    long long ld_t, ld_d;
    int32_t B, n_nodes, n_internal, V, n_entries, mode, pdl;
    float scale, scale_lo;
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
};

template <int DT>
__global__ void __launch_bounds__(kNodeThreads)
single_decide_kernel(const __grid_constant__ SingleParams P)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (P.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
    const long long n_items = static_cast<long long>(P.B) * P.n_internal;
    const long long warp_id = (static_cast<long long>(blockIdx.x) * kNodeThreads + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * kNodeThreads) >> 5;
    for (long long item = warp_id; item < n_items; item += n_warps) {
        const int b = static_cast<int>(item / P.n_internal), n = static_cast<int>(item - static_cast<long long>(b) * P.n_internal);
        if (P.child_count[n] != 1) continue;
        const long long node_idx = static_cast<long long>(b) * P.n_nodes + n;
        const int first = P.child_first[n];
        const float4 ent = lane < P.n_entries ? P.single_part[item * kLeafEntries + lane]
                                              : make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
        const float R_t = warp_max(ent.x), R_d = warp_max(ent.z);
        const float Z_t = warp_sum(ent.y * exp2i(ent.x - R_t));
        const float Z_d = warp_sum(ent.w * exp2i(ent.z - R_d));
        if (lane != 0) continue;
        const bool t_ok = Z_t > 0.f && Z_t < INFINITY, d_ok = Z_d > 0.f && Z_d < INFINITY;
        int status_bits = (!t_ok || !d_ok) ? MCSD_STATUS_DEGENERATE : 0;
        const long long ci = static_cast<long long>(b) * P.n_nodes + first;
        const int xi = P.cand[ci];
        const double ui = static_cast<double>(fminf(P.unif[2 * ci], 1.f));
        const bool valid = xi >= 0 && xi < P.V;
        if (!valid) status_bits |= MCSD_STATUS_BAD_TOKEN;
        const double K = static_cast<double>(Z_t) * static_cast<double>(Z_d);
        double px = 0.0, qx = 0.0;
        if (valid && t_ok && d_ok) {
            const float lt = E::load(reinterpret_cast<const unsigned char *>(P.target) + node_idx * P.ld_t * E::kBytes, xi);
            const float ld = E::load(reinterpret_cast<const unsigned char *>(P.draft) +
                                     (static_cast<long long>(b) * P.n_internal + n) * P.ld_d * E::kBytes, xi);
            int int_t, int_d;
            const float frac_t = split_exp2(lt, P.scale, P.scale_lo, int_t);
            const float frac_d = split_exp2(ld, P.scale, P.scale_lo, int_d);
            px = static_cast<double>(frac_t) * exp2i_d(int_t - static_cast<int>(R_t)) * static_cast<double>(Z_d);
            qx = static_cast<double>(frac_d) * exp2i_d(int_d - static_cast<int>(R_d)) * static_cast<double>(Z_t);
        }
        // the first test of a node: c = 0, S = 1, W = 1 (in units of K)
        const double Wk = K;
        const bool zero_q = !valid || !(qx > 0.0) || !(Wk > 0.0);
        const double Pn = px > 0.0 ? px : 0.0;
        const bool accept = !zero_q && ui * qx * K <= Pn * Wk;
        if (P.node_ratio) P.node_ratio[ci] = zero_q ? -1.f : static_cast<float>(Pn / (qx * K / Wk));
        // rejected: the residual moves on to c = S / W = 1 (0 where there is no q); its sum is the walk stage's
        const float c_final = accept ? 0.f : ((Wk > 0.0) ? 1.f : 0.f);
        P.node_accept[node_idx] = accept ? first : -1;
        reinterpret_cast<float4 *>(&P.stats[node_idx])[0] = make_float4(R_t, R_d, Z_t, Z_d);
        reinterpret_cast<float4 *>(&P.stats[node_idx])[1] = make_float4(c_final, 0.f, __int_as_float(status_bits), 0.f);
    }
}

}  // namespace mcsd
