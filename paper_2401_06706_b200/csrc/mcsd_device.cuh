// Device code of the MCSD verification library (sm_100a).
//
// Three kernels:
//   node_kernel      T > 0.  One thread-block cluster per tree node, persistent over the
//                    (sequence, node) items.  Each CTA of the cluster owns a contiguous
//                    slice of the vocabulary.  Its slice of the target row goes straight
//                    into registers with coalesced 128-bit loads; its slice of the draft
//                    row (nodes that have children) is brought into shared memory with
//                    one bulk async copy (TMA, to this CTA alone) and stays there.  Both are
//                    exponentiated once and then stay on chip while the k candidates of
//                    the node are tested in order (Algorithm 1 / Algorithm 2), so every
//                    logit row is read from HBM exactly once.  The rows of the cluster's
//                    next item are prefetched into L2 while the current one is computed.
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
// So one rejection costs one scalar-parameter reduction over the on-chip p and q,
// and nothing is written back.  c_1 = 1 whatever the candidates are, so the first
// reduction is started before the first test has been decided.
//
// Softmax references are integers (ceil of the scaled row maximum, in log2 units), so
// moving a partial sum from one reference to another is an exact multiplication by a
// power of two and every thread can exponentiate against its own maximum.
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
// Polls of a bounded wait before it gives up; with the back-off between polls the
// bound is about two seconds, far beyond any legitimate wait.
constexpr uint32_t kWaitPolls = 1u << 21;

struct __align__(16) NodeStats {
    float r_t, r_d;  // references of the sums: ceil(row maximum * scale), log2 units
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
    float *node_ratio;  // may be null
    NodeStats *stats;   // [B][n_nodes], written for nodes with children
    float2 *leaf_part;  // [B][n_nodes - n_internal][32] per-warp (reference, sum) of every leaf row
    int32_t *status;  // [B]
    long long ld_t, ld_d;
    int32_t B, n_nodes, n_internal, V;
    int32_t slice;   // vocabulary elements owned by one CTA of the cluster
    int32_t n_items; // B * n_nodes
    int32_t step_b, step_n;  // quotient and remainder of (clusters in the grid) / n_nodes
    // Path mode (one launch per tree level): the items are the sequences, item b works on node
    // path_cur[b] (negative: that walk has ended, nothing to do) and leaves in path_next[b] the
    // accepted child, or -1.  Null for the all-node form.  Then step_b = clusters, step_n = 0.
    const int32_t *path_cur;
    int32_t *path_next;
    int32_t mode;
    float scale;     // log2(e) / T rounded to float ...
    float scale_lo;  // ... and what the rounding dropped (for the candidates' own probabilities)
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
};

// ------------------------------------------------------------------ element types
// Three-input maximum (a NaN operand is ignored, as with fmaxf).
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d; asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c)); return d;
}

// Per element type: unpacking of one 16-byte vector, scalar access, and a running maximum
// over whole vectors that stays in the packed format for 2-byte types (two elements per
// instruction) and is turned into a float once at the end.
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
    // value of element i given the aligned 32-bit word that contains it
    static __device__ __forceinline__ float from_word(uint32_t w, long long) { return __uint_as_float(w); }
    typedef float2 MaxAcc;
    static __device__ __forceinline__ MaxAcc max_init() { return make_float2(-INFINITY, -INFINITY); }
    static __device__ __forceinline__ void max_step(MaxAcc &a, const uint4 &r) {
        a.x = max3(a.x, __uint_as_float(r.x), __uint_as_float(r.y));
        a.y = max3(a.y, __uint_as_float(r.z), __uint_as_float(r.w));
    }
    static __device__ __forceinline__ float max_final(const MaxAcc &a) { return fmaxf(a.x, a.y); }
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
    static __device__ __forceinline__ float from_word(uint32_t w, long long i) {
        return __uint_as_float((i & 1) ? (w & 0xffff0000u) : (w << 16));
    }
    // 16-bit pattern of a value that this type represents exactly
    static __device__ __forceinline__ uint32_t to_bits(float f) { return __float_as_uint(f) >> 16; }
    typedef uint32_t MaxAcc;
    static __device__ __forceinline__ uint32_t mx(uint32_t a, uint32_t b) {
        const __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&a),
                                         *reinterpret_cast<const __nv_bfloat162 *>(&b));
        return *reinterpret_cast<const uint32_t *>(&r);
    }
    static __device__ __forceinline__ MaxAcc max_init() { return 0xff80ff80u; }  // (-inf, -inf)
    static __device__ __forceinline__ void max_step(MaxAcc &a, const uint4 &r) {
        a = mx(a, mx(mx(r.x, r.y), mx(r.z, r.w)));
    }
    static __device__ __forceinline__ float max_final(const MaxAcc &a) { return fmaxf(from_word(a, 0), from_word(a, 1)); }
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
    static __device__ __forceinline__ float from_word(uint32_t w, long long i) {
        const unsigned short h = static_cast<unsigned short>((i & 1) ? (w >> 16) : (w & 0xffffu));
        return __half2float(__ushort_as_half(h));
    }
    static __device__ __forceinline__ uint32_t to_bits(float f) { return __half_as_ushort(__float2half_rn(f)); }
    typedef uint32_t MaxAcc;
    static __device__ __forceinline__ uint32_t mx(uint32_t a, uint32_t b) {
        const __half2 r = __hmax2(*reinterpret_cast<const __half2 *>(&a), *reinterpret_cast<const __half2 *>(&b));
        return *reinterpret_cast<const uint32_t *>(&r);
    }
    static __device__ __forceinline__ MaxAcc max_init() { return 0xfc00fc00u; }  // (-inf, -inf)
    static __device__ __forceinline__ void max_step(MaxAcc &a, const uint4 &r) {
        a = mx(a, mx(mx(r.x, r.y), mx(r.z, r.w)));
    }
    static __device__ __forceinline__ float max_final(const MaxAcc &a) { return fmaxf(from_word(a, 0), from_word(a, 1)); }
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
// Bounded wait with back-off (a waiting thread must not eat the issue slots of the
// working ones): false when the poll budget ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitPolls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(i < 64 ? 64 : 1000);
    }
    return false;
}
// One bulk async copy global -> this CTA's shared memory (TMA; the copy goes to this CTA alone);
// completion is signalled on an mbarrier of this CTA as a byte count.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Asks L2 to fetch a 16-byte-aligned range (size a multiple of 16); nothing waits on it.
__device__ __forceinline__ void bulk_prefetch_l2(const void *src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
// 4-byte asynchronous copy global -> shared (no register holds the value in flight).
// Orders this thread's earlier ordinary shared-memory accesses before later bulk
// (async-proxy) copies into the same locations.
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void cp_async4(void *smem_dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(smem_dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.wait_all;" ::: "memory");
}
// 128-bit streaming load (read once, do not keep in L1).
__device__ __forceinline__ uint4 ld_stream_v4(const void *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Asynchronous 16-byte store into a CTA of the cluster that reports its bytes to an
// mbarrier of that CTA: the data is visible to whoever sees the barrier's phase complete,
// no fence on either side.
__device__ __forceinline__ void st_async_f4(uint32_t addr, float4 v, uint32_t remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(remote_bar) : "memory");
}

// Packed pairs of floats: sm_100 executes fma and add on both halves of an aligned
// register pair with one instruction (each half rounds exactly like the scalar operation).
typedef float2 f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) { return make_float2(lo, hi); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) { return __fadd2_rn(a, b); }
// Warp-wide maximum in one instruction (NaN inputs are ignored).
__device__ __forceinline__ float warp_max(float v) {
    float d; asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(d) : "f"(v)); return d;
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
// 2^d for an integer-valued d (a difference of two references): exact; 0 when
// d < -126 (also for d = -inf), clamped to 2^127 above.
__device__ __forceinline__ float exp2i(float d) {
    d = fminf(fmaxf(d, -127.f), 127.f);
    // adding 1.5 * 2^23 leaves the integer in the low mantissa bits (no conversion instruction)
    const int i = __float_as_int(d + 12582912.f) - 0x4b400000;
    return __int_as_float((i + 127) << 23);
}
// The same in double for an integer e: 0 below 2^-1000.
__device__ __forceinline__ double exp2i_d(int e) {
    if (e < -1000) return 0.0;
    e = e > 1000 ? 1000 : e;
    return __hiloint2double((e + 1023) << 20, 0);
}
// 2^(l * (scale + scale_lo)) as 2^ip * (return value), ip an integer and the return value
// in [2^-0.51, 2^0.51], to about 1e-7 relative however large the exponent is: the
// product is formed exactly as a sum of two floats, its integer part goes to ip and only
// the fraction is exponentiated.  Infinite or NaN products give 0 (or +inf) with ip = 0.
__device__ __forceinline__ float split_exp2(float l, float scale, float scale_lo, int &ip) {
    const float ph = l * scale;
    ip = 0;
    if (!(fabsf(ph) < 1.0e9f)) return ph > 0.f ? INFINITY : 0.f;
    const float pe = fmaf(l, scale, -ph);      // exact error of the rounded product
    const float pl = fmaf(l, scale_lo, pe);    // plus the part of the scale that float drops
    const float ipf = rintf(ph);
    const float f = (ph - ipf) + pl;           // |f| <= 0.5 + tiny; the subtraction is exact
    ip = static_cast<int>(ipf);
    // Taylor series of exp(f ln 2), |f ln 2| <= 0.36: the degree-7 remainder is below 6e-9
    float y = 1.5252733804059841e-05f;
    y = fmaf(y, f, 1.5403530393381608e-04f);
    y = fmaf(y, f, 1.3333558146428443e-03f);
    y = fmaf(y, f, 9.6181291076284772e-03f);
    y = fmaf(y, f, 5.5504108664821580e-02f);
    y = fmaf(y, f, 2.4022650695910071e-01f);
    y = fmaf(y, f, 6.9314718055994531e-01f);
    return fmaf(y, f, 1.f);
}
// Integer reference of a set whose largest scaled logit is m (log2 units); -inf for
// an empty set.  NaN-free inputs give ceil(m), so that every exponent is <= 0.
__device__ __forceinline__ float int_ref(float m_scaled) {
    return (m_scaled == -INFINITY) ? -INFINITY : ceilf(m_scaled);
}

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

// ------------------------------------------------------------------ node kernel
// Warp totals of N values per lane in N-1 + (5 - log2 N) shuffles instead of 5 N: each
// halving step pairs lanes and splits the value indices between them.  On return
// every lane holds in `out` the warp total of value index `idx` (the return value),
// idx = lane / (32 / N).
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
    static_assert(N == 1 || N == 2 || N == 4 || N == 8 || N == 16, "unsupported count");
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
    if constexpr (N >= 16) halve_step<N / 16>(w, lane, 2, idx);
    else w[0] += __shfl_xor_sync(0xffffffffu, w[0], 2);
    w[0] += __shfl_xor_sync(0xffffffffu, w[0], 1);
    out = w[0];
    return idx;
}

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
// PATH: the items are the sequences, each at the node its walk stands on (see NodeParams).
//
// Ownership inside a CTA: the slice is cut into 16-byte groups of GV elements; thread
// (warp w, lane l) owns groups (w * NG + j) * 32 + l, j < NG, so that one warp-wide
// access is contiguous and a warp's elements are one contiguous run of the vocabulary.
// Groups past the end of the slice hold -inf (probability 0).
//
// Every decision of the rejection loop is taken by every warp of the cluster from
// bit-identical inputs, so all CTAs of a cluster execute the same number of exchange
// rounds (the byte counts the exchange barriers are armed with rely on it).
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
    constexpr bool kPrefetch = !DIRECT && E::kBytes == 2;
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

    const int tid = threadIdx.x, lane = tid & 31;
    // (broadcast from lane 0 so that the compiler knows the warp index is warp-uniform)
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const uint32_t crank = __clusterRelativeBlockRank(), csize = __clusterSizeInBlocks();
    const int cluster_id = blockIdx.x / csize;
    const int n_entries = static_cast<int>(csize) * NW;  // values per exchange round (<= 32)
    const float scale = P.scale;
    const uint32_t full_addr = smem_u32(&full_bar);
    const uint32_t xbar_addr[2] = {smem_u32(&xch.bar[0]), smem_u32(&xch.bar[1])};

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

    if (tid == 0) {
        mbar_init(full_addr, 1);
        mbar_init(xbar_addr[0], 1);
        mbar_init(xbar_addr[1], 1);
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
        if (tid == 0) mbar_arrive_expect_tx(xbar_addr[s], static_cast<uint32_t>(n_entries) * 16u);
        if (lane < static_cast<int>(csize)) {
            const uint32_t dst = map_to_rank(smem_u32(&xch.slot[s][crank * NW + warp]), lane);
            st_async_f4(dst, mine, map_to_rank(xbar_addr[s], lane));
        }
    };
    // leader (warp 0) only: waits for the round and returns entry `lane`
    auto exchange_leader_wait = [&](float4 identity) -> float4 {
        const uint32_t s = round & 1u;
        // once a wait has expired the results are void and later rounds do not wait again
        if (!poisoned && !mbar_wait(xbar_addr[s], (round >> 1) & 1u)) poisoned = 1;
        return lane < n_entries ? xch.slot[s][lane] : identity;
    };
    // all warps: ends the round (the other warps have been waiting here for the leader)
    auto exchange_release = [&]() {
        __syncthreads();
        ++round;
    };

    // (sequence, node) of the items this cluster visits: the current one and the two after
    // it, advanced by the precomputed quotient and remainder of the stride
    auto advance = [&](int &b, int &n) {
        b += P.step_b;
        n += P.step_n;
        if (n >= P.n_nodes) { n -= P.n_nodes; ++b; }
        if (PATH) n = b < P.B ? __ldg(P.path_cur + b) : 0;
    };

    // ---- candidate pipeline (the fetch warp only) -------------------------------------------
    auto fetch_tokens = [&](int b, int n, int slot3) {
        if (b < P.B) {
            const int k = ((!PATH || n >= 0) && n < P.n_internal) ? P.child_count[n] : 0;
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
            const int k = ((!PATH || n >= 0) && n < P.n_internal) ? P.child_count[n] : 0;
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

    int b = cluster_id / P.n_nodes, n = cluster_id - b * P.n_nodes;  // current item
    if (PATH) { b = cluster_id; n = b < P.B ? __ldg(P.path_cur + b) : 0; }
    int b1 = b, n1 = n;                                              // the next one
    advance(b1, n1);
    uint32_t it = 0;  // iteration count of this cluster
    bool prev_internal = false;
    if (warp == kFetchWarp) {
        fetch_tokens(b, n, 0);
        cp_async_wait_all();
        __syncwarp();
        fetch_logits(b, n, 0, 0);
        fetch_tokens(b1, n1, 1);
    }
    if (kPrefetch && tid == 0 && b < P.B && bulk_bytes) {
        bulk_prefetch_l2(t_slice(static_cast<long long>(b) * P.n_nodes + n), bulk_bytes);
        if (n < P.n_internal) bulk_prefetch_l2(d_slice(b, n), bulk_bytes);
    }

    for (; b < P.B; ++it) {
        const bool internal = (!PATH || n >= 0) && n < P.n_internal;
        const int k = internal ? P.child_count[n] : 0;
        const int first = P.child_first[n];
        const long long node_idx = static_cast<long long>(b) * P.n_nodes + n;
        const int s3 = it % 3u, s2 = it & 1u;
        int status_bits = 0;

        // this item's candidate data has landed (it was requested one item ago) ...
        if (warp == kFetchWarp) cp_async_wait_all();
        // ... and, around an item with children, all warps meet: they are done with the
        // previous item (its draft buffer and ring entries may be overwritten) and they
        // see this item's ring entries.  A run of leaves needs no meeting at all.
        if (internal || prev_internal) {
            if (!DIRECT) fence_proxy_async();
            __syncthreads();
        }
        prev_internal = internal;

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
            if (warp == kFetchWarp) {
                if (kPrefetch && lane == 0 && b1 < P.B && bulk_bytes) {
                    bulk_prefetch_l2(t_slice(static_cast<long long>(b1) * P.n_nodes + n1), bulk_bytes);
                    if (n1 < P.n_internal) bulk_prefetch_l2(d_slice(b1, n1), bulk_bytes);
                }
                fetch_logits(b1, n1, (it + 1) % 3u, s2 ^ 1);
                int b2 = b1, n2 = n1;
                advance(b2, n2);
                fetch_tokens(b2, n2, (it + 2) % 3u);
            }
        };
        auto next_item = [&]() {
            b = b1; n = n1;
            advance(b1, n1);
        };

        if (PATH && n < 0) {  // this walk ended at an earlier level
            if (crank == 0 && tid == 0) P.path_next[b] = -1;
            look_ahead();
            next_item();
            continue;
        }

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
        } else {
#pragma unroll
            for (int j = 0; j < NG; ++j) {
                const int g = g0 + j * 32;
                float f[GV];
                if (!DIRECT && g < n_full_groups) {
                    E::unpack(ld_stream_v4(t_row + static_cast<size_t>(g) * 16), f);
                } else if (g * GV >= n_mine) {  // wholly past the data
#pragma unroll
                    for (int e = 0; e < GV; ++e) f[e] = -INFINITY;
                } else {
#pragma unroll
                    for (int e = 0; e < GV; ++e) f[e] = (g * GV + e < n_mine) ? E::load(t_row, g * GV + e) : -INFINITY;
                }
#pragma unroll
                for (int e = 0; e < GV; e += 2) tv[(j * GV + e) / 2] = pack2(f[e], f[e + 1]);
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
                P.leaf_part[(static_cast<long long>(b) * (P.n_nodes - P.n_internal) + (n - P.n_internal)) * 32 +
                            crank * NW + warp] = make_float2(rt, st);
            if (crank == 0 && tid == 0) {
                P.node_accept[node_idx] = -1;
                if (PATH) P.path_next[b] = -1;
            }
            look_ahead();
            next_item();
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
        double px = 0.0, qx = 0.0;  // lane i of the leader: candidate i's p and q, times K
        int cand_i = 0, attempt = 0, accepted = -1, my_tok = -1;
        float u_acc = 2.f;
        // tests candidates from cand_i on until one is accepted (returns 0), all are rejected
        // (returns 0) or one is rejected and its residual sum is needed (returns 1, c_try set)
        auto leader_decide = [&]() -> int {
            while (cand_i < k) {
                const int i = cand_i;
                const int xi = __shfl_sync(0xffffffffu, my_tok, i);
                const double ui = static_cast<double>(__shfl_sync(0xffffffffu, u_acc, i));
                const double pxi = __shfl_sync(0xffffffffu, px, i), qxi = __shfl_sync(0xffffffffu, qx, i);
                const bool valid = xi >= 0 && xi < P.V;
                if (!valid) status_bits |= MCSD_STATUS_BAD_TOKEN;
                // Algorithm 2: a token rejected earlier at this node has draft probability 0 now
                const bool dup = P.mode == 1 &&
                    (__ballot_sync(0xffffffffu, lane < i && my_tok == xi) != 0u);
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
                attempt = 0;
                return 1;
            }
            return 0;
        };

        if (warp == 0) {
            // while the round is in flight: 2^(scaled logit) of the candidates' own logits as
            // 2^int * frac (lane i = candidate i)
            float frac_t = 0.f, frac_d = 0.f;
            int int_t = 0, int_d = 0;
            bool cand_ok = false;
            if (lane < k) {
                my_tok = ring.tok[s3][lane];
                u_acc = ring.u[s3][lane];
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
            if (!t_ok) status_bits |= MCSD_STATUS_NO_MASS;
            // candidates' probabilities, both multiplied by K so that no division is needed:
            // px' = 2^(l_t*scale - R_t) * Z_d, qx' = 2^(l_d*scale - R_d) * Z_t
            K = static_cast<double>(Z_t) * static_cast<double>(Z_d);
            Wk = K;
            if (cand_ok && t_ok && d_ok) {
                px = static_cast<double>(frac_t) * exp2i_d(int_t - static_cast<int>(R_t)) * static_cast<double>(Z_d);
                qx = static_cast<double>(frac_d) * exp2i_d(int_d - static_cast<int>(R_d)) * static_cast<double>(Z_t);
            }
            const int more = leader_decide();
            if (lane == 0) {
                act[round & 1u].stats = make_float4(R_t, R_d, t_ok ? 1.f / Z_t : 0.f, (t_ok && d_ok) ? Z_t / Z_d : 0.f);
                act[round & 1u].c_try = static_cast<float>(c_try);
                act[round & 1u].more = more;
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
                int next;
                if (S_new > 0.f) {
                    if (attempt == 0) { c = c_try; S = static_cast<double>(S_new); }
                    ++cand_i;
                    next = leader_decide();
                } else {
                    // zero residual mass: keep the previous residual (recompute its sums once)
                    status_bits |= MCSD_STATUS_DEGENERATE;
                    if (attempt == 0) { attempt = 1; c_try = c; next = 1; }
                    else { ++cand_i; next = leader_decide(); }
                }
                if (lane == 0) {
                    act[round & 1u].c_try = static_cast<float>(c_try);
                    act[round & 1u].more = next;
                }
            }
            exchange_release();
            more = act[(round - 1u) & 1u].more;
            c_next = act[(round - 1u) & 1u].c_try;
        }

        // ---- per-node results (the endpoint token is drawn by the walk kernel, and only
        // for the node where a walk stops)
        if (warp == 0) {
            if (crank == 0 && lane == 0) {
                P.node_accept[node_idx] = accepted;
                if (PATH) P.path_next[b] = accepted;
                reinterpret_cast<float4 *>(&P.stats[node_idx])[1] =
                    make_float4(static_cast<float>(c), static_cast<float>(S), 0.f, 0.f);
            }
        }
        if (poisoned) status_bits |= MCSD_STATUS_TIMEOUT;
        status_bits = __reduce_or_sync(0xffffffffu, status_bits);
        if (status_bits && lane == 0) atomicOr(P.status + b, status_bits);
        next_item();
    }

    if (warp == kFetchWarp) cp_async_wait_all();
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
                if (P.path_next) P.path_next[item] = acc;
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ walk + endpoint + residual
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
    float *out = P.out_residual ? P.out_residual + static_cast<long long>(b) * P.V : nullptr;

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

// ------------------------------------------------------------------ candidate sampling (Eq. 1)
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
    float scale;                  // log2(e)/T, or 0 for top-k
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
};

// One CTA per (sequence, node with children): draws the tokens of the node's k children from
// softmax(draft row / T) by inverse CDF in token order with one supplied uniform each
// (Section 3.2).  With replacement the k draws are independent; without (Eq. 1) every
// drawn token is taken out of the distribution before the next draw, which here means
// subtracting its weight from the partial sums of its lane, its warp's run and the
// element scan.  The row is read once (twice for its maximum, the second time from L2);
// temperature 0 takes the k largest logits instead (lowest index first on ties).
// NT threads per CTA: 512 (two CTAs per SM, two independent chains) when the vocabulary fits
// 16 steps per warp, else 1024.
template <int DT, int NT>
__global__ void __launch_bounds__(NT, NT == 512 ? 2 : 1)
sample_kernel(const __grid_constant__ SampleParams P)
{
    using E = Elem<DT>;
    constexpr int GV = E::kVec;
    constexpr int kStep = 32 * GV;
    constexpr int kW = NT / 32;  // warps
    constexpr int kMaxSteps = MCSD_MAX_VOCAB / 32 / kStep;  // steps of a warp's run (the host picks NT so that they suffice)
    __shared__ float s_wtot[32];
    __shared__ float s_red[32];
    __shared__ int s_redi[32];
    __shared__ int32_t s_rem_tok[MCSD_MAX_CHILDREN];
    __shared__ int s_pick;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / P.n_range, n = P.node_begin + (blockIdx.x - b * P.n_range);
    const int k = P.child_count[n], first = P.child_first[n];
    if (k == 0) return;
    int32_t *out = P.cand + static_cast<long long>(b) * P.n_nodes + first;
    const unsigned char *row = reinterpret_cast<const unsigned char *>(P.draft) +
        (static_cast<long long>(b) * P.n_internal + n) * P.ld_d * E::kBytes;
    auto load_group = [&](int x0, float *v) {   // GV logits from x0 on, -inf past the vocabulary
        if (P.vector_ok && x0 + GV <= P.V) {
            E::unpack(__ldg(reinterpret_cast<const uint4 *>(row + static_cast<size_t>(x0) * E::kBytes)), v);
        } else {
#pragma unroll
            for (int e = 0; e < GV; ++e) v[e] = x0 + e < P.V ? E::load(row, x0 + e) : -INFINITY;
        }
    };
    const int run = ((P.V + kW - 1) / kW + kStep - 1) / kStep * kStep;
    const int x_lo = warp * run;
    int x_hi = x_lo + run;
    x_hi = x_hi > P.V ? P.V : x_hi;

    if (P.scale == 0.f) {
        // ---- top-k: k block-wide maxima, each over the elements that come after the previous
        // pick in the order (logit descending, index ascending)
        float pv = INFINITY;
        int pi = -1;
        for (int i = 0; i < k; ++i) {
            float best = -INFINITY;
            int best_i = 0x7fffffff;
            for (int x0 = x_lo + lane * GV; x0 < x_hi; x0 += kStep) {
                float v[GV];
                load_group(x0, v);
#pragma unroll
                for (int e = 0; e < GV; ++e) {
                    const int x = x0 + e;
                    const bool after = i == 0 || v[e] < pv || (v[e] == pv && x > pi);
                    if (x < P.V && after && v[e] > best) { best = v[e]; best_i = x; }  // ascending x: ties keep the lowest
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best, o);
                const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
                if (ov > best || (ov == best && oi < best_i)) { best = ov; best_i = oi; }
            }
            if (lane == 0) { s_red[warp] = best; s_redi[warp] = best_i; }
            __syncthreads();
            best = lane < kW ? s_red[lane] : -INFINITY;
            best_i = lane < kW ? s_redi[lane] : 0x7fffffff;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best, o);
                const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
                if (ov > best || (ov == best && oi < best_i)) { best = ov; best_i = oi; }
            }
            pv = best;
            pi = best_i == 0x7fffffff ? -1 : best_i;
            if (tid == 0) out[i] = pi;
            __syncthreads();
        }
        return;
    }

    // ---- reference of the row: ceil(max * scale)
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
    const float ref = int_ref(warp_max(lane < kW ? s_red[lane] : -INFINITY) * P.scale);
    const float ref0 = ref == -INFINITY ? 0.f : ref;
    auto weights = [&](int x0, float *w) {
        float v[GV];
        load_group(x0, v);
#pragma unroll
        for (int e = 0; e < GV; ++e) w[e] = ex2f(fmaf(v[e], P.scale, -ref0));
    };
    // ---- unnormalised weights: per lane the sum of its group in every step, per warp its run
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
            for (int e = 0; e < GV; ++e) g[st] += w[e];
            mass += g[st];
        }
    }
    mass = warp_sum(mass);
    if (lane == 0) s_wtot[warp] = mass;
    __syncthreads();

    int n_rem = 0;  // tokens taken out so far (Eq. 1); the same in every thread
    for (int i = 0; i < k; ++i) {
        const float u = P.unif_draw[static_cast<long long>(b) * P.n_nodes + first + i];
        // the run that holds the quantile (every warp finds the same one)
        const float m = lane < kW ? s_wtot[lane] : 0.f;
        const float total = warp_sum(m);
        const float target = u * total;
        const float inc = warp_scan_incl(m, lane);
        const unsigned hit = __ballot_sync(0xffffffffu, m > 0.f && inc > target);
        const unsigned pos = __ballot_sync(0xffffffffu, m > 0.f);
        const int pick = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : -1);
        int found = -1;
        if (pick >= 0 && total > 0.f && warp == pick) {
            const float tgt = target - __shfl_sync(0xffffffffu, inc - m, pick);
            float tj;
            warp_multi_sum<kMaxSteps>(g, lane, tj);
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
            float t2 = tgt - ps_before;
            if (ps < 0) { ps = last_s; t2 = INFINITY; }   // rounding: take the run's last element with mass
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
                        const int x0 = x_lo + ps * kStep + lane * GV;
                        float w[GV];
                        weights(x0, w);
                        const float rem = t2 - (gi - gs);
                        float acc = 0.f;
#pragma unroll
                        for (int e = 0; e < GV; ++e) {
                            bool gone = false;
                            for (int j = 0; j < n_rem; ++j) gone |= s_rem_tok[j] == x0 + e;
                            if (!gone && w[e] > 0.f) {
                                acc += w[e];
                                last = e;
                                if (pe < 0 && acc > rem) pe = e;
                            }
                        }
                        if (pe < 0) pe = last;
                        if (pe >= 0 && P.mode == 1) {
                            // Eq. 1: the drawn token leaves the distribution.  The group's sum is
                            // formed again from the tokens that remain (subtracting would lose
                            // everything when the drawn token dominated the group)
                            float rest = 0.f;
#pragma unroll
                            for (int e = 0; e < GV; ++e) {
                                bool gone = e == pe;
                                for (int j = 0; j < n_rem; ++j) gone |= s_rem_tok[j] == x0 + e;
                                if (!gone) rest += w[e];
                            }
#pragma unroll
                            for (int st = 0; st < kMaxSteps; ++st)
                                if (st == ps) g[st] = rest;
                        }
                    }
                    found = __shfl_sync(0xffffffffu, pe < 0 ? -1 : x_lo + ps * kStep + lane * GV + pe, l);
                    if (P.mode == 1 && found >= 0) {
                        // ... and so is the run's total, from the lanes' current group sums
                        float rs = 0.f;
#pragma unroll
                        for (int st = 0; st < kMaxSteps; ++st) rs += g[st];
                        rs = warp_sum(rs);
                        if (lane == 0) s_wtot[warp] = rs;
                    }
                }
            }
            if (lane == 0) s_pick = found;
        }
        if (pick < 0 || !(total > 0.f)) { if (tid == 0) s_pick = -1; }
        __syncthreads();
        found = s_pick;
        if (tid == 0) {
            out[i] = found;
            if (found < 0 && P.status) atomicOr(P.status + b, MCSD_STATUS_NO_MASS);
            if (P.mode == 1) s_rem_tok[n_rem] = found;
        }
        if (P.mode == 1 && found >= 0) ++n_rem;
        __syncthreads();
    }
}

// ------------------------------------------------------------------ naive sampling (ablation baseline)
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

// Multi-candidate naive sampling, the baseline that Section 4.4 and Appendix C compare
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
    __shared__ float s_wtot[kWalkWarps];
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
            E::unpack(__ldg(reinterpret_cast<const uint4 *>(row + static_cast<size_t>(x0) * E::kBytes)), v);
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
        float mass = 0.f;
#pragma unroll
        for (int st = 0; st < kMaxSteps; ++st) {
            g[st] = 0.f;
            const int x0 = x_lo + st * kStep + lane * GV;
            if (x0 < x_hi) {
                float w[GV];
                weights(x0, w);
#pragma unroll
                for (int e = 0; e < GV; ++e) g[st] += w[e];
                mass += g[st];
            }
        }
        mass = warp_sum(mass);
        if (lane == 0) s_wtot[warp] = mass;
        if (tid == 0) s_pick = -1;
        __syncthreads();
        // the draw: run, step, lane, element
        const float u = P.unif[2 * (nb + n) + 1];
        const float m = s_wtot[lane];
        total = warp_sum(m);
        const float target = u * total;
        const float inc = warp_scan_incl(m, lane);
        const unsigned hit = __ballot_sync(0xffffffffu, m > 0.f && inc > target);
        const unsigned pos = __ballot_sync(0xffffffffu, m > 0.f);
        const int pick = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : -1);
        if (pick >= 0 && total > 0.f && warp == pick) {
            const float tgt = target - __shfl_sync(0xffffffffu, inc - m, pick);
            float tj;
            warp_multi_sum<kMaxSteps>(g, lane, tj);
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
            float t2 = tgt - ps_before;
            if (ps < 0) { ps = last_s; t2 = INFINITY; }
            if (ps >= 0) {
                float gs = g[0];
#pragma unroll
                for (int st = 1; st < kMaxSteps; ++st) gs = (ps == st) ? g[st] : gs;
                const float gi = warp_scan_incl(gs, lane);
                const unsigned h2 = __ballot_sync(0xffffffffu, gs > 0.f && gi > t2);
                const unsigned p2 = __ballot_sync(0xffffffffu, gs > 0.f);
                if (p2) {
                    const int l = h2 ? __ffs(h2) - 1 : 31 - __clz(p2);
                    if (lane == l) {
                        const int x0 = x_lo + ps * kStep + lane * GV;
                        float w[GV];
                        weights(x0, w);
                        const float rem = t2 - (gi - gs);
                        float acc = 0.f;
                        int pe = -1, last = -1;
#pragma unroll
                        for (int e = 0; e < GV; ++e) {
                            if (w[e] > 0.f) {
                                acc += w[e];
                                last = e;
                                if (pe < 0 && acc > rem) pe = e;
                            }
                        }
                        if (pe < 0) pe = last;
                        if (pe >= 0) s_pick = x0 + pe;
                    }
                }
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
        if (x < 0) atomicOr(P.status + b, MCSD_STATUS_NO_MASS);
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

// ------------------------------------------------------------------ tree attention layout
struct LayoutParams {
    uint8_t *mask;          // [n_nodes][n_nodes] or null
    int32_t *position_ids;  // [n_nodes] or null
    int32_t n_nodes, prefix_len;
    int16_t parent[MCSD_MAX_NODES];
};

// Section 3.3: row i of the mask marks node i and its ancestors; the position id of a node
// is the root's plus its depth.  One CTA per node: thread 0 climbs to the root marking the
// way in shared memory, then the CTA writes the row.
__global__ void __launch_bounds__(kThreads)
layout_kernel(const __grid_constant__ LayoutParams P)
{
    __shared__ uint8_t s_row[MCSD_MAX_NODES];
    const int i = blockIdx.x;
    for (int j = threadIdx.x; j < P.n_nodes; j += kThreads) s_row[j] = 0;
    __syncthreads();
    if (threadIdx.x == 0) {
        int depth = 0;
        int a = i;
        for (int hop = 0; hop < P.n_nodes && a >= 0; ++hop) {  // bounded even for a corrupt tree
            s_row[a] = 1;
            a = P.parent[a];
            if (a >= 0) ++depth;
        }
        if (P.position_ids) P.position_ids[i] = P.prefix_len + depth;
    }
    __syncthreads();
    if (P.mask)
        for (int j = threadIdx.x; j < P.n_nodes; j += kThreads) P.mask[static_cast<long long>(i) * P.n_nodes + j] = s_row[j];
}

}  // namespace mcsd
