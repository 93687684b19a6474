// Shared pieces of the MCSD device code (sm_100a): limits and bounded-wait constants, the
// per-node record and the parameter block of the node kernel, the element types (fp32,
// bf16, fp16) and the arithmetic, warp and PTX helpers that every kernel uses.
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
// Per-warp statistics entries a leaf row can have (cluster size * warps per CTA of the node kernel).
constexpr int kLeafEntries = kMaxCluster * 4;
// Polls of a bounded wait before it gives up; a poll suspends the thread for up to
// kWaitSuspendNs, so the bound is about two seconds, far beyond any legitimate wait.
constexpr uint32_t kWaitPolls = 1u << 21;
// Longest time one poll may keep a thread suspended (a hint to the hardware).
constexpr uint32_t kWaitSuspendNs = 1000u;

// What the node kernel leaves per node with children (32 bytes, two 16-byte stores).
struct __align__(16) NodeStats {
    float r_t, r_d;  // references of the sums: ceil(row maximum * scale), log2 units
    float z_t, z_d;  // sum_x exp2(l * scale - r)
    // The residual left when every candidate was rejected is max(p - c q, 0) (unnormalised).
    // The sum that follows the LAST rejection is not formed by the node kernel: nothing is
    // tested against that residual, only a walk that stops here draws from it, and the walk
    // kernel forms the sum then.  Should it be zero, the residual before that rejection,
    // max(p - c_prev q, 0), is the one that is kept.
    float c, c_prev;
    int32_t status;  // MCSD_STATUS_* bits met at this node
    int32_t pad;
};

struct NodeParams {
    const void *target;
    const void *draft;
    const int32_t *cand;
    const float *unif;
    int32_t *node_accept;
    float *node_ratio;  // may be null
    NodeStats *stats;   // [B][n_nodes], written for nodes with children
    float2 *leaf_part;  // [B][n_nodes - n_internal][kLeafEntries] per-warp (reference, sum) of every leaf row
    float4 *single_part; // [B][n_internal][kLeafEntries] per-warp (reference, sum) of both rows of every node
                         // with exactly one child (all-node form): such a node is decided by one test
                         // that needs no residual, so it is decided after the kernel, from these
    long long ld_t, ld_d;
    int32_t B, n_nodes, n_internal, V;
    int32_t slice;   // vocabulary elements owned by one CTA of the cluster
    int32_t n_items; // B * n_list
    // The nodes of a tree this launch evaluates, in ascending order: all of them, or (large
    // launches of the all-node form) only those with two or more children, the others being left
    // to stream_stats_kernel.  Item i is (sequence i / n_list, node item_node[i % n_list]).
    int32_t n_list;
    int32_t step_b, step_n;  // quotient and remainder of (clusters in the grid) / n_list
    // Path mode: the items are the sequences (step_b = clusters in the grid, step_n = 0); a cluster
    // follows each of its sequences from the root through the accepted children and evaluates
    // only the nodes on that walk.
    int32_t mode;
    uint32_t wait_polls;      // poll budget of the exchange wait (kWaitPolls unless a test shortens it)
    uint32_t test_extra_tx;   // 0; a test of the expiry path arms the exchange barrier for this many bytes nobody sends
    float scale;     // log2(e) / T rounded to float ...
    float scale_lo;  // ... and what the rounding dropped (for the candidates' own probabilities)
    uint16_t child_first[MCSD_MAX_NODES];
    uint8_t child_count[MCSD_MAX_NODES];
    uint16_t item_node[MCSD_MAX_NODES];
};

// ------------------------------------------------------------------ checked build
// With -DMCSD_DEBUG_BOUNDS (the library libmcsd_debug.so) every read of caller memory that goes
// through the helpers below is checked against the address ranges the host registered for the
// launch: a read outside them is not performed (the helper returns zeros, or its fill value) and
// is counted; nothing traps.  compute-sanitizer's memcheck stands behind this; the normal build
// compiles the checks away.
#ifdef MCSD_DEBUG_BOUNDS
struct DebugRanges {
    int n;                            // 0: nothing registered, nothing is checked
    unsigned long long lo[12], hi[12];
};
__device__ DebugRanges g_dbg_ranges;
__device__ unsigned long long g_dbg_hits;
__device__ __forceinline__ bool dbg_ok(const void *p, size_t bytes) {
    if (g_dbg_ranges.n == 0) return true;
    const unsigned long long a = reinterpret_cast<unsigned long long>(p);
    for (int i = 0; i < g_dbg_ranges.n; ++i)
        if (a >= g_dbg_ranges.lo[i] && a + bytes <= g_dbg_ranges.hi[i]) return true;
    atomicAdd(&g_dbg_hits, 1ull);
    return false;
}
#else
__device__ __forceinline__ constexpr bool dbg_ok(const void *, size_t) { return true; }
#endif

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
    static constexpr uint32_t kNegInfWord = 0xff800000u;  // 32 bits of -inf elements
    static __device__ __forceinline__ void unpack(const uint4 &r, float *o) {
        o[0] = __uint_as_float(r.x); o[1] = __uint_as_float(r.y);
        o[2] = __uint_as_float(r.z); o[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ float load(const void *base, long long i) {
        if (!dbg_ok(reinterpret_cast<const float *>(base) + i, 4)) return 0.f;
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
    static constexpr uint32_t kNegInfWord = 0xff80ff80u;
    static __device__ __forceinline__ void unpack(const uint4 &r, float *o) {
        o[0] = __uint_as_float(r.x << 16); o[1] = __uint_as_float(r.x & 0xffff0000u);
        o[2] = __uint_as_float(r.y << 16); o[3] = __uint_as_float(r.y & 0xffff0000u);
        o[4] = __uint_as_float(r.z << 16); o[5] = __uint_as_float(r.z & 0xffff0000u);
        o[6] = __uint_as_float(r.w << 16); o[7] = __uint_as_float(r.w & 0xffff0000u);
    }
    static __device__ __forceinline__ float load(const void *base, long long i) {
        if (!dbg_ok(reinterpret_cast<const unsigned short *>(base) + i, 2)) return 0.f;
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
    static constexpr uint32_t kNegInfWord = 0xfc00fc00u;
    static __device__ __forceinline__ void unpack(const uint4 &r, float *o) {
        const __half2 *h = reinterpret_cast<const __half2 *>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __half22float2(h[i]);
            o[2 * i] = f.x; o[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ float load(const void *base, long long i) {
        if (!dbg_ok(reinterpret_cast<const __half *>(base) + i, 2)) return 0.f;
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
    // the last operand lets the hardware keep the thread suspended for up to that many
    // nanoseconds while the phase is pending, instead of returning to a polling loop
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kWaitSuspendNs) : "memory");
    return ok != 0;
}
// Bounded wait: false when the poll budget ran out.  A poll that finds the phase pending
// suspends the thread in hardware (see above), so a waiting thread does not eat the issue
// slots of the working ones.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t polls = kWaitPolls) {
    for (uint32_t i = 0; i < polls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i >= 64) __nanosleep(1000);   // (whatever the hardware makes of the hint, a long wait backs off)
    }
    return false;
}
// One bulk async copy global -> this CTA's shared memory (TMA; the copy goes to this CTA alone);
// completion is signalled on an mbarrier of this CTA as a byte count.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    (void)dbg_ok(src, bytes);   // (counted only: the waiting side expects the bytes)
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Asks L2 to fetch a 16-byte-aligned range (size a multiple of 16); nothing waits on it.
__device__ __forceinline__ void bulk_prefetch_l2(const void *src, uint32_t bytes) {
    if (!dbg_ok(src, bytes)) return;
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
// 4-byte asynchronous copy global -> shared (no register holds the value in flight).
// Orders this thread's earlier ordinary shared-memory accesses before later bulk
// (async-proxy) copies into the same locations.
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void cp_async4(void *smem_dst, const void *src) {
    if (!dbg_ok(src, 4)) return;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(smem_dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.wait_all;" ::: "memory");
}
// 128-bit streaming load (read once, do not keep in L1).
__device__ __forceinline__ uint4 ld_stream_v4(const void *p) {
    uint4 r;
    if (!dbg_ok(p, 16)) return make_uint4(0u, 0u, 0u, 0u);
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
// The same under a predicate: where it is false nothing is read and all four words are `fill`.
// A run of these has no branch between the loads, so they are all in flight together.
__device__ __forceinline__ uint4 ld_stream_v4_if(const void *p, bool pred, uint32_t fill) {
    uint4 r;
    pred = pred && dbg_ok(p, 16);
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %5, 0;\n\t"
                 "mov.u32 %0, %6;\n\tmov.u32 %1, %6;\n\tmov.u32 %2, %6;\n\tmov.u32 %3, %6;\n\t"
                 "@q ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];\n\t}"
                 : "=&r"(r.x), "=&r"(r.y), "=&r"(r.z), "=&r"(r.w)
                 : "l"(p), "r"(static_cast<uint32_t>(pred)), "r"(fill));
    return r;
}
// Predicated 128-bit load that may stay in the caches (for data that is read again soon).
__device__ __forceinline__ uint4 ld_v4_if(const void *p, bool pred, uint32_t fill) {
    uint4 r;
    pred = pred && dbg_ok(p, 16);
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %5, 0;\n\t"
                 "mov.u32 %0, %6;\n\tmov.u32 %1, %6;\n\tmov.u32 %2, %6;\n\tmov.u32 %3, %6;\n\t"
                 "@q ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];\n\t}"
                 : "=&r"(r.x), "=&r"(r.y), "=&r"(r.z), "=&r"(r.w)
                 : "l"(p), "r"(static_cast<uint32_t>(pred)), "r"(fill));
    return r;
}
// 128-bit load through the read-only path (data that may be read again soon).
__device__ __forceinline__ uint4 ldg_v4(const void *p) {
    if (!dbg_ok(p, 16)) return make_uint4(0u, 0u, 0u, 0u);
    return __ldg(reinterpret_cast<const uint4 *>(p));
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

// ------------------------------------------------------------------ inverse CDF in token order
// "x ~ P" for non-negative weights P over the vocabulary, made deterministic by a supplied
// uniform u: the smallest x with sum_{y<=x} P(y) > u * sum_y P(y); tokens of weight 0 are
// never returned (Algorithm 1 / 2, "x_end ~ p"; Eq. 1 for the candidate draws).
// The vocabulary is cut into contiguous runs, one per warp; a run into S steps of 32
// groups (one group of 4 or 8 consecutive elements per lane).  Every lane keeps the float
// sums g[S] of its own groups.  The search goes run -> step -> lane -> element; everything
// that combines runs or steps (the prefix sums of the run totals, the position of the quantile
// inside the run, the prefix sums of the step totals) is carried in double, so that no rounding
// of the size of the whole distribution's ulp enters: the float roundings left are those of one
// run total (a sixteenth of the vocabulary or less) and of the sums inside one step.

// Total of every step of this warp's run: lane st * (32 / S) holds the total of step st.
template <int S>
__device__ __forceinline__ float step_totals(const float (&g)[S], int lane) {
    float tj;
    warp_multi_sum<S>(g, lane, tj);
    return tj;
}
// Total of the run (all lanes): the lanes' own sums over their groups, added across the warp.
template <int S>
__device__ __forceinline__ double run_total(const float (&g)[S]) {
    float t = 0.f;
#pragma unroll
    for (int st = 0; st < S; ++st) t += g[st];
    return static_cast<double>(warp_sum(t));
}
// The run that holds the quantile u of the whole distribution.  m: total of run `lane`
// (0 for lanes beyond the runs).  Every warp that calls this with the same totals finds the
// same run.  Returns the run index, or -1 if the distribution has no mass (total 0 or NaN);
// tgt receives the quantile's position inside the run.
__device__ __forceinline__ int pick_run(double m, float u, int lane, double &tgt) {
    double inc = m;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    const double total = __shfl_sync(0xffffffffu, inc, 31);
    const double target = static_cast<double>(u) * total;
    const unsigned hit = __ballot_sync(0xffffffffu, m > 0.0 && inc > target);
    const unsigned pos = __ballot_sync(0xffffffffu, m > 0.0);
    // (rounding, or u >= 1, may put the quantile past the end: the last run with mass)
    const int pick = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : -1);
    if (pick < 0 || !(total > 0.0)) return -1;
    tgt = target - __shfl_sync(0xffffffffu, inc - m, pick);
    return pick;
}
// Inside the run (called by the whole warp that owns it): the step ps and the lane l whose
// group holds the quantile; rem (meaningful in lane l) is the quantile's position inside that
// group.  False if the run has no mass.
template <int S>
__device__ __forceinline__ bool search_run(const float (&g)[S], float tj, double tgt, int lane,
                                           int &ps, int &l, float &rem) {
    ps = -1;
    int last_s = -1;
    double runsum = 0.0, before = 0.0;
#pragma unroll
    for (int st = 0; st < S; ++st) {
        const float ms = __shfl_sync(0xffffffffu, tj, st * (32 / S));
        if (ms > 0.f) {
            last_s = st;
            if (ps < 0 && runsum + static_cast<double>(ms) > tgt) { ps = st; before = runsum; }
        }
        runsum += static_cast<double>(ms);
    }
    float t2 = static_cast<float>(tgt - before);
    if (ps < 0) { ps = last_s; t2 = INFINITY; }   // past the run's own sum: its last element with mass
    if (ps < 0) return false;
    float gs = g[0];
#pragma unroll
    for (int st = 1; st < S; ++st) gs = (ps == st) ? g[st] : gs;
    const float gi = warp_scan_incl(gs, lane);
    const unsigned h2 = __ballot_sync(0xffffffffu, gs > 0.f && gi > t2);
    const unsigned p2 = __ballot_sync(0xffffffffu, gs > 0.f);
    if (!p2) return false;
    l = h2 ? __ffs(h2) - 1 : 31 - __clz(p2);
    rem = t2 - (gi - gs);
    return true;
}
// Inside one group: the first element whose running sum of positive weights exceeds rem,
// else the last element with positive weight, else -1.
template <int GV>
__device__ __forceinline__ int pick_element(const float (&w)[GV], float rem) {
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
    return pe < 0 ? last : pe;
}

}  // namespace mcsd
