// gather_kernel: the key/value rows of the accepted path move to their committed positions
// (Sections 3 and 3.3), in place.
#pragma once

#include "mcsd_common.cuh"

namespace mcsd {

struct GatherParams {
    unsigned char *cache;
    long long slab_stride, seq_stride, pos_stride;  // bytes
    long long n_items;                              // slabs * batch
    long long n_positions;                          // positions per sequence in the cache
    int32_t batch, gamma;
    int32_t row_units;                              // row length in units of UNIT bytes
    const int32_t *prefix_len;                      // [B]
    const int32_t *path_nodes;                      // [B][gamma + 1]
    const int32_t *accept_len;                      // [B]
};

// One CTA per (slab, sequence), grid-stride; a thread owns the same columns of every row.  The
// i-th accepted token's node sits at position prefix + path_nodes[i] and belongs at position
// prefix + 1 + i.  path_nodes[i] >= i + 1 and the nodes ascend, so a destination is never the
// source of a later move; a thread that handles its columns in ascending i therefore never reads
// a row it has overwritten, and no two threads touch the same bytes: in place, no staging buffer.
// Up to kBatch moves are read before any of them is written, so that the loads overlap.
template <typename T>
__global__ void __launch_bounds__(kThreads)
gather_kernel(const GatherParams P)
{
    constexpr int kBatch = 8;
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        const long long s = item / P.batch;
        const int b = static_cast<int>(item - s * P.batch);
        int len = P.accept_len[b];
        len = len < 0 ? 0 : (len > P.gamma ? P.gamma : len);
        const long long prefix = P.prefix_len[b];
        unsigned char *base = P.cache + s * P.slab_stride + b * P.seq_stride;
        const int32_t *nodes = P.path_nodes + static_cast<long long>(b) * (P.gamma + 1);
        for (int i0 = 0; i0 < len; i0 += kBatch) {
            for (int col = threadIdx.x; col < P.row_units; col += kThreads) {
                T v[kBatch];
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int i = i0 + u;
                    if (i < len) {
                        const int nd = nodes[i];
                        // (a node below i + 1 cannot come from a walk, one past the cache is not there:
                        // such entries are skipped)
                        if (nd >= i + 1 && prefix + nd < P.n_positions) v[u] = reinterpret_cast<const T *>(base + (prefix + nd) * P.pos_stride)[col];
                    }
                }
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int i = i0 + u;
                    if (i < len) {
                        const int nd = nodes[i];
                        if (nd > i + 1 && prefix + nd < P.n_positions) reinterpret_cast<T *>(base + (prefix + 1 + i) * P.pos_stride)[col] = v[u];
                    }
                }
            }
        }
    }
}

}  // namespace mcsd
