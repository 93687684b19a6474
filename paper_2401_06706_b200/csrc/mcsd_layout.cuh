// layout_kernel: ancestor mask and position ids of the tree attention of Section 3.3.
#pragma once

#include "mcsd_common.cuh"

namespace mcsd {

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
