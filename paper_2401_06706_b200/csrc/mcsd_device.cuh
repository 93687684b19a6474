// Device code of the MCSD verification library (sm_100a).
//
// The kernels, one file each:
//   node_kernel      (mcsd_node.cuh)  T > 0.  One thread-block cluster per tree node,
//                    persistent over the (sequence, node) items.  Each CTA of the cluster
//                    owns a contiguous slice of the vocabulary.  Its slice of the target
//                    row goes straight into registers with coalesced 128-bit loads; its
//                    slice of the draft row (nodes that have children) is brought into
//                    shared memory with one bulk async copy (TMA, to this CTA alone) and
//                    stays there.  Both are exponentiated once and then stay on chip while
//                    the k candidates of the node are tested in order (Algorithm 1 /
//                    Algorithm 2), so every logit row is read from HBM exactly once.
//   argmax_kernel    (mcsd_argmax.cuh)  T == 0.  One CTA per target row; argmax with lowest
//                    index on ties and the "candidate equals argmax" test (Section 4.5).
//   walk_kernel      (mcsd_walk.cuh)  One row of CTAs per sequence: follows the accepted
//                    children from the root (Section 3), writes the accepted tokens and the
//                    endpoint token, and rebuilds the residual distribution of the
//                    stopping node.
//   sample_kernel    (mcsd_sample.cuh)  The k candidate draws of a node, with or without
//                    replacement (Eq. 1).
//   naive_kernel     (mcsd_naive.cuh)  The sample-and-match baseline of Section 4.5.
//   layout_kernel    (mcsd_layout.cuh)  Mask and position ids of the tree attention
//                    (Section 3.3).
//   gather_kernel    (mcsd_gather.cuh)  Key/value cache rows of the accepted path to their
//                    committed positions.
//   shard_*_kernel   (mcsd_shard.cuh)  The verification with the vocabulary split over several
//                    devices: per-run partial statistics, decisions from the gathered partials,
//                    endpoint token and residual per shard.
// mcsd_common.cuh holds what they share.
//
// How the rejection loop avoids rewriting the residual.  After n rejections the
// unnormalised residual of Algorithm 1/2 is  P_n(x) = max(p(x) - c_n q(x), 0)  with
// c_0 = 0 and c_{n+1} = c_n + S_n / W_n, where S_n = sum_x P_n(x), and W_n = 1 for
// Algorithm 1 or 1 - (original draft mass of the tokens rejected so far) for
// Algorithm 2 (p and q are the ORIGINAL softmax outputs).  This follows from
// p_{n+1} ~ max(p_n - q_n, 0) by induction and holds for every rejection that can
// occur with r in (0,1).  The test of candidate n+1 is r <= [P_n(x~)/S_n]/[q(x~)/W_n].
// So one rejection costs one scalar-parameter reduction over the on-chip p and q,
// and nothing is written back; a node whose first candidate is accepted costs no
// reduction at all.
//
// Softmax references are integers (ceil of the scaled row maximum, in log2 units), so
// moving a partial sum from one reference to another is an exact multiplication by a
// power of two and every thread can exponentiate against its own maximum.
#pragma once

#include "mcsd_common.cuh"
#include "mcsd_node.cuh"
#include "mcsd_argmax.cuh"
#include "mcsd_walk.cuh"
#include "mcsd_sample.cuh"
#include "mcsd_naive.cuh"
#include "mcsd_layout.cuh"
#include "mcsd_gather.cuh"
#include "mcsd_shard.cuh"
