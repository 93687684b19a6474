/*
 * mcsd.h - C ABI of the B200 (sm_100a) multi-candidate speculative-decoding
 * verification library (libmcsd.so).
 *
 * One call verifies a batch of draft token trees that share one topology:
 * for every tree node it forms the target and draft next-token distributions
 * (temperature softmax over the full vocabulary), runs the k-candidate
 * rejection loop of Algorithm 1 (candidates drawn with replacement) or
 * Algorithm 2 (without replacement), and then walks every tree from the root
 * along accepted children (Section 3, "Multi-Candidate Speculative Decoding")
 * to return the accepted tokens, the endpoint ("bonus") token and the
 * distribution that token was drawn from.
 *
 * Conventions
 *   - "device" pointers are CUDA global-memory pointers on the current device;
 *     "host" pointers are ordinary CPU memory.  Nothing is allocated, freed or
 *     retained by the library except where an entry point says so; all device
 *     work is enqueued on desc->stream and the call returns without
 *     synchronising.
 *   - Tree layout: node 0 is the root (the last committed token); nodes are in
 *     generation (level) order, parent[n] < n, the children of a node are
 *     contiguous and are tested in ascending index, which is the order the draft
 *     model sampled them in (loop "for i = 1..k" of Algorithms 1 and 2); the
 *     nodes that have children are exactly 0 .. n_internal-1.  Every k-config
 *     tree k_1 x k_2 x ... (Section 4.3) has this form.
 *   - Randomness is supplied by the caller: uniforms[b][n][0] is the r of the
 *     acceptance test of node n as a candidate of its parent, uniforms[b][n][1]
 *     is the uniform used to draw the endpoint token if the walk stops at n.
 *     Uniforms are expected in the open interval (0, 1).  Other values have a
 *     defined outcome: an acceptance uniform that is not below 1 (NaN included)
 *     counts as 1, i.e. it accepts exactly when p(x) >= q(x); one that is <= 0
 *     accepts whenever q(x) > 0; an endpoint uniform >= 1 or NaN draws the last
 *     token of positive probability, one <= 0 the first.
 *   - Endpoint draw: inverse CDF in token order, the smallest x with
 *     sum_{y<=x} P(y) > u * sum_y P(y); tokens of probability 0 are never drawn.
 *   - Temperature 0 selects the argmax rule (Section 4.5): a candidate is
 *     accepted iff it equals the target argmax (lowest index on ties) and the
 *     endpoint token is the target argmax of the node where the walk stops;
 *     draft logits are not read.
 *   - Return value: MCSD_OK (0) or a negative MCSD_ERR_* code; on an error
 *     nothing has been enqueued.  Faults that only the device can see (token out
 *     of range, zero mass, expired bounded wait) set MCSD_STATUS_* bits in
 *     out_status[b]; kernels never trap and every wait in them is bounded.
 *     out_status[b] describes the walk of sequence b: it is the OR of what was
 *     met at the nodes the walk visited (the nodes the sequential procedure of
 *     Section 3 evaluates), the node where it stopped included; a fault at a node
 *     the walk never reached does not show.  The words are written, not
 *     accumulated: they need no clearing by the caller.
 *   - Logits: -inf is legal (probability 0).  A row from which no distribution
 *     can be formed (all -inf, a NaN or a +inf logit) is handled as follows: a
 *     target row without mass accepts nothing, a walk that stops there returns
 *     token -1 (MCSD_STATUS_NO_MASS | MCSD_STATUS_DEGENERATE); a draft row without
 *     mass rejects every candidate of its node and the endpoint is drawn from the
 *     untouched target distribution (MCSD_STATUS_DEGENERATE).
 */
#ifndef MCSD_H_
#define MCSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* 101: mcsd_desc gained node_residual at its end (a caller built against 100 must be rebuilt)
 * 102: out_status describes the walk only and is written, not accumulated; mcsd_set_option,
 *      mcsd_get_option, mcsd_release_host_staging; desc->reserved is checked; mcsd_shard_* */
#define MCSD_VERSION 102

/* logit element types (both logit tensors share one) */
#define MCSD_DTYPE_F32 0
#define MCSD_DTYPE_BF16 1
#define MCSD_DTYPE_F16 2

/* replacement_mode */
#define MCSD_MODE_WITH_REPLACEMENT 0    /* Algorithm 1 */
#define MCSD_MODE_WITHOUT_REPLACEMENT 1 /* Algorithm 2 */
#define MCSD_MODE_NAIVE 2 /* multi-candidate naive sampling, the ablation baseline of Section 4.5:
                             draw x from the target distribution (second uniform of the node);
                             accept the first child that carries x, else x is the endpoint token.
                             mcsd_verify, mcsd_verify_path and mcsd_verify_host only; draft_logits
                             are not read and may be NULL; out_residual is the stopping node's
                             target distribution; per-node outputs cover visited nodes */

/* limits */
#define MCSD_MAX_NODES 512     /* nodes per tree, root included            */
#define MCSD_MAX_CHILDREN 32   /* candidates per node (the paper uses <= 32) */
#define MCSD_MAX_VOCAB 65536   /* vocabulary size                          */

/* return codes */
#define MCSD_OK 0
#define MCSD_ERR_NULL (-1)        /* a required pointer is NULL                       */
#define MCSD_ERR_SHAPE (-2)       /* batch/n_nodes/n_internal/vocab out of range      */
#define MCSD_ERR_DTYPE (-3)
#define MCSD_ERR_MODE (-4)
#define MCSD_ERR_TEMPERATURE (-5) /* negative, NaN or infinite                        */
#define MCSD_ERR_TREE (-6)        /* tree_parent breaks the layout contract           */
#define MCSD_ERR_STRIDE (-7)      /* row stride smaller than vocab                    */
#define MCSD_ERR_WORKSPACE (-8)   /* workspace missing, misaligned or too small       */
#define MCSD_ERR_CUDA (-9)        /* a CUDA runtime call or kernel launch failed      */
#define MCSD_ERR_UNSUPPORTED (-10)/* beyond MCSD_MAX_*                                */
#define MCSD_ERR_STATIC_LIMIT (-11) /* mcsd_verify_static: scratch need > built-in array */

/* Bytes of the scratch array built into the library for mcsd_verify_static. */
#define MCSD_STATIC_WORKSPACE_BYTES (4u << 20)

/* bits of out_status[b] */
#define MCSD_STATUS_DEGENERATE 1 /* residual mass was 0 after a rejection; residual kept */
#define MCSD_STATUS_BAD_TOKEN 2  /* a candidate token outside [0, vocab): rejected       */
#define MCSD_STATUS_NO_MASS 4    /* endpoint draw from a distribution of mass 0 / NaN    */
#define MCSD_STATUS_TIMEOUT 8    /* a bounded on-chip wait expired; results invalid      */

/* Options of mcsd_set_option: process-wide tuning and test overrides, 0 = library default.
 * Some also take their initial value from the environment variable of the same
 * name (MCSD_CLUSTER, MCSD_EPT, MCSD_DIRECT, MCSD_SAMPLE_AHEAD, MCSD_PDL, MCSD_SPLIT, MCSD_TRACE, MCSD_WALK_CLUSTER), read once when
 * the library is loaded. */
#define MCSD_OPT_CLUSTER 0       /* CTAs per thread-block cluster of the node kernel (1..8)          */
#define MCSD_OPT_EPT 1           /* vocabulary elements per thread and row of the node kernel         */
#define MCSD_OPT_DIRECT 2        /* 1: plain element loads even where rows are 16-byte aligned        */
#define MCSD_OPT_SAMPLE_AHEAD 3  /* L2 look-ahead of the sampling kernel, percent of its default (100) */
#define MCSD_OPT_WAIT_POLLS 4    /* poll budget of the node kernel's exchange wait (0: about 2 s)     */
#define MCSD_OPT_TEST_EXTRA_TX 5 /* test of the expiry path only: the exchange barrier of every round
                                    expects this many bytes (a multiple of 16) that nobody sends, so
                                    the bounded wait runs out and MCSD_STATUS_TIMEOUT is reported      */
#define MCSD_OPT_PDL 6           /* 1 (default): the walk stage is launched as a programmatic dependent
                                    of the node stage; 0: plain stream order                         */
#define MCSD_OPT_TEST_SHRINK_RANGES 7 /* checked build only, test of the checker: every registered extent is
                                         cut short by this many bytes, so that valid reads of the last bytes of
                                         a tensor are reported (and skipped)                                  */
#define MCSD_OPT_SPLIT 8         /* the all-node form of mcsd_verify at temperature > 0 gives its cluster kernel only
                                    the nodes with two or more children and streams the rows of the others with a
                                    kernel of its own: 0 = for large launches (default), 1 = never, 2 = always    */
#define MCSD_OPT_TIME_KERNELS 9  /* 1: CUDA events are recorded around every kernel the verification entry points
                                    launch (on desc->stream); see mcsd_last_kernel_times.  With programmatic dependent
                                    launches a kernel's interval may overlap its predecessor's tail: measure with
                                    MCSD_OPT_PDL 0 for disjoint intervals                                          */
#define MCSD_OPT_TRACE 10        /* host-side tracing of the verification entry points and mcsd_sample_candidates:
                                    bit 0: one line per call on stderr (shape, temperature, mode, return code, kernel
                                    launches, layout of the node stage); bit 1: an NVTX range around every call     */
#define MCSD_OPT_WALK_CLUSTER 11 /* walk stage with a thread-block cluster of eight CTAs per sequence instead of one
                                    CTA (same results): 0 = library's choice (small batches), 1 = never, 2 = always  */
#define MCSD_OPT_COUNT 12

typedef struct mcsd_desc {
    int32_t batch;      /* B: number of trees                                         */
    int32_t n_nodes;    /* N+1: nodes per tree, root included                         */
    int32_t n_internal; /* nodes that have children (= rows of draft_logits per tree) */
    int32_t vocab;      /* V                                                          */
    int32_t dtype;      /* MCSD_DTYPE_*                                               */
    int32_t reserved;   /* must be 0 (MCSD_ERR_SHAPE otherwise)                       */
    int64_t ld_target;  /* elements between consecutive rows of target_logits, >= V   */
    int64_t ld_draft;   /* same for draft_logits                                      */
    void *stream;       /* cudaStream_t the work is enqueued on (0 = default stream)  */
    void *workspace;    /* device scratch, 256-byte aligned, caller-owned; at least   */
    size_t workspace_bytes; /* mcsd_workspace_bytes() bytes; contents are overwritten */
    /* Optional per-node outputs (device), NULL to skip; when NULL the library keeps
     * the first two in the workspace:                                              */
    int32_t *node_accept; /* [B][n_nodes] accepted child of each node, or -1          */
    int32_t *node_bonus;  /* [B][n_nodes] endpoint token of each node that can end a
                             walk (leaf, or all candidates rejected), else -1;
                             asking for it adds a pass over every such node       */
    float *node_ratio;    /* [B][n_nodes] p/q seen by the test of each draft node; -1
                             for a forced rejection; untouched if never tested      */
    int32_t *out_status;  /* [B] MCSD_STATUS_* bits of each walk (device), NULL to skip;
                             written by every call, no clearing needed              */
    int32_t *out_path_nodes; /* [B][gamma+1] (device), NULL to skip: entry i < accept_len
                             is the tree node whose token is out_tokens[i], the rest is
                             -1.  With the flattened-tree layout of Section 3.3 (node n
                             at sequence position prefix_len + n) these are the key/value
                             cache rows that stay after verification.                */
    float *node_residual; /* [B][n_nodes][V] float32 (device), NULL to skip: for every node
                             that can end a walk (as for node_bonus) the distribution its
                             endpoint token is drawn from, i.e. the residual p left by
                             Algorithm 1 / 2 after all k rejections, the target distribution
                             at a leaf, one-hot at temperature 0; rows of other nodes are
                             not written.  A debugging output: B * n_nodes * V * 4 bytes
                             and a pass over every such node; not produced by
                             mcsd_verify_path.                                        */
} mcsd_desc;

/*
 * The whole verification step (Algorithms 1 and 2 at every node, then the walk
 * of Section 3).  Equivalent to mcsd_verify_nodes followed by mcsd_verify_walk.
 *
 *   target_logits  device [B][n_nodes][ld_target]   logits of the target model at
 *                  the root and after every draft node
 *   draft_logits   device [B][n_internal][ld_draft] logits of the draft model at
 *                  every node that has children; may be NULL when temperature == 0
 *   tree_parent    HOST   [n_nodes] parent[0] = -1; shared by the whole batch
 *   cand_tokens    device [B][n_nodes] token carried by each draft node; entry 0
 *                  of a tree is ignored
 *   uniforms       device [B][n_nodes][2] float32, see "Randomness" above; may be
 *                  NULL when temperature == 0
 *   temperature    0 = argmax rule; > 0 = softmax(logits / temperature), both models
 *   replacement_mode  MCSD_MODE_*
 *   out_accept_len device [B] number of accepted draft tokens, 0 .. gamma
 *   out_tokens     device [B][gamma+1] accepted tokens, then the endpoint token,
 *                  then -1; gamma = depth of the tree
 *   out_residual   device [B][vocab] float32, the distribution the endpoint token
 *                  was drawn from (final residual p of the stopping node, its
 *                  target distribution for a leaf, one-hot at temperature 0);
 *                  NULL to skip
 * The call allocates nothing and does not synchronise: it enqueues its kernels on
 * desc->stream and returns.  After one ordinary call on a device (which looks up launch
 * attributes once per kernel) it can be captured in a CUDA graph and replayed (tested for
 * mcsd_verify and mcsd_verify_path).
 * Rows whose base address and stride are multiples of 16 bytes take the bulk-copy
 * (TMA) path; any other layout is accepted and takes a slower plain-load path.
 * All ld elements of every row, the last one included, must be readable memory: on
 * the bulk-copy path a row is loaded in 16-byte vectors, so up to 15 bytes of the
 * padding behind element vocab-1 may be read (their values are ignored).
 */
int mcsd_verify(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                float temperature, int replacement_mode, int32_t *out_accept_len,
                int32_t *out_tokens, float *out_residual);

/*
 * Stage 1: the per-node part (softmax statistics of both models at every node,
 * the rejection loop of Algorithm 1 / 2 at every node that has children).  Fills
 * node_accept (in the workspace when the descriptor leaves it NULL) and the
 * per-node statistics kept in the workspace; at temperature 0 also node_bonus
 * (the target argmax of every node that accepted nothing, else -1).  out_status is
 * written by stage 2.  Arguments as in mcsd_verify.
 */
int mcsd_verify_nodes(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                      const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                      float temperature, int replacement_mode);

/*
 * Stage 2: the walk of Section 3 from the root along accepted children, using
 * what stage 1 left in the workspace of the same descriptor; then, for the node
 * where each walk stops, the distribution its endpoint token is drawn from (the
 * final residual of Algorithm 1 / 2, rebuilt from that node's two logit rows and
 * the stored statistics) and the endpoint token itself ("x_end ~ p", last line
 * of both algorithms).  An endpoint token is only ever used at the node where a
 * walk stops, so it is drawn there and nowhere else; when the descriptor asks
 * for node_bonus, the same draw is also made at every node that accepted no
 * candidate, one CTA per node (a checking aid, not part of the timed path).
 * Arguments as in mcsd_verify.
 */
int mcsd_verify_walk(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int32_t *out_accept_len, int32_t *out_tokens, float *out_residual);

/*
 * The same result computed the way Section 3 describes the procedure: only the nodes a
 * walk actually visits are evaluated.  Every sequence starts at the root, evaluates the
 * node its walk stands on (softmax of that node's two rows, Algorithm 1 / 2 on its
 * candidates) and moves to the accepted child until a test sequence rejects all
 * candidates or a leaf is reached; then the walk stage runs as in mcsd_verify.  At
 * temperature > 0 one kernel launch does this for the whole batch (each sequence is
 * walked by one thread-block cluster); at temperature 0 there is one launch per level
 * of the tree.  At most 2 * gamma + 1 logit rows per tree are read instead of all of
 * them, so this is the form to use when the tree is large or latency matters more than
 * the node rate.  Outputs are identical to those of mcsd_verify (the same tests with
 * the same uniforms).  The optional per-node outputs of the descriptor are filled for
 * visited nodes only and node_bonus is not produced.  Arguments as in mcsd_verify.
 */
int mcsd_verify_path(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int replacement_mode, int32_t *out_accept_len,
                     int32_t *out_tokens, float *out_residual);

/*
 * The step before verification: drawing the candidate tokens (Section 3.2).  For every
 * node n in [node_begin, node_end) of every tree (node indices < n_internal) the tokens
 * of its k children are drawn from softmax(draft_logits[b][n] / temperature) by inverse
 * CDF in token order (see "Endpoint draw" above), child c with the uniform
 * uniforms_draw[b][c]:
 *   MCSD_MODE_WITH_REPLACEMENT     k independent draws (the input of Algorithm 1)
 *   MCSD_MODE_WITHOUT_REPLACEMENT  Eq. 1: every drawn token gets probability 0 before the
 *                                  next draw, so the k tokens are distinct
 *   temperature 0                  the k largest draft logits in descending order, lowest
 *                                  index first among equals; uniforms_draw may be NULL
 * A draft model produces the rows of one tree level at a time, hence the node range.
 *   draft_logits   device [B][n_internal][ld_draft]; as in mcsd_verify, all ld_draft elements
 *                  of the rows in range must be readable (16-byte vector loads)
 *   tree_parent    HOST   [n_nodes]
 *   uniforms_draw  device [B][n_nodes] float32 in (0, 1)
 *   cand_tokens    device [B][n_nodes], written for the children of the nodes in range
 * Of the descriptor only batch, n_nodes, n_internal, vocab, dtype, ld_draft, stream and
 * out_status (MCSD_STATUS_NO_MASS if a draw finds no mass; not cleared here) are read.
 */
int mcsd_sample_candidates(const mcsd_desc *desc, const void *draft_logits, const int32_t *tree_parent,
                           const float *uniforms_draw, float temperature, int replacement_mode,
                           int32_t node_begin, int32_t node_end, int32_t *cand_tokens);

/*
 * The same step for callers whose data lives in HOST memory: every pointer below
 * is a host pointer.  The library allocates device buffers for a slice of the
 * batch, copies the slice in, verifies it and copies the results back, slice
 * after slice on two internal streams so that copies overlap the kernels; it
 * synchronises before it returns.  The device staging buffers (two slices' worth:
 * about 2 x 256 MiB plus outputs) and the two streams are kept for the next call on
 * the same device and grown on demand; mcsd_release_host_staging frees them.  Calls
 * on one device are serialised.  Only batch, n_nodes, n_internal, vocab, dtype,
 * ld_target and ld_draft of the descriptor are read; node_* outputs are not produced.
 * out_status (host, [B]) may be NULL.  Host buffers in page-locked memory make the
 * copies asynchronous.  If a CUDA call fails part way (MCSD_ERR_CUDA) the outputs of
 * the slices not yet finished are undefined.
 */
int mcsd_verify_host(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                     const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                     float temperature, int replacement_mode, int32_t *out_accept_len,
                     int32_t *out_tokens, float *out_residual, int32_t *out_status);

/*
 * mcsd_verify for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of mcsd_verify, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a serving
 * loop that promised its memory pool a fixed footprint, in a plugin whose host
 * owns every allocation, or late in a process whose device memory is already
 * fully handed out - and that therefore has no buffer to put into
 * desc->workspace.  Here the scratch memory (per-node accept decisions, softmax
 * statistics, per-sequence status words) lives in an array of
 * MCSD_STATIC_WORKSPACE_BYTES bytes compiled into the library; every GPU that
 * loads the library carries that array until the process exits.  Inputs and
 * outputs are still the caller's buffers; desc->workspace and
 * desc->workspace_bytes are ignored.  Arguments, outputs and return codes are those of
 * mcsd_verify.
 *
 * Limits and rules
 *   - If mcsd_workspace_bytes(desc) exceeds MCSD_STATIC_WORKSPACE_BYTES the call
 *     returns MCSD_ERR_STATIC_LIMIT and enqueues nothing (roughly: batch * nodes
 *     per tree up to some tens of thousands; use mcsd_verify beyond that).
 *   - The first call on each device looks up the array's device address (once,
 *     with that device current).  Make that first call before any stream capture
 *     begins.
 *   - No cudaMalloc, cudaFree or other allocating routine is called.
 *   - All calls on one device share the one array, and it still holds what the
 *     previous call left; the call clears the part that has to start at zero (the
 *     status words) itself.  Two calls whose kernels can overlap on the GPU
 *     (different streams, no dependency between them) race on the array: order
 *     them.
 */
int mcsd_verify_static(const mcsd_desc *desc, const void *target_logits, const void *draft_logits,
                       const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                       float temperature, int replacement_mode, int32_t *out_accept_len,
                       int32_t *out_tokens, float *out_residual);

/*
 * Tree Attention layout (Section 3.3): the tree is fed to the target model as one flattened
 * sequence in node order, every node attending only to itself and its ancestors (and to the
 * whole prefix), with the position ids it would have in its own root-to-node sequence.
 *   tree_parent   HOST   [n_nodes]
 *   prefix_len    position id of the root (node 0 is the last committed token)
 *   mask          device [n_nodes][n_nodes] bytes: mask[i][j] = 1 iff j == i or j is an
 *                 ancestor of i, else 0
 *   position_ids  device [n_nodes]: prefix_len + depth of the node
 * Either output may be NULL.  stream: cudaStream_t the work is enqueued on.
 */
int mcsd_tree_attention_layout(const int32_t *tree_parent, int32_t n_nodes, int32_t prefix_len,
                               uint8_t *mask, int32_t *position_ids, void *stream);

/*
 * After verification (Sections 3 and 3.3): the target model ran over the flattened tree, so
 * its key/value cache holds one row per tree node, node n of sequence b at position
 * prefix_len[b] + n.  Only the rows of the accepted path stay.  This call moves, in place,
 * the row of the i-th accepted token's node (path_nodes[b][i], as mcsd_verify writes them to
 * desc->out_path_nodes) to position prefix_len[b] + 1 + i, for i < accept_len[b]; no other
 * row is written (rows behind the committed part keep stale tree rows).
 *   cache       device; row (slab s, sequence b, position t) starts at byte
 *               s * slab_stride + b * seq_stride + t * pos_stride and has row_bytes bytes.
 *               A slab is whatever shares this layout: a layer's keys, its values, one head.
 *               Rows are moved in the widest unit (16, 8, 4, 2 or 1 bytes) that divides the
 *               base address, the three strides and row_bytes.
 *   prefix_len  device [batch] int32: position of the root (the last committed token)
 *   path_nodes  device [batch][gamma + 1], accept_len device [batch]: outputs of mcsd_verify
 *   n_positions positions per sequence the cache holds
 * Entries of path_nodes below i + 1 (impossible for a walk) or at a position beyond the cache
 * are skipped; prefix_len must not be negative.
 */
int mcsd_gather_accepted_kv(void *cache, int64_t n_slabs, int64_t slab_stride, int32_t batch,
                            int64_t seq_stride, int64_t pos_stride, int64_t row_bytes,
                            int64_t n_positions, const int32_t *prefix_len, const int32_t *path_nodes,
                            const int32_t *accept_len, int32_t gamma, void *stream);

/*
 * Verification with the vocabulary split over several devices.  Section 4.1 runs its largest
 * target models across two GPUs; when the LM head stays column-split, device s holds only
 * columns [col_begin, col_begin + n_cols) of both logit tensors.  Algorithms 1 and 2 need, per
 * node, a handful of sums over the whole vocabulary (the two softmax normalisers, then one
 * residual sum per rejection that is followed by another test), so the step becomes a sequence
 * of rounds: every shard forms the partial sums of its columns, the CALLER gathers the partials
 * of all shards with a collective of its own (an all-gather of a few floats per node: NCCL,
 * MPI, ...; the library links none), and every shard takes the same decisions from the gathered
 * values.  Nothing but these partials, the candidates' own logits and, at the end, one token per
 * sequence crosses devices; no logit does.  The partials are formed over the same runs of columns
 * and in the same order as mcsd_verify forms them inside one device, so node_accept,
 * accept_len and the accepted tokens are identical to mcsd_verify's on the full tensors.
 *
 * One call sequence per step, the same on every shard (S = n_shards, R = mcsd_shard_rounds):
 *   mcsd_shard_partials(round 0)            -> part_out, cand_logits_out
 *   gather part_out -> stats_all [S][B*n_nodes][entries_per_shard] float4   (kept until the end)
 *   gather cand_logits_out -> cand_logits_all [S][B*n_nodes] float2
 *   mcsd_shard_decide(round 0, part_all = stats_all)
 *   for r = 1 .. R:  mcsd_shard_partials(round r) -> part_out; gather -> part_all;
 *                    mcsd_shard_decide(round r, part_all)
 *   for attempt = 0, 1:  mcsd_shard_endpoint(attempt) -> totals_out [B][entries_per_shard] double;
 *                    gather -> totals_all [S][B][entries_per_shard];  mcsd_shard_finish(attempt)
 *   reduce endpoint_part over the shards (maximum: the shard that holds the token wrote it, the
 *   others -1);  mcsd_shard_commit puts it behind the accepted tokens.
 * (attempt 1 only touches sequences whose residual after the last rejection had no mass and
 * returns at once for all others.)  All buffers are device memory of the caller; the partial
 * and gathered buffers may be reused from step to step.  Temperature must be > 0 (the argmax
 * rule needs no sums; MCSD_ERR_UNSUPPORTED) and the mode Algorithm 1 or 2.
 */
typedef struct mcsd_shard_desc {
    int32_t batch, n_nodes, n_internal;
    int32_t vocab;          /* V of the WHOLE vocabulary                                      */
    int32_t dtype;          /* MCSD_DTYPE_*                                                   */
    int32_t reserved;       /* must be 0                                                      */
    int32_t n_shards, shard;/* 1 <= n_shards <= 32, 0 <= shard < n_shards                     */
    int64_t ld_target;      /* elements between rows of this shard's target_slice, >= n_cols  */
    int64_t ld_draft;
    void *stream;
    void *workspace;        /* device scratch of this shard, 256-byte aligned, at least        */
    size_t workspace_bytes; /* mcsd_shard_workspace_bytes() bytes; must survive the whole step */
    float *node_ratio;      /* optional [B][n_nodes], as in mcsd_desc                          */
    int32_t *node_accept;   /* optional [B][n_nodes]: accepted child of every node with children,
                               or -1 (entries of leaves are not written); NULL: kept in the workspace */
} mcsd_shard_desc;

/* The column range shard `shard` of `n_shards` must hold, and the entries per shard of the
 * exchanged buffers.  Ranges are whole runs of the node kernel's column partition for this
 * vocabulary and dtype; trailing shards may be empty.  Host only, no device needed. */
int mcsd_shard_columns(int32_t vocab, int32_t dtype, int32_t n_shards, int32_t shard, int32_t *col_begin,
                       int32_t *n_cols, int32_t *entries_per_shard);
/* Bytes of mcsd_shard_desc.workspace; 0 for an invalid descriptor. */
size_t mcsd_shard_workspace_bytes(const mcsd_shard_desc *desc);
/* Rounds after round 0 a tree needs: (largest number of children of a node) - 1; negative
 * MCSD_ERR_* for a malformed tree. */
int mcsd_shard_rounds(const int32_t *tree_parent, int32_t n_nodes);
/* Partial sums of this shard's columns.  target_slice [B][n_nodes][ld_target], draft_slice
 * [B][n_internal][ld_draft] (device); part_out [B*n_nodes][entries_per_shard] float4;
 * cand_logits_out [B*n_nodes] float2 (round 0 only).  Round r >= 1 reads what
 * mcsd_shard_decide(round r - 1) left in the workspace. */
int mcsd_shard_partials(const mcsd_shard_desc *desc, const void *target_slice, const void *draft_slice,
                        const int32_t *tree_parent, const int32_t *cand_tokens, float temperature, int32_t round,
                        void *part_out, void *cand_logits_out);
/* Decisions of Algorithm 1 / 2 from the gathered partials (identical on every shard). */
int mcsd_shard_decide(const mcsd_shard_desc *desc, const int32_t *tree_parent, const int32_t *cand_tokens,
                      const float *uniforms, float temperature, int replacement_mode, int32_t round,
                      const void *part_all, const void *cand_logits_all);
/* Mass of every run of the residual of the node where each walk stops, and that residual
 * (unnormalised) in out_residual_slice [B][n_cols] (may be NULL). */
int mcsd_shard_endpoint(const mcsd_shard_desc *desc, const void *target_slice, const void *draft_slice,
                        const int32_t *tree_parent, float temperature, int32_t attempt, const void *stats_all,
                        void *totals_out, float *out_residual_slice);
/* Walk outputs (the same on every shard), this shard's part of the endpoint draw
 * (endpoint_part[b] = token or -1) and the scaling of out_residual_slice. */
int mcsd_shard_finish(const mcsd_shard_desc *desc, const void *target_slice, const void *draft_slice,
                      const int32_t *tree_parent, const int32_t *cand_tokens, const float *uniforms,
                      float temperature, int32_t attempt, const void *stats_all, const void *totals_all,
                      int32_t *out_accept_len, int32_t *out_tokens, int32_t *out_status, int32_t *out_path_nodes,
                      int32_t *endpoint_part, float *out_residual_slice);

/* out_tokens[b][accept_len[b]] = endpoint_all[b] (the reduced endpoint_part). */
int mcsd_shard_commit(const mcsd_shard_desc *desc, const int32_t *tree_parent, const int32_t *endpoint_all,
                      const int32_t *accept_len, int32_t *out_tokens);

/* Frees the device staging buffers and streams mcsd_verify_host keeps on the current
 * device (allocating again on its next call).  Returns MCSD_OK or MCSD_ERR_CUDA. */
int mcsd_release_host_staging(void);

/* Sets one of the MCSD_OPT_* overrides for the whole process (not synchronised with calls
 * running on other host threads).  value >= 0; 0 restores the default.  Returns MCSD_OK, or
 * MCSD_ERR_SHAPE for an unknown option or a negative value.  mcsd_get_option returns the
 * current value (or MCSD_ERR_SHAPE). */
int mcsd_set_option(int option, int value);
int mcsd_get_option(int option);

/* Bytes of device workspace mcsd_verify needs for this descriptor (batch, n_nodes and
 * n_internal are read: the need depends on the node counts only, not on the shape of the
 * tree); 0 if the descriptor is NULL or its shape is invalid. */
size_t mcsd_workspace_bytes(const mcsd_desc *desc);

/* Depth (gamma) of a tree given as a host parent array, or a negative MCSD_ERR_*
 * code if the array breaks the layout contract.  out_tokens has gamma+1 columns. */
int mcsd_tree_depth(const int32_t *tree_parent, int32_t n_nodes);

/* Number of kernel launches the last successful mcsd_verify / stage call on this
 * host thread enqueued (for launch accounting in benchmarks). */
int mcsd_last_launch_count(void);

/* With MCSD_OPT_TIME_KERNELS set: device time in milliseconds of the kernels the last mcsd_verify /
 * mcsd_verify_nodes / mcsd_verify_walk / mcsd_verify_path call of this host thread launched, from CUDA
 * events on its stream (waits for them): ms[0] cluster kernel (argmax kernel at temperature 0, naive
 * kernel in MCSD_MODE_NAIVE), ms[1] streaming statistics kernel, ms[2] single-test kernel, ms[3] walk
 * kernel; -1 where no such kernel ran.  Returns how many were filled, or a negative MCSD_ERR_*. */
int mcsd_last_kernel_times(float *ms, int32_t n);

/* The checked build of the library (libmcsd_debug.so, compiled with MCSD_DEBUG_BOUNDS) verifies every
 * read of caller memory by the verification, walk, argmax, naive-sampling and candidate-sampling
 * kernels against the extents the descriptor implies; a read outside them is skipped and counted,
 * nothing traps.  Returns the number of such reads since the last reset on the current device
 * (synchronises the device), resets the count if `reset` is not 0; -1 in the normal build. */
long long mcsd_debug_bounds_hits(int reset);

/* Static description of a return code. */
const char *mcsd_status_string(int code);

/* MCSD_VERSION the library was built from. */
int mcsd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MCSD_H_ */
