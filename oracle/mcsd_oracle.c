/*
 * CPU oracle for the verification step of Multi-Candidate Speculative Decoding.
 *
 * TEST INFRASTRUCTURE, NOT THE PRODUCT.  A plain, slow, float64 restatement of
 * what the paper defines, used to check the CUDA library and as the timed CPU
 * baseline.  It shares no code, header, table or helper with the CUDA path and
 * must never be called from it.
 *
 * What it follows:
 *   - Algorithm 1 (multi-candidate speculative sampling, candidates drawn with
 *     replacement) and Algorithm 2 (the variant without replacement), taken
 *     step by step in the paper's order: draw r, test r <= p(x~)/q(x~), on a
 *     rejection replace p by the normalised positive part of p - q, and in
 *     Algorithm 2 also zero q(x~) and renormalise q.
 *   - Section 3 (the verification walk): start at the root, run the sampling
 *     algorithm on that node's (p, q, candidates); move to the accepted child or
 *     stop; a node where everything is rejected returns a token from the final
 *     residual; a leaf returns a token from its own target distribution.
 *   - Section 3.2, Eq. 1 (how the k candidates of a node are drawn without replacement);
 *     the draws themselves are made deterministic by supplied uniforms.
 *   - Section 4.1 (sampling setups): temperature 1 is plain softmax sampling,
 *     temperature 0 is argmax.  Section 4.5 states that at temperature 0 the
 *     with-replacement algorithm degenerates to standard speculative decoding and
 *     the without-replacement one to naive sampling; both reduce to "accept a
 *     candidate iff it equals the target argmax".
 *
 * Readings taken where the paper is silent (the same list is kept in the design
 * document):
 *   - a candidate whose current draft probability is 0 is rejected (no 0/0 test);
 *   - the ratio in Algorithm 2 uses the renormalised q of the current iteration;
 *   - "x_end ~ p" is an inverse-CDF draw in token-index order from a supplied
 *     uniform u: the smallest x with sum_{y<=x} P(y) > u * sum_y P(y);
 *   - argmax ties go to the lowest token index;
 *   - the candidates of a node are its children, tested in ascending node index;
 *   - every test owns a pre-drawn uniform, indexed by the child node it tests;
 *   - if the residual mass is exactly 0 the residual is left unchanged and a
 *     status bit is set;
 *   - Algorithm 2's "q(x~) := 0; q := q / sum q" is the identity, and is skipped, where
 *     x~ is not a token or has draft probability 0 already (nothing is removed);
 *     as a consequence a draft row from which no distribution can be formed (its
 *     softmax is NaN) rejects every candidate of its node and leaves p as it is;
 *   - "r ~ U(0,1)" is an input of the verification step; a supplied r that is
 *     not below 1 (NaN included) counts as 1 there, so that every value a caller can pass has a defined
 *     outcome: such an r accepts exactly when p(x~) >= q(x~).  (An r <= 0 needs no
 *     rule: the ratio is never negative, so it accepts whenever q(x~) > 0.)
 *
 * All sums run left to right in double.  Inputs are float32 arrays holding the
 * exact (dtype-rounded) logits; every element is widened to double first.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_STATUS_DEGENERATE 1  /* residual mass was 0 after a rejection      */
#define ORACLE_STATUS_BAD_TOKEN 2   /* a candidate token outside [0, V)           */
#define ORACLE_STATUS_NO_MASS 4     /* endpoint draw from a distribution of mass 0 */

int32_t mcsd_oracle_num_threads(void)
{
#ifdef _OPENMP
    return (int32_t)omp_get_max_threads();
#else
    return 1;
#endif
}

/* Section 4.1: distribution of a model at temperature T > 0,
 * softmax(logits / T), with the row maximum subtracted before exponentiation. */
void mcsd_oracle_softmax(const float *logits, int32_t V, double T, double *out)
{
    double m = -INFINITY;
    for (int32_t x = 0; x < V; ++x) {
        double l = (double)logits[x];
        if (l > m) m = l;
    }
    double Z = 0.0;
    for (int32_t x = 0; x < V; ++x) {
        out[x] = exp(((double)logits[x] - m) / T);
        Z += out[x];
    }
    for (int32_t x = 0; x < V; ++x) out[x] /= Z;
}

/* Lowest index of the largest logit (temperature 0). */
int32_t mcsd_oracle_argmax(const float *logits, int32_t V)
{
    int32_t a = 0;
    double m = (double)logits[0];
    for (int32_t x = 1; x < V; ++x) {
        double l = (double)logits[x];
        if (l > m) { m = l; a = x; }
    }
    return a;
}

/* "x_end ~ p(x)" (last line of Algorithms 1 and 2) made deterministic by a
 * supplied uniform u: inverse CDF in token order over the (possibly
 * unnormalised) non-negative weights P.  Returns the smallest x whose running
 * sum exceeds u * total; tokens of weight 0 are never returned; if rounding
 * leaves no such x the last token of positive weight is returned; -1 if the
 * total is 0. */
int32_t mcsd_oracle_invcdf(const double *P, int32_t V, double u)
{
    double total = 0.0;
    for (int32_t x = 0; x < V; ++x) total += P[x];
    double target = u * total;
    double cum = 0.0;
    int32_t last = -1;
    for (int32_t x = 0; x < V; ++x) {
        if (P[x] > 0.0) {
            cum += P[x];
            last = x;
            if (cum > target) return x;
        }
    }
    return last;
}

/* Algorithm 1 (mode 0) and Algorithm 2 (mode 1) at one node.
 *
 *   p, q    [V]  in: the two distributions; out: their state when the loop ended
 *                (on an acceptance: as they were at the accepting test; when all
 *                k are rejected: p is the final residual the endpoint is drawn
 *                from).
 *   cand    [k]  candidate tokens in sampling order
 *   r       [k]  the uniform of each test
 *   ratio   [k]  out: p(x~)/q(x~) as seen by test i; -1 where q(x~) was 0 (forced
 *                rejection); NaN for tests that were never reached
 *   S       [k]  out: sum_x max(0, p(x)-q(x)) computed after rejection i (the
 *                normaliser of the residual); NaN where not reached
 *   status       out: OR of ORACLE_STATUS_* bits
 * Returns the index i in [0,k) of the accepted candidate, or -1.
 */
int32_t mcsd_oracle_mcss(double *p, double *q, int32_t V, const int32_t *cand,
                         const double *r, int32_t k, int32_t mode, double *ratio,
                         double *S, int32_t *status)
{
    for (int32_t i = 0; i < k; ++i) { ratio[i] = NAN; S[i] = NAN; }
    for (int32_t i = 0; i < k; ++i) {
        int32_t xt = cand[i];
        int32_t valid = (xt >= 0 && xt < V);
        double qx = valid ? q[xt] : 0.0;
        double px = valid ? p[xt] : 0.0;
        if (!valid) *status |= ORACLE_STATUS_BAD_TOKEN; /* not a token: rejected */
        if (qx > 0.0) {
            double rho = px / qx;
            ratio[i] = rho;
            if (r[i] <= rho) return i; /* accept x~^i */
        } else {
            ratio[i] = -1.0; /* never accept on a zero draft probability */
        }
        /* rejected: p := norm(max(0, p - q)) */
        double s = 0.0;
        for (int32_t x = 0; x < V; ++x) {
            double d = p[x] - q[x];
            if (d > 0.0) s += d;
        }
        S[i] = s;
        if (s > 0.0) {
            for (int32_t x = 0; x < V; ++x) {
                double d = p[x] - q[x];
                p[x] = (d > 0.0 ? d : 0.0) / s;
            }
        } else {
            *status |= ORACLE_STATUS_DEGENERATE;
        }
        if (mode == 1 && valid && q[xt] > 0.0) {
            /* Algorithm 2 only: q(x~) <- 0, q := q / sum q.  Where x~ is not a token, or has
             * draft probability 0 already, nothing is removed and the step is the identity:
             * q is left as it is (dividing it by its own sum, 1 up to rounding, would only
             * disturb the last bits, which matters when p and q are equal). */
            q[xt] = 0.0;
            double w = 0.0;
            for (int32_t x = 0; x < V; ++x) w += q[x];
            if (w > 0.0)
                for (int32_t x = 0; x < V; ++x) q[x] /= w;
        }
    }
    return -1;
}

/*
 * Drawing the k candidates of one node from the draft distribution q (Section 3.2).
 *   mode 0: k independent draws from q (sampling with replacement, the input of
 *           Algorithm 1): x_i is the inverse-CDF image of u[i] under q.
 *   mode 1: sampling without replacement, Eq. 1: x_1 is drawn from q; before each later
 *           draw the tokens already drawn get probability 0 and the rest is renormalised
 *           (the inverse CDF works on unnormalised weights, so zeroing is enough).
 * q [V] is used as scratch in mode 1 (drawn entries are zeroed).  Returns the number of
 * draws that found no mass (their token is -1).
 */
int32_t mcsd_oracle_draw(double *q, int32_t V, const double *u, int32_t k, int32_t mode, int32_t *x_out)
{
    int32_t failed = 0;
    for (int32_t i = 0; i < k; ++i) {
        int32_t x = mcsd_oracle_invcdf(q, V, u[i]);
        x_out[i] = x;
        if (x < 0) { ++failed; continue; }
        if (mode == 1) q[x] = 0.0;
    }
    return failed;
}

/* The k largest logits in descending order, equal logits by ascending index: what the
 * draws of a node become at temperature 0 (every draw takes the most probable token that
 * is still available). */
void mcsd_oracle_topk(const float *logits, int32_t V, int32_t k, int32_t *x_out)
{
    for (int32_t i = 0; i < k; ++i) {
        int32_t best = -1;
        for (int32_t x = 0; x < V; ++x) {
            int32_t taken = 0;
            for (int32_t j = 0; j < i; ++j) taken |= (x_out[j] == x);
            if (taken) continue;
            if (best < 0 || (double)logits[x] > (double)logits[best]) best = x;
        }
        x_out[i] = best;
    }
}

/*
 * Candidate tokens of every child of the nodes [node_begin, node_end) of every tree.
 *   draft  [B][n_internal][V]  float32 draft logits
 *   unif   [B][n_nodes]        the uniform that draws the token of each draft node
 *   cand   [B][n_nodes]        out: cand[b][c] for every child c of the nodes in range;
 *                              other entries are left untouched
 * T > 0: draws from softmax(draft / T) as in mcsd_oracle_draw; T == 0: top-k.
 * Returns 0, or -1 on malformed arguments.
 */
int32_t mcsd_oracle_sample(int32_t B, int32_t n_nodes, int32_t n_internal, int32_t V,
                           const float *draft, const int32_t *parent, const float *unif, double T,
                           int32_t mode, int32_t node_begin, int32_t node_end, int32_t *cand)
{
    if (B < 0 || n_nodes < 1 || V < 1 || n_internal < 0 || n_internal > n_nodes) return -1;
    if (!(T >= 0.0) || (mode != 0 && mode != 1)) return -1;
    if (node_begin < 0 || node_end > n_internal || node_begin > node_end) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        double *q = (double *)malloc((size_t)V * sizeof(double));
        for (int32_t n = node_begin; n < node_end; ++n) {
            int32_t first = -1, k = 0;
            for (int32_t c = n + 1; c < n_nodes; ++c)
                if (parent[c] == n) { if (k == 0) first = c; ++k; }
            if (k == 0 || k > 64) continue;
            const float *d = draft + ((size_t)b * n_internal + n) * V;
            int32_t x[64];
            if (T == 0.0) {
                mcsd_oracle_topk(d, V, k, x);
            } else {
                double u[64];
                for (int32_t i = 0; i < k; ++i) u[i] = (double)unif[(size_t)b * n_nodes + first + i];
                mcsd_oracle_softmax(d, V, T, q);
                mcsd_oracle_draw(q, V, u, k, mode, x);
            }
            for (int32_t i = 0; i < k; ++i) cand[(size_t)b * n_nodes + first + i] = x[i];
        }
        free(q);
    }
    return 0;
}

/* Children of node n in a level-ordered tree: the contiguous run of nodes whose
 * parent is n.  Returns the count and stores the first child. */
static int32_t children_of(const int32_t *parent, int32_t n_nodes, int32_t n, int32_t *first)
{
    int32_t cnt = 0;
    *first = -1;
    for (int32_t c = n + 1; c < n_nodes; ++c) {
        if (parent[c] == n) {
            if (cnt == 0) *first = c;
            ++cnt;
        }
    }
    return cnt;
}

static int32_t tree_depth(const int32_t *parent, int32_t n_nodes)
{
    int32_t gamma = 0;
    for (int32_t n = 1; n < n_nodes; ++n) {
        int32_t d = 0;
        for (int32_t a = n; a > 0; a = parent[a]) ++d;
        if (d > gamma) gamma = d;
    }
    return gamma;
}

/* Everything the verification computes at node n of sequence b.
 * residual [V] receives the distribution the endpoint token of this node is
 * drawn from (final residual for an internal node, target distribution for a
 * leaf, one-hot argmax at temperature 0).  Returns the accepted child or -1. */
static int32_t verify_node(int32_t n, int32_t n_nodes, int32_t n_internal, int32_t V,
                           const float *target_b, const float *draft_b,
                           const int32_t *parent, const int32_t *cand_b,
                           const float *unif_b, double T, int32_t mode, double *residual,
                           double *qbuf, int32_t *bonus, double *ratio_b, int32_t *status)
{
    const float *t = target_b + (size_t)n * V;
    int32_t first, k = children_of(parent, n_nodes, n, &first);
    (void)n_internal;
    if (T == 0.0) {
        int32_t a = mcsd_oracle_argmax(t, V);
        for (int32_t x = 0; x < V; ++x) residual[x] = 0.0;
        residual[a] = 1.0;
        *bonus = a;
        for (int32_t i = 0; i < k; ++i) {
            /* ratio of one-hot target to one-hot draft is not defined; report
             * 1 for a match and 0 otherwise */
            int32_t match = cand_b[first + i] == a;
            if (ratio_b) ratio_b[first + i] = match ? 1.0 : 0.0;
            if (match) { *bonus = -1; return first + i; }
        }
        return -1;
    }
    mcsd_oracle_softmax(t, V, T, residual); /* p */
    if (mode == 2 && k > 0) {
        /* Naive sampling (the baseline of Section 2 that Section 4.5 and Appendix C compare
         * with): draw x from the target distribution itself; if one of the candidates
         * carries x the walk moves to (the first) such child, otherwise x is the endpoint
         * token.  The draft distribution plays no part. */
        int32_t x = mcsd_oracle_invcdf(residual, V, (double)unif_b[2 * n + 1]);
        if (x < 0) { *status |= ORACLE_STATUS_NO_MASS; *bonus = -1; return -1; }
        for (int32_t i = 0; i < k; ++i) {
            int32_t match = cand_b[first + i] == x;
            if (ratio_b) ratio_b[first + i] = match ? 1.0 : 0.0;
            if (match) { *bonus = -1; return first + i; }
        }
        *bonus = x;
        return -1;
    }
    if (k == 0) {
        /* leaf: endpoint from its own target distribution */
        *bonus = mcsd_oracle_invcdf(residual, V, (double)unif_b[2 * n + 1]);
        if (*bonus < 0) *status |= ORACLE_STATUS_NO_MASS;
        return -1;
    }
    mcsd_oracle_softmax(draft_b + (size_t)n * V, V, T, qbuf); /* q */
    int32_t cands[64];
    double r[64], ratio[64], S[64];
    for (int32_t i = 0; i < k; ++i) {
        cands[i] = cand_b[first + i];
        r[i] = (double)unif_b[2 * (first + i)];
        if (!(r[i] < 1.0)) r[i] = 1.0; /* supplied in place of r ~ U(0,1): not below 1 counts as 1 */
    }
    int32_t acc = mcsd_oracle_mcss(residual, qbuf, V, cands, r, k, mode, ratio, S, status);
    if (ratio_b)
        for (int32_t i = 0; i < k; ++i) ratio_b[first + i] = ratio[i];
    if (acc >= 0) {
        *bonus = -1;
        return first + acc;
    }
    *bonus = mcsd_oracle_invcdf(residual, V, (double)unif_b[2 * n + 1]);
    if (*bonus < 0) *status |= ORACLE_STATUS_NO_MASS;
    return -1;
}

/*
 * Whole verification step for a batch of trees that share one topology.
 *
 *   target  [B][n_nodes][V]     float32 (exact widening of the rounded logits)
 *   draft   [B][n_internal][V]  float32; nodes with children are 0..n_internal-1;
 *                               may be NULL when T == 0
 *   parent  [n_nodes]           parent[0] = -1, parent[n] < n, level order,
 *                               children of a node contiguous; every node has at
 *                               most 64 children
 *   cand    [B][n_nodes]        token carried by each draft node (entry 0 unused)
 *   unif    [B][n_nodes][2]     [..][0]: uniform of the test of node n as a
 *                               candidate; [..][1]: uniform of the endpoint draw
 *                               when the walk stops at n
 *   mode 0 / 1: Algorithm 1 / Algorithm 2; mode 2: naive sampling (draw from the target
 *   distribution, accept if a candidate carries the drawn token; draft unused, may be NULL)
 *   sequential = 0: evaluate every node, then walk (the data-parallel form);
 *   sequential = 1: the paper's literal procedure, evaluating only the nodes the
 *                   walk stands on.  Per-node outputs of unvisited nodes are then
 *                   -2 (accept, bonus) and NaN (ratio).
 * Outputs (any of the per-node ones may be NULL):
 *   out_accept_len [B]            number of accepted draft tokens, 0..gamma
 *   out_tokens     [B][gamma+1]   accepted tokens, then the endpoint token, then -1
 *   out_residual   [B][V] double  distribution the endpoint token was drawn from
 *   node_accept    [B][n_nodes]   accepted child of each node or -1
 *   node_bonus     [B][n_nodes]   endpoint token of each node that can end a walk
 *                                 (leaf, or every candidate rejected), else -1
 *   node_ratio     [B][n_nodes]   p/q seen by the test of each draft node
 *   out_status     [B]            OR of ORACLE_STATUS_* bits
 * Returns 0, or -1 on malformed arguments.
 */
int32_t mcsd_oracle_verify(int32_t B, int32_t n_nodes, int32_t n_internal, int32_t V,
                           const float *target, const float *draft, const int32_t *parent,
                           const int32_t *cand, const float *unif, double T, int32_t mode,
                           int32_t sequential, int32_t *out_accept_len,
                           int32_t *out_tokens, double *out_residual, int32_t *node_accept,
                           int32_t *node_bonus, double *node_ratio, int32_t *out_status)
{
    if (B < 0 || n_nodes < 1 || V < 1 || n_internal < 0 || n_internal > n_nodes) return -1;
    if (!(T >= 0.0) || (mode != 0 && mode != 1 && mode != 2)) return -1;
    if (parent[0] != -1) return -1;
    for (int32_t n = 1; n < n_nodes; ++n)
        if (parent[n] < 0 || parent[n] >= n || parent[n] < parent[n - 1]) return -1;
    for (int32_t n = 0; n < n_nodes; ++n) {
        int32_t first, k = children_of(parent, n_nodes, n, &first);
        if (k > 64) return -1;
        if ((k > 0) != (n < n_internal)) return -1;
    }
    if (T > 0.0 && mode != 2 && n_internal > 0 && !draft) return -1;
    const int32_t gamma = tree_depth(parent, n_nodes);
    int32_t fail = 0;

#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        const float *target_b = target + (size_t)b * n_nodes * V;
        const float *draft_b = draft ? draft + (size_t)b * n_internal * V : NULL;
        const int32_t *cand_b = cand + (size_t)b * n_nodes;
        const float *unif_b = unif + (size_t)b * n_nodes * 2;
        double *ratio_b = node_ratio ? node_ratio + (size_t)b * n_nodes : NULL;
        int32_t status = 0;
        size_t n_keep = sequential ? 1 : (size_t)n_nodes;
        double *res = (double *)malloc(n_keep * V * sizeof(double));
        double *qbuf = (double *)malloc((size_t)V * sizeof(double));
        int32_t *acc = (int32_t *)malloc((size_t)n_nodes * sizeof(int32_t));
        int32_t *bon = (int32_t *)malloc((size_t)n_nodes * sizeof(int32_t));
        if (!res || !qbuf || !acc || !bon) {
            fail = 1;
            free(res); free(qbuf); free(acc); free(bon);
            continue;
        }
        for (int32_t n = 0; n < n_nodes; ++n) { acc[n] = -2; bon[n] = -2; }
        if (ratio_b)
            for (int32_t n = 0; n < n_nodes; ++n) ratio_b[n] = NAN;

        if (!sequential) {
            for (int32_t n = 0; n < n_nodes; ++n)
                acc[n] = verify_node(n, n_nodes, n_internal, V, target_b, draft_b, parent,
                                     cand_b, unif_b, T, mode, res + (size_t)n * V, qbuf,
                                     &bon[n], ratio_b, &status);
        }
        /* the walk: from the root, follow accepted children */
        int32_t n = 0, len = 0;
        int32_t *tok = out_tokens + (size_t)b * (gamma + 1);
        for (int32_t i = 0; i <= gamma; ++i) tok[i] = -1;
        for (;;) {
            if (sequential)
                acc[n] = verify_node(n, n_nodes, n_internal, V, target_b, draft_b, parent,
                                     cand_b, unif_b, T, mode, res, qbuf, &bon[n], ratio_b,
                                     &status);
            if (acc[n] < 0) break;
            n = acc[n];
            tok[len++] = cand_b[n];
        }
        tok[len] = bon[n];
        out_accept_len[b] = len;
        if (out_residual)
            memcpy(out_residual + (size_t)b * V, sequential ? res : res + (size_t)n * V,
                   (size_t)V * sizeof(double));
        if (node_accept) memcpy(node_accept + (size_t)b * n_nodes, acc, (size_t)n_nodes * sizeof(int32_t));
        if (node_bonus) memcpy(node_bonus + (size_t)b * n_nodes, bon, (size_t)n_nodes * sizeof(int32_t));
        if (out_status) out_status[b] = status;
        free(res); free(qbuf); free(acc); free(bon);
    }
    return fail ? -2 : 0;
}
