/*
 * CPU oracle for Fast Feedforward (FFF) networks -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, float64 restatement of what the paper defines.  It exists to
 * check the CUDA library and to be timed as a CPU baseline.  It shares no code
 * with the CUDA path and must never be called from it.
 *
 * Conventions (all arrays row-major, all floating point in double):
 *   node_w [2^d-1][D], node_b [2^d-1]      node N_{m,n} is row 2^m - 1 + n
 *   w1 [2^d][l][D], b1 [2^d][l]            leaf N_{d,j} hidden weights / biases
 *   w2 [2^d][O][l], b2 [2^d][O]            leaf output weights / biases
 *   x  [B][D], y [B][O]
 *
 * A node is one neuron with a sigmoid head (node size n = 1, Section
 * "Algorithm", Definition and the paragraph on region boundaries): its output
 * is c = sigmoid(<w, x> + b).  A leaf is a <D, l, O> feedforward network:
 * y = W2 act(W1 x + b1) + b2.
 *
 * Parity status of each function is listed next to it: every function below is
 * pinned by tests that do not call this file's own formulae (brute-force path
 * enumeration, hand-computed cases, library routines, identities from the
 * paper).  The numerical values of y on the five benchmark configurations are
 * not printed anywhere in the paper, so they are pinned only through those
 * structural checks.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { FFF_ORACLE_RELU = 0, FFF_ORACLE_GELU = 1, FFF_ORACLE_GELU_TANH = 2, FFF_ORACLE_SILU = 3 };

/*
 * The leaf's hidden activation.  The paper never names one (Definition: the
 * leaves are plain <D, l, O> feedforward networks), so it is a parameter:
 *   RELU       max(v, 0)
 *   GELU       v * Phi(v), Phi the standard normal CDF (exact erf form)
 *   GELU_TANH  the published tanh approximation of GELU,
 *              v/2 * (1 + tanh(sqrt(2/pi) * (v + 0.044715 v^3)))
 *   SILU       v * sigmoid(v)
 * Pinned by: library routines (torch), table values of Phi, the identity
 * f(v) - f(-v) = v that the last three share, values at 0 and far from 0.
 */
static double act_fn(int act, double v)
{
    if (act == FFF_ORACLE_RELU) return v > 0.0 ? v : 0.0;
    if (act == FFF_ORACLE_GELU_TANH)
        return 0.5 * v * (1.0 + tanh(sqrt(2.0 / 3.14159265358979323846) * (v + 0.044715 * v * v * v)));
    if (act == FFF_ORACLE_SILU) return v / (1.0 + exp(-v));
    return 0.5 * v * (1.0 + erf(v / sqrt(2.0)));
}

/* <w, x> + b, k ascending. */
static double node_logit(int D, const double *w, double b, const double *x)
{
    double s = b;
    for (int k = 0; k < D; ++k) s += w[k] * x[k];
    return s;
}

/* Leaf network N_{d,j}(x) = W2_j act(W1_j x + b1_j) + b2_j  (Definition, set L). */
static void leaf_eval(int D, int O, int l, int act,
                      const double *w1, const double *b1,
                      const double *w2, const double *b2,
                      long j, const double *x, double *y)
{
    double *h = (double *)malloc(sizeof(double) * (size_t)(l > 0 ? l : 1));
    const double *w1j = w1 + (size_t)j * l * D, *b1j = b1 + (size_t)j * l;
    const double *w2j = w2 + (size_t)j * O * l, *b2j = b2 + (size_t)j * O;
    for (int i = 0; i < l; ++i) {
        double s = b1j[i];
        for (int k = 0; k < D; ++k) s += w1j[(size_t)i * D + k] * x[k];
        h[i] = act_fn(act, s);
    }
    for (int o = 0; o < O; ++o) {
        double s = b2j[o];
        for (int i = 0; i < l; ++i) s += w2j[(size_t)o * l + i] * h[i];
        y[o] = s;
    }
    free(h);
}

/*
 * Hard descent of Algorithm 1, FORWARD_I, non-leaf branch, for one token: at
 * N_{m,n} take the right child N_{m+1,2n+1} when c >= 1/2, otherwise the left
 * child N_{m+1,2n}.  sigmoid is increasing with sigmoid(0) = 1/2, so c >= 1/2
 * exactly when the logit is >= 0 (the paper's own implementation note likewise
 * tests the sign of the logit: Section "Algorithm", paragraph on inference
 * complexity).  Returns n of the leaf N_{d,n} reached.
 */
static long descend_one(int D, int depth, const double *node_w, const double *node_b,
                        const double *xt, double *min_abs, long *node_evals)
{
    long n = 0;                          /* current node is N_{m,n} */
    double mn = INFINITY;
    for (long m = 0; m < depth; ++m) {
        long row = ((long)1 << m) - 1 + n;
        double logit = node_logit(D, node_w + (size_t)row * D, node_b[row], xt);
        if (node_evals) ++*node_evals;
        if (fabs(logit) < mn) mn = fabs(logit);
        n = (logit >= 0.0) ? 2 * n + 1 : 2 * n;
    }
    if (min_abs) *min_abs = mn;
    return n;
}

/*
 * Descent only, tokens [t0, t1).
 * leaf_idx[t]  = n of the leaf N_{d,n} reached.
 * min_abs[t]   = smallest |logit| met on the path (NULL to skip); +inf if d = 0.
 * node_evals   = incremented once per node network executed (NULL to skip).
 * Pinned by: brute-force path enumeration, zero-weight tie case, hand case
 * (leaf indices and the per-token smallest |logit|).
 */
void fff_oracle_descend(int D, int depth, const double *node_w, const double *node_b,
                        const double *x, long t0, long t1,
                        int32_t *leaf_idx, double *min_abs, long *node_evals)
{
    for (long t = t0; t < t1; ++t)
        leaf_idx[t] = (int32_t)descend_one(D, depth, node_w, node_b, x + (size_t)t * D,
                                           min_abs ? min_abs + t : NULL, node_evals);
}

/*
 * FORWARD_I of Algorithm 1 for tokens [t0, t1): descend, then evaluate the one
 * leaf reached.  Exactly `depth` node networks and one leaf network run per
 * token (paragraph on inference complexity); the counters record that.
 * Pinned by: depth-0 == plain feedforward layer, hand case, saturated soft
 * mixture, all-leaves-masked evaluation.
 */
void fff_oracle_forward_i(int D, int O, int depth, int l, int act,
                          const double *node_w, const double *node_b,
                          const double *w1, const double *b1,
                          const double *w2, const double *b2,
                          const double *x, long t0, long t1,
                          double *y, int32_t *leaf_idx,
                          long *node_evals, long *leaf_evals)
{
    for (long t = t0; t < t1; ++t) {
        long j = descend_one(D, depth, node_w, node_b, x + (size_t)t * D, NULL, node_evals);
        if (leaf_idx) leaf_idx[t] = (int32_t)j;
        leaf_eval(D, O, l, act, w1, b1, w2, b2, j, x + (size_t)t * D, y + (size_t)t * O);
        if (leaf_evals) ++*leaf_evals;
    }
}

/* FORWARD_T of Algorithm 1 at node N_{m,n}: recursive soft mixture into out[O]. */
static void forward_t_rec(int D, int O, int depth, int l, int act,
                          const double *node_w, const double *node_b,
                          const double *w1, const double *b1,
                          const double *w2, const double *b2,
                          const double *x, long m, long n, double *out)
{
    if (m == depth) {
        leaf_eval(D, O, l, act, w1, b1, w2, b2, n, x, out);
        return;
    }
    long row = ((long)1 << m) - 1 + n;
    double logit = node_logit(D, node_w + (size_t)row * D, node_b[row], x);
    double c = 1.0 / (1.0 + exp(-logit));
    double *right = (double *)malloc(sizeof(double) * (size_t)O);
    double *left = (double *)malloc(sizeof(double) * (size_t)O);
    forward_t_rec(D, O, depth, l, act, node_w, node_b, w1, b1, w2, b2, x, m + 1, 2 * n + 1, right);
    forward_t_rec(D, O, depth, l, act, node_w, node_b, w1, b1, w2, b2, x, m + 1, 2 * n, left);
    for (int o = 0; o < O; ++o) out[o] = c * right[o] + (1.0 - c) * left[o];
    free(right);
    free(left);
}

/*
 * FORWARD_T of Algorithm 1 (training-time soft mixture over all 2^d leaves).
 * Only used to check FORWARD_I against its soft limit; cost is 2^d leaves per
 * token, so small trees only.
 * Pinned by: zero node weights == mean of all leaves; mixture weights sum to 1.
 */
void fff_oracle_forward_t(int D, int O, int depth, int l, int act,
                          const double *node_w, const double *node_b,
                          const double *w1, const double *b1,
                          const double *w2, const double *b2,
                          const double *x, long B, double *y)
{
    for (long t = 0; t < B; ++t)
        forward_t_rec(D, O, depth, l, act, node_w, node_b, w1, b1, w2, b2,
                      x + (size_t)t * D, 0, 0, y + (size_t)t * O);
}

/*
 * Mixture weights of FORWARD_T written as products over root paths: unrolling the recursion of Algorithm 1,
 * leaf N_{d,j} enters the output with weight  prod_m (bit_m ? c_m : 1 - c_m), where the ancestor of leaf j at
 * level m is N_{m, j >> (d-m)}, c_m its choice and bit_m = (j >> (d-m-1)) & 1 the child on j's path
 * (1 = right, the child that c weighs).  For each token the 2^d weights form a stochastic vector (Section
 * "Algorithm", paragraph on the soft mixture).  mix: [B][2^d].
 * Pinned by: weights sum to 1; sum_j mix_j * leaf_j(x) equals the recursive FORWARD_T; d = 1 by hand.
 */
void fff_oracle_mixture_weights(int D, int depth, const double *node_w, const double *node_b,
                                const double *x, long t0, long t1, double *mix)
{
    long nl = (long)1 << depth;
    for (long t = t0; t < t1; ++t) {
        const double *xt = x + (size_t)t * D;
        for (long j = 0; j < nl; ++j) {
            double p = 1.0;
            for (long m = 0; m < depth; ++m) {
                long n = j >> (depth - m);
                long row = ((long)1 << m) - 1 + n;
                double c = 1.0 / (1.0 + exp(-node_logit(D, node_w + (size_t)row * D, node_b[row], xt)));
                long bit = (j >> (depth - m - 1)) & 1;
                p *= bit ? c : 1.0 - c;
            }
            mix[(size_t)t * nl + j] = p;
        }
    }
}

/*
 * Batch mean of the entropy of every node's choice (Section "Training", hardening: the hardening loss is
 * the sum over the batch and the nodes of the entropies of the Bernoulli choices, and the batch means are
 * what the paper monitors):  H(c) = -c ln c - (1 - c) ln(1 - c), with 0 ln 0 = 0, c = N_{m,n}(x) evaluated
 * for EVERY token at EVERY node (not only along the token's path).  ent: [2^d - 1].
 * Pinned by: c = 1/2 gives ln 2; saturated nodes give 0; a library entropy routine on a hand case.
 */
void fff_oracle_node_entropy(int D, int depth, const double *node_w, const double *node_b,
                             const double *x, long B, double *ent)
{
    long nn = ((long)1 << depth) - 1;
    for (long r = 0; r < nn; ++r) {
        double sum = 0.0;
        for (long t = 0; t < B; ++t) {
            double c = 1.0 / (1.0 + exp(-node_logit(D, node_w + (size_t)r * D, node_b[r], x + (size_t)t * D)));
            double h = 0.0;
            if (c > 0.0) h -= c * log(c);
            if (c < 1.0) h -= (1.0 - c) * log(1.0 - c);
            sum += h;
        }
        ent[r] = B > 0 ? sum / (double)B : 0.0;
    }
}

/*
 * Conditional execution written the wasteful way: evaluate every leaf, keep
 * the one whose region contains the token (each leaf is responsible for
 * exactly one region of the partition).  y = sum_j [j == leaf_idx] * L_j(x).
 */
void fff_oracle_forward_all_leaves_masked(int D, int O, int depth, int l, int act,
                                          const double *w1, const double *b1,
                                          const double *w2, const double *b2,
                                          const double *x, long B,
                                          const int32_t *leaf_idx, double *y)
{
    long nl = (long)1 << depth;
    double *tmp = (double *)malloc(sizeof(double) * (size_t)O);
    for (long t = 0; t < B; ++t) {
        double *yt = y + (size_t)t * O;
        for (int o = 0; o < O; ++o) yt[o] = 0.0;
        for (long j = 0; j < nl; ++j) {
            leaf_eval(D, O, l, act, w1, b1, w2, b2, j, x + (size_t)t * D, tmp);
            double mask = (j == leaf_idx[t]) ? 1.0 : 0.0;
            for (int o = 0; o < O; ++o) yt[o] += mask * tmp[o];
        }
    }
    free(tmp);
}

/*
 * Region membership by brute force: leaf N_{d,j} owns the inputs for which
 * every node on its root path decides toward it.  The ancestor of leaf j at
 * level m is N_{m, j >> (d-m)}, and it must choose child bit (j >> (d-m-1)) & 1
 * (1 = right = c >= 1/2).  Returns the number of leaves whose region contains
 * x_row and stores the last such leaf in *leaf (a partition gives exactly 1).
 */
int fff_oracle_brute_force_leaf(int D, int depth, const double *node_w, const double *node_b,
                                const double *x_row, int32_t *leaf)
{
    long nl = (long)1 << depth;
    int hits = 0;
    for (long j = 0; j < nl; ++j) {
        int ok = 1;
        for (int m = 0; m < depth && ok; ++m) {
            long n = j >> (depth - m);
            int want_right = (int)((j >> (depth - m - 1)) & 1);
            long row = ((long)1 << m) - 1 + n;
            double c = 1.0 / (1.0 + exp(-node_logit(D, node_w + (size_t)row * D, node_b[row], x_row)));
            int right = (c >= 0.5);
            if (right != want_right) ok = 0;
        }
        if (ok) { ++hits; *leaf = (int32_t)j; }
    }
    return hits;
}

/*
 * Leaf bucketing: stable counting sort of token ids by leaf index.
 *   offsets[j]   = number of tokens with leaf < j          (offsets[n_leaves] = B)
 *   perm[offsets[j] + r] = r-th smallest token id with leaf j
 * Pinned by: library stable argsort, permutation / monotonicity properties.
 */
void fff_oracle_bucket(const int32_t *leaf_idx, long B, long n_leaves,
                       int32_t *offsets, int32_t *perm)
{
    long *cursor = (long *)calloc((size_t)n_leaves + 1, sizeof(long));
    for (long j = 0; j <= n_leaves; ++j) offsets[j] = 0;
    for (long t = 0; t < B; ++t) offsets[leaf_idx[t] + 1] += 1;
    for (long j = 0; j < n_leaves; ++j) offsets[j + 1] += offsets[j];
    for (long t = 0; t < B; ++t) {
        long j = leaf_idx[t];
        perm[offsets[j] + cursor[j]] = (int32_t)t;
        cursor[j] += 1;
    }
    free(cursor);
}

/* Section "Size and width": neuron counts of an FFF with depth d, node size n, leaf size l. */
long fff_oracle_training_size(int d, int n, int l) { return (((long)1 << d) - 1) * n + ((long)1 << d) * l; }
long fff_oracle_inference_size(int d, int n, int l) { return (long)d * n + l; }
long fff_oracle_training_width(int d, int l) { return ((long)1 << d) * l; }
long fff_oracle_inference_width(int l) { return l; }
