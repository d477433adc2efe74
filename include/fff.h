/*
 * fff.h -- C ABI of the B200 (sm_100a) library for hard-routed inference of
 * Fast Feedforward (FFF) networks.
 *
 * The library computes FORWARD_I of Algorithm 1 ("FFF forward pass") for a
 * batch of B independent tokens: every token descends a depth-d balanced
 * binary tree of single-neuron nodes, taking the right child when the node
 * output c = sigmoid(<w, x> + b) is >= 1/2 (i.e. when the logit is >= 0) and
 * the left child otherwise, and is then evaluated by the one leaf network
 * N_{d,j} it reaches:  y = W2_j act(W1_j x + b1_j) + b2_j.
 *
 * Conventions shared by all calls
 *  - Every pointer is a DEVICE pointer unless its name ends in _host.  Device
 *    pointers must be 16-byte aligned and belong to the CUDA device that was
 *    current when the handle was created.  The caller owns every buffer it
 *    passes in.
 *  - All tensors are dense and row-major.  One element type per handle: all of
 *    x, y and the weights are float32 (FFF_DTYPE_F32) or bfloat16
 *    (FFF_DTYPE_BF16, products accumulated in float32).  Index arrays are
 *    int32.
 *  - Node N_{m,n} (level m, position n) is row 2^m - 1 + n of the node arrays;
 *    its children are N_{m+1,2n} (left) and N_{m+1,2n+1} (right) (Section
 *    "Algorithm", Definition).  leaf_idx is n of the leaf N_{d,n}: the d
 *    decisions read from the root as a binary number, 1 = right.
 *  - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *    Calls that take a stream only enqueue work on it and return without
 *    waiting, unless stated otherwise.
 *  - Every call returns an fff_status_t; nothing throws, aborts or traps.
 *    Argument errors are detected on the host before anything is launched.
 *  - A handle serves one forward at a time (its workspace is shared by its
 *    calls); different handles are independent.
 *  - Results are bit-reproducible from run to run for fixed inputs.
 */
#ifndef FFF_H
#define FFF_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fff_handle_s *fff_handle_t;

typedef enum {
    FFF_OK = 0,
    FFF_ERR_INVALID_ARG = 1,     /* NULL / misaligned pointer, non-positive size, unknown enum, B < 0 */
    FFF_ERR_UNSUPPORTED = 2,     /* valid request this build cannot serve (e.g. depth > FFF_MAX_DEPTH, B > FFF_MAX_TOKENS) */
    FFF_ERR_ALLOC = 3,           /* device or host allocation failed */
    FFF_ERR_CUDA = 4,            /* a CUDA runtime call failed */
    FFF_ERR_DEVICE_TIMEOUT = 5,  /* a bounded device-side wait ran out (read by fff_get_last_status) */
    FFF_ERR_BAD_HANDLE = 6,      /* NULL, destroyed or corrupted handle */
    FFF_ERR_TOO_LARGE = 7        /* request exceeds the fixed capacity of fff_leaf_bucketing_static */
} fff_status_t;

typedef enum {
    FFF_ACT_RELU = 0,            /* max(v, 0) */
    FFF_ACT_GELU = 1,            /* v * Phi(v), erf form (not the tanh approximation); the bf16 tensor-core
                                    kernels evaluate erf to 1.5e-7 absolute, below bf16 resolution */
    FFF_ACT_GELU_TANH = 2,       /* v/2 * (1 + tanh(sqrt(2/pi) * (v + 0.044715 v^3))): a different function from
                                    FFF_ACT_GELU (up to 5e-4 apart), not a cheaper evaluation of it */
    FFF_ACT_SILU = 3             /* v * sigmoid(v) */
} fff_activation_t;              /* the leaf networks' hidden activation: the paper's Definition (leaves are
                                    <dim_I, l, dim_O> feedforward networks) names none */

typedef enum {
    FFF_DTYPE_F32 = 0,
    FFF_DTYPE_BF16 = 1           /* bf16 storage, float32 accumulation, y rounded to nearest even */
} fff_dtype_t;

#define FFF_MAX_DEPTH 20
/* Largest batch any call accepts (2^31 - 4096: token numbers and slice bounds are int32). */
#define FFF_MAX_TOKENS 2147479552

/* Kernel families a handle may be pinned to with fff_set_path (testing / tuning). */
typedef enum {
    FFF_PATH_AUTO = 0,           /* library picks per stage from shapes and B */
    FFF_PATH_WARP = 1,           /* CUDA-core warp kernels for descent and leaf evaluation */
    FFF_PATH_TENSOR = 2,         /* tensor-core kernels wherever the shapes allow them */
    FFF_PATH_FUSED = 3           /* the one-launch kernel for small trees with leaves of at most 32 neurons */
} fff_path_t;

/*
 * Create an FFF layer (Section "Algorithm", Definition: a pair <N, L> of
 * 2^d - 1 node networks of node size 1 and 2^d leaf networks of leaf size l).
 *
 *   D, O          dim_I and dim_O, >= 1
 *   depth         d, 0 <= d <= FFF_MAX_DEPTH; d = 0 is a single leaf, no nodes
 *   leaf_width    l >= 1
 *   node_w        [2^d-1, D]   may be NULL iff depth == 0
 *   node_b        [2^d-1]      NULL = all zero
 *   leaf_w1       [2^d, l, D]
 *   leaf_b1       [2^d, l]     NULL = all zero
 *   leaf_w2       [2^d, O, l]
 *   leaf_b2       [2^d, O]     NULL = all zero
 *
 * The weights are copied (and re-laid-out for the kernels) into memory owned
 * by the handle before the call returns; the caller's buffers may be freed
 * afterwards.  The call synchronises the device.  On failure *out is NULL.
 */
fff_status_t fff_create(fff_handle_t *out, int D, int O, int depth, int leaf_width,
                        fff_activation_t act, fff_dtype_t dtype,
                        const void *node_w, const void *node_b,
                        const void *leaf_w1, const void *leaf_b1,
                        const void *leaf_w2, const void *leaf_b2);

/*
 * The same layer with its leaf weights stored as 8-bit floats: leaf_w1_e4m3 [2^d, l, D] and leaf_w2_e4m3
 * [2^d, O, l] hold e4m3 codes (4 exponent bits with bias 7, 3 mantissa bits, no infinities), leaf_w1_scale and
 * leaf_w2_scale [2^d] one float32 scale per leaf: the weight a code stands for is its e4m3 value times the
 * scale of its leaf.  Everything else (x, y, node weights, biases) is bfloat16; products are accumulated in
 * float32 and the scales are applied to the sums, so the result is FORWARD_I of the layer with exactly those
 * weights.  (The paper stores its weights in one floating-point type; this halves the bytes of the leaf
 * weights, the largest stream of a layer with many thin leaves.)  Runs on the tcgen05 kernels only:
 * FFF_ERR_UNSUPPORTED unless D % 128 == 0, O % 16 == 0 and l <= 64; fff_forward_train, the warp path and the
 * one-launch kernel are not available on such a handle.
 */
fff_status_t fff_create_w8(fff_handle_t *out, int D, int O, int depth, int leaf_width, fff_activation_t act,
                           const void *node_w, const void *node_b,
                           const uint8_t *leaf_w1_e4m3, const float *leaf_w1_scale, const void *leaf_b1,
                           const uint8_t *leaf_w2_e4m3, const float *leaf_w2_scale, const void *leaf_b2);

/*
 * FORWARD_I of Algorithm 1 for B tokens, enqueued on `cuda_stream`.
 *
 *   x         [B, D]  in
 *   y         [B, O]  out
 *   leaf_idx  [B]     out, may be NULL: the region / leaf each token was routed to
 *
 * B == 0 is FFF_OK and enqueues nothing.  If B exceeds what fff_reserve was
 * given, the workspace is grown first (this allocates and synchronises).
 * Otherwise the call only enqueues kernels (and at most a small memset) and
 * returns: after fff_reserve(B) and one ordinary call of the same size, it may
 * be captured into a CUDA graph and replayed on new contents of x (tested).
 */
fff_status_t fff_forward_infer(fff_handle_t h, const void *x, void *y, int32_t *leaf_idx,
                               int64_t B, void *cuda_stream);

/*
 * FORWARD_T of Algorithm 1 for B tokens: the training-time forward pass, in which every token is evaluated by
 * ALL leaves and the outputs are mixed with the node choices, y = sum_j mix_j N_{d,j}(x), where mix_j is the
 * product over the root path of leaf j of c = sigmoid(<w, x> + b) (where the path goes right) or 1 - c (left).
 * A dense contraction over all 2^d l hidden neurons, run as three tensor-core GEMMs (bf16 products, float32
 * accumulation; the weighted hidden activations are rounded to bf16 between the last two).
 *
 *   x             [B, D]       in
 *   y             [B, O]       out
 *   mixture       [B, 2^d]     out, float32, may be NULL: the weight of every leaf (each row sums to 1)
 *   node_entropy  [2^d - 1]    out, float32, may be NULL: for every node, the batch mean of the entropy
 *                 -c ln c - (1 - c) ln(1 - c) of its choice (Section "Training": the hardening loss is B times the
 *                 sum of these; the batch means are what the paper monitors)
 *
 * bf16 layers with D % 64 == 0 only (FFF_ERR_UNSUPPORTED otherwise).  The first call of a size allocates a
 * workspace of B (2^d l + 2^d) bf16 and B 2^(d+1) float32 and synchronises; later calls only enqueue.
 * No gradients are computed: this is the forward half of a training step.
 */
fff_status_t fff_forward_train(fff_handle_t h, const void *x, void *y, float *mixture, float *node_entropy,
                               int64_t B, void *cuda_stream);

/*
 * The same computation for buffers in HOST memory (pinned or pageable):
 * copies x to the device, runs fff_forward_infer, copies y (and leaf_idx when
 * not NULL) back, and returns after `cuda_stream` has completed.  Batches of
 * 16384 tokens or more are cut into up to 16 chunks whose copies (on two
 * library-owned streams, ordered after what `cuda_stream` already holds) and
 * kernels overlap; with pinned host buffers this takes about the time of the
 * slower copy direction.  Results do not depend on the chunking.  After a
 * chunked call fff_debug_get_bucketing has nothing to report
 * (FFF_ERR_INVALID_ARG) until the next fff_forward_infer.
 */
fff_status_t fff_forward_infer_host(fff_handle_t h, const void *x_host, void *y_host,
                                    int32_t *leaf_idx_host, int64_t B, void *cuda_stream);

/* Free everything the handle owns.  Synchronises the device first; no work of
 * this handle may be enqueued afterwards. */
fff_status_t fff_destroy(fff_handle_t h);

/* Size the workspace for batches of up to max_B tokens so that later forwards
 * allocate nothing.  Allocates and synchronises.  The workspace is a few
 * int32 per token, plus, on the tensor-core path, a table of per-leaf token
 * lists of 2^depth * max_B int32 (only while that is at most 1 GiB; larger
 * layers run a bucketing kernel instead), of which a forward touches B entries;
 * trees whose descent runs as two tensor-core stages add a table of per-node
 * lists between the stages (at most 256 * max_B int32, same rule). */
fff_status_t fff_reserve(fff_handle_t h, int64_t max_B);

/* Pin the handle to one kernel family (FFF_PATH_*).  FFF_ERR_UNSUPPORTED if
 * the shapes of this handle cannot run on it. */
fff_status_t fff_set_path(fff_handle_t h, fff_path_t path);

/* Switches between kernels that compute the same thing, for A/B timing and tests.  Every switch is on (1) by
 * default, which is the measured best; results never depend on them.  The paper describes no such choices.
 * FFF_ERR_INVALID_ARG for an unknown key or a value other than 0 or 1. */
typedef enum {
    FFF_TUNE_TCGEN05_DESCENT = 0, /* first descent stage of up to 8 levels on tcgen05 (0: stages of <= 6 levels on mma.sync) */
    FFF_TUNE_TCGEN05_GROUPED = 1, /* later descent stages on tcgen05 when their groups fill 128-row tiles (0: mma.sync) */
    FFF_TUNE_TCGEN05_LEAF = 2,    /* leaf evaluation on tcgen05 (0: mma.sync kernel) */
    FFF_TUNE_CTA_PAIRS = 3,       /* first descent stage with 128 or 256 nodes on pairs of CTAs (0: single CTAs) */
    FFF_TUNE_DIRECT_LISTS = 4,    /* descent stages file the tokens under the nodes / leaves they reach, for the kernel
                                     that follows (0: bucketing kernels) */
    FFF_TUNE_FUSED_SMALL = 5,     /* small trees with thin leaves in one launch: descent, grid barrier, leaf evaluation
                                     by groups of 32 hidden neurons kept in shared memory (0: descent, bucketing and
                                     leaf kernels).  Taken by default by layers without a tensor-core leaf path */
    FFF_TUNE_GROUP_TILES = 6,     /* leaf kernel tiles of tokens that share the node three levels above the leaves: the
                                     first descent stage stops there, the leaf kernel walks the last three levels from
                                     7 extra accumulator columns and evaluates the node's 8 leaves side by side, each
                                     row keeping its own leaf's hidden units (0: tiles of one leaf).  Taken for bf16
                                     layers with 8 <= leaf_width < 16 and 9 <= depth <= 11 (where it replaces the
                                     second descent stage and its node bucketing), when those nodes receive at least
                                     128 tokens each on average */
    FFF_TUNE_COUNT = 7
} fff_tuning_t;
fff_status_t fff_set_tuning(fff_handle_t h, fff_tuning_t key, int value);

/*
 * Stage entry points.  fff_forward_infer computes what these three compute
 * when called in this order.
 */

/* Tree descent (Algorithm 1, FORWARD_I, non-leaf branch; paragraph on
 * inference complexity: d steps, one node network each).
 *   x [B, D] in;  leaf_idx [B] out. */
fff_status_t fff_tree_descent(fff_handle_t h, const void *x, int32_t *leaf_idx,
                              int64_t B, void *cuda_stream);

/* Leaf bucketing: the stable counting sort of token ids by leaf.  Not a step
 * of the paper (its implementation gathers weights per token); it groups the
 * tokens so that each leaf's weights are fetched once per batch.
 *   leaf_idx [B] in, values in [0, 2^depth); ids outside that range are
 *            ignored and leave their perm entries unwritten
 *   offsets  [2^depth + 1] out: offsets[j] = #tokens with leaf < j
 *   perm     [B] out: perm[offsets[j] + r] = r-th smallest token id routed to leaf j
 * Uses the handle's workspace. */
fff_status_t fff_leaf_bucketing(fff_handle_t h, const int32_t *leaf_idx, int32_t *offsets,
                                int32_t *perm, int64_t B, void *cuda_stream);

/*
 * Leaf bucketing without any allocation.  (The paper has no counterpart of
 * this call; it exists for the callers described below.)
 *
 * Some callers must not allocate device memory at the point where they need
 * the bucketing: code running between the begin and end of a memory-pool
 * accounting window, plugins of a host application that owns all device
 * memory and forbids cudaMalloc, or latency-critical loops in which an
 * allocation (which may synchronise the device) is unacceptable.  Such callers
 * cannot create an fff handle, whose workspace is allocated.  This entry point
 * returns exactly what fff_leaf_bucketing returns, bit for bit (the stable
 * order is unique), through different kernels (a histogram, then a placement
 * pass over ranges of leaves); it takes no handle and keeps its scratch (the
 * per-leaf token counts) in a fixed array compiled into the library:
 * 2 * FFF_STATIC_MAX_BINS int32 counters = 512 KiB, resident on every GPU
 * that loads the library, for the life of the process.
 *
 *   leaf_idx [B] in, values in [0, 2^depth); ids outside are ignored (they
 *            are not counted in offsets and take no perm entry, so the last
 *            B - offsets[2^depth] entries of perm stay unwritten)
 *   offsets  [2^depth + 1] out,  perm [B] out      (as for fff_leaf_bucketing)
 *   depth    0 <= depth <= FFF_STATIC_MAX_DEPTH;  B <= FFF_MAX_TOKENS
 *
 * Larger requests return FFF_ERR_TOO_LARGE and launch nothing.  The call uses
 * the current device; all pointers are device pointers on it.  It calls no
 * cudaMalloc / cudaFree and no allocating library routine.
 *
 * The first call on each device looks up the device address of the array
 * (and sets a kernel attribute); make that first call before starting any
 * stream capture.  The array is shared by every call in the process and
 * keeps the previous call's counts, so each call first clears the part it
 * uses, on `cuda_stream`.  Two calls whose work overlaps on the GPU (different
 * streams, or different host threads) race on the array: serialise them.
 */
#define FFF_STATIC_MAX_DEPTH 16
#define FFF_STATIC_MAX_BINS (1 << FFF_STATIC_MAX_DEPTH)
fff_status_t fff_leaf_bucketing_static(const int32_t *leaf_idx, int32_t *offsets, int32_t *perm,
                                       int64_t B, int depth, void *cuda_stream);

/* Grouped leaf evaluation with un-permuting write-back (Algorithm 1,
 * FORWARD_I, leaf branch: return N_{d,j}(x)):
 * for every i, with t = perm[i] and j = leaf_idx[t]:
 *   y[t, :] = W2_j act(W1_j x[t, :] + b1_j) + b2_j.
 *   x [B, D], leaf_idx [B], offsets [2^depth + 1], perm [B] in;  y [B, O] out. */
fff_status_t fff_grouped_leaf_ff(fff_handle_t h, const void *x, const int32_t *leaf_idx,
                                 const int32_t *offsets, const int32_t *perm, void *y,
                                 int64_t B, void *cuda_stream);

/* Copy the bucketing of the handle's most recent forward into caller buffers
 * (device): perm [B], offsets [2^depth + 1].  Enqueued on `cuda_stream`.  Two kinds
 * of forward do not make the stable bucketing themselves: one with fewer than
 * about 4 tokens per leaf, which evaluates the leaves one token at a time, and one
 * whose descent files the tokens under their leaves directly for the tensor-core
 * leaf kernel (in an order that is not the stable one).  The bucketing is then
 * computed here, from the leaf indices the forward kept in the handle's workspace. */
fff_status_t fff_debug_get_bucketing(fff_handle_t h, int32_t *perm, int32_t *offsets,
                                     void *cuda_stream);

/* Synchronise the device and report the device-side status word of the handle:
 * FFF_OK, or FFF_ERR_DEVICE_TIMEOUT if a bounded wait in a kernel expired since
 * the last call (the word is cleared). */
fff_status_t fff_get_last_status(fff_handle_t h);

/* Self-test of the error path behind FFF_ERR_DEVICE_TIMEOUT (no counterpart in the paper).  Enqueues a
 * one-CTA kernel whose threads wait, with the library's bounded-wait helpers, on a barrier that nothing
 * ever signals; after limit_cycles (1 .. 2^24 SM clock cycles, i.e. at most about 10 ms) the wait gives
 * up and the kernel records the timeout in the handle's status word and ends.  The next
 * fff_get_last_status then returns FFF_ERR_DEVICE_TIMEOUT once, and FFF_OK after that.  Nothing faults
 * and the context stays usable. */
fff_status_t fff_selftest_bounded_wait(fff_handle_t h, int64_t limit_cycles, void *cuda_stream);

/* Which kernel families the shapes of this layer admit (a bit set; -1 for a bad handle).  A bf16 layer whose
 * D is no multiple of 128, whose O is no multiple of 8 or whose leaves are wider than 64 has no tensor-core
 * kernels: its forward runs on CUDA-core kernels (the one-launch kernel when FFF_CAP_FUSED_SMALL is set, else
 * one warp per token), which is several times slower per token; float32 layers never have them.  Callers
 * that depend on tensor-core speed can check here instead of timing. */
typedef enum {
    FFF_CAP_TENSOR_DESCENT = 1,   /* staged descent on tensor cores (bf16, D % 128 == 0, depth > 0) */
    FFF_CAP_TCGEN05_DESCENT = 2,  /* ... its first stage on tcgen05 */
    FFF_CAP_TENSOR_LEAF = 4,      /* grouped leaf evaluation on tensor cores (also O % 8 == 0, l <= 64) */
    FFF_CAP_TCGEN05_LEAF = 8,     /* ... on tcgen05 (also O % 16 == 0) */
    FFF_CAP_FUSED_SMALL = 16,     /* the one-launch kernel (l <= 32, at most one group of 32 neurons per SM) */
    FFF_CAP_FORWARD_TRAIN = 32,   /* fff_forward_train (bf16, D % 64 == 0) */
    FFF_CAP_GROUP_TILES = 64      /* leaf tiles of 8 sibling leaves (FFF_TUNE_GROUP_TILES: 8 <= leaf_width < 16, 9 <= depth <= 11) */
} fff_capability_t;
int fff_capabilities(fff_handle_t h);

/* Number of kernels the most recent forward / stage call of this handle enqueued
 * (-1 for a bad handle). */
int fff_last_launch_count(fff_handle_t h);

/*
 * Per-launch timing of forwards, for benchmarks.  After fff_profile_begin the
 * next max_steps calls of fff_forward_infer record a CUDA event on their stream
 * before the first and after every kernel they launch (at most 16 per forward).
 * fff_profile_end synchronises the device, writes the mean duration in
 * milliseconds of each launch position into mean_ms[0 .. fff_profile_launches)
 * and the number of recorded forwards into *steps, and stops recording.
 * fff_profile_launch_name(h, i) names the kernel at position i ("" if out of
 * range); the string is static.
 */
fff_status_t fff_profile_begin(fff_handle_t h, int max_steps);
fff_status_t fff_profile_end(fff_handle_t h, double *mean_ms, int *steps);
int fff_profile_launches(fff_handle_t h);
const char *fff_profile_launch_name(fff_handle_t h, int i);

/*
 * Several FFF layers behind one handle (Section "Fast feedforward layers as building blocks": FFF layers in
 * place of the feedforward layers of a transformer, each behind a layer normalisation and inside a residual
 * connection; the attention layers between them are not part of this library).  For token x_0 and K layers:
 *     z_k     = layer_norm ? (x_k - mean) / sqrt(var + eps) * gamma_k + beta_k : x_k      (over the D features)
 *     x_{k+1} = residual ? x_k + FFF_k(z_k) : FFF_k(z_k)                                   (FORWARD_I per layer)
 * and y = x_K.  z_k and x_k are stored in the layers' element type between the kernels.
 *
 *   layers     n_layers distinct live handles on one device, one element type, D == O == the same width
 *   ln_gamma   NULL, or n_layers device pointers to [D] vectors in the element type (an entry may be NULL = ones)
 *   ln_beta    likewise (NULL = zeros); both are copied.  Ignored when layer_norm == 0
 * The stack does not own the layers: destroy it before them, and run no other forward on them while one of
 * the stack's is in flight.  fff_set_path / fff_set_tuning on the layers stay in effect.
 */
typedef struct fff_stack_s *fff_stack_t;
fff_status_t fff_stack_create(fff_stack_t *out, int n_layers, const fff_handle_t *layers, int layer_norm,
                              const void *const *ln_gamma, const void *const *ln_beta, float eps, int residual);

/* x [B, D] in, y [B, D] out, leaf_idx [n_layers, B] out (may be NULL), all device; enqueued on `cuda_stream`.
 * The first call of a size allocates the buffers between the layers (and synchronises). */
fff_status_t fff_stack_forward(fff_stack_t s, const void *x, void *y, int32_t *leaf_idx, int64_t B, void *cuda_stream);

/* on = 1: the stack records its forward into a CUDA graph the second time it is called with the same x, y,
 * leaf_idx, B and stream, and replays that graph on every later call with those arguments (new contents of x
 * are read; the addresses are part of the recording).  Other arguments run as plain launches and start a new
 * recording.  If the forward cannot be recorded (the legacy default stream cannot be captured, for one), plain
 * launches are used from then on; fff_stack_set_graph(s, 1) again allows another attempt.  Default 0. */
fff_status_t fff_stack_set_graph(fff_stack_t s, int on);

/* Kernels the most recent plain (not replayed) forward enqueued, and whether the most recent forward was a
 * replay (-1 for a bad handle). */
int fff_stack_last_launch_count(fff_stack_t s);
int fff_stack_last_was_replay(fff_stack_t s);

fff_status_t fff_stack_destroy(fff_stack_t s);

/* Static, never NULL. */
const char *fff_status_string(fff_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* FFF_H */
