/* cmoe.h — C ABI of the B200 (sm_100a) forward pass of a SwiGLU FFN restructured
 * into a sparse mixture of experts (shared + routed experts with an analytical
 * router).
 *
 * Method (paper notation): an FFN with hidden width d_h is split, by a neuron
 * partition, into N experts of m = d_h/N neurons, N_s shared (always on) and
 * N_r = N - N_s routed (Section 4.1).  For a token x
 *     F_MoE(x) = E^s(x) + sum_{i<=N_r} g_i E_i^r(x)                 (Eq. moe_output)
 * where every expert is the SwiGLU FFN restricted to its neurons
 *     E(x) = W_down[S]^T ( Swish(W_gate[S]^T x) * (W_up[S]^T x) )   (Eq. ori_ffn_method)
 * the router scores are the SwiGLU activations of one representative neuron
 * per routed expert
 *     s = Swish(W_gate^{R T} x) * (W_up^{R T} x)                    (Eq. router)
 * and, with s' = Softmax(s) over all N_r scores,
 *     g_i = 1 + s'_i u_i  if s'_i + b_i is among the N_k largest keys, else 0
 *                                                                   (Eq. final_gate).
 * Equal keys: the lower expert index wins.  NaN keys rank below every number.
 *
 * All functions return CMOE_OK (0) or a negative cmoe_status; none throws,
 * aborts or prints.  "device" pointers are CUDA global memory of the device
 * that was current at create time; "host" pointers are ordinary memory that
 * is only read (or written) during the call.  A stream argument is a
 * cudaStream_t passed as void* (NULL = the legacy default stream).
 */
#ifndef CMOE_H_
#define CMOE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cmoe_layer cmoe_layer;   /* opaque; owns device memory */

typedef enum {
  CMOE_OK = 0,
  CMOE_ERR_INVALID_ARG = -1,     /* null pointer, negative size, unsupported shape */
  CMOE_ERR_BAD_PARTITION = -2,   /* d_ff % n_experts != 0, or neuron_perm is not a bijection */
  CMOE_ERR_BAD_REP = -3,         /* a representative lies outside its routed expert's slice */
  CMOE_ERR_CAPACITY = -4,        /* T > max_tokens, or a size beyond a stated maximum */
  CMOE_ERR_CUDA = -5,            /* a CUDA runtime/driver call failed (see cmoe_last_error) */
  CMOE_ERR_DEVICE_TIMEOUT = -6,  /* a bounded device-side wait gave up (see cmoe_layer_status) */
  CMOE_ERR_UNSUPPORTED = -7      /* the device is not compute capability 10.x, or a size beyond a stated limit */
} cmoe_status;

typedef enum { CMOE_BF16 = 0, CMOE_FP32 = 1 } cmoe_dtype;

typedef struct {
  int32_t d_model;      /* d */
  int32_t d_ff;         /* d_h */
  int32_t n_experts;    /* N ; m = d_ff / N must divide exactly */
  int32_t n_shared;     /* N_s >= 0 */
  int32_t top_k;        /* N_k, 0 <= N_k <= N_r = N - N_s ; N_r <= 32, N_k <= 8 */
  int32_t max_tokens;   /* the workspace is sized for this many tokens at create */
  int32_t dtype;        /* cmoe_dtype of x, out and every weight matrix */
} cmoe_config;

/* Build a layer from the dense FFN's weights, the neuron partition and the
 * representative neurons (Sections 4.1 and 4.2).
 *   w_gate, w_up : device, [d_ff, d_model] row-major; row n is neuron n's vector
 *                  (column n of the paper's W_gate / W_up).
 *   w_down       : device, [d_model, d_ff] row-major; column n is neuron n's output
 *                  vector (row n of the paper's W_down).
 *   neuron_perm  : host, [d_ff]; expert e owns original neurons
 *                  neuron_perm[e*m .. (e+1)*m); experts 0..N_s-1 are shared and
 *                  form one always-on expert of N_s*m neurons.
 *   rep_idx      : host, [N_r]; ORIGINAL index of routed expert j's representative
 *                  neuron R_j (Eq. rep_neuron); must lie in expert N_s+j's slice.
 *   gate_scale_u : host, [N_r] or NULL (zeros, i.e. unit gates)   (Section 4.3)
 *   select_bias_b: host, [N_r] or NULL (zeros)                     (Eq. final_gate)
 * The weights are copied into expert-contiguous operand layouts on `stream`;
 * the call synchronises that stream before returning, so the caller may free
 * its arrays afterwards.  Requires d_model % 8 == 0.
 * Errors: INVALID_ARG, BAD_PARTITION, BAD_REP, CUDA, UNSUPPORTED. */
int cmoe_layer_create(const cmoe_config* cfg, const void* w_gate, const void* w_up,
                      const void* w_down, const int32_t* neuron_perm, const int32_t* rep_idx,
                      const float* gate_scale_u, const float* select_bias_b, void* stream,
                      cmoe_layer** out_layer);

/* Hierarchical restructuring of an existing MoE layer (Section 4.4): every one
 * of the n_outer experts has been restructured into its own shared + routed
 * sub-experts (inner[i], all created with the same cmoe_config); a top-level
 * router picks outer_top_k of them per token:
 *     logits = W_r x, selected = the outer_top_k largest logits (ties: lower
 *     index), weights w = softmax over the selected logits,
 *     out = sum_{i selected} w_i (E_i^s(x) + sum_j g'_{i,j} E^r_{i,j}(x)).
 *   w_router : device, [n_outer, d_model] row-major, same dtype as the layers.
 *   inner    : host array of n_outer layers; on success their device memory has
 *              been moved into the new layer and the handles are dead (do not
 *              destroy them); on failure they are untouched.
 *   max_tokens: capacity in tokens of the new layer.
 * forward / destroy / get_routing / status of the result are the calls below. */
int cmoe_hier_create(int32_t n_outer, int32_t outer_top_k, const void* w_router,
                     cmoe_layer* const* inner, int32_t max_tokens, void* stream,
                     cmoe_layer** out_layer);

/* out = F_MoE(x) for T tokens (Eq. moe_output with Eq. router and Eq. final_gate).
 *   x   : device, [T, d_model] row-major, 16-byte aligned.
 *   out : device, [T, d_model] row-major, 32-byte aligned (the combine step writes 32 bytes
 *         per store), must not overlap x.
 * Asynchronous on `stream`; allocates nothing; T == 0 is a no-op.  A layer owns
 * one workspace: do not run two forwards of the same layer concurrently.
 * Errors: INVALID_ARG (null, misaligned or overlapping buffers), CAPACITY (T > max_tokens), CUDA. */
int cmoe_ffn_forward(cmoe_layer* layer, const void* x, int32_t T, void* out, void* stream);

/* The same forward for buffers in HOST memory (Eq. moe_output is per token, so a batch may be
 * cut anywhere): the T tokens are processed in chunks; chunk c+1 is copied to the device and
 * chunk c-1 back to the host on two internal copy streams while chunk c runs on `stream`
 * through the kernels of cmoe_ffn_forward.  Each token's result is what cmoe_ffn_forward
 * gives for it in a batch of the chunk's size.
 *   x_host, out_host : host, [T, d_model] row-major; page-locked memory is needed for the
 *                      copies to overlap (pageable memory works, serially).  The buffers
 *                      belong to the caller and must stay valid until `stream` has passed
 *                      this call; out_host is complete when work enqueued on `stream` after
 *                      the call runs (or after synchronising `stream`).
 *   chunk_tokens     : tokens per chunk, clamped to [1, max_tokens]; <= 0 picks a sixteenth
 *                      of the batch rounded up to 128 rows, at least 512 (the first copy in and
 *                      the last copy out are not overlapped, so more chunks hide more of them).
 * The first call (and any later call with a larger chunk) allocates the staging: two device
 * buffers each for x and out of chunk_tokens rows, two streams and a few events, all freed by
 * cmoe_layer_destroy; other calls allocate nothing.  Routing read-back afterwards (cmoe_get_routing)
 * describes the LAST chunk only.  Errors: INVALID_ARG, CUDA. */
int cmoe_ffn_forward_host(cmoe_layer* layer, const void* x_host, int32_t T, void* out_host,
                          int32_t chunk_tokens, void* stream);

/* FP8 weight-only quantisation of the expert weights (the paper's Section 6, "Compatibility with
 * Other Efficiency Techniques", states that the restructured FFN composes with post-training
 * quantisation and names no format; this library's format is: OCP E4M3 codes — 1 sign, 4 exponent
 * bits with bias 7, 3 mantissa bits, subnormals, largest value 448 — with one power-of-two scale
 * per output channel, code = round-to-nearest-even(w / scale), scale = the smallest power of two
 * with max|w| / scale <= 448, 1 for an all-zero channel).
 *
 * cmoe_quantise_rows_fp8: the stand-alone operation on a matrix.
 *   w           : device, bf16 [rows, cols] row-major; a row is an output channel.
 *   codes       : device, uint8 [rows, cols], receives the E4M3 codes.
 *   scale       : device, float [rows], receives the power-of-two scales.
 *   dequantised : device, bf16 [rows, cols] or NULL; receives code * scale (exact in bf16); may be w itself.
 * Asynchronous on `stream`, allocates nothing.  Errors: INVALID_ARG, CUDA. */
int cmoe_quantise_rows_fp8(const void* w, int32_t rows, int32_t cols, uint8_t* codes, float* scale,
                           void* dequantised, void* stream);

/* cmoe_layer_quantise_fp8: quantise a bf16 layer's expert weights in that format.  Output channels:
 * a neuron's row of W_gate and of W_up; a model dimension's row of each expert's block of W_down
 * (the N_s shared experts form one block), so W_down has one scale per (expert, model dimension).
 * The router's representative rows keep their original values, so the routing does not change.
 * Afterwards every forward of the layer computes with the dequantised weights code * scale:
 * batches of at most 64 rows stream the FP8 codes (half the weight bytes of bf16) into FP8
 * tensor-core instructions, with every bf16 token row split into two E4M3 planes whose sum is
 * the bf16 value itself; larger batches read bf16 copies holding exactly the same weight values.
 * The layer then owns 1.5x the weight memory.  Plain and hierarchical layers; needs d_model, the
 * expert width and the shared width to be multiples of 16.  Allocates (a set-up call, like create)
 * and synchronises `stream`.  Idempotent.  Errors: INVALID_ARG, UNSUPPORTED (fp32 layer, shape), CUDA. */
int cmoe_layer_quantise_fp8(cmoe_layer* layer, void* stream);

/* Replace the learnable gate scaling u and the selection bias b (Section 4.3).
 * host arrays [n_routed_groups] (N_r, or n_outer*N_r for a hierarchical layer,
 * outer-major) or NULL for zeros.  Synchronises `stream`. */
int cmoe_layer_set_gate_params(cmoe_layer* layer, const float* gate_scale_u,
                               const float* select_bias_b, void* stream);

/* Read the current gate scaling u and selection bias b back (host arrays
 * [n_routed_groups]; either may be NULL).  Synchronises `stream`. */
int cmoe_layer_get_gate_params(cmoe_layer* layer, float* gate_scale_u, float* select_bias_b,
                               void* stream);

/* One step of the load-balancing rule (Section 4.3) on the device, from the token counts
 * of the LAST forward: with p_i the fraction of the routed assignments of an (outer)
 * layer that went to its expert i, b_i -= gamma if p_i > p*_i and b_i += gamma if
 * p_i < p*_i.  The paper's target is uniform, p* = 1/N_r, and gamma = 1e-3.
 *   target_share: host, [n_routed_groups] or NULL (uniform); fractions per (outer) layer.
 *   utilisation : host, [n_routed_groups] or NULL; receives p_i (the call then
 *                 synchronises `stream`; otherwise it is asynchronous unless a target is given).
 * Call it on the stream of the last forward (or after synchronising it).
 * Errors: INVALID_ARG (no routed experts, no forward yet, negative gamma), CUDA. */
int cmoe_layer_update_bias(cmoe_layer* layer, float gamma, const float* target_share,
                           float* utilisation, void* stream);

/* Activation profiling, steps 1-3 of the paper's pipeline (Section 4.1 "Activation Profiling";
 * Appendix "Complete Activation Analysis Pipeline", Eq. h_matrix_appendix, Eq. atopk_appendix,
 * Eq. mu_appendix): for n_tokens calibration rows x, H = Swish(x W_gate) * (x W_up), then per
 * token the k_a hidden activations of largest magnitude (equal magnitudes at the cut go to the
 * lower neuron index; NaN ranks last).  Neuron i of a selected pair (token, i) gets bit
 * (token0 + t) % 32 of word act_bits[i * words_per_neuron + (token0 + t) / 32] set (its
 * activation feature vector c_i, bit-packed) and act_count[i] incremented (q * mu_i).
 *   layer    : a plain layer created with n_shared == n_experts and top_k == 0, i.e. the dense
 *              FFN itself; neuron index i means position i of the neuron_perm it was created
 *              with (the identity gives original neuron numbers).  H is held in the layer's
 *              storage type (bf16 or fp32) and the selection is taken on those stored values.
 *   x        : device, [n_tokens, d_model] in the layer's dtype, 16-byte aligned; 0 <= n_tokens <= max_tokens.
 *   token0   : position of x's first row in the calibration set, so that a set larger than
 *              max_tokens is profiled in chunks.
 *   act_bits : device, uint32 [d_ff, words_per_neuron], words_per_neuron * 32 >= token0 + n_tokens.
 *   act_count: device, int32 [d_ff].
 * Both outputs accumulate: the caller zeroes them before the first chunk.  Asynchronous on
 * `stream`; the buffers belong to the caller.  Errors: INVALID_ARG (layer has routed experts or
 * is hierarchical, k_a outside [1, d_ff], null or misaligned pointers), CAPACITY, UNSUPPORTED
 * (d_ff above 20352 for bf16 or 10176 for fp32: a row's keys and the candidate arrays share 48 KB
 * of shared memory), CUDA. */
int cmoe_profile_activations(cmoe_layer* layer, const void* x, int32_t n_tokens, int32_t k_a, int32_t token0,
                             uint32_t* act_bits, int32_t words_per_neuron, int32_t* act_count, void* stream);

/* Step 4 (Eq. S_Ns_appendix): the n_select = N_s * m neurons with the highest activation
 * count, written to shared_idx[0 .. n_select) from the highest count down; equal counts go
 * to the lower neuron index.  act_count: device int32 [d_ff]; shared_idx: device int32
 * [n_select].  No layer and no scratch memory are involved.  Asynchronous on `stream`.
 * Errors: INVALID_ARG (n_select outside [0, d_ff], null pointers), CUDA. */
int cmoe_select_shared(const int32_t* act_count, int32_t d_ff, int32_t n_select, int32_t* shared_idx,
                       void* stream);

/* Data-parallel pieces of the balanced K-means that partitions the non-shared neurons into
 * routed experts (Appendix "Balanced Clustering Algorithm for Routed Experts") and of the
 * representative-neuron choice (Eq. rep_neuron).  They work on the bit rows act_bits written
 * by cmoe_profile_activations (row i = activation feature vector c_i over n_tokens calibration
 * tokens) for the n neurons listed in neuron_idx (device int32 [n], rows of act_bits).  A
 * centroid, being the mean of binary vectors, is held exactly: centroid_count[j][k] = number
 * of cluster j's members active for token k (device int32 [n_clusters, n_tokens]) and
 * cluster_size[j] = its member count (device int32 [n_clusters]); chat_j = count_j / size_j.
 * The balanced assignment itself (a sequential O(n^3) solver in the paper) is not provided.
 * Limits: n_clusters <= 32, n_tokens * n < 2^31.  All three calls are asynchronous on `stream`,
 * allocate nothing, and leave their buffers to the caller.  Errors: INVALID_ARG, CAPACITY, CUDA.
 *
 * cmoe_cluster_update (the cluster-update rule): assign[i] in [0, n_clusters) is neuron
 *   neuron_idx[i]'s cluster, any other value means unassigned.  Every cluster with at least one
 *   member gets its count vector and size rebuilt; a cluster without members keeps both, as
 *   the paper's rule keeps the old centroid.  (Initial centroids: n_clusters neurons, assign[i] = i.) */
int cmoe_cluster_update(const uint32_t* act_bits, int32_t words_per_neuron, int32_t n_tokens,
                        const int32_t* neuron_idx, const int32_t* assign, int32_t n, int32_t n_clusters,
                        int32_t* centroid_count, int32_t* cluster_size, void* stream);

/* cmoe_cluster_distances (the distance matrix D): scaled_sq_dist[i, j] (device int64
 *   [n, n_clusters]) = size_j^2 * || c_i - chat_j ||_2^2, an exact integer; d_ij =
 *   sqrt(scaled_sq_dist[i, j]) / size_j.  With binary centroids (size 1) it is the Hamming
 *   distance.  centroid_sqnorm: device int64 [n_clusters], written by the call (||count_j||^2).
 *   Every cluster_size[j] must be at least 1. */
int cmoe_cluster_distances(const uint32_t* act_bits, int32_t words_per_neuron, int32_t n_tokens,
                           const int32_t* neuron_idx, int32_t n, const int32_t* centroid_count,
                           const int32_t* cluster_size, int32_t n_clusters, int64_t* centroid_sqnorm,
                           int64_t* scaled_sq_dist, void* stream);

/* cmoe_cluster_representatives (Eq. rep_neuron): rep_neuron[j] (device int32 [n_clusters]) =
 *   neuron_idx[i] of the member i of cluster j with the smallest scaled_sq_dist[i, j]; equal
 *   distances go to the lower position i; -1 for a cluster without members. */
int cmoe_cluster_representatives(const int64_t* scaled_sq_dist, const int32_t* neuron_idx, const int32_t* assign,
                                 int32_t n, int32_t n_clusters, int32_t* rep_neuron, void* stream);

/* Choose the expert-GEMM implementation: 0 = automatic (tensor-core path when the
 * dtype is bf16 and the shape allows, else the plain SIMT path; for batches of at least 256
 * rows each of the two GEMMs may run on CTA pairs: below 1024 rows when the experts are at least
 * 1024 neurons wide (a pair fetches a third less operand data per SM), from 1024 rows when the
 * padding of the expert groups to 256-row tiles is expected to stay small; batches of 65 to 128 rows stream the bf16 weights through the
 * decode-shaped kernels, weights on the MMA's M side; a single row of a plain layer
 * runs on the CUDA cores with plain-load weight streams, down projection and combine in one
 * launch), 1 = always SIMT, 2 = tensor-core with
 * single-CTA token-major tiles only (decode-shaped kernels up to 64 rows), 3 = tensor-core on CTA
 * pairs (cta_group::2) for batches of at least 256 rows;
 * 2 and 3 return CMOE_ERR_INVALID_ARG if the layer cannot take the tensor-core path. */
int cmoe_layer_set_gemm_path(cmoe_layer* layer, int32_t path);

/* Launch chaining (on by default): on the bf16 tensor-core path every kernel of a forward
 * after the expert router is launched as a programmatic dependent of its predecessor, so it
 * may become resident (and fetch what does not depend on the predecessor) while the
 * predecessor drains, and waits on the device before touching anything the predecessor
 * produces.  Results are bit-identical either way; 0 restores ordinary stream-ordered
 * launches.  Has no effect on fp32 layers or while per-stage timing is enabled, and the
 * prologue of a hierarchical layer (top-level router, its permutation, the row copy) always
 * uses ordinary launches.  Error: INVALID_ARG (null layer). */
int cmoe_layer_set_launch_chaining(cmoe_layer* layer, int32_t on);

/* Sizes a caller needs to read the routing state back.  n_outer / outer_top_k
 * are 0 for a plain layer. */
int cmoe_layer_dims(const cmoe_layer* layer, int32_t* n_routed_groups, int32_t* top_k,
                    int32_t* n_outer, int32_t* outer_top_k);

/* Copy the routing state of the LAST forward (T tokens) to host buffers; any
 * pointer may be NULL.  Synchronises the stream of that forward.  R = T for a
 * plain layer, T*outer_top_k for a hierarchical one (outer rows); G = routed groups.
 *   keys      [R, N_r] fp32  s'_i + b_i of every routed expert of the row's (outer) layer
 *   scores    [R, N_r] fp32  s_i (Eq. router)
 *   topk_idx  [R, N_k] int32 selected routed GROUP (outer*N_r + j), descending key
 *   topk_gate [R, N_k] fp32  g_i = 1 + s'_i u_i
 *   counts    [G] , offsets [G+1] int32  rows per routed group and their exclusive scan
 *   row_token [R*N_k] int32  row r of the expert-contiguous order holds outer row row_token[r]
 *                            (= token for a plain layer); ascending inside a group
 *   row_of    [R, N_k] int32 inverse map: row of pair (r, j)
 *   outer_idx [T, outer_top_k] int32, outer_w [T, outer_top_k] fp32, outer_row_token [R] int32
 *                            hierarchical layers only. */
int cmoe_get_routing(cmoe_layer* layer, float* keys, float* scores, int32_t* topk_idx,
                     float* topk_gate, int32_t* counts, int32_t* offsets, int32_t* row_token,
                     int32_t* row_of, int32_t* outer_idx, float* outer_w,
                     int32_t* outer_row_token);

/* Device-side error word of the last forward: 0, or a code written by a kernel whose
 * bounded wait (mbarrier) ran out.  Synchronises the last stream.  Returns
 * CMOE_ERR_DEVICE_TIMEOUT when the word is non-zero; the output of the forward that timed out
 * is undefined.  Recovery is part of this call: after reporting a timeout it clears the error
 * word and the K-slice tickets a part-finished kernel may have left taken, so the layer can be
 * used again (the next status call reports CMOE_OK unless another wait runs out). */
int cmoe_layer_status(cmoe_layer* layer, int32_t* device_error_word);

/* Self-test of the give-up path (no paper counterpart: failure detection of this library).
 * Enqueues one warp that waits on a barrier nobody arrives on through the same bounded wait the
 * tensor-core kernels use, with a limit of limit_cycles SM clock cycles (1e3 .. 2e9; 2e6 is
 * about a millisecond).  The wait gives up, writes its code to the layer's error word and the
 * kernel returns normally: nothing traps, no copy is in flight, the context stays usable.
 * cmoe_layer_status then returns CMOE_ERR_DEVICE_TIMEOUT once.  Asynchronous on `stream`. */
int cmoe_layer_selftest_wait_timeout(cmoe_layer* layer, int64_t limit_cycles, void* stream);

/* Number of this library's kernels the last forward launched. */
int cmoe_layer_launch_count(const cmoe_layer* layer, int32_t* n_launches);

/* Per-stage device timing with CUDA events on the forward's stream.  ring_steps > 0
 * creates a ring of events covering that many forwards (0 switches timing off);
 * while on, every forward records CMOE_N_STAGES+1 events and allocates nothing.
 * Stages: 0 routing (top-level router and its permutation for hierarchical layers,
 * analytical router + gates), 1 histogram/scan/permute + row gather, 2 gate/up GEMM
 * with the SwiGLU epilogue, 3 down GEMM, 4 combine.
 * cmoe_layer_stage_times synchronises the last stream and returns, per stage, the
 * summed milliseconds over the last n_steps forwards held in the ring. */
#define CMOE_N_STAGES 5
int cmoe_layer_enable_stage_timing(cmoe_layer* layer, int32_t ring_steps);
int cmoe_layer_stage_times(cmoe_layer* layer, float* ms_sum /*[CMOE_N_STAGES]*/, int32_t* n_steps);

int cmoe_layer_destroy(cmoe_layer* layer);

/* Stand-alone token histogram / exclusive scan / stable permutation: the
 * expert-contiguous order of the selected (token, expert) pairs — the paper only
 * states that the top-N_k routed experts of a token are activated (Eq. moe_output);
 * the canonical listing is "sorted by (expert, token)".
 *   topk_idx : device int32 [n_rows, n_k], entries in [0, n_groups); a row never
 *              names the same group twice (entries out of range are ignored).
 *   counts [n_groups], offsets [n_groups+1], row_token [n_rows*n_k], row_of [n_rows, n_k]:
 *              device int32 outputs, as in cmoe_get_routing.
 *   scratch  : device, at least cmoe_token_permute_scratch_bytes(n_rows, n_groups) bytes,
 *              256-byte aligned; contents need not be initialised; may be NULL when
 *              n_rows <= 256.
 * Asynchronous on `stream`; allocates nothing.  n_groups <= 1024, n_k <= 8. */
int64_t cmoe_token_permute_scratch_bytes(int32_t n_rows, int32_t n_groups);
int cmoe_token_permute(const int32_t* topk_idx, int32_t n_rows, int32_t n_k, int32_t n_groups,
                       int32_t* counts, int32_t* offsets, int32_t* row_token, int32_t* row_of,
                       void* scratch, int64_t scratch_bytes, void* stream);

/* cmoe_token_permute for callers that cannot allocate device memory.  (The paper has
 * no counterpart; this is a packaging variant of the call above.)
 *
 * Who needs it: code that runs where cudaMalloc is unavailable or forbidden — inside a
 * serving loop whose memory pool is frozen after start-up, in a plug-in that was handed
 * only its input and output buffers, or in a process that must not touch the allocator
 * because another component owns all of the device's free memory.  Such a caller cannot
 * provide the `scratch` buffer of cmoe_token_permute, so this variant keeps the
 * chunk-count matrix in a fixed 1 MiB array that is part of the library image: every GPU
 * that loads the library holds that 1 MiB from load until the process exits.
 *
 * Same inputs, outputs and result as cmoe_token_permute.  Differences:
 *   - limit: ceil(n_rows / 256) * n_groups <= CMOE_STATIC_PERMUTE_MAX_CELLS when
 *     n_rows > 256 (e.g. 65,536 rows with 1024 groups, or 4 M rows with 16 groups);
 *     larger problems are refused with CMOE_ERR_CAPACITY and nothing is launched.
 *   - it calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - the first call on each device looks up the array's device address (a one-off,
 *     host-side query made with that device current); make that first call outside any
 *     stream capture.
 *   - all calls on one device share the array.  Its contents carry over from call to
 *     call, which is harmless (each call overwrites every cell before reading it), but two
 *     calls that overlap in time on the GPU — different streams, or the same call from
 *     two threads — race on it and return garbage: serialise them. */
#define CMOE_STATIC_PERMUTE_MAX_CELLS 262144
int cmoe_token_permute_static(const int32_t* topk_idx, int32_t n_rows, int32_t n_k,
                              int32_t n_groups, int32_t* counts, int32_t* offsets,
                              int32_t* row_token, int32_t* row_of, void* stream);

const char* cmoe_status_string(int status);
/* Text of the most recent error seen by this library on the calling thread. */
const char* cmoe_last_error(void);

#ifdef __cplusplus
}
#endif
#endif  /* CMOE_H_ */
