/*
 * moev.h -- C ABI of the B200 (sm_100a) MoE verification layer.
 *
 * One call, moev_verify(), runs the MoE expert layer of the target model's
 * verification pass over the gamma tokens of a speculative draft tree:
 *
 *   router top-k per token  ->  expert union + token->expert grouping
 *   ->  grouped gated-SwiGLU expert FFN over the union, each active expert's
 *       weights read from HBM once  ->  routing-weighted combine,
 *
 * and reports the per-layer active-expert count.
 *
 * Paper passages the operations follow:
 *   - Sec. 1: top-k routing -- the router scores the E experts for every token and the
 *     token is processed by its k best-scoring experts only.
 *   - Eq. 1 (Sec. 3): the verification footprint is the union over the gamma
 *     verified tokens of their expert sets; its size -- not gamma -- drives the
 *     cost, because the verifier fetches every expert of the union from HBM and
 *     reuses it for all tokens routed to it.
 *   - Table 1 / Table 3 metric "average active experts": the size of that union
 *     per MoE layer per verification step (n_active here; shared experts are not
 *     counted, as the autoregressive rows of Table 1 show).
 *   - Table 13: experts per layer, top-k and the always-on shared expert.
 *   - Fig. 1(c): bytes of one expert (moev_expert_bytes).
 * The paper does not print the expert FFN; it is the bias-free gated SwiGLU
 *   FFN_e(x) = W_down,e ( silu(W_gate,e x) * (W_up,e x) ),  silu(z) = z/(1+exp(-z)),
 *   y_t = sum_j w[t,j] FFN_{ids[t,j]}(x_t) + sum_s FFN_shared,s(x_t).
 *
 * Conventions
 *   - No exceptions, aborts or traps cross this boundary: every entry point
 *     returns a moev_status; moev_last_error() gives the text of the last failure.
 *   - Unless a parameter says HOST, pointers are DEVICE pointers, borrowed for the
 *     duration of the call; the library never frees or retains caller memory.
 *   - moev_verify() is asynchronous on the given CUDA stream, allocates nothing
 *     and never synchronises; outputs are valid once the stream reaches that point.
 *   - One context per host thread / stream (calls on one context must not overlap).
 */
#ifndef MOEV_H_
#define MOEV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moev_ctx moev_ctx; /* opaque; owns the device workspace */

typedef enum {
  MOEV_OK = 0,
  MOEV_EINVAL = 1,       /* bad argument (null, out of range, misaligned, shape granularity) */
  MOEV_EUNSUPPORTED = 2, /* device is not sm_100 */
  MOEV_ECUDA = 3,        /* a CUDA runtime/driver call failed; see moev_last_error */
  MOEV_ENOMEM = 4,       /* workspace allocation failed in moev_create */
  MOEV_ETIMEOUT = 5      /* a bounded device-side wait expired (reported by moev_status_sync) */
} moev_status;

/* Expert-weight storage formats (K = contraction dimension, always contiguous). */
typedef enum {
  MOEV_W_FP32 = 0,         /* float32 */
  MOEV_W_BF16 = 1,         /* bfloat16 */
  MOEV_W_FP8E4M3_B128 = 2, /* e4m3fn codes + float32 scale per 128x128 block: W = code * s */
  MOEV_W_MXFP4 = 3         /* e2m1 codes, two per byte (even k in the low nibble) + e8m0
                              scale per 32 along K: W = code * 2^(s-127) */
} moev_wfmt;

typedef enum { MOEV_ACT_FP32 = 0, MOEV_ACT_BF16 = 1 } moev_afmt;

/* Router weights over the k selected experts (selection itself is always on raw logits,
 * descending, exact ties to the lower expert id):
 *   SOFTMAX: w_j = exp(l_j - l_max) / sum_{j<k} exp(l_j - l_max)
 *   SIGMOID: s_j = 1/(1+exp(-l_j)),  w_j = routed_scale * s_j / (sum_j s_j + 1e-20)      */
typedef enum { MOEV_SCORE_SOFTMAX = 0, MOEV_SCORE_SIGMOID = 1 } moev_score;

/* Which expert-FFN kernels moev_verify uses. */
typedef enum {
  MOEV_IMPL_AUTO = 0,   /* tensor-core (TMA + tcgen05) path when the shape allows, else SIMT */
  MOEV_IMPL_SIMT = 1,   /* CUDA-core kernels (all formats, all shapes) */
  MOEV_IMPL_TCGEN05 = 2 /* tensor-core path; MOEV_EINVAL if the shape does not allow it */
} moev_impl;

/* Expert form.  The paper does not print the FFN; the benchmark configurations use the bias-free
 * gated SwiGLU  down(silu(gate x) * (up x)).  MOEV_FFN_GPTOSS is the published GPT-OSS expert:
 *   g = min(gate x + b_gate, 7),  u = clamp(up x + b_up, -7, 7),
 *   h = g * sigmoid(1.702 g) * (u + 1),  out = down h + b_down   (weighted by the router weight). */
typedef enum { MOEV_FFN_SWIGLU = 0, MOEV_FFN_GPTOSS = 1 } moev_ffn_kind;

/* Group-limited routing (n_group > 0), the rule of the published DeepSeek-V3 models; the paper's
 * routing is the plain top-k.  s_e = sigmoid(logit_e), c_e = s_e + router_bias_e; the E experts
 * form n_group contiguous groups; a group's score is the sum of its two largest c; the topk_group
 * best groups are kept (ties: lower index); among their experts the top_k by c (ties: lower id) are
 * selected and emitted in that order; weights use the unbiased scores:
 * w_j = routed_scale * s_j / (sum_j s_j + 1e-20). */

/* FP8 activations in front of both expert GEMMs (what deployed DeepSeek-V3 inference does; the
 * paper does not print the expert FFN).  The input x of the gate / up projections and the input h
 * of the down projection are quantised on the fly per token and per block of 128 consecutive
 * elements of the contraction axis: amax = max |v| over the block, s = amax / 448 (binary32; with
 * POW2 the smallest power of two that is not below it; 1 for an all-zero block), code = e4m3(v / s)
 * rounded to nearest even, and the GEMM sees decode(code) * s.  The router sees the unquantised x.
 * Tensor-core kernels: MOEV_W_FP8E4M3_B128 with H <= 8192 and I <= 4096; other configurations run
 * on the CUDA-core kernels. */
typedef enum { MOEV_ACTQ_NONE = 0, MOEV_ACTQ_FP8_B128 = 1, MOEV_ACTQ_FP8_B128_POW2 = 2 } moev_act_quant;

typedef struct {
  int32_t H;          /* hidden size; multiple of 32 */
  int32_t I;          /* expert intermediate size; multiple of 32 */
  int32_t E;          /* routed experts, 1..512 */
  int32_t top_k;      /* 1..min(E,32) */
  int32_t n_shared;   /* always-on shared experts (weight 1), >= 0 */
  int32_t max_tokens; /* largest gamma this context will be asked to verify, 1..1024 */
  int32_t wfmt;       /* moev_wfmt */
  int32_t afmt;       /* moev_afmt: type of x and y */
  int32_t score;      /* moev_score */
  int32_t impl;       /* moev_impl */
  float routed_scale; /* c in the SIGMOID rule; ignored for SOFTMAX */
  int32_t ffn_kind;   /* moev_ffn_kind; MOEV_FFN_GPTOSS needs n_shared == 0 */
  int32_t n_group;    /* 0 = plain top-k; > 0: group-limited routing (below), needs MOEV_SCORE_SIGMOID, E % n_group == 0 */
  int32_t topk_group; /* groups kept per token, 1..n_group; top_k <= topk_group * E / n_group */
  int32_t act_quant;  /* moev_act_quant */
} moev_config;

/* One layer's parameters.  Layouts, row-major, last index contiguous:
 *   router_w            [E, H]  float32
 *   w_gate, w_up        [E, I, H]   in wfmt     (K = H)
 *   w_down              [E, H, I]   in wfmt     (K = I)
 *   s_*   FP8 : float32 [E, ceil(N/128), ceil(K/128)]   (N = rows of the matrix)
 *         MXFP4: uint8  [E, N, K/32]                     else NULL
 *   sh_*  the same for the n_shared shared experts (leading dim n_shared), NULL if none.
 * Every pointer must be 16-byte aligned; on the tensor-core path (moev_resolved_impl ==
 * MOEV_IMPL_TCGEN05) the six expert weight tensors w_* and sh_* must be 32-byte aligned (they
 * are read through TMA descriptors).  A misaligned pointer is rejected with MOEV_EINVAL. */
typedef struct {
  const float* router_w;
  const void *w_gate, *w_up, *w_down;
  const void *s_gate, *s_up, *s_down;
  const void *sh_gate, *sh_up, *sh_down;
  const void *sh_s_gate, *sh_s_up, *sh_s_down;
  const float *b_gate, *b_up, *b_down; /* MOEV_FFN_GPTOSS: fp32 biases [E,I], [E,I], [E,H]; NULL = zero */
  const float* router_bias;            /* n_group > 0: fp32 score-correction bias [E]; NULL = zero */
  /* Optional prefetch hint (Sec. 4.1, Eq. 4: the predictor's expert set for this layer): DEVICE list of
   * n_predicted expert ids whose weights the first routing kernel pulls into the L2 while the router
   * runs, next to the shared experts' (only when moev_prefetch_enable switched the prefetch on).  A wrong prediction costs only
   * bandwidth; results never depend on the hint.  At most what fits an 80 MB share of the L2 is taken
   * (the first entries of the list).  NULL / 0 = no hint. */
  const int32_t* predicted_ids;
  int32_t n_predicted;
} moev_layer;

/* Outputs.  y and n_active are required; the others are diagnostics and may be NULL.
 *   y          [gamma, H] in afmt
 *   topk_ids   [gamma, k] int32   expert ids in descending-logit order
 *   topk_w     [gamma, k] float32 router weights
 *   union_ids  [E]        int32   first U entries: active experts, ascending (Eq. 1)
 *   offsets    [E+1]      int32   first U+1 entries: exclusive scan of tokens per active expert
 *   perm       [gamma*k]  int32   assignments a = t*k+j stably sorted by expert id
 *   n_active   [1]        int32   U = size of the union (shared experts not counted)       */
typedef struct {
  void* y;
  int32_t* topk_ids;
  float* topk_w;
  int32_t* union_ids;
  int32_t* offsets;
  int32_t* perm;
  int32_t* n_active;
} moev_out;

/* Create a context for one layer shape on the current CUDA device; allocates the device
 * workspace (router logits, grouping tables, fp32 intermediates).  MOEV_EINVAL on a bad
 * config, MOEV_EUNSUPPORTED when the device is not compute capability 10.x, MOEV_ENOMEM /
 * MOEV_ECUDA on allocation failure.  *out is NULL on failure. */
moev_status moev_create(const moev_config* cfg, moev_ctx** out);

/* Free the workspace.  The caller must have synchronised the streams it used. */
moev_status moev_destroy(moev_ctx* ctx);

/* Verify gamma tokens (1 <= gamma <= max_tokens): x [gamma, H] in afmt (device).
 * Enqueues the whole path on cuda_stream (a cudaStream_t, may be NULL for the default
 * stream) and returns without waiting.  Invalid arguments are rejected with MOEV_EINVAL
 * before anything is launched. */
moev_status moev_verify(moev_ctx* ctx, const moev_layer* layer, const void* x, int32_t gamma,
                        const moev_out* out, void* cuda_stream);

/* The same path for callers whose activations live in HOST memory: x_host [gamma, H]
 * (pinned memory recommended) is copied to the device, the layer runs, and y_host
 * [gamma, H] plus *n_active_host are copied back, all on cuda_stream; the call waits for
 * the stream before returning so the host buffers are valid.  Weights stay on the device. */
moev_status moev_verify_host(moev_ctx* ctx, const moev_layer* layer, const void* x_host,
                             int32_t gamma, void* y_host, int32_t* n_active_host,
                             void* cuda_stream);

/* Wait for cuda_stream and read the device status word: MOEV_OK, or MOEV_ETIMEOUT if a
 * bounded device-side wait gave up (the outputs of that call are then undefined). */
moev_status moev_status_sync(moev_ctx* ctx, void* cuda_stream);

/* Text of the last error on this context ("" if none).  Owned by the context. */
const char* moev_last_error(const moev_ctx* ctx);

/* Bytes of one expert's three matrices including scale factors (Fig. 1(c): the FP8
 * DeepSeek-V3.1 expert is 3*7168*2048 = 44 040 192 code bytes, + 10 752 scale bytes). */
size_t moev_expert_bytes(const moev_config* cfg);

/* Code bytes only (the paper's 44.04 MB figure). */
size_t moev_expert_code_bytes(const moev_config* cfg);

/* Number of kernels one moev_verify call launches on this context (for launch accounting; calls
 * of at most 32 tokens with plain top-k routing take two routing launches, others three -- a
 * context whose max_tokens exceeds 32 reports the larger figure), and which FFN implementation
 * it resolved to (a moev_impl value, never AUTO). */
int32_t moev_launches_per_call(const moev_ctx* ctx);
int32_t moev_resolved_impl(const moev_ctx* ctx);

/* Per-kernel device time of a call, measured with CUDA events recorded on the call's
 * stream between its kernels.  moev_profile_enable(ctx, 1) turns the event records on (at
 * most 512 calls are kept between reads), 0 off.  moev_profile_read waits for the stream and
 * writes mean_us[0..5], the mean duration in microseconds of: router partial logits, top-k
 * with exact refinement, grouping (union / permutation), first FFN kernel (the fused
 * tensor-core kernel, or SIMT gate/up), second FFN kernel (SIMT down; 0 on the fused path),
 * finalize; then the number of calls averaged, and resets the accumulator. */
moev_status moev_profile_enable(moev_ctx* ctx, int32_t on);
moev_status moev_profile_read(moev_ctx* ctx, void* cuda_stream, double* mean_us /*[6]*/,
                              int32_t* calls);

/* Working time of the tensor-core expert kernel inside a call as the call really runs (the event
 * records above switch the dependent launches off, so their interval for a kernel includes its
 * launch gap and its set-up, which a real call hides behind the routing kernels).  With
 * moev_ffn_span_enable(ctx, 1) every CTA of the expert kernel stores the device's global timer when
 * the routing kernels release it and when it leaves (two 8-byte stores per CTA and call; nothing
 * else changes).  moev_ffn_span_read waits for the stream and writes to span_us (host) the time in
 * microseconds from the earliest release to the latest exit in the most recent call, or 0 when no
 * tensor-core expert kernel has run with the stamps on (the CUDA-core path does not stamp).  The
 * paper has no counterpart: a measurement aid for its Fig. 1(a) quantity, latency against the
 * number of active experts. */
moev_status moev_ffn_span_enable(moev_ctx* ctx, int32_t on);
moev_status moev_ffn_span_read(moev_ctx* ctx, void* cuda_stream, double* span_us);

/* Weight prefetch by the first routing kernel (off by default): the shared experts' matrices and
 * those of the layer's predicted_ids are pulled into the L2 while the routing kernels run, so the
 * expert kernel finds them on chip (Sec. 3: the verification cost is expert-weight traffic from
 * HBM; what is known to be needed before the router decides need not wait for it).  Measured on
 * B200 it does not pay: the L2 delivers these bytes only slightly faster than HBM does, and the
 * prefetch traffic delays the latency-bound routing kernels by more than the expert kernel gains. */
moev_status moev_prefetch_enable(moev_ctx* ctx, int32_t on);

/* Several independent layers in one call (multi-layer pipelining; the paper has no counterpart:
 * its prototype runs layer by layer).  Equivalent to n_layers calls of moev_verify on the same
 * stream with layers[l], x[l], outs[l] and the same gamma, except that the first kernel of layer
 * l + 1 is enqueued as a programmatic dependent launch: its CTAs occupy the SMs that layer l's
 * expert kernel has already left, so the router of the next layer overlaps the tail of the
 * previous one.  The inputs x[l] must not depend on the outputs of earlier layers of the same
 * call (independent requests, or hidden states that are already available); results are the same
 * as those of separate calls.  layers / x / outs are HOST arrays of n_layers entries whose
 * pointers are DEVICE pointers.  Errors as moev_verify; nothing is enqueued for layers after the
 * first failing one. */
moev_status moev_verify_pipeline(moev_ctx* ctx, int32_t n_layers, const moev_layer* layers,
                                 const void* const* x, int32_t gamma, const moev_out* outs,
                                 void* cuda_stream);

/* Consecutive dependent layers in one call: layer l + 1 verifies the output of layer l (Sec. 5 /
 * Table 13: a verification pass runs the model's 36 - 94 MoE layers one after another; the
 * attention between them is outside this library and is the identity here).  x0 [gamma, H] is the
 * input of layers[0]; outs[l].y [gamma, H] (afmt, required for every layer) is both the result of
 * layer l and the input of layer l + 1.  Same results as n_layers calls of moev_verify with those
 * inputs; every kernel of the call is a programmatic dependent launch of its predecessor, the
 * first kernel of a layer included: it is scheduled while the previous layer drains, starts the
 * optional weight prefetch at once, and waits for the previous layer's output before it reads it.
 * layers / outs are HOST arrays whose pointers are DEVICE pointers.  Errors as moev_verify. */
moev_status moev_verify_chain(moev_ctx* ctx, int32_t n_layers, const moev_layer* layers, const void* x0,
                              int32_t gamma, const moev_out* outs, void* cuda_stream);

/* Cost-aware draft selection: Algorithm 1 of the paper (Sec. 4.2, Eqs. 7-10), the step that
 * runs between drafting and verification and decides which gamma draft-tree nodes are verified.
 *   n, parent [n]   draft tree in topological order: parent[i] < i, parent[root] = -1
 *   P [n]           cumulative draft probability of every node (float32)
 *   pred [n, W]     predicted expert set of every node as a bitmap over (layer, expert) pairs,
 *                   bit l*E + e, W = ceil(L*E / 32) 32-bit words (Eq. 4)
 *   buffer0 [W]     initial expert buffer B_0, or NULL for the empty set
 *   E_traj(i) = OR of pred along root -> i (Eq. 7);  cost = |E_traj(i) \ B| (Eq. 8);
 *   score = P(i) / (cost + eps) (Eq. 9), evaluated in binary32;  gamma rounds of arg-max
 *   (exact ties: the lowest index, so a parent precedes its children), each followed by
 *   B |= E_traj(chosen).  global_cost != 0 selects the ablation variant of Eq. 10: cost =
 *   |E_traj(i)|, buffer not updated.
 * Outputs: selected [gamma] (first min(gamma, n) entries, in selection order), costs [gamma]
 * (cost of each choice when it was made; may be NULL), buffer_out [W] (final B; may be NULL),
 * n_selected [1] (may be NULL; -1 if a bounded device wait expired).  traj_workspace is
 * caller-provided scratch of n * W + 516 32-bit words (the path footprints, then control words);
 * it must be 16-byte aligned (the control words are accessed as 64-bit and 128-bit quantities),
 * otherwise MOEV_EINVAL.
 * All pointers are DEVICE pointers; one kernel (for bitmaps too long for one CTA's shared memory:
 * one memset and one cooperative kernel over several CTAs) is enqueued on cuda_stream; nothing is
 * allocated.
 * MOEV_EINVAL for n outside 1..4096, W < 1, gamma < 1, eps <= 0, null required pointers, or
 * tables too large for shared memory (3 n + 4 W words above ~50 000). */
moev_status moev_select_drafts(int32_t n, int32_t W, const int32_t* parent, const float* P,
                               const uint32_t* pred, const uint32_t* buffer0, int32_t gamma, float eps,
                               int32_t global_cost, uint32_t* traj_workspace, int32_t* selected,
                               int32_t* costs, uint32_t* buffer_out, int32_t* n_selected,
                               void* cuda_stream);

/* Router top-k without any allocation.  (The paper has no counterpart: this entry point
 * exists for the integration constraints of some callers, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is forbidden or unavailable -- inside a
 * memory-pool-managed serving process that has handed all device memory to its own allocator,
 * in a latency-critical thread that may not take the allocator's lock, or before a framework
 * has set up its caching allocator.  Such callers cannot create a moev_ctx (moev_create
 * allocates the workspace), but may still want the routing decision of a layer.
 *
 * Computes, for the gamma tokens x [gamma, H] (afmt of cfg), the same topk_ids [gamma, k] and
 * topk_w [gamma, k] that moev_verify writes for plain top-k routing.  Of cfg it reads H, E,
 * top_k, afmt, score, routed_scale and max_tokens (gamma <= max_tokens); the other fields must
 * merely be valid.  Group-limited routing needs the layer's score-correction bias, which this
 * entry point does not take: cfg->n_group > 0 is rejected with MOEV_EINVAL.  All pointers are
 * DEVICE pointers owned by the caller.  The split-K partial logits live in a fixed 20 MiB array compiled into the
 * library (held by every GPU that loads it until the process exits) instead of a context
 * workspace; moev_route_topk_static_scratch_floats() returns how many of its 5 242 880 floats a
 * problem needs, and problems that need more are rejected with MOEV_EINVAL.  The call itself
 * calls no cudaMalloc/cudaFree and no allocating library routine; it enqueues two kernels on
 * cuda_stream and returns without waiting.
 *
 * The first call on a device looks up the device address of the array (once per device, with
 * that device current); make that first call before starting any stream capture.  All calls
 * share the one array: nothing in it has to be cleared between calls (each call overwrites
 * what it reads), but two calls whose kernels overlap on the GPU (different streams, or
 * several host threads) race on it and give undefined results -- serialise them. */
moev_status moev_route_topk_static(const moev_config* cfg, const float* router_w, const void* x,
                                   int32_t gamma, int32_t* topk_ids, float* topk_w,
                                   void* cuda_stream);
size_t moev_route_topk_static_scratch_floats(int32_t H, int32_t E, int32_t gamma);

#ifdef __cplusplus
}
#endif
#endif /* MOEV_H_ */
