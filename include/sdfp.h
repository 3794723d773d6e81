/*
 * sdfp.h — C ABI of the SDFP speculative-decode library for NVIDIA B200 (sm_100a).
 *
 * The library runs the online stage of SDFP (Algorithm 1, Stage B, "Speculative
 * Decoding with Pruned Draft Model"; Section II-A for the accept/reject rule):
 * a Llama-style decoder drafts k tokens with a subset of its own layers, the
 * full stack verifies k+1 positions in one pass, the longest accepted prefix
 * plus one corrected/bonus token is committed, and both KV caches roll back.
 *
 * Conventions
 *   - Every function returns 0 on success or a negative sdfp_status; nothing is
 *     thrown, nothing aborts.  sdfp_last_error() gives the text of the last
 *     failure on that context (or of the last failed sdfp_create when ctx is NULL).
 *   - "device" pointers are CUDA global-memory addresses valid on the device
 *     that is current when sdfp_create is called; "host" pointers are ordinary
 *     host memory.  The library never frees or writes caller-owned memory
 *     except the documented outputs.
 *   - All work is issued on the CUDA stream given to sdfp_create (borrowed, the
 *     caller keeps ownership; NULL = the legacy default stream).
 *   - Deterministic: same config, weights, mask, prompts, k, temperature and
 *     seed give bit-identical outputs, and a sequence's tokens do not depend on
 *     what else is in the batch nor on how many rows a pass carries.  (A context
 *     takes one arithmetic path for all its passes: bf16 contexts whose widest
 *     pass, max_batch*max(k_max+1, 2) rows, fits 16 rows run every pass in the
 *     persistent whole-pass kernel, all others run one kernel per operation.)
 *   - A context belongs to the device that was current at sdfp_create; calls made
 *     with another device current fail with SDFP_ESTATE before touching the GPU.
 *   - Kernels that wait on one another (the whole-pass kernel's grid barriers and
 *     hand-offs) bound every wait; a wait that runs out ends the call with
 *     SDFP_ETIMEOUT, the outputs of that call are invalid, and the context can be
 *     used again.
 *   - There is no CPU fallback: without a usable CUDA device every entry point
 *     that computes fails with SDFP_ECUDA.
 */
#ifndef SDFP_H_
#define SDFP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sdfp_ctx sdfp_ctx; /* opaque, library-owned */

typedef enum {
  SDFP_OK = 0,
  SDFP_EINVAL = -1, /* bad argument or unsupported shape            */
  SDFP_ENOMEM = -2, /* device or host allocation failed             */
  SDFP_ECUDA = -3,  /* a CUDA call failed (text in sdfp_last_error) */
  SDFP_ESTATE = -4, /* call not valid in the context's state        */
  SDFP_ETIMEOUT = -5 /* a bounded wait inside a kernel ran out; the context stays usable */
} sdfp_status;

typedef enum { SDFP_F32 = 0, SDFP_BF16 = 1 } sdfp_dtype;

/* sdfp_config.flags */
#define SDFP_FLAG_NO_GRAPH 1u /* launch kernels directly instead of replaying CUDA graphs    */
#define SDFP_FLAG_NO_PDL 2u   /* no programmatic dependent launch between consecutive kernels */
#define SDFP_FLAG_FMA_GEMM 4u /* bf16 models: CUDA-core FMA GEMM instead of the tensor path  */
#define SDFP_FLAG_NO_PASS_KERNEL 8u /* bf16 models: one kernel per operation instead of the
                                       persistent whole-pass kernel                            */
#define SDFP_FLAG_NO_DENSE 16u      /* bf16 models: no tcgen05 path (the prompt goes through the
                                       decode kernels in chunks; contexts too wide for the
                                       whole-pass kernel run mma.sync kernels per operation)  */

/*
 * Model and capacity description.  The decoder is the LLaMA-2 architecture the
 * paper evaluates (Section IV-A): RMSNorm(eps inside the root), rotary
 * embeddings on pairs (i, i + head_dim/2) with base rope_theta, multi-head
 * causal attention (n_kv_heads == n_heads), SwiGLU FFN, untied lm-head, no bias.
 * Requirements: d_model == n_heads*head_dim; head_dim in {64, 128}; d_model,
 * d_ffn and vocab multiples of 16; max_batch <= 16, k_max <= 15 and
 * max_batch*max(k_max+1, 2) <= 80 rows per pass (8 sequences with k = 8: 72).
 */
typedef struct {
  int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_theta;
  int32_t max_seq;   /* KV-cache capacity per sequence, tokens              */
  int32_t max_batch; /* sequences per sdfp_generate call                    */
  int32_t k_max;     /* largest draft length k that will be requested       */
  int32_t dtype;     /* sdfp_dtype: storage type of weights and of the KV cache */
  int32_t eos_id;    /* < 0: never stop on a token                          */
  uint32_t flags;
} sdfp_config;

/*
 * Weights: DEVICE pointers, every matrix row-major [out_features, in_features]
 * in the storage type of the config.  The per-layer members point to HOST
 * arrays of n_layers device pointers.  sdfp_create re-packs everything into
 * library-owned buffers (fused QKV, interleaved gate/up, tensor-core fragment
 * order) and does not keep the caller's pointers: the caller may free its
 * tensors after sdfp_create returns.
 */
typedef struct {
  const void *tok_embed;  /* [vocab, d_model] */
  const void *final_norm; /* [d_model]        */
  const void *lm_head;    /* [vocab, d_model] */
  const void *const *wq, *const *wk, *const *wv, *const *wo; /* [d_model, d_model] each */
  const void *const *w_gate, *const *w_up;                   /* [d_ffn, d_model]        */
  const void *const *w_down;                                 /* [d_model, d_ffn]        */
  const void *const *attn_norm, *const *ffn_norm;            /* [d_model]               */
} sdfp_weights;

/* One speculative round of one sequence (Algorithm 1, loop body). */
typedef struct {
  int32_t drafted;   /* k                                                    */
  int32_t accepted;  /* j = length of the accepted prefix (Eq. 2), 0..k      */
  int32_t committed; /* tokens appended this round after truncation, <= j+1  */
} sdfp_round_stat;

/* Timing and traffic of the last sdfp_generate call (CUDA events on the stream). */
typedef struct {
  float prefill_ms;         /* prompt pass(es) of target and draft                     */
  float decode_ms;          /* first round's first kernel .. last round's last kernel  */
  int32_t n_rounds;         /* rounds (speculative) or steps (k = 0)                   */
  int32_t n_draft_passes;   /* draft forward passes in the decode phase                */
  int32_t n_target_passes;  /* verify (or autoregressive) passes in the decode phase   */
  int64_t kernel_launches;  /* kernels of this library launched in the decode phase    */
  int64_t weight_bytes;     /* weight bytes the decode-phase passes had to read        */
  int64_t kv_bytes;         /* KV-cache bytes read + written in the decode phase       */
  int64_t tokens_committed; /* over all sequences                                      */
} sdfp_timing;

/*
 * Create a context: validates the config, packs the weights, allocates both KV
 * caches (target: all layers; draft: its own cache for the kept layers, Section
 * III-C "architecture-compatible") and all scratch.  `cuda_stream` is a
 * cudaStream_t.  The draft initially keeps every layer.
 */
int sdfp_create(const sdfp_config *cfg, const sdfp_weights *w, void *cuda_stream, sdfp_ctx **out);

/*
 * Select the draft model (Algorithm 1: "construct draft model by removing
 * layers in P"): keep_mask is a HOST array of n_layers bytes, 1 = the draft runs
 * the layer, 0 = the layer is the identity for the draft.  At least one layer
 * must be kept.  Takes effect at the next sdfp_generate.
 */
int sdfp_set_draft_layers(sdfp_ctx *ctx, const uint8_t *keep_mask);

/*
 * The same at sub-layer granularity (Section IV-A, implementation details: attention layers and
 * FFN layers are pruned at separate ratios, e.g. 50 % and 35 % for the 13B model).  A decoder
 * layer is two residual blocks, h += Attn(norm(h)) and h += FFN(norm(h)); keep_attn and keep_ffn
 * are HOST arrays of n_layers bytes each, 1 = the draft runs that block, 0 = the block is the
 * identity for the draft.  At least one block must be kept.  The draft's KV cache is used for
 * the layers whose attention block runs.  sdfp_set_draft_layers(m) is
 * sdfp_set_draft_sublayers(m, m).  Takes effect at the next sdfp_generate.
 */
int sdfp_set_draft_sublayers(sdfp_ctx *ctx, const uint8_t *keep_attn, const uint8_t *keep_ffn);

/*
 * KV reuse between draft and target (Section III-C: the pruned draft stays architecture-
 * compatible with the target, "enabling efficient KV reuse during verification").  share = 0
 * (default): the draft has its own cache, filled by its own prompt pass.  share != 0: the draft
 * keeps no cache; in the layers it runs it attends the TARGET's K/V for the committed prefix and
 * writes the K/V of the tokens it drafts into the same cache behind the committed length, where
 * the verification pass overwrites them.  No prompt pass of the draft, no second cache to read,
 * and each round's first draft pass feeds one token instead of two.  The generated tokens are
 * the target's either way; the acceptance counts differ unless every pruned block lies behind
 * every kept one (then both modes are the same computation).  Takes effect at the next
 * sdfp_generate.  With share != 0 the test hook sdfp_forward_logits(draft = 1) writes the
 * target's cache.
 */
int sdfp_set_draft_kv_sharing(sdfp_ctx *ctx, int32_t share);

/*
 * Generate (Algorithm 1, Stage B).  Synchronous: returns when the outputs are
 * in host memory.
 *   prompts     host int32 [batch, prompt_len], ids in [0, vocab); prompt_len >= 1
 *   k           draft length per round, 1..k_max; 0 = plain autoregressive decoding
 *               with the full model (the "vanilla" baseline of Table I)
 *   max_new     tokens to produce per sequence (fewer if eos_id is produced)
 *   temperature 0 = greedy (accept iff the draft token is the target's argmax, ties
 *               to the lowest id); > 0 = sampling from softmax(logits/temperature)
 *               with the accept rule of Eq. 2 and residual resampling (Eq. 3 read as
 *               normalised max(0, p − q))
 *   seed        key of the Philox4x32-10 streams (sampling only)
 *   out_tokens  host int32 [batch, max_new]; entries beyond out_len[b] are −1
 *   out_len     host int32 [batch]
 *   stats       host [max_rounds, batch] or NULL; round r of sequence b at
 *               stats[r*batch + b]; sequences that were already finished in a
 *               round report {0,0,0}
 *   n_rounds    host int32, rounds executed (may be NULL)
 * Fails with SDFP_EINVAL when prompt_len + max_new + k + 1 > max_seq,
 * batch > max_batch, k > k_max, temperature < 0 or a pointer is NULL.
 */
int sdfp_generate(sdfp_ctx *ctx, const int32_t *prompts, int32_t batch, int32_t prompt_len,
                  int32_t k, int32_t max_new, float temperature, uint64_t seed,
                  int32_t *out_tokens, int32_t *out_len, sdfp_round_stat *stats,
                  int32_t max_rounds, int32_t *n_rounds);

/*
 * Test hook: run `rows` tokens of ONE sequence at positions start.. through the
 * target (draft == 0) or the draft (draft != 0) model on sequence slot 0,
 * writing K/V into that model's cache from `start` on, and copy the logits
 * [rows, vocab] (fp32) to host.  rows <= 80.  Lets a test compare logits with
 * the oracle position by position, in chunks of any size.
 */
int sdfp_forward_logits(sdfp_ctx *ctx, int32_t draft, const int32_t *tokens, int32_t rows,
                        int32_t start, float *host_logits);

/*
 * sdfp_forward_logits without any allocation behind it.  (The paper has no counterpart:
 * this is a packaging variant of the test hook above, not a step of the method.)
 *
 * Who needs it: code that is not allowed to reach a device allocator when it calls into the
 * library.  Examples are a serving process whose own pool has claimed all of HBM, so that a
 * later cudaMalloc fails or stalls the device; a real-time loop that must not take the
 * implicit device-wide synchronisation cudaMalloc and cudaFree imply; and a thread that runs
 * while another one captures a CUDA graph, during which allocation calls are illegal.  The
 * split-KV attention kernel needs scratch in global memory (per (row, head, 64-key chunk) a
 * partial max, sum and output vector, plus one arrival counter per head).  Here that scratch
 * is a fixed array of SDFP_STATIC_SCRATCH_BYTES bytes compiled into the library, which every
 * GPU that loads the library holds until the process exits.  The call uses no cudaMalloc,
 * cudaFree, pool or framework allocator, directly or through another library.
 *
 * Arguments, results and errors are those of sdfp_forward_logits, and the logits are the same
 * bit for bit.  In addition:
 *   - SDFP_EINVAL when R x n_heads x P x (head_dim + 2) x 4 bytes, plus the counters, exceed
 *     SDFP_STATIC_SCRATCH_BYTES.  R is the number of rows of the widest pass the call runs and
 *     P the number of partials per (row, head): for bf16 models on the whole-pass kernel
 *     R <= 16 and P = 8, which always fits; for bf16 contexts that decode on the dense path
 *     R = rows (rounded up to a multiple of 16 beyond 16) and P = 8; with
 *     SDFP_FLAG_NO_PASS_KERNEL, SDFP_FLAG_FMA_GEMM or SDFP_FLAG_NO_DENSE and for fp32 models
 *     R likewise and P = ceil((start + rows) / 64).  The message states both sizes.
 *   - The first call on a device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and keeps it.  Make that first call
 *     before starting any stream capture, and from one thread: two threads making the first
 *     call on a device at the same time both store the (same) address without synchronisation.
 *   - All contexts of the process on one device share the array, and it keeps what the last
 *     call left in it.  The call clears the part that must start at zero itself, but two such
 *     calls whose GPU work overlaps (different streams, different threads) race on it:
 *     serialise them.
 */
#define SDFP_STATIC_SCRATCH_BYTES (8u << 20)
int sdfp_forward_logits_static(sdfp_ctx *ctx, int32_t draft, const int32_t *tokens, int32_t rows,
                               int32_t start, float *host_logits);

/*
 * Stage A of Algorithm 1 ("FIT-based pruning"): the layer scores from which the prune set P is
 * chosen.  No context is needed; the weights are read where the caller has them (same structure
 * and storage type as for sdfp_create, row-major [out, in]) and nothing is kept.
 *   tokens     host int32 [n_seq, seq_len]: the calibration set D, one sequence = one sample z_i;
 *              f(z_i, theta) = mean cross-entropy of token t+1 under the logits at position t
 *   out_trace  host double [n_layers]: T_l = (1/N) sum_i ||grad_{theta_l} f(z_i, theta)||^2, the
 *              empirical-Fisher trace of layer l (Eq. 11; Eq. 8-9), over the layer's seven
 *              matrices and two norm gains
 *   out_fit    host double [n_layers] or NULL: sum over the layer's tensors of T_t * mean(theta_t^2),
 *              the layer-wise FIT form (Eq. 7) with the perturbation of removing the layer,
 *              delta theta = -theta
 * Algorithm 1 then sorts ascending and prunes the floor(r L) lowest layers; feed the result to
 * sdfp_set_draft_layers.  One forward and one backward pass per sequence in fp32 (squared norms
 * accumulated in fp64); device memory for the activations of one sequence is allocated and freed
 * inside the call, which is synchronous.  Errors as for sdfp_create (message via
 * sdfp_last_error(NULL)).
 */
int sdfp_fit_scores(const sdfp_config *cfg, const sdfp_weights *w, void *cuda_stream, const int32_t *tokens,
                    int32_t n_seq, int32_t seq_len, double *out_trace, double *out_fit);

/* Timing of the last successful sdfp_generate. */
int sdfp_get_timing(const sdfp_ctx *ctx, sdfp_timing *out);

/*
 * Micro-benchmark hook for the roofline report: launches the library's
 * weight-streaming linear kernel of layer `layer` (which: 0 = QKV, 1 = O,
 * 2 = gate/up, 3 = down, 4 = lm-head) with `rows` activation rows `iters`
 * times back to back on the context's stream, layer advancing cyclically so
 * that consecutive launches read different weights, and returns the average
 * duration of one launch in milliseconds (CUDA events) and the weight bytes one
 * launch reads.  Scratch activations are used; caches are not touched.
 */
int sdfp_time_linear(sdfp_ctx *ctx, int32_t which, int32_t rows, int32_t iters,
                     float *ms_per_launch, int64_t *weight_bytes_per_launch);

/*
 * Micro-benchmark hook for the roofline report of the whole-pass kernel (bf16 models without
 * SDFP_FLAG_NO_PASS_KERNEL; SDFP_ESTATE otherwise).  Runs `iters` forward passes of `rows`
 * rows (1..16) of sequence slot 0 at positions position.. through the target (draft == 0) or
 * the draft model, lm-head included, and returns the average duration of ONE launch of the
 * pass kernel in milliseconds (a CUDA-event pair around every launch, on the context's stream)
 * together with the bytes such a launch has to move: the weights of the layers it runs and of
 * the lm-head, the K/V of those layers for positions 0..position+rows-1, and the K/V rows it
 * writes.  The token ids fed are 0; the K/V cache of slot 0 is overwritten from `position` on
 * (in Section II-A's terms: a timing-only verification pass whose result is discarded).
 */
int sdfp_time_pass(sdfp_ctx *ctx, int32_t draft, int32_t rows, int32_t position, int32_t iters,
                   float *ms_per_launch, int64_t *bytes_per_launch);

/*
 * Failure-path test hook (bf16 contexts whose passes run in the whole-pass kernel or on the
 * dense path; SDFP_ESTATE otherwise).  Section II-A's loop has no counterpart: this exercises
 * the library's own bounded waits.  Whole-pass kernel: after the call, the grid barriers of the
 * next pass expect one arrival more than the grid can provide.  Dense path: in the next
 * sdfp_forward_logits or sdfp_forward_logits_static call (other entry points are not affected),
 * the CTAs of the linear kernels that hold the middle of a feature tile raise their "partial
 * sum posted" flags where nobody looks, so the CTA that finishes the tile waits for a post that
 * never comes.  Either way every wait gives up after wait_limit_ns (1 ms .. 2 s) instead of
 * the default 2 s: that pass winds down in an orderly way (nothing faults, nothing spins on),
 * the entry point that launched it returns SDFP_ETIMEOUT with the name of the wait in
 * sdfp_last_error, and in doing so puts everything back to normal, so the next call on the
 * context works.
 */
int sdfp_debug_expire_next_wait(sdfp_ctx *ctx, uint64_t wait_limit_ns);

const char *sdfp_last_error(const sdfp_ctx *ctx);
void sdfp_destroy(sdfp_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* SDFP_H_ */
