// Host engine and C ABI of the SDFP speculative-decode library (see include/sdfp.h).
//
// One forward pass = plan+embed, then per running layer
//   [RMSNorm + QKV + RoPE + KV append] -> [split-KV attention] -> [O-proj + residual]
//   -> [RMSNorm + gate/up + SwiGLU] -> [down-proj + residual],
// then [final RMSNorm + lm-head] and a token decision.  A speculative round is
// k draft passes (kept layers, own KV cache), one verify pass over k+1 rows (all
// layers) and one accept/commit kernel; all lengths live on the device, so a round
// is a fixed kernel sequence that is captured once as a CUDA graph and replayed.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <tuple>
#include <vector>

#include "../../include/sdfp.h"
#include "attention.cuh"
#include "common.cuh"
#include "dense_attention.cuh"
#include "fit.cuh"
#include "linear_fma.cuh"
#include "linear_mma.cuh"
#include "misc_kernels.cuh"
#include "pass_kernel.cuh"
#include "prefill_attention.cuh"
#include "sampling.cuh"
#include "umma_linear.cuh"

using namespace sdfp;
static_assert(kAmaxRows == kPassMaxRows, "the partial-argmax array is indexed by the whole-pass kernel's rows");

namespace {

thread_local std::string g_create_error;

struct LayerWeights {
  void* qkv = nullptr;   // packed [3d, d]
  void* wo = nullptr;    // packed [d, d]
  void* gu = nullptr;    // packed [2f, d]
  void* down = nullptr;  // packed [d, f]
  // the same matrices as tcgen05 operand images (dense path), null when that path is off
  void *um_qkv = nullptr, *um_wo = nullptr, *um_gu = nullptr, *um_down = nullptr;
  float* attn_gain = nullptr;
  float* ffn_gain = nullptr;
};

struct KvCache {
  std::vector<void*> k, v;  // per layer: [max_batch][heads][max_seq][head_dim]
};

}  // namespace

struct sdfp_ctx {
  sdfp_config cfg{};
  cudaStream_t stream = nullptr;
  std::string err;
  bool bf16 = false, use_mma = false, use_pdl = true, use_graph = true;
  size_t esz = 4;  // bytes per stored element
  int num_sms = 148;
  int device = -1;  // ordinal that was current at sdfp_create; every computing call checks it is still current

  std::vector<LayerWeights> layers;
  void* embed = nullptr;
  void* lm_head = nullptr;
  float* final_gain = nullptr;
  float *rope_cos = nullptr, *rope_sin = nullptr;
  KvCache cache_t, cache_d;
  std::vector<uint8_t> keep_attn, keep_ffn;  // draft: which attention blocks and which FFN blocks run
  bool share_kv = false;  // the draft reads and writes the target's cache instead of its own

  // activations / scratch
  float *h = nullptr, *q = nullptr, *att = nullptr, *u = nullptr, *logits = nullptr;
  float* h_fork = nullptr;  // dense prompt pass: the residual rows where the draft leaves the target
  float *part_o = nullptr, *part_ml = nullptr;
  int* attn_counters = nullptr;
  int n_chunks_cap = 0;
  RowPlan plan{};
  int *seq_tok = nullptr, *draft_tok = nullptr, *tgt_tok = nullptr, *row_argmax = nullptr, *out_tok = nullptr;
  int* fwd_tok = nullptr;
  float* qprob = nullptr;  // sampling: unnormalised draft probabilities [max_batch][kMaxK][vocab]
  double* qsum = nullptr;  // [max_batch][kMaxK]
  GenState* gs = nullptr;
  RoundStat* stats = nullptr;
  int stats_cap = 0;
  int* pinned_flag = nullptr;  // host pinned: [all_done, round]

  std::vector<void*> allocs;
  struct RoundGraph {
    cudaGraphExec_t exec;
    long long launches;
  };
  std::map<std::tuple<int, int, int, int>, RoundGraph> graphs;  // (k, batch, sampled, n_chunks)
  long long launches = 0;
  Launcher L{};

  // persistent pass kernel (bf16 tensor path, passes of up to kPassMaxRows rows)
  bool use_pass = false;
  StageDesc *prog_t = nullptr, *prog_d = nullptr;  // device: stage lists of the target and of the draft
  int n_prog_t = 0, n_prog_d = 0;
  PassSync* psync = nullptr;
  ulonglong2* split_partials = nullptr;
  float* ssq_part = nullptr;
  int2* amax_part = nullptr;  // greedy decision fused into the lm-head: (largest logit, index) per (group of the vocabulary, row)
  int amax_groups = 0;
  int pass_slots[3] = {0, 0, 0};  // ring slots of the instantiation with 1 and with 2 column groups
  size_t pass_smem = 0;
  int pass_grid = 0;
  // dense path on tcgen05 (bf16 tensor path): the prompt pass of every context, and every pass of
  // a context whose widest pass does not fit the whole-pass kernel
  bool use_dense = false;
  bool dense_decode = false;       // ... this context's decode passes run on it as well
  int attn_splits = 1;             // its attention kernel: CTAs per (sequence, head), fixed for the life of the context
  void* um_lm_head = nullptr;
  unsigned char* um_x = nullptr;   // activation image, rows_cap (rounded to 128) x widest K
  unsigned char *um_pa = nullptr, *um_pu = nullptr;  // prompt pass: images of the attention output and of u
  // decode on the dense path: images of gain * h, of the attention output and of u; sums of squares
  unsigned char *um_xh = nullptr, *um_xa = nullptr, *um_xu = nullptr;
  float* um_ssq = nullptr;
  float* um_partial = nullptr;
  int *um_flags = nullptr, *um_error = nullptr;
  int* um_flags_dummy = nullptr;          // failure-path test hook: where posts go to be lost
  unsigned long long um_expire_ns = 0;    // hook armed: the next sdfp_forward_logits call runs with ...
  unsigned long long um_sabotage_ns = 0;  // ... lost posts and this wait limit
  int rows_cap = kMaxRows;         // rows the activation buffers h, q, att, u and the row plan hold
  int max_smem_optin = 0;
  bool own_stream = false;
  sdfp_timing timing{};
  cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
};

namespace {

int fail(sdfp_ctx* c, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c)
    c->err = buf;
  else
    g_create_error = buf;
  return code;
}

// The context's memory, stream and kernels belong to the device that was current at sdfp_create.
// With another device current a launch on the legacy default stream (or a symbol lookup) would land
// on the wrong GPU, so every entry point that touches the device checks first.
int check_device(sdfp_ctx* c, const char* who) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return fail(c, SDFP_ECUDA, "%s: cudaGetDevice failed", who);
  }
  if (dev != c->device)
    return fail(c, SDFP_ESTATE, "%s: the context was created on device %d but device %d is current", who, c->device, dev);
  return 0;
}

#define CU_OK(c, call)                                                                          \
  do {                                                                                          \
    cudaError_t e_ = (call);                                                                    \
    if (e_ != cudaSuccess)                                                                      \
      return fail((c), e_ == cudaErrorMemoryAllocation ? SDFP_ENOMEM : SDFP_ECUDA, "%s: %s", #call, \
                  cudaGetErrorString(e_));                                                      \
  } while (0)

template <typename T>
int dev_alloc(sdfp_ctx* c, T** p, size_t n, bool zero = false) {
  void* q = nullptr;
  CU_OK(c, cudaMalloc(&q, std::max<size_t>(n * sizeof(T), 16)));
  c->allocs.push_back(q);
  if (zero) CU_OK(c, cudaMemsetAsync(q, 0, std::max<size_t>(n * sizeof(T), 16), c->stream));
  *p = reinterpret_cast<T*>(q);
  return 0;
}

template <typename... KArgs, typename... Args>
cudaError_t launch(sdfp_ctx* c, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
  return launch_kernel(c->L, kernel, grid, block, smem, std::forward<Args>(args)...);
}

// ---- linear layer dispatch ---------------------------------------------------------

struct LinearCall {
  const void* w;
  const float* x;
  int ldx, rows, K, n_pairs;
  const float* gain;  // non-null: RMSNorm of x with this gain first
  EpiParams ep;
};

int linear_grid_fma(const sdfp_ctx* c, int n_pairs) {
  const int want = (n_pairs + 7) / 8;
  return std::max(1, std::min(want, c->num_sms * 8));
}

UmmaParams dense_params(const sdfp_ctx* c, const void* w_img, const unsigned char* x_img, int rows, int RB, int KB, int n_pairs,
                        const EpiParams& ep) {
  UmmaParams p{};
  p.W = reinterpret_cast<const unsigned char*>(w_img);
  p.X = x_img;
  p.n_ft = (n_pairs + 63) / 64;
  p.n_rb = (rows + RB - 1) / RB;
  p.KB = KB;
  p.RB = RB;
  p.M = rows;
  p.n_pairs = n_pairs;
  p.n_stages = umma_stages_for(RB, c->max_smem_optin);
  p.partial = c->um_partial;
  p.flags = c->um_flags;
  p.flags_post = c->um_sabotage_ns ? c->um_flags_dummy : c->um_flags;  // test hook: posts that never arrive
  p.error = c->um_error;
  p.wait_limit_ns = c->um_sabotage_ns ? c->um_sabotage_ns : kWaitLimitNs;
  p.ssq_ld = kMaxRows;
  p.inv_k = 1.0f;
  p.eps = c->cfg.rms_eps;
  p.ep = ep;
  return p;
}

// One CTA per SM.  Launched with the programmatic-dependent-launch attribute like every other
// kernel: the kernel requests its first weights before it waits for its predecessor.
cudaError_t launch_dense(sdfp_ctx* c, const UmmaParams& p) {
  return launch(c, umma_linear_kernel, dim3(c->num_sms), dim3(kUmThreads), umma_smem_bytes(p.RB, p.n_stages), p);
}

// Linear layer on the tcgen05 path from fp32 rows: activation image (RMSNorm folded in) by a
// conversion kernel, then the stream-K kernel.  (The prompt pass; decode passes on the dense path
// chain the kernels image to image instead, see enqueue_dense_pass.)
cudaError_t run_dense_linear(sdfp_ctx* c, const void* w_img, const float* x, int ldx, int rows, int K, int n_pairs,
                             const float* gain, const EpiParams& ep) {
  const int RB = rows >= kUmMaxRB ? kUmMaxRB : ((rows + 15) / 16) * 16;
  const int KB = (K + kUmBK - 1) / kUmBK;
  cudaError_t e = launch(c, prep_rows_kernel, dim3((rows + 7) / 8), dim3(kPrepThreads), 0, x, ldx, rows, K, gain, c->cfg.rms_eps,
                         c->um_x, RB, KB);
  if (e != cudaSuccess) return e;
  const UmmaParams p = dense_params(c, w_img, c->um_x, rows, RB, KB, n_pairs, ep);
  return launch_dense(c, p);
}

cudaError_t run_linear(sdfp_ctx* c, const LinearCall& lc) {
  if (c->dense_decode)
    return run_dense_linear(c, lc.w, lc.x, lc.ldx, lc.rows, lc.K, lc.n_pairs, lc.gain, lc.ep);
  if (c->use_mma)
    return launch_linear_mma(c->L, c->num_sms, lc.w, lc.x, lc.ldx, lc.rows, lc.K, lc.n_pairs, lc.gain, c->cfg.rms_eps, lc.ep);
  const dim3 grid(linear_grid_fma(c, lc.n_pairs)), block(kFmaThreads);
  if (c->bf16)
    return launch(c, linear_fma_kernel<__nv_bfloat16, __nv_bfloat16>, grid, block, 0,
                  reinterpret_cast<const __nv_bfloat16*>(lc.w), lc.x, lc.ldx, lc.rows, lc.K, lc.n_pairs, lc.gain,
                  c->cfg.rms_eps, lc.ep);
  return launch(c, linear_fma_kernel<float, float>, grid, block, 0, reinterpret_cast<const float*>(lc.w), lc.x,
                lc.ldx, lc.rows, lc.K, lc.n_pairs, lc.gain, c->cfg.rms_eps, lc.ep);
}

EpiParams base_epi(const sdfp_ctx* c, int mode, float* out, int ld) {
  EpiParams ep{};
  ep.mode = mode;
  ep.out = out;
  ep.out_ld = ld;
  ep.rope_cos = c->rope_cos;
  ep.rope_sin = c->rope_sin;
  ep.row_pos = c->plan.row_pos;
  ep.row_seq = c->plan.row_seq;
  ep.n_heads = c->cfg.n_heads;
  ep.head_dim = c->cfg.head_dim;
  ep.max_seq = c->cfg.max_seq;
  return ep;
}

template <typename KT, int HD>
cudaError_t launch_attention_t(sdfp_ctx* c, const AttnParams& ap, int n_groups) {
  const size_t smem = attention_smem_bytes<KT, HD>();
  return launch(c, attention_kernel<KT, HD>, dim3(ap.n_chunks, ap.n_heads, n_groups), dim3(kAttnThreads), smem, ap);
}

cudaError_t run_attention(sdfp_ctx* c, const KvCache& kv, int layer, int rows, int rows_per_seq, int n_chunks,
                          unsigned char* img = nullptr, int img_rb = 0, int img_kb = 0) {
  AttnParams ap{};
  ap.img = img;
  ap.img_rb = img_rb;
  ap.img_kb = img_kb;
  ap.q = c->q;
  ap.kcache = kv.k[layer];
  ap.vcache = kv.v[layer];
  ap.out = c->att;
  ap.part_o = c->part_o;
  ap.part_ml = c->part_ml;
  ap.counters = c->attn_counters;
  ap.row_pos = c->plan.row_pos;
  ap.row_seq = c->plan.row_seq;
  ap.rows_per_seq = rows_per_seq;
  ap.n_heads = c->cfg.n_heads;
  ap.max_seq = c->cfg.max_seq;
  ap.n_chunks = n_chunks;
  ap.scale = 1.0f / std::sqrt((float)c->cfg.head_dim);
  const int n_groups = rows / rows_per_seq;
  const bool hd128 = c->cfg.head_dim == 128;
  if (c->dense_decode) {
    ap.n_splits = c->attn_splits;
    const dim3 grid(ap.n_splits, ap.n_heads, n_groups);
    if (hd128) return launch(c, attention_mma_kernel<128>, grid, dim3(kAmThreads), attention_mma_smem<128>(), ap, rows);
    return launch(c, attention_mma_kernel<64>, grid, dim3(kAmThreads), attention_mma_smem<64>(), ap, rows);
  }
  if (c->bf16)
    return hd128 ? launch_attention_t<__nv_bfloat16, 128>(c, ap, n_groups)
                 : launch_attention_t<__nv_bfloat16, 64>(c, ap, n_groups);
  return hd128 ? launch_attention_t<float, 128>(c, ap, n_groups) : launch_attention_t<float, 64>(c, ap, n_groups);
}

template <typename KT, int HD>
cudaError_t configure_attention_t() {
  return cudaFuncSetAttribute(attention_kernel<KT, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)attention_smem_bytes<KT, HD>());
}

cudaError_t configure_kernels(const sdfp_ctx* c) {
  const bool hd128 = c->cfg.head_dim == 128;
  cudaError_t e;
  if (c->bf16)
    e = hd128 ? configure_attention_t<__nv_bfloat16, 128>() : configure_attention_t<__nv_bfloat16, 64>();
  else
    e = hd128 ? configure_attention_t<float, 128>() : configure_attention_t<float, 64>();
  return e;
}

// ---- persistent pass kernel: stage lists and launch ---------------------------------------------

StageDesc linear_desc(const void* w, const float* x, int K, int n_pairs, const float* gain, const EpiParams& ep) {
  StageDesc s{};
  s.kind = ST_LINEAR;
  s.K = K;
  s.KT = K / 16;
  s.NT = n_pairs / 8;
  s.n_groups = (s.NT + kUnitTiles - 1) / kUnitTiles;
  s.ldx = K;
  s.x_mode = X_PLAIN;
  s.rms_mode = gain ? RMS_FROM_PARTS : RMS_NONE;
  s.write_ssq = ep.mode == EPI_RESID ? 1 : 0;
  s.W = reinterpret_cast<const uint4*>(w);
  s.X = x;
  s.gain = gain;
  s.ep = ep;
  return s;
}

// The stage list of one forward pass: the target runs every layer, the draft the kept ones
// (Algorithm 1: the draft is the model with the pruned layers removed).  The lm-head is the
// last stage, so a pass that needs no logits runs the list without its last entry.
int build_program(sdfp_ctx* c, bool draft, StageDesc** dev, int* n_out) {
  const sdfp_config& g = c->cfg;
  const int d = g.d_model, f = g.d_ffn;
  const int resid_groups = (d / 16 + kUnitTiles - 1) / kUnitTiles;  // groups of the stages that write the residual stream
  const KvCache& kv = (draft && !c->share_kv) ? c->cache_d : c->cache_t;
  std::vector<StageDesc> prog;
  for (int l = 0; l < g.n_layers; ++l) {
    const LayerWeights& lw = c->layers[l];
    if (!draft || c->keep_attn[l]) {  // the attention block: h += Wo * Attn(norm(h))
      EpiParams qkv = base_epi(c, EPI_QKV, c->q, d);
      qkv.kcache = kv.k[l];
      qkv.vcache = kv.v[l];
      prog.push_back(linear_desc(lw.qkv, c->h, d, 3 * d / 2, lw.attn_gain, qkv));
      StageDesc at{};
      at.kind = ST_ATTN;
      at.X = c->q;
      at.ep = base_epi(c, EPI_RESID, nullptr, d);
      at.ep.kcache = kv.k[l];
      at.ep.vcache = kv.v[l];
      prog.push_back(at);
      // the O-projection reads the attention output as kAttnSplits partials per (row, head)
      prog.push_back(linear_desc(lw.wo, nullptr, d, d / 2, nullptr, base_epi(c, EPI_RESID, c->h, d)));
      prog.back().x_mode = X_ATTN_FOLD;
    }
    if (!draft || c->keep_ffn[l]) {   // the FFN block: h += Wdown * SwiGLU(norm(h))
      prog.push_back(linear_desc(lw.gu, c->h, d, f, lw.ffn_gain, base_epi(c, EPI_SWIGLU, c->u, f)));
      prog.push_back(linear_desc(lw.down, c->u, f, d / 2, nullptr, base_epi(c, EPI_RESID, c->h, d)));
    }
  }
  prog.push_back(linear_desc(c->lm_head, c->h, d, g.vocab / 2, c->final_gain, base_epi(c, EPI_LOGITS, c->logits, g.vocab)));
  // the embedding rows come from another kernel: the first norm of a pass sums its rows itself
  prog.front().rms_mode = RMS_DIRECT;
  for (StageDesc& sd : prog) sd.ssq_groups = resid_groups;
  if (*dev == nullptr)
    if (int r = dev_alloc(c, dev, (size_t)5 * g.n_layers + 1)) return r;
  CU_OK(c, cudaMemcpyAsync(*dev, prog.data(), prog.size() * sizeof(StageDesc), cudaMemcpyHostToDevice, c->stream));
  CU_OK(c, cudaStreamSynchronize(c->stream));  // prog is a local
  *n_out = (int)prog.size();
  return 0;
}

int build_programs(sdfp_ctx* c) {
  if (!c->use_pass) return 0;
  if (int r = build_program(c, false, &c->prog_t, &c->n_prog_t)) return r;
  return build_program(c, true, &c->prog_d, &c->n_prog_d);
}

template <int CG, int HD>
size_t pass_smem_bytes(int n_slots) {
  return (size_t)n_slots * kSlotBytes + pass_work_bytes<CG, HD>() + sizeof(PassShared);
}

template <int CG, int HD>
int pass_slots_that_fit(int max_smem_optin) {
  // Measured on B200 (7B shape): what matters most is the total shared-memory footprint, which
  // decides how much of the SM's 256 KB is left as L1: up to 164 KB (three 32 KB slots with one
  // column group, two with two) a pass is 4-6% faster than with four or five slots, although the
  // ring is shallower; the refill burst at a stage end, which slows every L2 round trip of the
  // barrier chain, is shorter as well.  Two slots with one column group are too few (+8%).
#ifndef SDFP_MAX_SLOTS2
#define SDFP_MAX_SLOTS2 2
#endif
  int n_slots = CG == 1 ? 3 : SDFP_MAX_SLOTS2;
  while (n_slots > 2 && pass_smem_bytes<CG, HD>(n_slots) > (size_t)max_smem_optin) --n_slots;
  return n_slots;
}

// Each instantiation gets the largest ring that fits beside its work area.
template <int HD>
cudaError_t configure_pass_t(sdfp_ctx* c, int max_smem_optin) {
  c->pass_slots[1] = pass_slots_that_fit<1, HD>(max_smem_optin);
  c->pass_slots[2] = pass_slots_that_fit<2, HD>(max_smem_optin);
  c->pass_smem = std::max(pass_smem_bytes<1, HD>(c->pass_slots[1]), pass_smem_bytes<2, HD>(c->pass_slots[2]));
  if (c->pass_smem > (size_t)max_smem_optin) return cudaErrorLaunchOutOfResources;
  cudaError_t e = cudaFuncSetAttribute(pass_kernel<1, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->pass_smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(pass_kernel<2, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->pass_smem);
  if (e != cudaSuccess) return e;
  // The kernel moves registers from its producer group to its consumers; the amounts are fixed
  // numbers that only add up if it was compiled to the launch size they assume.  Otherwise the
  // consumers would wait for registers that never come: refuse rather than launch.
  for (const void* fn : {(const void*)pass_kernel<1, HD>, (const void*)pass_kernel<2, HD>}) {
    cudaFuncAttributes fa{};
    e = cudaFuncGetAttributes(&fa, fn);
    if (e != cudaSuccess) return e;
    if (fa.numRegs != kPassLaunchRegs) return cudaErrorInvalidDeviceFunction;
  }
  // a cooperative launch needs every CTA resident at once: one per SM
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pass_kernel<2, HD>, kPassThreads, c->pass_smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  c->pass_grid = c->num_sms;
  return cudaSuccess;
}

template <int CG, int HD>
cudaError_t launch_pass_t(sdfp_ctx* c, const PassParams& pp) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(c->pass_grid);
  lc.blockDim = dim3(kPassThreads);
  lc.dynamicSmemBytes = c->pass_smem;
  lc.stream = c->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  c->launches += 1;
  return cudaLaunchKernelEx(&lc, pass_kernel<CG, HD>, pp, c->pass_slots[CG]);
}

// Chunks (32 KB per CTA) of weights the producer asks into L2 ahead of the ring.  Measured on the
// 7B shape, single-row pass: 0 -> 3.68 ms, 4 -> 3.42, 8 -> 3.38, 10 -> 3.50, 12 -> 3.60, 16 -> 3.89:
// a ring of three slots refills from L2 only ~1.5x faster than from memory, so a window the
// consumers cannot drain soon only takes bandwidth from the loads the running stage waits for.
#ifndef SDFP_PREFETCH_CHUNKS
#define SDFP_PREFETCH_CHUNKS 8
#endif

cudaError_t run_pass(sdfp_ctx* c, bool draft, int rows, int rows_per_seq, bool with_lm_head, bool fused_argmax = false) {
  PassParams pp{};
  pp.prog = draft ? c->prog_d : c->prog_t;
  pp.n_stages = (draft ? c->n_prog_d : c->n_prog_t) - (with_lm_head ? 0 : 1);
  pp.M = rows;
  pp.rows_per_seq = rows_per_seq;
  pp.row_pos = c->plan.row_pos;
  pp.row_seq = c->plan.row_seq;
  pp.eps = c->cfg.rms_eps;
  pp.attn_scale = 1.0f / std::sqrt((float)c->cfg.head_dim);
  pp.zero = 0u;
  pp.pf_chunks = SDFP_PREFETCH_CHUNKS;
  pp.part_o = c->part_o;
  pp.part_ml = c->part_ml;
  pp.split_partials = c->split_partials;
  pp.ssq_part = c->ssq_part;
  pp.amax_part = fused_argmax ? c->amax_part : nullptr;
  pp.sync = c->psync;
  const bool hd128 = c->cfg.head_dim == 128;
  if (rows <= 8) return hd128 ? launch_pass_t<1, 128>(c, pp) : launch_pass_t<1, 64>(c, pp);
  return hd128 ? launch_pass_t<2, 128>(c, pp) : launch_pass_t<2, 64>(c, pp);
}

// ---- one forward pass ------------------------------------------------------------------

// prompts shorter than this go through the decode kernels in chunks (a handful of launches)
constexpr int kDenseMinRows = 16;

int enqueue_dense_pass(sdfp_ctx* c, const PassDesc& pd, bool draft, int rows, int attn_rows_per_seq, int n_chunks, int decide);

enum Decide { DECIDE_NONE = 0, DECIDE_LOGITS = 1, DECIDE_ARGMAX = 2, DECIDE_SAMPLE_DRAFT = 3 };

// rows: total rows; rows_per_seq for the attention grouping; n_chunks bounds the context.
int enqueue_pass(sdfp_ctx* c, const PassDesc& pd, bool draft, int rows, int attn_rows_per_seq, int n_chunks,
                 int decide) {
  const sdfp_config& g = c->cfg;
  const int d = g.d_model, f = g.d_ffn;
  if (c->dense_decode) return enqueue_dense_pass(c, pd, draft, rows, attn_rows_per_seq, n_chunks, decide);
  if (c->bf16)
    CU_OK(c, launch(c, plan_embed_kernel<__nv_bfloat16>, dim3(rows), dim3(128), 0, pd, (const GenState*)c->gs,
                    (const int*)c->seq_tok, g.max_seq, (const int*)c->draft_tok, c->plan,
                    reinterpret_cast<const __nv_bfloat16*>(c->embed), c->h, d, EmbedImage{}));
  else
    CU_OK(c, launch(c, plan_embed_kernel<float>, dim3(rows), dim3(128), 0, pd, (const GenState*)c->gs,
                    (const int*)c->seq_tok, g.max_seq, (const int*)c->draft_tok, c->plan,
                    reinterpret_cast<const float*>(c->embed), c->h, d, EmbedImage{}));
  const KvCache& kv = (draft && !c->share_kv) ? c->cache_d : c->cache_t;
  const bool whole_pass = c->use_pass;  // a context takes ONE path for all its passes (see sdfp_create)
  if (whole_pass && rows > kPassMaxRows) return fail(c, SDFP_ESTATE, "a pass of %d rows reached the whole-pass kernel", rows);
  // greedy decisions of the rounds are taken inside the pass kernel's lm-head (pd.amax_part set by enqueue_round)
  const bool fused_argmax = whole_pass && decide == DECIDE_ARGMAX && pd.amax_part != nullptr;
  if (whole_pass) CU_OK(c, run_pass(c, draft, rows, attn_rows_per_seq, decide != DECIDE_NONE, fused_argmax));
  if (fused_argmax) return 0;
  for (int l = 0; l < g.n_layers && !whole_pass; ++l) {
    // Algorithm 1: pruned layers are removed from the draft, attention and FFN blocks separately
    const bool run_attn = !draft || c->keep_attn[l], run_ffn = !draft || c->keep_ffn[l];
    const LayerWeights& lw = c->layers[l];
    if (run_attn) {
      LinearCall lc{lw.qkv, c->h, d, rows, d, 3 * d / 2, lw.attn_gain, base_epi(c, EPI_QKV, c->q, d)};
      lc.ep.kcache = kv.k[l];
      lc.ep.vcache = kv.v[l];
      CU_OK(c, run_linear(c, lc));
      CU_OK(c, run_attention(c, kv, l, rows, attn_rows_per_seq, n_chunks));
      LinearCall lo{lw.wo, c->att, d, rows, d, d / 2, nullptr, base_epi(c, EPI_RESID, c->h, d)};
      CU_OK(c, run_linear(c, lo));
    }
    if (!run_ffn) continue;
    {
      LinearCall lc{lw.gu, c->h, d, rows, d, f, lw.ffn_gain, base_epi(c, EPI_SWIGLU, c->u, f)};
      CU_OK(c, run_linear(c, lc));
    }
    {
      LinearCall lc{lw.down, c->u, f, rows, f, d / 2, nullptr, base_epi(c, EPI_RESID, c->h, d)};
      CU_OK(c, run_linear(c, lc));
    }
  }
  if (decide == DECIDE_NONE) return 0;
  if (!whole_pass) {
    LinearCall lc{c->lm_head, c->h, d, rows, d, g.vocab / 2, c->final_gain, base_epi(c, EPI_LOGITS, c->logits, g.vocab)};
    CU_OK(c, run_linear(c, lc));
  }
  if (decide == DECIDE_ARGMAX)
    CU_OK(c, launch(c, argmax_kernel, dim3(rows), dim3(kArgmaxThreads), 0, (const float*)c->logits, g.vocab, pd,
                    c->draft_tok, c->tgt_tok, c->row_argmax));
  else if (decide == DECIDE_SAMPLE_DRAFT)
    CU_OK(c, launch(c, sample_draft_kernel, dim3(rows), dim3(kSampleThreads), 0, (const float*)c->logits, g.vocab, pd,
                    (const GenState*)c->gs, c->draft_tok, c->qprob, c->qsum));
  return 0;
}

// One forward pass of a context that decodes on the dense path: every linear layer is one launch of
// the tcgen05 kernel, and the kernels hand the activations on as operand images: the embedding
// kernel and the epilogues that write the residual stream leave (next norm's gain) * h as bf16
// hi + lo plus partial sums of squares, the next linear layer applies 1/rms to its accumulators;
// the SwiGLU epilogue leaves the image of u, the attention kernel the image of its output.
int enqueue_dense_pass(sdfp_ctx* c, const PassDesc& pd, bool draft, int rows, int attn_rows_per_seq, int n_chunks, int decide) {
  const sdfp_config& g = c->cfg;
  const int d = g.d_model, f = g.d_ffn;
  const int RB = ((rows + 15) / 16) * 16;
  const int KBd = (d + kUmBK - 1) / kUmBK, KBf = (f + kUmBK - 1) / kUmBK;
  const KvCache& kv = (draft && !c->share_kv) ? c->cache_d : c->cache_t;
  struct Block {
    int layer;
    bool attn;
  };
  std::vector<Block> blocks;
  for (int l = 0; l < g.n_layers; ++l) {
    if (!draft || c->keep_attn[l]) blocks.push_back({l, true});
    if (!draft || c->keep_ffn[l]) blocks.push_back({l, false});
  }
  auto gain_of = [&](size_t i) -> const float* {  // the gain of the norm in front of block i (the final norm behind the last)
    if (i >= blocks.size()) return c->final_gain;
    const LayerWeights& lw = c->layers[blocks[i].layer];
    return blocks[i].attn ? lw.attn_gain : lw.ffn_gain;
  };
  CU_OK(c, launch(c, plan_embed_kernel<__nv_bfloat16>, dim3(rows), dim3(128), 0, pd, (const GenState*)c->gs, (const int*)c->seq_tok,
                  g.max_seq, (const int*)c->draft_tok, c->plan, reinterpret_cast<const __nv_bfloat16*>(c->embed), c->h, d,
                  EmbedImage{c->um_xh, gain_of(0), c->um_ssq, RB, KBd}));
  int groups = 1;  // partial sums of squares per row the next norm has to add
  const int resid_tiles = 4 * ((d / 2 + 63) / 64);  // a sum of squares per (32 features, row): four per tile
  auto normed = [&](UmmaParams& p) {
    p.ssq_in = c->um_ssq;
    p.ssq_groups = groups;
    p.inv_k = 1.0f / (float)d;
  };
  auto resid_out = [&](UmmaParams& p, size_t next_block) {
    p.img_out = c->um_xh;
    p.img_KB = KBd;
    p.gain_out = gain_of(next_block);
    p.ssq_out = c->um_ssq;
  };
  for (size_t i = 0; i < blocks.size(); ++i) {
    const int l = blocks[i].layer;
    const LayerWeights& lw = c->layers[l];
    if (blocks[i].attn) {
      EpiParams qkv = base_epi(c, EPI_QKV, c->q, d);
      qkv.kcache = kv.k[l];
      qkv.vcache = kv.v[l];
      UmmaParams p = dense_params(c, lw.um_qkv, c->um_xh, rows, RB, KBd, 3 * d / 2, qkv);
      normed(p);
      CU_OK(c, launch_dense(c, p));
      CU_OK(c, run_attention(c, kv, l, rows, attn_rows_per_seq, n_chunks, c->um_xa, RB, KBd));
      UmmaParams o = dense_params(c, lw.um_wo, c->um_xa, rows, RB, KBd, d / 2, base_epi(c, EPI_RESID, c->h, d));
      resid_out(o, i + 1);
      CU_OK(c, launch_dense(c, o));
    } else {
      UmmaParams p = dense_params(c, lw.um_gu, c->um_xh, rows, RB, KBd, f, base_epi(c, EPI_SWIGLU, nullptr, f));
      normed(p);
      p.img_out = c->um_xu;
      p.img_KB = KBf;
      CU_OK(c, launch_dense(c, p));
      UmmaParams dn = dense_params(c, lw.um_down, c->um_xu, rows, RB, KBf, d / 2, base_epi(c, EPI_RESID, c->h, d));
      resid_out(dn, i + 1);
      CU_OK(c, launch_dense(c, dn));
    }
    groups = resid_tiles;
  }
  if (decide == DECIDE_NONE) return 0;
  UmmaParams lm = dense_params(c, c->um_lm_head, c->um_xh, rows, RB, KBd, g.vocab / 2, base_epi(c, EPI_LOGITS, c->logits, g.vocab));
  normed(lm);
  CU_OK(c, launch_dense(c, lm));
  if (decide == DECIDE_ARGMAX)
    CU_OK(c, launch(c, argmax_kernel, dim3(rows), dim3(kArgmaxThreads), 0, (const float*)c->logits, g.vocab, pd, c->draft_tok,
                    c->tgt_tok, c->row_argmax));
  else if (decide == DECIDE_SAMPLE_DRAFT)
    CU_OK(c, launch(c, sample_draft_kernel, dim3(rows), dim3(kSampleThreads), 0, (const float*)c->logits, g.vocab, pd,
                    (const GenState*)c->gs, c->draft_tok, c->qprob, c->qsum));
  return 0;
}

int enqueue_round(sdfp_ctx* c, int k, int batch, bool sampled, int n_chunks) {
  PassDesc pd{};
  pd.n_seq = batch;
  const bool fused = c->use_pass && !sampled;  // the lm-head leaves argmax partials; consumers finish them
  if (fused) {
    pd.amax_part = c->amax_part;
    pd.amax_groups = c->amax_groups;
  }
  if (k > 0) {
    // The draft's own cache lags one token after a fully accepted round, so its first pass feeds
    // the last two committed tokens; a draft that shares the target's cache feeds the last one.
    const int first_rows = c->share_kv ? 1 : 2;
    pd.kind = PASS_DRAFT_FIRST;
    pd.rows_per_seq = first_rows;
    if (int r = enqueue_pass(c, pd, true, first_rows * batch, first_rows, n_chunks, sampled ? DECIDE_SAMPLE_DRAFT : DECIDE_ARGMAX))
      return r;
    for (int s = 1; s < k; ++s) {
      pd.kind = PASS_DRAFT_NEXT;
      pd.step = s;
      pd.prev_rows_per_seq = fused ? (s == 1 ? first_rows : 1) : 0;
      pd.rows_per_seq = 1;
      if (int r = enqueue_pass(c, pd, true, batch, 1, n_chunks, sampled ? DECIDE_SAMPLE_DRAFT : DECIDE_ARGMAX)) return r;
    }
  }
  pd.kind = PASS_VERIFY;
  pd.step = 0;
  pd.prev_rows_per_seq = (fused && k > 0) ? (k == 1 ? (c->share_kv ? 1 : 2) : 1) : 0;
  pd.rows_per_seq = k + 1;
  if (int r = enqueue_pass(c, pd, false, (k + 1) * batch, k + 1, n_chunks, sampled ? DECIDE_LOGITS : DECIDE_ARGMAX))
    return r;
  const int* pass_err = c->use_pass ? &c->psync->error : nullptr;
  if (sampled)
    CU_OK(c, launch(c, accept_sampled_kernel, dim3(1), dim3(kSampleThreads), 0, c->gs, (const float*)c->logits,
                    c->cfg.vocab, (const int*)c->draft_tok, (const float*)c->qprob, (const double*)c->qsum, c->seq_tok,
                    c->cfg.max_seq, c->out_tok, c->stats, pass_err));
  else
    CU_OK(c, launch(c, accept_greedy_kernel, dim3(1), dim3(kAcceptThreads), 0, c->gs, (const int*)c->draft_tok,
                    (const int*)c->tgt_tok, c->seq_tok, c->cfg.max_seq, c->out_tok, c->stats, pass_err,
                    (const int2*)(fused ? c->amax_part : nullptr), c->amax_groups));
  return 0;
}

// ---- weights ------------------------------------------------------------------------------

// the tcgen05 operand image of a matrix (see umma_linear.cuh)
int pack_dense_image(sdfp_ctx* c, void** dst, PackSrc ps, int n_pairs, int K) {
  const int n_ft = (n_pairs + 63) / 64, KB = (K + kUmBK - 1) / kUmBK;
  __nv_bfloat16* p = nullptr;
  if (int r = dev_alloc(c, &p, (size_t)n_ft * KB * (kUmABytes / 2))) return r;
  pack_umma_kernel<<<1184, 256, 0, c->stream>>>(p, ps, n_pairs, K, n_ft, KB);
  CU_OK(c, cudaGetLastError());
  *dst = p;
  return 0;
}

// A matrix in the layout(s) this context's kernels read: `dst` for the whole-pass / per-operation
// kernels, `img` (may be null) for the dense path.  A context whose decode passes run on the dense
// path reads only images: `dst` then points to the image as well.
template <typename WT>
int pack_matrix(sdfp_ctx* c, void** dst, void** img, PackSrc ps, int n_pairs, int K) {
  if (c->use_dense && img) {
    if (int r = pack_dense_image(c, img, ps, n_pairs, K)) return r;
    if (c->dense_decode) {
      *dst = *img;
      return 0;
    }
  }
  const int n_groups = (n_pairs / 8 + kUnitTiles - 1) / kUnitTiles;
  const size_t n = c->use_mma ? (size_t)n_groups * (K / 16) * (kUnitBytes / 2) : (size_t)n_pairs * 2 * K;
  WT* p = nullptr;
  if (int r = dev_alloc(c, &p, n)) return r;
  if (c->use_mma) {
    pack_units_kernel<<<1184, 256, 0, c->stream>>>(reinterpret_cast<__nv_bfloat16*>(p), ps, n_pairs, K, n_groups);
  } else {
    pack_pairs_kernel<WT><<<1184, 256, 0, c->stream>>>(p, ps, n_pairs, K);
  }
  CU_OK(c, cudaGetLastError());
  *dst = p;
  return 0;
}

template <typename WT>
int widen_gain(sdfp_ctx* c, float** dst, const void* src, int n) {
  if (int r = dev_alloc(c, dst, (size_t)n)) return r;
  widen_vector_kernel<WT><<<(n + 255) / 256, 256, 0, c->stream>>>(*dst, reinterpret_cast<const WT*>(src), n);
  CU_OK(c, cudaGetLastError());
  return 0;
}

template <typename WT>
int load_weights(sdfp_ctx* c, const sdfp_weights* w) {
  const sdfp_config& g = c->cfg;
  const int d = g.d_model, f = g.d_ffn, H = g.n_heads, hd = g.head_dim;
  c->layers.resize(g.n_layers);
  for (int l = 0; l < g.n_layers; ++l) {
    LayerWeights& lw = c->layers[l];
    if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->w_gate[l] || !w->w_up[l] || !w->w_down[l] ||
        !w->attn_norm[l] || !w->ffn_norm[l])
      return fail(c, SDFP_EINVAL, "layer %d has a NULL weight pointer", l);
    if (int r = pack_matrix<WT>(c, &lw.qkv, &lw.um_qkv, PackSrc{w->wq[l], w->wk[l], w->wv[l], 0, H, hd}, 3 * d / 2, d)) return r;
    if (int r = pack_matrix<WT>(c, &lw.wo, &lw.um_wo, PackSrc{w->wo[l], nullptr, nullptr, 2, H, hd}, d / 2, d)) return r;
    if (int r = pack_matrix<WT>(c, &lw.gu, &lw.um_gu, PackSrc{w->w_gate[l], w->w_up[l], nullptr, 1, H, hd}, f, d)) return r;
    if (int r = pack_matrix<WT>(c, &lw.down, &lw.um_down, PackSrc{w->w_down[l], nullptr, nullptr, 2, H, hd}, d / 2, f)) return r;
    if (int r = widen_gain<WT>(c, &lw.attn_gain, w->attn_norm[l], d)) return r;
    if (int r = widen_gain<WT>(c, &lw.ffn_gain, w->ffn_norm[l], d)) return r;
  }
  // the prompt pass needs no logits: only contexts that decode on the dense path get an lm-head image
  if (int r = pack_matrix<WT>(c, &c->lm_head, c->dense_decode ? &c->um_lm_head : nullptr,
                              PackSrc{w->lm_head, nullptr, nullptr, 2, H, hd}, g.vocab / 2, d))
    return r;
  if (int r = widen_gain<WT>(c, &c->final_gain, w->final_norm, d)) return r;
  WT* e = nullptr;
  if (int r = dev_alloc(c, &e, (size_t)g.vocab * d)) return r;
  CU_OK(c, cudaMemcpyAsync(e, w->tok_embed, (size_t)g.vocab * d * sizeof(WT), cudaMemcpyDeviceToDevice, c->stream));
  c->embed = e;
  return 0;
}

int alloc_cache(sdfp_ctx* c, KvCache& kv) {
  const sdfp_config& g = c->cfg;
  const size_t bytes = (size_t)g.max_batch * g.n_heads * g.max_seq * g.head_dim * c->esz;
  kv.k.resize(g.n_layers);
  kv.v.resize(g.n_layers);
  for (int l = 0; l < g.n_layers; ++l) {
    unsigned char *pk = nullptr, *pv = nullptr;
    if (int r = dev_alloc(c, &pk, bytes, true)) return r;
    if (int r = dev_alloc(c, &pv, bytes, true)) return r;
    kv.k[l] = pk;
    kv.v[l] = pv;
  }
  return 0;
}

int64_t attn_block_bytes(const sdfp_ctx* c) { return 4LL * c->cfg.d_model * c->cfg.d_model * (int64_t)c->esz; }
int64_t ffn_block_bytes(const sdfp_ctx* c) { return 3LL * c->cfg.d_model * c->cfg.d_ffn * (int64_t)c->esz; }
int64_t lm_head_bytes(const sdfp_ctx* c) { return (int64_t)c->cfg.vocab * c->cfg.d_model * (int64_t)c->esz; }
int kept_blocks(const std::vector<uint8_t>& keep) {
  int n = 0;
  for (uint8_t x : keep) n += x ? 1 : 0;
  return n;
}
// weight bytes one pass of the draft / of the target has to read, lm-head excluded
int64_t pass_weight_bytes(const sdfp_ctx* c, bool draft) {
  const int64_t na = draft ? kept_blocks(c->keep_attn) : c->cfg.n_layers, nf = draft ? kept_blocks(c->keep_ffn) : c->cfg.n_layers;
  return na * attn_block_bytes(c) + nf * ffn_block_bytes(c);
}
// layers whose K/V a pass reads and writes
int64_t pass_kv_layers(const sdfp_ctx* c, bool draft) { return draft ? kept_blocks(c->keep_attn) : c->cfg.n_layers; }

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================

extern "C" const char* sdfp_last_error(const sdfp_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

extern "C" void sdfp_destroy(sdfp_ctx* c) {
  if (!c) return;
  cudaStreamSynchronize(c->stream);
  for (auto& kv : c->graphs) cudaGraphExecDestroy(kv.second.exec);
  for (void* p : c->allocs) cudaFree(p);
  if (c->pinned_flag) cudaFreeHost(c->pinned_flag);
  for (auto& e : c->ev)
    if (e) cudaEventDestroy(e);
  if (c->own_stream) cudaStreamDestroy(c->stream);
  delete c;
}

extern "C" int sdfp_create(const sdfp_config* cfg, const sdfp_weights* w, void* cuda_stream, sdfp_ctx** out) {
  if (!cfg || !w || !out) return fail(nullptr, SDFP_EINVAL, "sdfp_create: NULL argument");
  *out = nullptr;
  const sdfp_config& g = *cfg;
  if (g.n_layers < 1 || g.n_layers > 1024 || g.d_model < 16 || g.n_heads < 1 || g.d_ffn < 16 || g.vocab < 16)
    return fail(nullptr, SDFP_EINVAL, "sdfp_create: non-positive model dimension");
  if (g.head_dim != 64 && g.head_dim != 128) return fail(nullptr, SDFP_EINVAL, "head_dim must be 64 or 128");
  if (g.d_model != g.n_heads * g.head_dim) return fail(nullptr, SDFP_EINVAL, "d_model must equal n_heads*head_dim");
  if (g.d_model % 16 || g.d_ffn % 16 || g.vocab % 16)
    return fail(nullptr, SDFP_EINVAL, "d_model, d_ffn and vocab must be multiples of 16");
  if (g.dtype != SDFP_F32 && g.dtype != SDFP_BF16) return fail(nullptr, SDFP_EINVAL, "unknown dtype");
  if (g.max_batch < 1 || g.max_batch > kMaxBatch) return fail(nullptr, SDFP_EINVAL, "max_batch must be 1..%d", kMaxBatch);
  if (g.k_max < 0 || g.k_max > kMaxK) return fail(nullptr, SDFP_EINVAL, "k_max must be 0..%d", kMaxK);
  if (g.max_batch * (g.k_max + 1) > kMaxRows || g.max_batch * 2 > kMaxRows)
    return fail(nullptr, SDFP_EINVAL, "max_batch*(k_max+1) = %d exceeds the %d rows a pass can carry",
                g.max_batch * std::max(g.k_max + 1, 2), kMaxRows);
  if (g.max_seq < 4 || !(g.rms_eps > 0.f) || !(g.rope_theta > 0.f)) return fail(nullptr, SDFP_EINVAL, "bad max_seq, rms_eps or rope_theta");
  if (!w->tok_embed || !w->final_norm || !w->lm_head || !w->wq || !w->wk || !w->wv || !w->wo || !w->w_gate || !w->w_up ||
      !w->w_down || !w->attn_norm || !w->ffn_norm)
    return fail(nullptr, SDFP_EINVAL, "sdfp_create: NULL weight pointer");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
    cudaGetLastError();
    return fail(nullptr, SDFP_ECUDA, "no CUDA device: this library has no CPU path");
  }
  sdfp_ctx* c = new (std::nothrow) sdfp_ctx();
  if (!c) return fail(nullptr, SDFP_ENOMEM, "host allocation failed");
  auto bail = [&](int code) {
    g_create_error = c->err;
    sdfp_destroy(c);
    return code;
  };
  c->cfg = g;
  c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (c->stream == nullptr) {
    // the legacy default stream cannot be captured into a graph: use a stream of our own,
    // after everything the caller queued so far (its weight tensors) has completed
    if (cudaDeviceSynchronize() != cudaSuccess || cudaStreamCreateWithFlags(&c->stream, cudaStreamNonBlocking) != cudaSuccess) {
      c->stream = nullptr;
      c->err = "could not create a stream";
      return bail(SDFP_ECUDA);
    }
    c->own_stream = true;
  }
  c->L.stream = c->stream;
  c->L.count = &c->launches;
  c->bf16 = (g.dtype == SDFP_BF16);
  c->esz = c->bf16 ? 2 : 4;
  c->use_mma = c->bf16 && !(g.flags & SDFP_FLAG_FMA_GEMM);
  c->use_pdl = !(g.flags & SDFP_FLAG_NO_PDL);
  c->use_graph = !(g.flags & SDFP_FLAG_NO_GRAPH);
  c->L.pdl = c->use_pdl;
  c->keep_attn.assign(g.n_layers, 1);
  c->keep_ffn.assign(g.n_layers, 1);
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    c->err = "cudaGetDeviceProperties failed";
    return bail(SDFP_ECUDA);
  }
  if (prop.major < 10) {
    c->err = "this library is built for sm_100a (B200) only";
    return bail(SDFP_ECUDA);
  }
  c->num_sms = prop.multiProcessorCount;
  c->device = dev;
  // One arithmetic path per context.  The whole-pass kernel and the per-operation kernels add a
  // dot product's terms in different orders, so a context whose widest pass (a verify pass of
  // max_batch sequences, or the two-row draft pass) does not fit the whole-pass kernel runs
  // every pass, narrow ones included, on the per-operation kernels: only then is a row's
  // result independent of the pass it sits in, and speculative output equal to autoregressive
  // output bit for bit.
  const int widest = g.max_batch * std::max(g.k_max + 1, 2);
  c->amax_groups = (g.vocab / 16 + kUnitTiles - 1) / kUnitTiles;
  c->use_pass = c->use_mma && !(g.flags & SDFP_FLAG_NO_PASS_KERNEL) && prop.cooperativeLaunch && g.d_model >= 64 &&
                g.n_heads <= kPassMaxHeads && g.d_model / 128 + 1 <= kSsqMaxGroups && widest <= kPassMaxRows;
  int optin = 0;
  cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  c->max_smem_optin = optin;
  c->use_dense = c->use_mma && !(g.flags & SDFP_FLAG_NO_DENSE);
  c->dense_decode = c->use_dense && !c->use_pass && !(g.flags & SDFP_FLAG_NO_PASS_KERNEL);
  if (c->use_dense) {
    c->rows_cap = std::max((int)kMaxRows, g.max_seq);
    if (cudaFuncSetAttribute(umma_linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin) != cudaSuccess ||
        cudaFuncSetAttribute(prefill_attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)prefill_attention_smem<64>()) != cudaSuccess ||
        cudaFuncSetAttribute(prefill_attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)prefill_attention_smem<128>()) != cudaSuccess) {
      c->err = "dense-path kernel configuration failed";
      return bail(SDFP_ECUDA);
    }
  }
  if (c->dense_decode) {
    // As many splits as still give one wave of CTAs (two per SM) when every sequence slot is in
    // use: more CTAs than that only add set-up and fold time (7B shape, batch 8, context ~600: 4.11 /
    // 4.34 / 4.61 ms per 8-row pass at 1 / 2 / 4 splits).  One number for all passes of the context,
    // because the order in which a row's keys are added depends on it.
    c->attn_splits = std::min((int)kAttnSplits, std::max(1, 2 * c->num_sms / (g.max_batch * g.n_heads)));
    auto cfg_attn = [](auto kernel, size_t sm) {
      return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) == cudaSuccess;
    };
    const bool ok = g.head_dim == 128 ? cfg_attn(attention_mma_kernel<128>, attention_mma_smem<128>())
                                       : cfg_attn(attention_mma_kernel<64>, attention_mma_smem<64>());
    if (!ok) {
      c->err = "dense-path attention kernel configuration failed";
      return bail(SDFP_ECUDA);
    }
  }
  if (c->use_pass) {
    const cudaError_t pe = g.head_dim == 128 ? configure_pass_t<128>(c, optin) : configure_pass_t<64>(c, optin);
    if (pe != cudaSuccess) {
      c->err = std::string("pass kernel configuration failed: ") + cudaGetErrorString(pe);
      return bail(SDFP_ECUDA);
    }
  }
  if (cudaError_t ke = configure_kernels(c)) {
    c->err = std::string("kernel configuration failed: ") + cudaGetErrorString(ke);
    return bail(SDFP_ECUDA);
  }
  int r = c->bf16 ? load_weights<__nv_bfloat16>(c, w) : load_weights<float>(c, w);
  if (r) return bail(r);
  if ((r = alloc_cache(c, c->cache_t)) || (r = alloc_cache(c, c->cache_d))) return bail(r);

  // rotary tables in fp64, rounded to fp32
  {
    const int hp = g.head_dim / 2;
    std::vector<float> cs((size_t)g.max_seq * hp), sn((size_t)g.max_seq * hp);
    for (int i = 0; i < hp; ++i) {
      const double inv = std::pow((double)g.rope_theta, -2.0 * i / g.head_dim);
      for (int p = 0; p < g.max_seq; ++p) {
        cs[(size_t)p * hp + i] = (float)std::cos(p * inv);
        sn[(size_t)p * hp + i] = (float)std::sin(p * inv);
      }
    }
    if ((r = dev_alloc(c, &c->rope_cos, cs.size())) || (r = dev_alloc(c, &c->rope_sin, sn.size()))) return bail(r);
    if (cudaMemcpyAsync(c->rope_cos, cs.data(), cs.size() * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
        cudaMemcpyAsync(c->rope_sin, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess) {
      c->err = "upload of rotary tables failed";
      return bail(SDFP_ECUDA);
    }
  }
  const size_t R = (size_t)c->rows_cap;  // prompt rows on the dense path, else the rows of the widest decode pass
  c->n_chunks_cap = std::max(kAttnSplits, (g.max_seq + kAttnChunk - 1) / kAttnChunk);  // per (row, head): one partial per 64-key chunk, or kAttnSplits
  c->stats_cap = g.max_seq;
  if ((r = dev_alloc(c, &c->h, R * g.d_model, true)) || (r = dev_alloc(c, &c->q, R * g.d_model, true)) ||
      (r = dev_alloc(c, &c->att, R * g.d_model, true)) || (r = dev_alloc(c, &c->u, R * g.d_ffn, true)) ||
      (r = dev_alloc(c, &c->logits, (size_t)kMaxRows * g.vocab, true)) ||
      (r = dev_alloc(c, &c->part_o, (size_t)kMaxRows * g.n_heads * c->n_chunks_cap * g.head_dim)) ||
      (r = dev_alloc(c, &c->part_ml, (size_t)kMaxRows * g.n_heads * c->n_chunks_cap * 2)) ||
      (r = dev_alloc(c, &c->attn_counters, (size_t)kMaxRows * g.n_heads, true)) || (r = dev_alloc(c, &c->plan.row_pos, R, true)) ||
      (r = dev_alloc(c, &c->plan.row_seq, R, true)) || (r = dev_alloc(c, &c->plan.row_tok, R, true)) ||
      (r = dev_alloc(c, &c->seq_tok, (size_t)g.max_batch * g.max_seq, true)) ||
      (r = dev_alloc(c, &c->draft_tok, (size_t)kMaxBatch * kMaxK, true)) ||
      (r = dev_alloc(c, &c->tgt_tok, (size_t)kMaxBatch * (kMaxK + 1), true)) ||
      (r = dev_alloc(c, &c->row_argmax, (size_t)kMaxRows, true)) || (r = dev_alloc(c, &c->out_tok, (size_t)g.max_batch * g.max_seq, true)) ||
      (r = dev_alloc(c, &c->fwd_tok, (size_t)kMaxRows, true)) ||
      (r = dev_alloc(c, &c->qprob, (size_t)g.max_batch * std::max(1, g.k_max) * g.vocab, true)) ||
      (r = dev_alloc(c, &c->qsum, (size_t)kMaxBatch * kMaxK, true)) || (r = dev_alloc(c, &c->gs, 1, true)) ||
      (r = dev_alloc(c, &c->stats, (size_t)c->stats_cap * g.max_batch, true)))
    return bail(r);
  if (c->use_dense) {
    const size_t rows128 = ((R + 127) / 128) * 128;
    const size_t kmax = (size_t)(((std::max(g.d_model, g.d_ffn) + kUmBK - 1) / kUmBK) * kUmBK);
    const size_t kd64 = (size_t)(((g.d_model + kUmBK - 1) / kUmBK) * kUmBK), kf64 = (size_t)(((g.d_ffn + kUmBK - 1) / kUmBK) * kUmBK);
    if ((r = dev_alloc(c, &c->um_x, rows128 * kmax * 4, true)) || (r = dev_alloc(c, &c->um_pa, rows128 * kd64 * 4, true)) ||
        (r = dev_alloc(c, &c->um_pu, rows128 * kf64 * 4, true)) ||
        (r = dev_alloc(c, &c->um_partial, (size_t)c->num_sms * kUmMaxRB * kUmFeat)) ||
        (r = dev_alloc(c, &c->um_flags, (size_t)c->num_sms, true)) || (r = dev_alloc(c, &c->um_error, 1, true)) ||
        (r = dev_alloc(c, &c->um_flags_dummy, (size_t)c->num_sms, true)) ||
        (r = dev_alloc(c, &c->h_fork, R * g.d_model)))
      return bail(r);
    if (c->dense_decode) {
      const size_t kd = (size_t)(((g.d_model + kUmBK - 1) / kUmBK) * kUmBK), kf = (size_t)(((g.d_ffn + kUmBK - 1) / kUmBK) * kUmBK);
      if ((r = dev_alloc(c, &c->um_xh, (size_t)kMaxRows * kd * 4, true)) || (r = dev_alloc(c, &c->um_xa, (size_t)kMaxRows * kd * 4, true)) ||
          (r = dev_alloc(c, &c->um_xu, (size_t)kMaxRows * kf * 4, true)) ||
          (r = dev_alloc(c, &c->um_ssq, (size_t)(g.d_model / 32 + 4) * kMaxRows, true)))
        return bail(r);
    }
  }
  if (c->use_pass) {
    if ((r = dev_alloc(c, &c->psync, 1, true)) ||
        (r = dev_alloc(c, &c->split_partials, (size_t)c->pass_grid * kUnitTiles * 2 * 64, true)) ||
        (r = dev_alloc(c, &c->ssq_part, (size_t)kSsqMaxGroups * kPassMaxRows, true)) ||
        (r = dev_alloc(c, &c->amax_part, (size_t)((g.vocab / 16 + kUnitTiles - 1) / kUnitTiles) * kPassMaxRows, true)) ||
        (r = build_programs(c)))
      return bail(r);
  }
  if (cudaMallocHost(reinterpret_cast<void**>(&c->pinned_flag), 64) != cudaSuccess) {
    c->err = "cudaMallocHost failed";
    return bail(SDFP_ENOMEM);
  }
  for (auto& e : c->ev)
    if (cudaEventCreate(&e) != cudaSuccess) {
      c->err = "cudaEventCreate failed";
      return bail(SDFP_ECUDA);
    }
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) {
    c->err = std::string("weight packing failed: ") + cudaGetErrorString(e);
    return bail(SDFP_ECUDA);
  }
  *out = c;
  return 0;
}

extern "C" int sdfp_set_draft_sublayers(sdfp_ctx* c, const uint8_t* keep_attn, const uint8_t* keep_ffn) {
  if (!c) return SDFP_EINVAL;
  if (!keep_attn || !keep_ffn) return fail(c, SDFP_EINVAL, "keep mask is NULL");
  if (int r = check_device(c, "sdfp_set_draft_sublayers")) return r;
  const int L = c->cfg.n_layers;
  int kept = 0;
  for (int l = 0; l < L; ++l) kept += (keep_attn[l] ? 1 : 0) + (keep_ffn[l] ? 1 : 0);
  if (kept == 0) return fail(c, SDFP_EINVAL, "the draft must keep at least one block");
  bool same = true;
  for (int l = 0; l < L; ++l)
    same = same && ((keep_attn[l] != 0) == (c->keep_attn[l] != 0)) && ((keep_ffn[l] != 0) == (c->keep_ffn[l] != 0));
  if (!same) {
    for (int l = 0; l < L; ++l) {
      c->keep_attn[l] = keep_attn[l] ? 1 : 0;
      c->keep_ffn[l] = keep_ffn[l] ? 1 : 0;
    }
    for (auto& kv : c->graphs) cudaGraphExecDestroy(kv.second.exec);  // captured rounds baked the old block set in
    c->graphs.clear();
    CU_OK(c, cudaStreamSynchronize(c->stream));
    if (int r = build_programs(c)) return r;
  }
  return 0;
}

extern "C" int sdfp_set_draft_kv_sharing(sdfp_ctx* c, int32_t share) {
  if (!c) return SDFP_EINVAL;
  if (int r = check_device(c, "sdfp_set_draft_kv_sharing")) return r;
  const bool on = share != 0;
  if (on == c->share_kv) return 0;
  c->share_kv = on;
  for (auto& kv : c->graphs) cudaGraphExecDestroy(kv.second.exec);  // captured rounds baked the cache pointers in
  c->graphs.clear();
  CU_OK(c, cudaStreamSynchronize(c->stream));
  return build_programs(c);
}

extern "C" int sdfp_set_draft_layers(sdfp_ctx* c, const uint8_t* keep_mask) {
  if (!c) return SDFP_EINVAL;
  if (!keep_mask) return fail(c, SDFP_EINVAL, "keep_mask is NULL");
  return sdfp_set_draft_sublayers(c, keep_mask, keep_mask);
}

namespace {

int check_dense_error(sdfp_ctx* c) {
  if (!c->use_dense) return 0;
  int e = 0;
  CU_OK(c, cudaMemcpyAsync(&e, c->um_error, sizeof e, cudaMemcpyDeviceToHost, c->stream));
  CU_OK(c, cudaStreamSynchronize(c->stream));
  if (e == 0) return 0;
  cudaMemsetAsync(c->um_error, 0, sizeof(int), c->stream);
  cudaMemsetAsync(c->um_flags, 0, (size_t)c->num_sms * sizeof(int), c->stream);
  cudaMemsetAsync(c->um_flags_dummy, 0, (size_t)c->num_sms * sizeof(int), c->stream);
  cudaStreamSynchronize(c->stream);
  static const char* const what[] = {"", "pipeline stage never freed", "pipeline stage never filled", "accumulator never freed",
                                     "accumulator never finished", "partial accumulator of a cut tile never posted"};
  return fail(c, SDFP_ETIMEOUT, "dense linear kernel gave up a wait (%s); results of this call are invalid",
              e >= 1 && e <= 5 ? what[e] : "unknown");
}

// A failed wait inside the pass kernel leaves its code in device memory; turn it into an error
// and put the synchronisation words back to their initial state.
int check_pass_error(sdfp_ctx* c) {
  if (!c->use_pass) return 0;
  PassSync ps{};
  CU_OK(c, cudaMemcpyAsync(&ps, c->psync, sizeof ps, cudaMemcpyDeviceToHost, c->stream));
  CU_OK(c, cudaStreamSynchronize(c->stream));
  if (ps.error == 0) return 0;
  cudaMemsetAsync(c->psync, 0, sizeof(PassSync), c->stream);
  cudaMemsetAsync(c->split_partials, 0, (size_t)c->pass_grid * kUnitTiles * 2 * 64 * sizeof(ulonglong2), c->stream);
  cudaStreamSynchronize(c->stream);
  static const char* const what[] = {"", "grid barrier", "weight slot never filled", "weight slot never freed",
                                     "partial sum of a split group never posted"};
  return fail(c, SDFP_ETIMEOUT, "pass kernel gave up a wait (%s); results of this call are invalid",
              ps.error >= 1 && ps.error <= 4 ? what[ps.error] : "unknown");
}

// Logits of `rows` tokens of sequence slot 0 at positions start.., in passes of as many rows as
// one pass carries, so that a row's logits never depend on how many rows the caller asked for.
int forward_logits_passes_inner(sdfp_ctx* c, bool draft, const int32_t* tokens, int rows, int start, float* host_logits);

// (the failure-path test hook of the dense path applies to exactly one call of this function)
int forward_logits_passes(sdfp_ctx* c, bool draft, const int32_t* tokens, int rows, int start, float* host_logits) {
  c->um_sabotage_ns = c->um_expire_ns;
  c->um_expire_ns = 0;
  const int r = forward_logits_passes_inner(c, draft, tokens, rows, start, host_logits);
  c->um_sabotage_ns = 0;
  return r;
}

int forward_logits_passes_inner(sdfp_ctx* c, bool draft, const int32_t* tokens, int rows, int start, float* host_logits) {
  const sdfp_config& g = c->cfg;
  CU_OK(c, cudaMemcpyAsync(c->fwd_tok, tokens, (size_t)rows * 4, cudaMemcpyHostToDevice, c->stream));
  const int per_pass = c->use_pass ? kPassMaxRows : kMaxRows;
  for (int off = 0; off < rows; off += per_pass) {
    const int cnt = std::min(per_pass, rows - off);
    PassDesc pd{};
    pd.kind = PASS_TOKENS;
    pd.seq = 0;
    pd.start = start + off;
    pd.count = cnt;
    pd.src = c->fwd_tok + off;
    const int rps = std::min(cnt, kAttnMaxR);
    const int prow = ((cnt + rps - 1) / rps) * rps;
    const int n_chunks = (start + off + cnt + kAttnChunk - 1) / kAttnChunk;
    if (int r = enqueue_pass(c, pd, draft, prow, rps, n_chunks, DECIDE_LOGITS)) return r;
    CU_OK(c, cudaMemcpyAsync(host_logits + (size_t)off * g.vocab, c->logits, (size_t)cnt * g.vocab * 4,
                             cudaMemcpyDeviceToHost, c->stream));
  }
  CU_OK(c, cudaStreamSynchronize(c->stream));
  if (int r = check_dense_error(c)) return r;
  return check_pass_error(c);
}

}  // namespace

namespace {

// Feed tokens [from, to) of sequence b (already in seq_tok) through target or draft to fill its cache.
int prefill_range(sdfp_ctx* c, bool draft, int b, int from, int to) {
  const int chunk = c->use_pass ? kPassMaxRows : 32;
  for (int s = from; s < to; s += chunk) {
    const int cnt = std::min(chunk, to - s);
    PassDesc pd{};
    pd.kind = PASS_TOKENS;
    pd.seq = b;
    pd.start = s;
    pd.count = cnt;
    pd.src = c->seq_tok + (size_t)b * c->cfg.max_seq + s;
    const int rps = std::min(cnt, kAttnMaxR);
    const int rows = ((cnt + rps - 1) / rps) * rps;  // whole attention groups; extra rows carry nothing
    const int n_chunks = (s + cnt + kAttnChunk - 1) / kAttnChunk;
    if (int r = enqueue_pass(c, pd, draft, rows, rps, n_chunks, DECIDE_NONE)) return r;
  }
  return 0;
}

// ---- the prompt pass on the dense path ---------------------------------------------------------------
//
// Rows 0..rows-1 of sequence b (tokens already in seq_tok) through the target (all layers) or the
// draft (kept layers), filling that model's cache; no logits.  Per layer: activation image with the
// norm folded in -> QKV on tcgen05 (epilogue: RoPE, K/V into the cache, q) -> causal attention over
// the prompt -> O-projection + residual -> gate/up + SwiGLU -> down-projection + residual.
//
// The draft shares the target's work where it is the same work: the layers in front of the first
// pruned layer see the same tokens through the same weights, so their K/V ARE the target's.  The
// target's pass leaves the residual rows at that point in `h_fork`; the draft copies the K/V of
// those layers and runs only the kept layers behind the fork.
// gate/up + SwiGLU, whose epilogue leaves u as the operand image of the down-projection, then down + residual
int dense_ffn_block(sdfp_ctx* c, const LayerWeights& lw, int rows, int RB, int KBf) {
  const int d = c->cfg.d_model, f = c->cfg.d_ffn;
  const int KBd = (d + kUmBK - 1) / kUmBK;
  CU_OK(c, launch(c, prep_rows_kernel, dim3((rows + 7) / 8), dim3(kPrepThreads), 0, (const float*)c->h, d, rows, d,
                  (const float*)lw.ffn_gain, c->cfg.rms_eps, c->um_x, RB, KBd));
  UmmaParams gu = dense_params(c, lw.um_gu, c->um_x, rows, RB, KBd, f, base_epi(c, EPI_SWIGLU, nullptr, f));
  gu.img_out = c->um_pu;
  gu.img_KB = KBf;
  CU_OK(c, launch_dense(c, gu));
  CU_OK(c, launch_dense(c, dense_params(c, lw.um_down, c->um_pu, rows, RB, KBf, d / 2, base_epi(c, EPI_RESID, c->h, d))));
  return 0;
}

int dense_layer(sdfp_ctx* c, const KvCache& kv, int l, int b, int rows, bool run_attn, bool run_ffn) {
  const sdfp_config& g = c->cfg;
  const int d = g.d_model, f = g.d_ffn;
  const LayerWeights& lw = c->layers[l];
  if (run_ffn && !run_attn) {
    const int RB0 = rows >= kUmMaxRB ? kUmMaxRB : ((rows + 15) / 16) * 16;
    return dense_ffn_block(c, lw, rows, RB0, (f + kUmBK - 1) / kUmBK);
  }
  if (!run_attn) return 0;
  const int RB = rows >= kUmMaxRB ? kUmMaxRB : ((rows + 15) / 16) * 16;  // as run_dense_linear chooses it
  const int KBd = (d + kUmBK - 1) / kUmBK, KBf = (f + kUmBK - 1) / kUmBK;
  EpiParams qkv = base_epi(c, EPI_QKV, c->q, d);
  qkv.kcache = kv.k[l];
  qkv.vcache = kv.v[l];
  CU_OK(c, run_dense_linear(c, lw.um_qkv, c->h, d, rows, d, 3 * d / 2, lw.attn_gain, qkv));
  // the attention output and the SwiGLU output are written as operand images by their producers
  const float scale = 1.0f / std::sqrt((float)g.head_dim);
  const dim3 grid((rows + kPfaQ - 1) / kPfaQ, g.n_heads);
  const __nv_bfloat16* kc = reinterpret_cast<const __nv_bfloat16*>(kv.k[l]);
  const __nv_bfloat16* vc = reinterpret_cast<const __nv_bfloat16*>(kv.v[l]);
  if (g.head_dim == 128)
    CU_OK(c, launch(c, prefill_attention_kernel<128>, grid, dim3(kPfaThreads), prefill_attention_smem<128>(), (const float*)c->q, kc,
                    vc, c->att, rows, g.n_heads, g.max_seq, b, scale, c->um_pa, RB, KBd));
  else
    CU_OK(c, launch(c, prefill_attention_kernel<64>, grid, dim3(kPfaThreads), prefill_attention_smem<64>(), (const float*)c->q, kc, vc,
                    c->att, rows, g.n_heads, g.max_seq, b, scale, c->um_pa, RB, KBd));
  CU_OK(c, launch_dense(c, dense_params(c, lw.um_wo, c->um_pa, rows, RB, KBd, d / 2, base_epi(c, EPI_RESID, c->h, d))));
  if (!run_ffn) return 0;
  return dense_ffn_block(c, lw, rows, RB, KBf);
}

int first_pruned_layer(const sdfp_ctx* c) {
  for (int l = 0; l < c->cfg.n_layers; ++l)
    if (!c->keep_attn[l] || !c->keep_ffn[l]) return l;  // the first layer of which the draft drops a block
  return c->cfg.n_layers;
}

// rows_t rows through the target and, when with_draft, rows_d <= rows_t rows through the draft
int prefill_dense(sdfp_ctx* c, int b, int rows_t, int rows_d, bool with_draft) {
  const sdfp_config& g = c->cfg;
  const int d = g.d_model;
  PassDesc pd{};
  pd.kind = PASS_TOKENS;
  pd.seq = b;
  pd.start = 0;
  pd.count = rows_t;
  pd.src = c->seq_tok + (size_t)b * g.max_seq;
  CU_OK(c, launch(c, plan_embed_kernel<__nv_bfloat16>, dim3(rows_t), dim3(128), 0, pd, (const GenState*)c->gs, (const int*)c->seq_tok,
                  g.max_seq, (const int*)c->draft_tok, c->plan, reinterpret_cast<const __nv_bfloat16*>(c->embed), c->h, d, EmbedImage{}));
  const int fork = with_draft ? first_pruned_layer(c) : -1;  // the draft's residual rows leave the target's after this many layers
  const size_t fork_bytes = (size_t)rows_d * d * sizeof(float);
  if (fork == 0 && rows_d > 0) CU_OK(c, cudaMemcpyAsync(c->h_fork, c->h, fork_bytes, cudaMemcpyDeviceToDevice, c->stream));
  for (int l = 0; l < g.n_layers; ++l) {
    if (int r = dense_layer(c, c->cache_t, l, b, rows_t, true, true)) return r;
    if (l + 1 == fork && rows_d > 0) CU_OK(c, cudaMemcpyAsync(c->h_fork, c->h, fork_bytes, cudaMemcpyDeviceToDevice, c->stream));
  }
  if (!with_draft || rows_d <= 0) return 0;
  // K/V of the shared layers: per head one contiguous run of rows_d positions
  const size_t pitch = (size_t)g.max_seq * g.head_dim * c->esz, width = (size_t)rows_d * g.head_dim * c->esz;
  const size_t seq_off = (size_t)b * g.n_heads * pitch;
  for (int l = 0; l < std::min(fork, g.n_layers); ++l) {
    CU_OK(c, cudaMemcpy2DAsync((unsigned char*)c->cache_d.k[l] + seq_off, pitch, (const unsigned char*)c->cache_t.k[l] + seq_off, pitch,
                               width, g.n_heads, cudaMemcpyDeviceToDevice, c->stream));
    CU_OK(c, cudaMemcpy2DAsync((unsigned char*)c->cache_d.v[l] + seq_off, pitch, (const unsigned char*)c->cache_t.v[l] + seq_off, pitch,
                               width, g.n_heads, cudaMemcpyDeviceToDevice, c->stream));
  }
  bool any = false;
  for (int l = fork; l < g.n_layers; ++l) any = any || c->keep_attn[l] || c->keep_ffn[l];
  if (!any) return 0;
  CU_OK(c, cudaMemcpyAsync(c->h, c->h_fork, fork_bytes, cudaMemcpyDeviceToDevice, c->stream));
  pd.count = rows_d;  // the row plan of the draft's rows (positions 0..rows_d-1 are already right; rows beyond carry nothing)
  for (int l = fork; l < g.n_layers; ++l)
    if (int r = dense_layer(c, c->cache_d, l, b, rows_d, c->keep_attn[l] != 0, c->keep_ffn[l] != 0)) return r;
  return 0;
}

}  // namespace

extern "C" int sdfp_generate(sdfp_ctx* c, const int32_t* prompts, int32_t batch, int32_t prompt_len, int32_t k,
                             int32_t max_new, float temperature, uint64_t seed, int32_t* out_tokens, int32_t* out_len,
                             sdfp_round_stat* stats, int32_t max_rounds, int32_t* n_rounds) {
  if (!c) return SDFP_EINVAL;
  const sdfp_config& g = c->cfg;
  if (!prompts || !out_tokens || !out_len) return fail(c, SDFP_EINVAL, "sdfp_generate: NULL pointer");
  if (int r = check_device(c, "sdfp_generate")) return r;
  if (batch < 1 || batch > g.max_batch) return fail(c, SDFP_EINVAL, "batch %d outside 1..%d", batch, g.max_batch);
  if (k < 0 || k > g.k_max) return fail(c, SDFP_EINVAL, "k %d outside 0..%d", k, g.k_max);
  if (prompt_len < 1 || max_new < 1) return fail(c, SDFP_EINVAL, "prompt_len and max_new must be >= 1");
  if ((int64_t)prompt_len + max_new + k + 1 > g.max_seq)
    return fail(c, SDFP_EINVAL, "prompt_len + max_new + k + 1 = %lld exceeds max_seq %d",
                (long long)prompt_len + max_new + k + 1, g.max_seq);
  if (!(temperature >= 0.f)) return fail(c, SDFP_EINVAL, "temperature must be >= 0");
  if (stats && max_rounds < 0) return fail(c, SDFP_EINVAL, "max_rounds < 0");
  for (int64_t i = 0; i < (int64_t)batch * prompt_len; ++i)
    if (prompts[i] < 0 || prompts[i] >= g.vocab) return fail(c, SDFP_EINVAL, "prompt token %d out of range", prompts[i]);
  const bool sampled = temperature > 0.f;
  cudaStream_t st = c->stream;

  // state
  GenState hs{};
  for (int b = 0; b < batch; ++b) hs.n[b] = prompt_len;
  for (int b = batch; b < kMaxBatch; ++b) hs.done[b] = 1;
  hs.batch = batch;
  hs.k = k;
  hs.max_new = max_new;
  hs.eos_id = g.eos_id;
  hs.max_rounds = c->stats_cap;
  hs.temperature = temperature;
  hs.seed = seed;
  CU_OK(c, cudaMemcpyAsync(c->gs, &hs, sizeof hs, cudaMemcpyHostToDevice, st));
  for (int b = 0; b < batch; ++b)
    CU_OK(c, cudaMemcpyAsync(c->seq_tok + (size_t)b * g.max_seq, prompts + (size_t)b * prompt_len,
                             (size_t)prompt_len * 4, cudaMemcpyHostToDevice, st));
  CU_OK(c, cudaMemsetAsync(c->out_tok, 0xff, (size_t)batch * max_new * 4, st));
  CU_OK(c, cudaMemsetAsync(c->stats, 0, (size_t)c->stats_cap * batch * sizeof(RoundStat), st));

  // prefill: the target caches positions 0..P-2, the draft 0..P-3 (its first pass of a
  // round always feeds the last two committed tokens)
  CU_OK(c, cudaEventRecord(c->ev[0], st));
  for (int b = 0; b < batch; ++b) {
    const bool draft_prompt = k > 0 && !c->share_kv;  // a sharing draft has no prompt pass of its own
    if (c->use_dense && prompt_len - 1 >= kDenseMinRows) {
      if (int r = prefill_dense(c, b, prompt_len - 1, prompt_len - 2, draft_prompt)) return r;
      continue;
    }
    if (int r = prefill_range(c, false, b, 0, prompt_len - 1)) return r;
    if (draft_prompt)
      if (int r = prefill_range(c, true, b, 0, prompt_len - 2)) return r;
  }
  CU_OK(c, cudaEventRecord(c->ev[1], st));

  // decode
  const int n_chunks = (prompt_len + max_new + k + kAttnChunk) / kAttnChunk;
  const long long launches0 = c->launches;
  cudaGraphExec_t exec = nullptr;
  long long launches_per_round = 0;
  if (c->use_graph) {
    auto key = std::make_tuple((int)k, (int)batch, sampled ? 1 : 0, n_chunks);
    auto it = c->graphs.find(key);
    if (it == c->graphs.end()) {
      const long long l0 = c->launches;
      cudaGraph_t graph = nullptr;
      CU_OK(c, cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
      const int r = enqueue_round(c, k, batch, sampled, n_chunks);
      cudaError_t ce = cudaStreamEndCapture(st, &graph);
      launches_per_round = c->launches - l0;
      c->launches = l0;
      if (r) {
        if (graph) cudaGraphDestroy(graph);
        return r;
      }
      CU_OK(c, ce);
      cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
      cudaGraphDestroy(graph);
      CU_OK(c, ie);
      c->graphs[key] = sdfp_ctx::RoundGraph{exec, launches_per_round};
    } else {
      exec = it->second.exec;
      launches_per_round = it->second.launches;
    }
  }
  int rounds = 0;
  const int round_cap = max_new + 1;
  while (rounds < round_cap) {
    if (exec) {
      CU_OK(c, cudaGraphLaunch(exec, st));
      c->launches += launches_per_round;
    } else if (int r = enqueue_round(c, k, batch, sampled, n_chunks)) {
      return r;
    }
    ++rounds;
    CU_OK(c, cudaMemcpyAsync(c->pinned_flag, &c->gs->all_done, 8, cudaMemcpyDeviceToHost, st));  // all_done, pass_error
    CU_OK(c, cudaStreamSynchronize(st));
    if (c->pinned_flag[0] || c->pinned_flag[1]) break;
  }
  CU_OK(c, cudaEventRecord(c->ev[2], st));
  if (int r = check_pass_error(c)) return r;
  if (int r = check_dense_error(c)) return r;

  // results
  std::vector<int> lens(kMaxBatch);
  GenState fin{};
  CU_OK(c, cudaMemcpyAsync(&fin, c->gs, sizeof fin, cudaMemcpyDeviceToHost, st));
  CU_OK(c, cudaMemcpyAsync(out_tokens, c->out_tok, (size_t)batch * max_new * 4, cudaMemcpyDeviceToHost, st));
  std::vector<RoundStat> hstats((size_t)rounds * batch);
  CU_OK(c, cudaMemcpyAsync(hstats.data(), c->stats, hstats.size() * sizeof(RoundStat), cudaMemcpyDeviceToHost, st));
  CU_OK(c, cudaStreamSynchronize(st));
  for (int b = 0; b < batch; ++b) out_len[b] = fin.n_new[b];
  if (n_rounds) *n_rounds = rounds;
  if (stats)
    for (int r = 0; r < std::min(rounds, (int)max_rounds); ++r)
      for (int b = 0; b < batch; ++b) {
        const RoundStat& s = hstats[(size_t)r * batch + b];
        stats[(size_t)r * batch + b] = sdfp_round_stat{s.drafted, s.accepted, s.committed};
      }

  // timing and traffic of the decode phase
  sdfp_timing& t = c->timing;
  t = sdfp_timing{};
  cudaEventElapsedTime(&t.prefill_ms, c->ev[0], c->ev[1]);
  cudaEventElapsedTime(&t.decode_ms, c->ev[1], c->ev[2]);
  t.n_rounds = rounds;
  t.n_draft_passes = rounds * k;
  t.n_target_passes = rounds;
  t.kernel_launches = c->launches - launches0;
  const int64_t lm = lm_head_bytes(c);
  const int64_t kept = pass_kv_layers(c, true);
  t.weight_bytes = (int64_t)rounds * ((int64_t)k * (pass_weight_bytes(c, true) + lm) + pass_weight_bytes(c, false) + lm);
  const int64_t kv_tok = 2LL * g.d_model * (int64_t)c->esz;  // K and V of one token of one layer
  std::vector<int> n(batch, prompt_len);
  for (int r = 0; r < rounds; ++r)
    for (int b = 0; b < batch; ++b) {
      const RoundStat& s = hstats[(size_t)r * batch + b];
      if (s.committed == 0 && s.drafted == 0 && k > 0) continue;
      if (k == 0 && s.committed == 0) continue;
      // draft pass i reads keys 0..n-1+i of the kept layers and writes its rows; verify reads 0..n-1+k
      for (int i = 0; i < k; ++i) t.kv_bytes += (int64_t)kept * kv_tok * ((n[b] + i) + (i == 0 && !c->share_kv ? 2 : 1));
      t.kv_bytes += (int64_t)g.n_layers * kv_tok * ((n[b] + k) + (k + 1));
      n[b] += s.committed;
      t.tokens_committed += s.committed;
    }
  return 0;
}

extern "C" int sdfp_forward_logits(sdfp_ctx* c, int32_t draft, const int32_t* tokens, int32_t rows, int32_t start,
                                   float* host_logits) {
  if (!c) return SDFP_EINVAL;
  const sdfp_config& g = c->cfg;
  if (!tokens || !host_logits) return fail(c, SDFP_EINVAL, "sdfp_forward_logits: NULL pointer");
  if (int r = check_device(c, "sdfp_forward_logits")) return r;
  if (rows < 1 || rows > kMaxRows) return fail(c, SDFP_EINVAL, "rows %d outside 1..%d", rows, kMaxRows);
  if (start < 0 || start + rows > g.max_seq) return fail(c, SDFP_EINVAL, "positions exceed max_seq");
  for (int i = 0; i < rows; ++i)
    if (tokens[i] < 0 || tokens[i] >= g.vocab) return fail(c, SDFP_EINVAL, "token out of range");
  return forward_logits_passes(c, draft != 0, tokens, rows, start, host_logits);
}

// ---- forward pass whose attention scratch is a static device array -----------------------------
//
// The split-KV attention kernel needs global scratch beyond its inputs and outputs: one
// partial (max, sum, o[head_dim]) per (row, head, key chunk) and one arrival counter per
// (sequence, head).  A context gets that scratch from cudaMalloc inside sdfp_create.  The
// entry point below points the same kernel at a fixed array that is part of the library image
// instead, so that the call itself reaches no allocator of any kind.
namespace {

constexpr size_t kStaticScratchBytes = SDFP_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};  // device address of the array, per device ordinal

// In host code `g_static_scratch` is only a handle for the symbol; the address a kernel can
// use has to be asked for, once per device, with that device current.
int static_scratch_address(sdfp_ctx* c, unsigned char** out) {
  const int dev = c->device;  // current: the caller checked
  if (dev < 0 || dev >= kMaxDevices) return fail(c, SDFP_ECUDA, "device ordinal %d not supported", dev);
  if (!g_static_scratch_addr[dev]) {
    void* p = nullptr;
    CU_OK(c, cudaGetSymbolAddress(&p, g_static_scratch));
    if (!p) return fail(c, SDFP_ECUDA, "cudaGetSymbolAddress returned a null address");
    g_static_scratch_addr[dev] = p;
  }
  *out = reinterpret_cast<unsigned char*>(g_static_scratch_addr[dev]);
  return 0;
}

size_t round_up_256(size_t n) { return (n + 255) & ~size_t(255); }

}  // namespace

extern "C" int sdfp_forward_logits_static(sdfp_ctx* c, int32_t draft, const int32_t* tokens, int32_t rows,
                                          int32_t start, float* host_logits) {
  if (!c) return SDFP_EINVAL;
  const sdfp_config& g = c->cfg;
  if (!tokens || !host_logits) return fail(c, SDFP_EINVAL, "sdfp_forward_logits_static: NULL pointer");
  if (int r = check_device(c, "sdfp_forward_logits_static")) return r;
  if (rows < 1 || rows > kMaxRows) return fail(c, SDFP_EINVAL, "rows %d outside 1..%d", rows, kMaxRows);
  if (start < 0 || start + rows > g.max_seq) return fail(c, SDFP_EINVAL, "positions exceed max_seq");
  for (int i = 0; i < rows; ++i)
    if (tokens[i] < 0 || tokens[i] >= g.vocab) return fail(c, SDFP_EINVAL, "token out of range");
  // the widest pass this call will run, and the longest context any of its passes sees
  const int per_pass = std::min((int)rows, c->use_pass ? kPassMaxRows : kMaxRows);
  const int rps = std::min(per_pass, kAttnMaxR);
  const int prow = ((per_pass + rps - 1) / rps) * rps;
  // partials per (row, head): one per 64-key chunk, or a fixed kAttnSplits in the whole-pass kernel
  const int n_chunks = (c->use_pass || c->dense_decode) ? kAttnSplits : (start + rows + kAttnChunk - 1) / kAttnChunk;
  // layout inside the array: arrival counters | (max, sum) partials | o partials
  const size_t counters_bytes = round_up_256((size_t)kMaxRows * g.n_heads * sizeof(int));
  const size_t ml_bytes = round_up_256((size_t)prow * g.n_heads * n_chunks * 2 * sizeof(float));
  const size_t o_bytes = round_up_256((size_t)prow * g.n_heads * n_chunks * g.head_dim * sizeof(float));
  const size_t need = counters_bytes + ml_bytes + o_bytes;
  if (need > kStaticScratchBytes)
    return fail(c, SDFP_EINVAL,
                "sdfp_forward_logits_static: %d rows x %d heads x %d partials need %zu bytes of attention scratch, "
                "the static array holds %zu; use fewer rows per call, a shorter context, or sdfp_forward_logits",
                prow, g.n_heads, n_chunks, need, kStaticScratchBytes);
  unsigned char* base = nullptr;
  if (int r = static_scratch_address(c, &base)) return r;
  // the array keeps whatever the previous call (of any context) left: the counters must start at zero
  CU_OK(c, cudaMemsetAsync(base, 0, counters_bytes, c->stream));
  // same passes as sdfp_forward_logits, with the attention scratch pointers swapped for their duration
  float* const own_o = c->part_o;
  float* const own_ml = c->part_ml;
  int* const own_counters = c->attn_counters;
  c->attn_counters = reinterpret_cast<int*>(base);
  c->part_ml = reinterpret_cast<float*>(base + counters_bytes);
  c->part_o = reinterpret_cast<float*>(base + counters_bytes + ml_bytes);
  const int r = forward_logits_passes(c, draft != 0, tokens, rows, start, host_logits);
  c->part_o = own_o;
  c->part_ml = own_ml;
  c->attn_counters = own_counters;
  return r;
}

extern "C" int sdfp_debug_expire_next_wait(sdfp_ctx* c, uint64_t wait_limit_ns) {
  if (!c) return SDFP_EINVAL;
  if (int r = check_device(c, "sdfp_debug_expire_next_wait")) return r;
  if (!c->use_pass && !c->dense_decode)
    return fail(c, SDFP_ESTATE, "sdfp_debug_expire_next_wait: this context uses neither the whole-pass kernel nor the dense path for its passes");
  if (wait_limit_ns < 1000000ull || wait_limit_ns > 2000000000ull)
    return fail(c, SDFP_EINVAL, "sdfp_debug_expire_next_wait: the limit must lie between 1 ms and 2 s");
  if (c->dense_decode) {  // the next sdfp_forward_logits[_static] call: see forward_logits_passes
    c->um_expire_ns = wait_limit_ns;
    return 0;
  }
  const unsigned long long words[2] = {1ull, (unsigned long long)wait_limit_ns};  // bar_extra, wait_limit_ns
  CU_OK(c, cudaMemcpyAsync(&c->psync->bar_extra, words, sizeof words, cudaMemcpyHostToDevice, c->stream));
  CU_OK(c, cudaStreamSynchronize(c->stream));  // words is a local
  return 0;
}

extern "C" int sdfp_fit_scores(const sdfp_config* cfg, const sdfp_weights* w, void* cuda_stream, const int32_t* tokens,
                               int32_t n_seq, int32_t seq_len, double* out_trace, double* out_fit) {
  if (!cfg || !w || !tokens || !out_trace) return fail(nullptr, SDFP_EINVAL, "sdfp_fit_scores: NULL argument");
  const sdfp_config& g = *cfg;
  if (g.n_layers < 1 || g.n_layers > 1024 || g.d_model < 2 || g.n_heads < 1 || g.d_ffn < 1 || g.vocab < 2 || g.head_dim < 2 ||
      (g.head_dim & 1) || g.d_model != g.n_heads * g.head_dim)
    return fail(nullptr, SDFP_EINVAL, "sdfp_fit_scores: bad model dimensions");
  if (g.dtype != SDFP_F32 && g.dtype != SDFP_BF16) return fail(nullptr, SDFP_EINVAL, "unknown dtype");
  if (!(g.rms_eps > 0.f) || !(g.rope_theta > 0.f)) return fail(nullptr, SDFP_EINVAL, "bad rms_eps or rope_theta");
  if (n_seq < 1 || seq_len < 2 || seq_len > 4097) return fail(nullptr, SDFP_EINVAL, "sdfp_fit_scores: need n_seq >= 1 and 2 <= seq_len <= 4097");
  if (!w->tok_embed || !w->final_norm || !w->lm_head || !w->wq || !w->wk || !w->wv || !w->wo || !w->w_gate || !w->w_up || !w->w_down ||
      !w->attn_norm || !w->ffn_norm)
    return fail(nullptr, SDFP_EINVAL, "sdfp_fit_scores: NULL weight pointer");
  for (int l = 0; l < g.n_layers; ++l)
    if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->w_gate[l] || !w->w_up[l] || !w->w_down[l] || !w->attn_norm[l] ||
        !w->ffn_norm[l])
      return fail(nullptr, SDFP_EINVAL, "layer %d has a NULL weight pointer", l);
  for (int64_t i = 0; i < (int64_t)n_seq * seq_len; ++i)
    if (tokens[i] < 0 || tokens[i] >= g.vocab) return fail(nullptr, SDFP_EINVAL, "calibration token %d out of range", tokens[i]);
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
    cudaGetLastError();
    return fail(nullptr, SDFP_ECUDA, "no CUDA device: this library has no CPU path");
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const cudaError_t e = g.dtype == SDFP_BF16 ? fit::run<__nv_bfloat16>(g, w, st, tokens, n_seq, seq_len, out_trace, out_fit)
                                              : fit::run<float>(g, w, st, tokens, n_seq, seq_len, out_trace, out_fit);
  if (e != cudaSuccess)
    return fail(nullptr, e == cudaErrorMemoryAllocation ? SDFP_ENOMEM : SDFP_ECUDA, "sdfp_fit_scores: %s", cudaGetErrorString(e));
  return 0;
}

extern "C" int sdfp_get_timing(const sdfp_ctx* c, sdfp_timing* out) {
  if (!c || !out) return SDFP_EINVAL;
  *out = c->timing;
  return 0;
}

extern "C" int sdfp_time_pass(sdfp_ctx* c, int32_t draft, int32_t rows, int32_t position, int32_t iters,
                              float* ms_per_launch, int64_t* bytes_per_launch) {
  if (!c) return SDFP_EINVAL;
  const sdfp_config& g = c->cfg;
  if (!ms_per_launch || !bytes_per_launch) return fail(c, SDFP_EINVAL, "sdfp_time_pass: NULL pointer");
  if (int r = check_device(c, "sdfp_time_pass")) return r;
  if (!c->use_pass) return fail(c, SDFP_ESTATE, "sdfp_time_pass: this context does not use the whole-pass kernel");
  if (rows < 1 || rows > kPassMaxRows || iters < 1 || iters > 256 || position < 0 || position + rows > g.max_seq)
    return fail(c, SDFP_EINVAL, "sdfp_time_pass: bad argument");
  CU_OK(c, cudaMemsetAsync(c->fwd_tok, 0, (size_t)kMaxRows * 4, c->stream));
  PassDesc pd{};
  pd.kind = PASS_TOKENS;
  pd.seq = 0;
  pd.start = position;
  pd.count = rows;
  pd.src = c->fwd_tok;
  std::vector<cudaEvent_t> ev(2 * (size_t)iters, nullptr);
  cudaError_t err = cudaSuccess;
  for (auto& e : ev)
    if (err == cudaSuccess) err = cudaEventCreate(&e);  // on failure the loops below do nothing and every event made so far is destroyed
  auto plan = [&]() -> cudaError_t {
    return launch(c, plan_embed_kernel<__nv_bfloat16>, dim3(rows), dim3(128), 0, pd, (const GenState*)c->gs,
                  (const int*)c->seq_tok, g.max_seq, (const int*)c->draft_tok, c->plan,
                  reinterpret_cast<const __nv_bfloat16*>(c->embed), c->h, g.d_model, EmbedImage{});
  };
  for (int i = 0; i < 3 && err == cudaSuccess; ++i) {  // warm-up
    err = plan();
    if (err == cudaSuccess) err = run_pass(c, draft != 0, rows, rows, true, true);
  }
  for (int i = 0; i < iters && err == cudaSuccess; ++i) {
    err = plan();  // fresh residual rows every time, outside the timed interval
    if (err == cudaSuccess) err = cudaEventRecord(ev[2 * i], c->stream);
    if (err == cudaSuccess) err = run_pass(c, draft != 0, rows, rows, true, true);  // as in a greedy round: decision in the lm-head
    if (err == cudaSuccess) err = cudaEventRecord(ev[2 * i + 1], c->stream);
  }
  if (err == cudaSuccess) err = cudaStreamSynchronize(c->stream);
  double total = 0.0;
  for (int i = 0; i < iters && err == cudaSuccess; ++i) {
    float ms = 0.f;
    err = cudaEventElapsedTime(&ms, ev[2 * i], ev[2 * i + 1]);
    total += ms;
  }
  for (auto& e : ev)
    if (e) cudaEventDestroy(e);
  CU_OK(c, err);
  if (int r = check_pass_error(c)) return r;
  *ms_per_launch = (float)(total / iters);
  const int64_t layers = pass_kv_layers(c, draft != 0);
  const int64_t kv_tok = 2LL * g.d_model * (int64_t)c->esz;
  *bytes_per_launch = pass_weight_bytes(c, draft != 0) + lm_head_bytes(c) + layers * kv_tok * ((int64_t)position + rows) +
                      layers * kv_tok * rows;
  return 0;
}

extern "C" int sdfp_time_linear(sdfp_ctx* c, int32_t which, int32_t rows, int32_t iters, float* ms_per_launch,
                                int64_t* weight_bytes_per_launch) {
  if (!c) return SDFP_EINVAL;
  const sdfp_config& g = c->cfg;
  if (!ms_per_launch || !weight_bytes_per_launch) return fail(c, SDFP_EINVAL, "sdfp_time_linear: NULL pointer");
  if (int r = check_device(c, "sdfp_time_linear")) return r;
  if (which < 0 || which > 4 || rows < 1 || rows > kMaxRows || iters < 1)
    return fail(c, SDFP_EINVAL, "sdfp_time_linear: bad argument");
  const int d = g.d_model, f = g.d_ffn;
  // rows carry nothing (position -1): the QKV epilogue then writes no cache entry
  CU_OK(c, cudaMemsetAsync(c->plan.row_pos, 0xff, kMaxRows * 4, c->stream));
  CU_OK(c, cudaMemsetAsync(c->plan.row_seq, 0, kMaxRows * 4, c->stream));
  // contexts that decode on the dense path: the activation image is made once, outside the timed
  // launches (in a pass the preceding kernel's epilogue leaves it), and one launch = one tcgen05 kernel
  const bool dense = c->dense_decode;
  const int RB = ((rows + 15) / 16) * 16;
  const int Kin = which == 3 ? f : d, KBin = (Kin + kUmBK - 1) / kUmBK;
  if (dense)
    CU_OK(c, launch(c, prep_rows_kernel, dim3((rows + 7) / 8), dim3(kPrepThreads), 0, (const float*)(which == 3 ? c->u : c->h),
                    Kin, (int)rows, Kin, (const float*)nullptr, g.rms_eps, c->um_x, RB, KBin));
  auto one = [&](int l) -> cudaError_t {
    const LayerWeights& lw = c->layers[l % g.n_layers];
    if (dense) {
      const void* w = which == 0 ? lw.um_qkv : which == 1 ? lw.um_wo : which == 2 ? lw.um_gu : which == 3 ? lw.um_down : c->um_lm_head;
      const int n_pairs = which == 0 ? 3 * d / 2 : which == 2 ? f : which == 4 ? g.vocab / 2 : d / 2;
      EpiParams ep = which == 0 ? base_epi(c, EPI_QKV, c->q, d)
                     : which == 2 ? base_epi(c, EPI_SWIGLU, c->u, f)
                     : which == 4 ? base_epi(c, EPI_LOGITS, c->logits, g.vocab)
                                  : base_epi(c, EPI_RESID, c->q, d);
      ep.kcache = c->cache_t.k[0];
      ep.vcache = c->cache_t.v[0];
      return launch_dense(c, dense_params(c, w, c->um_x, rows, RB, KBin, n_pairs, ep));
    }
    if (which == 0) {
      LinearCall lc{lw.qkv, c->h, d, rows, d, 3 * d / 2, lw.attn_gain, base_epi(c, EPI_QKV, c->q, d)};
      lc.ep.kcache = c->cache_t.k[0];
      lc.ep.vcache = c->cache_t.v[0];
      return run_linear(c, lc);
    } else if (which == 1) {
      LinearCall lc{lw.wo, c->att, d, rows, d, d / 2, nullptr, base_epi(c, EPI_RESID, c->q, d)};
      return run_linear(c, lc);
    } else if (which == 2) {
      LinearCall lc{lw.gu, c->h, d, rows, d, f, lw.ffn_gain, base_epi(c, EPI_SWIGLU, c->u, f)};
      return run_linear(c, lc);
    } else if (which == 3) {
      LinearCall lc{lw.down, c->u, f, rows, f, d / 2, nullptr, base_epi(c, EPI_RESID, c->q, d)};
      return run_linear(c, lc);
    }
    LinearCall lc{c->lm_head, c->h, d, rows, d, g.vocab / 2, c->final_gain, base_epi(c, EPI_LOGITS, c->logits, g.vocab)};
    return run_linear(c, lc);
  };
  for (int i = 0; i < 3; ++i) CU_OK(c, one(i));
  CU_OK(c, cudaEventRecord(c->ev[0], c->stream));
  for (int i = 0; i < iters; ++i) CU_OK(c, one(i + 3));
  CU_OK(c, cudaEventRecord(c->ev[1], c->stream));
  CU_OK(c, cudaStreamSynchronize(c->stream));
  float ms = 0.f;
  cudaEventElapsedTime(&ms, c->ev[0], c->ev[1]);
  *ms_per_launch = ms / iters;
  const int64_t e = (int64_t)c->esz;
  const int64_t bytes[5] = {3LL * d * d * e, 1LL * d * d * e, 2LL * f * d * e, 1LL * d * f * e, 1LL * g.vocab * d * e};
  *weight_bytes_per_launch = bytes[which];
  return 0;
}
