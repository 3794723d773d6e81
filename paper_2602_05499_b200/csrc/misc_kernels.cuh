// Small kernels around the linear and attention kernels: row planning + embedding
// gather, argmax over the vocabulary, greedy accept/commit (Algorithm 1, loop body).
#pragma once

#include "common.cuh"

namespace sdfp {

constexpr int kMaxBatch = 16;
constexpr int kMaxK = 15;

// Device-resident generation state: a round never needs the host.
struct GenState {
  int n[kMaxBatch];      // committed length (prompt + generated) per sequence
  int n_new[kMaxBatch];  // generated so far
  int done[kMaxBatch];
  int round;
  int all_done;
  int pass_error;  // directly after all_done: the host reads both with one copy per round
  // parameters of the running sdfp_generate call
  int batch, k, max_new, eos_id, max_rounds;
  float temperature;
  unsigned long long seed;
};

enum PassKind {
  PASS_TOKENS = 0,       // rows r = 0..count-1 of one sequence: token src[r], position start + r
  PASS_DRAFT_FIRST = 1,  // rows_per_seq (2, or 1 when the draft shares the target's cache) rows per sequence: the last committed tokens
  PASS_DRAFT_NEXT = 2,   // 1 row per sequence: draft token number `step` (1-based step >= 1)
  PASS_VERIFY = 3        // k+1 rows per sequence: last committed token, then the k drafts
};

struct PassDesc {
  int kind, step, rows_per_seq, n_seq;
  int seq, start, count;  // PASS_TOKENS
  const int* src;         // PASS_TOKENS: device token ids
  // Greedy decision fused into the lm-head (whole-pass kernel): the previous pass left, per row and
  // per 128-feature group of the vocabulary, the largest logit and its index; the kernel that needs
  // the token finishes the argmax.  prev_rows_per_seq = rows per sequence of that previous pass
  // (0: tokens come from draft_tok / tgt_tok as written by argmax_kernel).
  int prev_rows_per_seq;
  const int2* amax_part;  // [group][kAmaxRows] (float bits, index)
  int amax_groups;
};

constexpr int kAmaxRows = 16;  // rows per group in the partial-argmax array (the whole-pass kernel's row capacity)

// Largest logit of row `row` over all groups, ties to the lowest index; one warp, every lane gets the result.
__device__ __forceinline__ int amax_finish(const int2* part, int n_groups, int row) {
  const int lane = threadIdx.x & 31;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int g = lane; g < n_groups; g += 32) {
    const int2 v = __ldcg(part + (size_t)g * kAmaxRows + row);
    const float x = __int_as_float(v.x);
    if (x > best || (x == best && v.y < bi)) {
      best = x;
      bi = v.y;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ob > best || (ob == best && oi < bi)) {
      best = ob;
      bi = oi;
    }
  }
  return bi;
}

struct RowPlan {
  int* row_pos;  // [kMaxRows]
  int* row_seq;
  int* row_tok;
};

// Dense path: the embedding rows also go out as the activation image of the first linear layer
// (gain * h as bf16 hi + lo, layout of umma_linear.cuh) together with each row's sum of squares.
struct EmbedImage {
  unsigned char* img;  // null: none
  const float* gain;
  float* ssq;          // [rows]
  int rb, kb;
};

// One CTA per row: decide which token sits in the row and where, then gather its
// embedding into the residual stream h[row, :].
template <typename WT>
__global__ void __launch_bounds__(128)
plan_embed_kernel(PassDesc pd, const GenState* gs, const int* seq_tok, int max_seq,
                  const int* draft_tok, RowPlan plan, const WT* __restrict__ embed, float* __restrict__ h,
                  int d_model, EmbedImage im) {
  __shared__ int s_tok, s_pos;
  __shared__ float s_sq[128];
  pdl_wait();
  pdl_launch_dependents();
  const int m = blockIdx.x;
  // a draft token the previous pass decided but nobody has written down yet (fused argmax)
  int pending = -1;
  if (pd.prev_rows_per_seq > 0 && threadIdx.x < 32) {
    const int R = pd.rows_per_seq;
    const int b = m / R, i = m - b * R;
    const bool mine = (pd.kind == PASS_DRAFT_NEXT) || (pd.kind == PASS_VERIFY && R > 1 && i == R - 1);
    if (mine && !ld_act(&gs->done[b])) {
      const int pr = pd.prev_rows_per_seq;
      pending = amax_finish(pd.amax_part, pd.amax_groups, b * pr + pr - 1);
      const int slot = (pd.kind == PASS_DRAFT_NEXT) ? pd.step - 1 : R - 2;
      if (threadIdx.x == 0) const_cast<int*>(draft_tok)[b * kMaxK + slot] = pending;
    }
  }
  if (threadIdx.x == 0) {
    int tok = 0, pos = -1, seq = 0;
    if (pd.kind == PASS_TOKENS) {
      seq = pd.seq;
      if (m < pd.count) {
        tok = ld_act(pd.src + m);
        pos = pd.start + m;
      }
    } else {
      const int R = pd.rows_per_seq;
      const int b = m / R, i = m - b * R;
      seq = b;
      if (!ld_act(&gs->done[b])) {
        const int n = ld_act(&gs->n[b]);
        if (pd.kind == PASS_DRAFT_FIRST) {
          pos = n - R + i;
          if (pos >= 0) tok = ld_act(seq_tok + (size_t)b * max_seq + pos);
        } else if (pd.kind == PASS_DRAFT_NEXT) {
          pos = n - 1 + pd.step;
          tok = pending >= 0 ? pending : ld_act(draft_tok + b * kMaxK + pd.step - 1);
        } else {
          pos = n - 1 + i;
          tok = (i == 0) ? ld_act(seq_tok + (size_t)b * max_seq + n - 1)
                         : (pending >= 0 ? pending : ld_act(draft_tok + b * kMaxK + i - 1));
        }
      }
    }
    plan.row_pos[m] = pos;
    plan.row_seq[m] = seq;
    plan.row_tok[m] = tok;
    s_tok = tok;
    s_pos = pos;
  }
  __syncthreads();
  const WT* e = embed + (size_t)s_tok * d_model;
  float* dst = h + (size_t)m * d_model;
  float sq = 0.f;
  for (int k = threadIdx.x * 4; k < d_model; k += blockDim.x * 4) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (s_pos >= 0) v = load4(e + k);
    *reinterpret_cast<float4*>(dst + k) = v;
    if (im.img != nullptr) {
      sq = fmaf(v.x, v.x, sq);
      sq = fmaf(v.y, v.y, sq);
      sq = fmaf(v.z, v.z, sq);
      sq = fmaf(v.w, v.w, sq);
      const float4 g = *reinterpret_cast<const float4*>(im.gain + k);
      const float x0 = v.x * g.x, x1 = v.y * g.y, x2 = v.z * g.z, x3 = v.w * g.w;
      const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1), h2 = __float2bfloat16_rn(x2), h3 = __float2bfloat16_rn(x3);
      const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0)), l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
      const __nv_bfloat16 l2 = __float2bfloat16_rn(x2 - __bfloat162float(h2)), l3 = __float2bfloat16_rn(x3 - __bfloat162float(h3));
      const int rb = m / im.rb, tm = m - rb * im.rb, kg = k >> 3;
      unsigned char* p = im.img + ((size_t)rb * im.kb + (kg >> 3)) * ((size_t)im.rb * 256) + (size_t)(kg & 7) * (im.rb * 32) +
                         (size_t)(tm >> 3) * 128 + (tm & 7) * 16 + (k & 7) * 2;
      uint2 hv, lv;
      hv.x = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
      hv.y = (uint32_t)__bfloat16_as_ushort(h2) | ((uint32_t)__bfloat16_as_ushort(h3) << 16);
      lv.x = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
      lv.y = (uint32_t)__bfloat16_as_ushort(l2) | ((uint32_t)__bfloat16_as_ushort(l3) << 16);
      *reinterpret_cast<uint2*>(p) = hv;
      *reinterpret_cast<uint2*>(p + (size_t)im.rb * 16) = lv;
    }
  }
  if (im.img != nullptr) {  // the row's sum of squares, thread partials added in thread order
    s_sq[threadIdx.x] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
      for (int i = 0; i < (int)blockDim.x; ++i) t += s_sq[i];
      im.ssq[m] = t;
    }
  }
}

// argmax over the vocabulary of every row; ties go to the lowest token id.
// The result lands where the next kernel of the round expects it.
constexpr int kArgmaxThreads = 512;
__global__ void __launch_bounds__(kArgmaxThreads)
argmax_kernel(const float* logits, int vocab, PassDesc pd, int* draft_tok, int* tgt_tok, int* row_argmax) {
  __shared__ float s_val[kArgmaxThreads / 32];
  __shared__ int s_idx[kArgmaxThreads / 32];
  pdl_wait();
  pdl_launch_dependents();
  const int m = blockIdx.x;
  const float* l = logits + (size_t)m * vocab;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int v = threadIdx.x; v < vocab; v += kArgmaxThreads) {
    const float x = ld_act(l + v);
    if (x > best || (x == best && v < bi)) {
      best = x;
      bi = v;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ob > best || (ob == best && oi < bi)) {
      best = ob;
      bi = oi;
    }
  }
  if ((threadIdx.x & 31) == 0) {
    s_val[threadIdx.x >> 5] = best;
    s_idx[threadIdx.x >> 5] = bi;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kArgmaxThreads / 32; ++w)
      if (s_val[w] > best || (s_val[w] == best && s_idx[w] < bi)) {
        best = s_val[w];
        bi = s_idx[w];
      }
    row_argmax[m] = bi;
    const int R = pd.rows_per_seq;
    const int b = m / R, i = m - b * R;
    if (pd.kind == PASS_DRAFT_FIRST) {
      if (i == R - 1) draft_tok[b * kMaxK + 0] = bi;
    } else if (pd.kind == PASS_DRAFT_NEXT) {
      draft_tok[b * kMaxK + pd.step] = bi;
    } else if (pd.kind == PASS_VERIFY) {
      tgt_tok[b * (kMaxK + 1) + i] = bi;
    }
  }
}

struct RoundStat {
  int drafted, accepted, committed;
};

// Commit step shared by greedy and sampled decoding: append d_1..d_j and the extra
// token, truncated to max_new and at EOS, advance the lengths (that is the whole
// rollback: cache entries beyond the new length are never read before being
// rewritten), record the round.  Called by one thread per sequence.
__device__ __forceinline__ void commit_tokens(volatile GenState* gs, int b, int k, int j, int extra, const int* d,
                                              int* seq_tok, int max_seq, int* out_tok, RoundStat* stats) {
  const int n = gs->n[b];
  const int room = gs->max_new - gs->n_new[b];
  int cnt = 0;
  bool eos = false;
  for (int t = 0; t <= j && cnt < room && !eos; ++t) {
    const int tok = (t < j) ? ld_act(d + t) : extra;
    seq_tok[(size_t)b * max_seq + n + cnt] = tok;
    out_tok[(size_t)b * gs->max_new + gs->n_new[b] + cnt] = tok;
    ++cnt;
    if (gs->eos_id >= 0 && tok == gs->eos_id) eos = true;
  }
  gs->n[b] = n + cnt;
  gs->n_new[b] += cnt;
  if (eos || gs->n_new[b] >= gs->max_new) gs->done[b] = 1;
  if (gs->round < gs->max_rounds) {
    RoundStat* st = stats + (size_t)gs->round * gs->batch + b;
    st->drafted = k;
    st->accepted = j;
    st->committed = cnt;
  }
}

// Greedy accept (Eq. 2 degenerates to "draft token == target argmax"); k = 0 is a
// plain autoregressive step.
constexpr int kAcceptThreads = 256;
__global__ void __launch_bounds__(kAcceptThreads)
accept_greedy_kernel(GenState* gs_, const int* draft_tok, const int* tgt_tok, int* seq_tok, int max_seq,
                     int* out_tok, RoundStat* stats, const int* pass_error, const int2* amax_part, int amax_groups) {
  volatile GenState* gs = gs_;
  __shared__ int s_tgt[kMaxBatch * (kMaxK + 1)];
  pdl_wait();
  pdl_launch_dependents();
  const int B = gs->batch, k = gs->k;
  // the target's argmax of every verify row: finished here from the lm-head's per-group partials
  // (whole-pass kernel), else read where argmax_kernel left it
  for (int r = threadIdx.x >> 5; r < B * (k + 1); r += kAcceptThreads / 32) {
    const int b2 = r / (k + 1), i2 = r - b2 * (k + 1);
    const int v = amax_part ? amax_finish(amax_part, amax_groups, r) : ld_act(tgt_tok + b2 * (kMaxK + 1) + i2);
    if ((threadIdx.x & 31) == 0) s_tgt[b2 * (kMaxK + 1) + i2] = v;
  }
  __syncthreads();
  if (threadIdx.x >= 32) return;
  const int b = threadIdx.x;
  if (b < B) {
    if (gs->done[b]) {
      if (gs->round < gs->max_rounds) stats[(size_t)gs->round * B + b] = RoundStat{0, 0, 0};
    } else {
      const int* d = draft_tok + b * kMaxK;
      const int* t = s_tgt + b * (kMaxK + 1);
      int j = 0;
      while (j < k && ld_act(d + j) == t[j]) ++j;
      commit_tokens(gs, b, k, j, t[j], d, seq_tok, max_seq, out_tok, stats);
    }
  }
  __syncwarp();
  const int fin = (b < B) ? gs->done[b] : 1;
  const unsigned all = __all_sync(0xffffffffu, fin);
  if (threadIdx.x == 0) {
    gs->round += 1;
    gs->all_done = all ? 1 : 0;
    gs->pass_error = pass_error ? ld_act(pass_error) : 0;  // a pass of this round gave up a wait
  }
}

}  // namespace sdfp
