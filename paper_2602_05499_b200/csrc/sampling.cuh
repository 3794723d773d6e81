// Sampled decoding: Philox4x32-10 uniforms, categorical draws by inverse CDF in
// token-id order, the accept test of Eq. 2 and the corrected distribution of Eq. 3
// (read as max(0, p − q) normalised, the rule of the speculative-sampling work the
// paper cites; the printed "p − α_j q" can go negative and is not lossless).
#pragma once

#include "common.cuh"
#include "misc_kernels.cuh"

namespace sdfp {

constexpr int kSampleThreads = 1024;

// Philox4x32-10 (Salmon et al., SC'11), written from the published round function.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0;
    c1 = lo1;
    c2 = n2;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

// purposes: 0 = draft-token draw, 1 = accept test, 2 = corrected / bonus / autoregressive draw.
// u = (top 23 bits + 1/2) * 2^-23: inside (0,1) and exact in fp32.
__device__ __forceinline__ double draw_u(unsigned long long seed, int seq, int position, int purpose) {
  uint32_t o[4];
  philox4x32_10((uint32_t)position, (uint32_t)purpose, (uint32_t)seq, 0u, (uint32_t)(seed & 0xffffffffull),
                (uint32_t)(seed >> 32), o);
  return ((double)(o[0] >> 9) + 0.5) * (1.0 / 8388608.0);
}

__device__ __forceinline__ float block_max(float v, float* s_red) {
  v = warp_max(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = s_red[0];
  for (int w = 1; w < kSampleThreads / 32; ++w) r = fmaxf(r, s_red[w]);
  return r;
}

// Inverse-CDF draw over weights wf(v) >= 0, v = 0..V-1: the smallest v whose cumulative
// weight exceeds u * total.  Thread t sums the contiguous segment it owns in order;
// segment totals are scanned in a fixed order; the owner walks its segment.  All in
// fp64, so the association order changes the result only at the 1e-16 level.
// Returns (to every thread) the drawn index and writes the total to *total_out.
template <typename WF>
__device__ int block_categorical(WF wf, int V, double u, double* s_scan, int* s_pick, double* total_out) {
  const int t = threadIdx.x;
  const int seg = (V + kSampleThreads - 1) / kSampleThreads;
  const int lo = min(V, t * seg), hi = min(V, lo + seg);
  double s = 0.0;
  for (int v = lo; v < hi; ++v) s += wf(v);
  // inclusive scan over threads: warp shuffles, then warp totals
  double x = s;
  const int lane = t & 31, warp = t >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();
  if (lane == 31) s_scan[kSampleThreads + warp] = x;
  __syncthreads();
  double base = 0.0;
  for (int w = 0; w < warp; ++w) base += s_scan[kSampleThreads + w];
  const double incl = base + x;
  s_scan[t] = incl - s;  // exclusive prefix of this thread's segment
  if (t == kSampleThreads - 1) s_scan[kSampleThreads + 32] = incl;
  if (t == 0) *s_pick = -1;
  __syncthreads();
  const double total = s_scan[kSampleThreads + 32];
  const double target = u * total;
  // owner = the last thread whose segment starts at or below the target and is not empty
  const bool cand = (hi > lo) && (s_scan[t] <= target);
  const bool next_cand = (t + 1 < kSampleThreads) && (min(V, (t + 1) * seg) < V) && (s_scan[t + 1] <= target);
  if (cand && !next_cand) {
    const double rem = target - s_scan[t];
    double c = 0.0;
    int pick = -1, last_pos = -1;
    for (int v = lo; v < hi; ++v) {
      const double w = wf(v);
      c += w;
      if (w > 0.0) last_pos = v;
      if (c > rem) {
        pick = v;
        break;
      }
    }
    if (pick < 0) pick = (last_pos >= 0) ? last_pos : hi - 1;  // rounding at a segment end
    *s_pick = pick;
  }
  __syncthreads();
  if (total_out) *total_out = total;
  return *s_pick;
}

// After a draft pass in sampling mode: q = softmax(logits / T) of the deciding row is
// kept (unnormalised exponentials + their fp64 sum) for the accept test, and the draft
// token is drawn from it (Eq. 1).
__global__ void __launch_bounds__(kSampleThreads)
sample_draft_kernel(const float* logits, int vocab, PassDesc pd, const GenState* gs_, int* draft_tok, float* qprob,
                    double* qsum) {
  const volatile GenState* gs = gs_;
  __shared__ float s_red[kSampleThreads / 32];
  __shared__ double s_scan[kSampleThreads + 33];
  __shared__ int s_pick;
  pdl_wait();
  pdl_launch_dependents();
  const int m = blockIdx.x;
  const int R = pd.rows_per_seq;
  const int b = m / R, i = m - b * R;
  int s;
  if (pd.kind == PASS_DRAFT_FIRST) {
    if (i != R - 1) return;
    s = 0;
  } else {
    s = pd.step;
  }
  if (gs->done[b]) return;
  const float* l = logits + (size_t)m * vocab;
  float mx = -INFINITY;
  for (int v = threadIdx.x; v < vocab; v += kSampleThreads) mx = fmaxf(mx, ld_act(l + v));
  mx = block_max(mx, s_red);
  const float inv_t = 1.0f / gs->temperature;
  float* q = qprob + ((size_t)b * gs->k + s) * vocab;
  for (int v = threadIdx.x; v < vocab; v += kSampleThreads) q[v] = __expf((ld_act(l + v) - mx) * inv_t);
  __syncthreads();
  const double u = draw_u(gs->seed, b, gs->n[b] + s, 0);
  double total;
  const int tok = block_categorical([&](int v) { return (double)q[v]; }, vocab, u, s_scan, &s_pick, &total);
  if (threadIdx.x == 0) {
    draft_tok[b * kMaxK + s] = tok;
    qsum[b * kMaxK + s] = total;
  }
}

// Verify in sampling mode, one CTA, sequences in turn.  logits rows b*(k+1)+i, i = 0..k,
// are the target's for the token after row i.
__global__ void __launch_bounds__(kSampleThreads)
accept_sampled_kernel(GenState* gs_, const float* logits, int vocab, const int* draft_tok, const float* qprob,
                      const double* qsum, int* seq_tok, int max_seq, int* out_tok, RoundStat* stats,
                      const int* pass_error) {
  volatile GenState* gs = gs_;
  __shared__ float s_red[kSampleThreads / 32];
  __shared__ double s_scan[kSampleThreads + 33];
  __shared__ int s_pick;
  pdl_wait();
  pdl_launch_dependents();
  const int B = gs->batch, k = gs->k;
  const float inv_t = 1.0f / gs->temperature;
  for (int b = 0; b < B; ++b) {
    if (gs->done[b]) {
      if (threadIdx.x == 0 && gs->round < gs->max_rounds) stats[(size_t)gs->round * B + b] = RoundStat{0, 0, 0};
      continue;
    }
    const int n = gs->n[b];
    const int* d = draft_tok + b * kMaxK;
    int j = 0, extra = 0;
    for (;; ++j) {
      const float* l = logits + ((size_t)b * (k + 1) + j) * vocab;
      float mx = -INFINITY;
      for (int v = threadIdx.x; v < vocab; v += kSampleThreads) mx = fmaxf(mx, ld_act(l + v));
      mx = block_max(mx, s_red);
      auto pe = [&](int v) { return (double)__expf((ld_act(l + v) - mx) * inv_t); };
      if (j == k) {  // every draft accepted: bonus token from the target's distribution
        extra = block_categorical(pe, vocab, draw_u(gs->seed, b, n + j, 2), s_scan, &s_pick, nullptr);
        break;
      }
      // S_p with the same segment/scan order a draw would use
      double sp;
      block_categorical(pe, vocab, 0.5, s_scan, &s_pick, &sp);
      const float* q = qprob + ((size_t)b * k + j) * vocab;
      const double sq = ld_act(qsum + b * kMaxK + j);
      const int tok = ld_act(d + j);
      const double pd_ = pe(tok) / sp, qd_ = (double)ld_act(q + tok) / sq;
      const double u = draw_u(gs->seed, b, n + j, 1);
      if (u * qd_ < pd_) continue;  // accepted (Eq. 2)
      // first rejection: draw from max(0, p − q), falling back to p if that is all zero
      auto res = [&](int v) {
        const double r = pe(v) / sp - (double)ld_act(q + v) / sq;
        return r > 0.0 ? r : 0.0;
      };
      const double u2 = draw_u(gs->seed, b, n + j, 2);
      double tot;
      extra = block_categorical(res, vocab, u2, s_scan, &s_pick, &tot);
      if (!(tot > 0.0)) extra = block_categorical(pe, vocab, u2, s_scan, &s_pick, nullptr);
      break;
    }
    __syncthreads();
    if (threadIdx.x == 0) commit_tokens(gs, b, k, j, extra, d, seq_tok, max_seq, out_tok, stats);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    int all = 1;
    for (int b = 0; b < B; ++b) all &= gs->done[b];
    gs->round += 1;
    gs->all_done = all;
    gs->pass_error = pass_error ? ld_act(pass_error) : 0;
  }
}

}  // namespace sdfp
