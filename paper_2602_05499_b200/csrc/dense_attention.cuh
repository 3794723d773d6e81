// Split-KV decode / verify attention for the passes of a batch on the dense path.
//
// One CTA = (split j of kAttnSplits, head, sequence): it runs the whole-pass kernel's attention
// item (attention_item in pass_kernel.cuh: the rows a sequence carries in this pass share one sweep
// over the 64-key chunks j, j + kAttnSplits, ... of the head, running max and sum per row, K
// straight to registers, V by asynchronous copies), which leaves one un-normalised partial (max,
// sum, o) per (row, head, split).  The CTA that arrives last for a (sequence, head) folds the
// kAttnSplits partials of every row in split order and writes the result, as bf16 hi + lo into the
// activation image of the O-projection or as fp32 rows.  A row's numbers depend on its own
// position alone (chunks beyond it are skipped entirely), so a verify row equals the same token
// decoded alone, whatever else is in the batch.
#pragma once

#include "attention.cuh"
#include "pass_kernel.cuh"

namespace sdfp {

// RM = row capacity of the item (its per-row registers are arrays of RM entries): one kernel per
// capacity, so that the narrow passes (one or two rows per sequence) keep several CTAs per SM.
template <int HD, int RM>
__global__ void __launch_bounds__(kHalfThreads, RM <= 2 ? 3 : (RM <= 8 ? 2 : 1)) attention_split_kernel(AttnParams ap, int M) {
  extern __shared__ __align__(16) unsigned char das_smem[];
  __shared__ PassShared sh;
  __shared__ StageDesc st;
  __shared__ int s_last;
  const int tid = threadIdx.x;
  const int split = blockIdx.x, head = blockIdx.y, b = blockIdx.z;
  const int R = ap.rows_per_seq, row0 = b * R;

  pdl_wait();
  pdl_launch_dependents();

  if (tid < kPassMaxRows) {  // the item sees this sequence's rows as rows 0..R-1
    const bool live = tid < R && row0 + tid < M;
    sh.row_pos[tid] = live ? ld_act(ap.row_pos + row0 + tid) : -1;
    sh.row_seq[tid] = live ? ld_act(ap.row_seq + row0 + tid) : ld_act(ap.row_seq + row0);
  }
  if (tid == 0) {
    st = StageDesc{};
    st.X = ap.q + (size_t)row0 * ap.n_heads * HD;
    st.ep.kcache = const_cast<void*>(ap.kcache);
    st.ep.vcache = const_cast<void*>(ap.vcache);
    st.ep.n_heads = ap.n_heads;
    st.ep.max_seq = ap.max_seq;
  }
  __syncthreads();
  PassParams pp{};
  pp.M = min(R, M - row0);
  pp.rows_per_seq = R;
  pp.attn_scale = ap.scale;
  pp.part_o = ap.part_o + (size_t)row0 * ap.n_heads * kAttnSplits * HD;
  pp.part_ml = ap.part_ml + (size_t)row0 * ap.n_heads * kAttnSplits * 2;
  attention_item<HD, RM>(st, pp, &sh, das_smem, 0, tid, head, split, 0);

  // the last CTA of this (sequence, head) folds the splits
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int prev = atomicAdd(&ap.counters[b * ap.n_heads + head], 1);
    s_last = (prev == kAttnSplits - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid == 0) ap.counters[b * ap.n_heads + head] = 0;
  const size_t d_model = (size_t)ap.n_heads * HD;
  for (int e = tid; e < R * HD; e += kHalfThreads) {
    const int i = e / HD, d = e - i * HD;
    const int m = row0 + i;
    if (m >= M) continue;
    const float* ml = ap.part_ml + ((size_t)m * ap.n_heads + head) * kAttnSplits * 2;
    const float* po = ap.part_o + ((size_t)m * ap.n_heads + head) * kAttnSplits * HD + d;
    float mj[kAttnSplits], lj[kAttnSplits], oj[kAttnSplits];
#pragma unroll
    for (int j = 0; j < kAttnSplits; ++j) {
      mj[j] = __ldcg(ml + 2 * j);
      lj[j] = __ldcg(ml + 2 * j + 1);
      oj[j] = __ldcg(po + (size_t)j * HD);
    }
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < kAttnSplits; ++j)
      if (lj[j] > 0.f) mx = fmaxf(mx, mj[j]);
    float l = 0.f, o = 0.f;
#pragma unroll
    for (int j = 0; j < kAttnSplits; ++j) {
      const float w = lj[j] > 0.f ? __expf(mj[j] - mx) : 0.f;
      l = fmaf(lj[j], w, l);
      o = fmaf(w, oj[j], o);
    }
    const float v = l > 0.f ? o / l : 0.f;  // a row that carries nothing has no keys: zero
    attn_store(ap, ap.out + (size_t)m * d_model, m, head * HD + d, v);
  }
}

}  // namespace sdfp
