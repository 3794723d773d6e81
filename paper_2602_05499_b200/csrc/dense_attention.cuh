// Decode / verify attention for the passes of a batch on the dense path: the rows a sequence
// carries in a pass attend the keys of its cache up to their own positions; the result goes out as
// bf16 hi + lo into the activation image of the O-projection (or as fp32 rows).
//
// One CTA = (split j of n_splits, head, sequence), four warps.  The rows the sequence carries in
// the pass (at most 16) are the M tile of mma.sync.m16n8k16: q is split q = hi + lo into bf16 once
// (shared memory), and so is every block of probabilities, so nothing is rounded to 8 mantissa bits
// that the other kernels keep in fp32; K and V are bf16 in the cache.  The CTA walks the 64-key
// chunks j, j + n_splits, ... through a three-deep ring of shared-memory tiles (16-byte asynchronous
// copies, rows padded by 16 bytes for ldmatrix); warp w owns keys 16w..16w+15 of every chunk:
//   S = Q K^T  (16 rows x 16 keys, 2 x HD/16 MMAs each for hi and lo),  mask, running max / sum,
//   O += P V   (16 rows x HD, HD/8 MMAs each for hi and lo),
// with its own running state, so the warps never wait for one another inside a chunk; their four
// partial results are combined in warp order at the end, and with more than one split the CTA that
// arrives last for its (sequence, head) folds the splits in split order.  The tensor work does not
// depend on how many of the 16 rows are in use, and each row's numbers depend on its own position
// alone (a key a row cannot see gets probability exactly zero), so a verify row equals the same
// token decoded alone, whatever else is in the batch.
#pragma once

#include "attention.cuh"
#include "pass_kernel.cuh"
#include "prefill_attention.cuh"

namespace sdfp {

constexpr int kAmThreads = 128;
constexpr int kAmWarps = 4;
constexpr int kAmRows = 16;
constexpr int kAmKeys = 64;   // keys per chunk: 16 per warp
constexpr int kAmStages = 3;

template <int HD>
__host__ __device__ constexpr size_t attention_mma_smem() {
  return (size_t)(2 * kAmRows + kAmStages * 2 * kAmKeys) * (HD + 8) * 2;  // Q hi, Q lo, stages x (K, V)
}

template <int HD>
__global__ void __launch_bounds__(kAmThreads, 2) attention_mma_kernel(AttnParams ap, int M) {
  constexpr int LD = HD + 8;
  static_assert((size_t)kAmWarps * kAmRows * (HD + 2) * 4 <= (size_t)kAmStages * 2 * kAmKeys * LD * 2, "merge area");
  extern __shared__ __align__(16) unsigned char am_smem[];
  __shared__ int s_pos[kAmRows];
  __shared__ int s_last;
  __nv_bfloat16* sQh = reinterpret_cast<__nv_bfloat16*>(am_smem);
  __nv_bfloat16* sQl = sQh + kAmRows * LD;
  __nv_bfloat16* sKV = sQl + kAmRows * LD;  // [stage][K | V][64][LD]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, qd = lane & 3;
  const int split = blockIdx.x, head = blockIdx.y, b = blockIdx.z, n_splits = ap.n_splits;
  const int R = ap.rows_per_seq, row0 = b * R;
  const size_t d_model = (size_t)ap.n_heads * HD;

  pdl_wait();  // q and the newest K/V rows are the preceding kernel's output
  pdl_launch_dependents();

  if (tid < kAmRows) s_pos[tid] = (tid < R && row0 + tid < M) ? ld_act(ap.row_pos + row0 + tid) : -1;
  const int seq = ld_act(ap.row_seq + row0);
  __syncthreads();
  int max_pos = -1;
#pragma unroll
  for (int r = 0; r < kAmRows; ++r) max_pos = max(max_pos, s_pos[r]);
  const int nc = (max_pos + kAmKeys) / kAmKeys;  // chunks that hold a visible key
  const int n_my = nc > split ? (nc - split + n_splits - 1) / n_splits : 0;
  const size_t base = ((size_t)seq * ap.n_heads + head) * (size_t)ap.max_seq * HD;
  const __nv_bfloat16* gK = reinterpret_cast<const __nv_bfloat16*>(ap.kcache) + base;
  const __nv_bfloat16* gV = reinterpret_cast<const __nv_bfloat16*>(ap.vcache) + base;

  auto load_kv = [&](int i) {  // chunk number i of this CTA into stage i % kAmStages; always one commit group
    if (i < n_my) {
      const int key0 = (split + i * n_splits) * kAmKeys;
      __nv_bfloat16* dK = sKV + (size_t)(i % kAmStages) * 2 * kAmKeys * LD;
      __nv_bfloat16* dV = dK + kAmKeys * LD;
      constexpr int VPR = HD / 8;  // 16-byte vectors per row
      for (int v = tid; v < kAmKeys * VPR; v += kAmThreads) {
        const int key = v / VPR, j = v - key * VPR;
        if (key0 + key <= max_pos) {
          cp_async16(dK + key * LD + j * 8, gK + (size_t)(key0 + key) * HD + j * 8);
          cp_async16(dV + key * LD + j * 8, gV + (size_t)(key0 + key) * HD + j * 8);
        } else {  // no row sees it: keep the tile finite (its probabilities are exactly zero)
          *reinterpret_cast<uint4*>(dK + key * LD + j * 8) = make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4*>(dV + key * LD + j * 8) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    }
    cp_async_commit();
  };
#pragma unroll
  for (int i = 0; i < kAmStages - 1; ++i) load_kv(i);

  // q rows of this sequence and head: fp32 -> bf16 hi + lo (rows not in use: zero)
  for (int e = tid; e < kAmRows * (HD / 4); e += kAmThreads) {
    const int i = e / (HD / 4), d = (e - i * (HD / 4)) * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (s_pos[i] >= 0) v = ld_act4(ap.q + (size_t)(row0 + i) * d_model + head * HD + d);
    uint2 hi, lo;
    split_pack(v.x, v.y, hi.x, lo.x);
    split_pack(v.z, v.w, hi.y, lo.y);
    *reinterpret_cast<uint2*>(sQh + i * LD + d) = hi;
    *reinterpret_cast<uint2*>(sQl + i * LD + d) = lo;
  }

  float o[HD / 8][4];
#pragma unroll
  for (int j = 0; j < HD / 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[j][e] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // rows g and g + 8
  const int pos_a = s_pos[g], pos_b = s_pos[g + 8];

  for (int i = 0; i < n_my; ++i) {
    cp_async_wait_group<kAmStages - 2>();
    __syncthreads();       // chunk i (and, the first time, q) is visible; everyone has left chunk i - 1
    load_kv(i + kAmStages - 1);  // into the stage chunk i - 1 occupied
    const __nv_bfloat16* tK = sKV + (size_t)(i % kAmStages) * 2 * kAmKeys * LD;
    const __nv_bfloat16* tV = tK + kAmKeys * LD;
    const int key0 = (split + i * n_splits) * kAmKeys + warp * 16;

    // ---- S = Q K^T: 16 rows x this warp's 16 keys ----
    float s[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[j][e] = 0.f;
#pragma unroll
    for (int k16 = 0; k16 < HD / 16; ++k16) {
      uint32_t ah[4], al[4], kb[4];
      const int arow = (lane & 7) + ((lane >> 3) & 1) * 8, acol = k16 * 16 + (lane >> 4) * 8;
      ldsm_x4(ah, sQh + arow * LD + acol);
      ldsm_x4(al, sQl + arow * LD + acol);
      const int key = warp * 16 + (lane & 7) + (lane >> 4) * 8, dim = k16 * 16 + ((lane >> 3) & 1) * 8;
      ldsm_x4(kb, tK + key * LD + dim);
      mma_16816(s[0], ah, kb[0], kb[1]);
      mma_16816(s[0], al, kb[0], kb[1]);
      mma_16816(s[1], ah, kb[2], kb[3]);
      mma_16816(s[1], al, kb[2], kb[3]);
    }
    // ---- scale, mask, running max and sum ----
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = key0 + j * 8 + 2 * qd + (e & 1);
        const float v = (key <= ((e < 2) ? pos_a : pos_b)) ? s[j][e] * ap.scale : -INFINITY;
        s[j][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    float alpha[2], m_use[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r]);
      const bool none = m_new == -INFINITY;          // this warp has not met a key the row can see
      alpha[r] = none ? 1.0f : __expf(m_run[r] - m_new);  // exp(-inf) = 0 the first time
      m_use[r] = none ? 0.0f : m_new;
      m_run[r] = m_new;
    }
    float ps[2] = {0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float pv = __expf(s[j][e] - m_use[e >> 1]);  // masked entries: exp(-inf) = 0
        s[j][e] = pv;
        ps[e >> 1] += pv;
      }
#pragma unroll
    for (int r = 0; r < 2; ++r) l_run[r] = fmaf(l_run[r], alpha[r], ps[r]);
#pragma unroll
    for (int j = 0; j < HD / 8; ++j) {
      o[j][0] *= alpha[0];
      o[j][1] *= alpha[0];
      o[j][2] *= alpha[1];
      o[j][3] *= alpha[1];
    }
    // ---- O += P V ----
    uint32_t ph[4], pl[4];
    split_pack(s[0][0], s[0][1], ph[0], pl[0]);
    split_pack(s[0][2], s[0][3], ph[1], pl[1]);
    split_pack(s[1][0], s[1][1], ph[2], pl[2]);
    split_pack(s[1][2], s[1][3], ph[3], pl[3]);
#pragma unroll
    for (int d2 = 0; d2 < HD / 16; ++d2) {  // two dimension groups of 8 per ldmatrix
      uint32_t vb[4];
      const int key = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, dim = d2 * 16 + (lane >> 4) * 8;
      ldsm_x4_trans(vb, tV + key * LD + dim);
      mma_16816(o[2 * d2], ph, vb[0], vb[1]);
      mma_16816(o[2 * d2], pl, vb[0], vb[1]);
      mma_16816(o[2 * d2 + 1], ph, vb[2], vb[3]);
      mma_16816(o[2 * d2 + 1], pl, vb[2], vb[3]);
    }
  }
  cp_async_wait_group<0>();
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }

  // ---- the four warps' partial results, combined in warp order ----
  __syncthreads();  // every warp has left the ring
  float* mo = reinterpret_cast<float*>(sKV);           // [warp][row][HD]
  float* mml = mo + (size_t)kAmWarps * kAmRows * HD;   // [warp][row][2]
#pragma unroll
  for (int j = 0; j < HD / 8; ++j) {
    const int d = j * 8 + 2 * qd;
    *reinterpret_cast<float2*>(mo + ((size_t)warp * kAmRows + g) * HD + d) = make_float2(o[j][0], o[j][1]);
    *reinterpret_cast<float2*>(mo + ((size_t)warp * kAmRows + g + 8) * HD + d) = make_float2(o[j][2], o[j][3]);
  }
  if (qd == 0) {
    mml[((size_t)warp * kAmRows + g) * 2] = m_run[0];
    mml[((size_t)warp * kAmRows + g) * 2 + 1] = l_run[0];
    mml[((size_t)warp * kAmRows + g + 8) * 2] = m_run[1];
    mml[((size_t)warp * kAmRows + g + 8) * 2 + 1] = l_run[1];
  }
  __syncthreads();
  const int nr = min(R, kAmRows);
  for (int e = tid; e < nr * HD; e += kAmThreads) {
    const int r = e / HD, d = e - r * HD;
    const int m = row0 + r;
    if (m >= M) continue;
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < kAmWarps; ++w)
      if (mml[((size_t)w * kAmRows + r) * 2 + 1] > 0.f) mx = fmaxf(mx, mml[((size_t)w * kAmRows + r) * 2]);
    float l = 0.f, ov = 0.f;
#pragma unroll
    for (int w = 0; w < kAmWarps; ++w) {
      const float lw = mml[((size_t)w * kAmRows + r) * 2 + 1];
      const float wt = lw > 0.f ? __expf(mml[((size_t)w * kAmRows + r) * 2] - mx) : 0.f;
      l = fmaf(lw, wt, l);
      ov = fmaf(wt, mo[((size_t)w * kAmRows + r) * HD + d], ov);
    }
    if (n_splits == 1) {
      attn_store(ap, ap.out + (size_t)m * d_model, m, head * HD + d, l > 0.f ? ov / l : 0.f);  // no visible key: zero
    } else {
      const size_t slot = ((size_t)m * ap.n_heads + head) * kAttnSplits + split;
      ap.part_o[slot * HD + d] = ov;
      if (d == 0) {
        ap.part_ml[slot * 2] = mx;
        ap.part_ml[slot * 2 + 1] = l;
      }
    }
  }
  if (n_splits == 1) return;

  // ---- the last CTA of this (sequence, head) folds the splits ----
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int prev = atomicAdd(&ap.counters[b * ap.n_heads + head], 1);
    s_last = (prev == n_splits - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid == 0) ap.counters[b * ap.n_heads + head] = 0;
  for (int e = tid; e < nr * HD; e += kAmThreads) {
    const int r = e / HD, d = e - r * HD;
    const int m = row0 + r;
    if (m >= M) continue;
    const float* ml = ap.part_ml + ((size_t)m * ap.n_heads + head) * kAttnSplits * 2;
    const float* po = ap.part_o + ((size_t)m * ap.n_heads + head) * kAttnSplits * HD + d;
    float mj[kAttnSplits], lj[kAttnSplits], oj[kAttnSplits];
#pragma unroll
    for (int j = 0; j < kAttnSplits; ++j) {
      const bool have = j < n_splits;
      mj[j] = have ? __ldcg(ml + 2 * j) : 0.f;
      lj[j] = have ? __ldcg(ml + 2 * j + 1) : 0.f;
      oj[j] = have ? __ldcg(po + (size_t)j * HD) : 0.f;
    }
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < kAttnSplits; ++j)
      if (lj[j] > 0.f) mx = fmaxf(mx, mj[j]);
    float l = 0.f, ov = 0.f;
#pragma unroll
    for (int j = 0; j < kAttnSplits; ++j) {
      const float w = lj[j] > 0.f ? __expf(mj[j] - mx) : 0.f;
      l = fmaf(lj[j], w, l);
      ov = fmaf(w, oj[j], ov);
    }
    attn_store(ap, ap.out + (size_t)m * d_model, m, head * HD + d, l > 0.f ? ov / l : 0.f);
  }
}

}  // namespace sdfp
