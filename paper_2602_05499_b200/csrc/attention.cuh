// Split-KV decode / verify attention over a contiguous per-sequence KV cache.
//
// One CTA = (key chunk c of kAttnChunk keys, head, sequence).  The R query rows a
// sequence carries in this pass (1 in a draft or autoregressive step, k+1 in a
// verify pass, up to kMaxRows in prefill) share the one sweep over the chunk's K
// and V.  Each (row, chunk) yields a partial (max, sum, o[head_dim]); the CTA that
// arrives last for a (sequence, head) folds the chunks of every row in chunk order.
//
// A row's result is independent of the other rows: a row at position pos sees keys
// 0..pos, the chunk grid is fixed in absolute key index, every (row, chunk) partial
// runs the same instruction sequence, and the fold walks chunks 0..pos/kAttnChunk
// in order.  So a verify row is bit-identical to the same token decoded alone.
#pragma once

#include "common.cuh"

namespace sdfp {

constexpr int kAttnThreads = 128;
constexpr int kAttnMaxR = 16;  // rows of one sequence handled per launch slice

struct AttnParams {
  const float* q;    // [rows, n_heads*head_dim]
  const void* kcache;  // this layer: [seq][head][max_seq][head_dim]
  const void* vcache;
  float* out;        // [rows, n_heads*head_dim]
  float* part_o;     // [rows][head][n_chunks][head_dim]
  float* part_ml;    // [rows][head][n_chunks][2]
  int* counters;     // [max_batch][head], zero between launches
  const int* row_pos;  // [rows]
  int rows_per_seq;  // R: rows b*R .. b*R+R-1 belong to sequence slot row_seq[b*R]
  const int* row_seq;
  int n_heads, max_seq, n_chunks;
  float scale;       // 1/sqrt(head_dim)
  // non-null: leave the result as bf16 hi + lo in the activation image of the O-projection on the
  // dense path instead of fp32 rows (row block img_rb, img_kb k blocks of 64; 16-byte piece of
  // (row m, columns 8*kg..) at byte (m / rb * kb + kg / 8) * rb * 256 + (kg % 8) * rb * 32 +
  // (m % rb / 8) * 128 + (m % 8) * 16, low parts rb * 16 bytes further)
  unsigned char* img;
  int img_rb, img_kb;
  // dense path only: CTAs per (sequence, head), each taking every n_splits-th 64-key chunk
  int n_splits;
};

__device__ __forceinline__ void attn_store(const AttnParams& ap, float* dst, int m, int col, float v) {
  if (ap.img == nullptr) {
    dst[col] = v;
    return;
  }
  const int rb = m / ap.img_rb, tm = m - rb * ap.img_rb, kg = col >> 3;
  unsigned char* p = ap.img + ((size_t)rb * ap.img_kb + (kg >> 3)) * ((size_t)ap.img_rb * 256) + (size_t)(kg & 7) * (ap.img_rb * 32) +
                     (size_t)(tm >> 3) * 128 + (tm & 7) * 16 + (col & 7) * 2;
  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
  *reinterpret_cast<__nv_bfloat16*>(p) = hi;
  *reinterpret_cast<__nv_bfloat16*>(p + (size_t)ap.img_rb * 16) = __float2bfloat16_rn(v - __bfloat162float(hi));
}

template <typename KT, int HD>
__global__ void __launch_bounds__(kAttnThreads) attention_kernel(AttnParams ap) {
  constexpr int C = kAttnChunk;
  constexpr int KV_LD = HD + 8;  // padded row, in elements, to spread shared-memory banks
  extern __shared__ __align__(16) unsigned char smem_raw[];
  KT* sK = reinterpret_cast<KT*>(smem_raw);
  KT* sV = sK + C * KV_LD;
  float* sQ = reinterpret_cast<float*>(sV + C * KV_LD);  // [R][HD]
  float* sS = sQ + kAttnMaxR * HD;                        // [R][C] scores, then probabilities
  __shared__ int s_pos[kAttnMaxR];
  __shared__ int s_last;

  pdl_wait();
  pdl_launch_dependents();

  const int c = blockIdx.x, head = blockIdx.y, b = blockIdx.z;
  const int R = ap.rows_per_seq;
  const int tid = threadIdx.x;
  const int row0 = b * R;
  const int key0 = c * C;

  if (tid < R) s_pos[tid] = ld_act(ap.row_pos + row0 + tid);
  __syncthreads();
  int max_pos = -1;
  for (int i = 0; i < R; ++i) max_pos = max(max_pos, s_pos[i]);

  const size_t d_model = (size_t)ap.n_heads * HD;
  if (max_pos >= key0) {
    const int seq = ld_act(ap.row_seq + row0);
    const int nk_all = min(C, max_pos + 1 - key0);  // keys of this chunk any row can see
    const KT* gK = reinterpret_cast<const KT*>(ap.kcache) + (((size_t)seq * ap.n_heads + head) * ap.max_seq + key0) * HD;
    const KT* gV = reinterpret_cast<const KT*>(ap.vcache) + (((size_t)seq * ap.n_heads + head) * ap.max_seq + key0) * HD;
    // stage K, V (16-byte vectors) and q
    constexpr int VEC = 16 / sizeof(KT);
    constexpr int VPR = HD / VEC;  // vectors per row
    for (int v = tid; v < nk_all * VPR; v += kAttnThreads) {
      const int key = v / VPR, j = v - key * VPR;
      *reinterpret_cast<uint4*>(sK + key * KV_LD + j * VEC) = __ldcg(reinterpret_cast<const uint4*>(gK + (size_t)key * HD + j * VEC));
      *reinterpret_cast<uint4*>(sV + key * KV_LD + j * VEC) = __ldcg(reinterpret_cast<const uint4*>(gV + (size_t)key * HD + j * VEC));
    }
    for (int e = tid; e < R * HD; e += kAttnThreads) {
      const int i = e / HD, d = e - i * HD;
      sQ[e] = (s_pos[i] >= 0) ? ld_act(ap.q + (size_t)(row0 + i) * d_model + head * HD + d) : 0.f;
    }
    __syncthreads();

    // scores: thread (key, half) does half of the dot product of every row with its key
    {
      const int key = tid >> 1, half = tid & 1;
      float acc[kAttnMaxR];
#pragma unroll
      for (int i = 0; i < kAttnMaxR; ++i) acc[i] = 0.f;
      if (key < nk_all) {
        const KT* kr = sK + key * KV_LD + half * (HD / 2);
        const float* qh = sQ + half * (HD / 2);
#pragma unroll 4
        for (int d = 0; d < HD / 2; d += 4) {
          const float4 kv = load4(kr + d);
#pragma unroll
          for (int i = 0; i < kAttnMaxR; ++i) {
            if (i < R) {
              const float4 qv = *reinterpret_cast<const float4*>(qh + i * HD + d);
              acc[i] = fmaf(kv.x, qv.x, acc[i]);
              acc[i] = fmaf(kv.y, qv.y, acc[i]);
              acc[i] = fmaf(kv.z, qv.z, acc[i]);
              acc[i] = fmaf(kv.w, qv.w, acc[i]);
            }
          }
        }
      }
#pragma unroll
      for (int i = 0; i < kAttnMaxR; ++i) {
        if (i < R) {
          const float other = __shfl_xor_sync(0xffffffffu, acc[i], 1);
          const float lo = half ? other : acc[i];
          const float hi = half ? acc[i] : other;
          if (half == 0 && key < C) sS[i * C + key] = (lo + hi) * ap.scale;
        }
      }
    }
    __syncthreads();

    // per-row softmax statistics inside the chunk: warp w takes rows w, w+4, ...
    {
      const int warp = tid >> 5, lane = tid & 31;
      for (int i = warp; i < R; i += kAttnThreads / 32) {
        const int nk = min(C, s_pos[i] + 1 - key0);  // <= 0: the row sees nothing here
        float s0 = (lane < nk) ? sS[i * C + lane] : -INFINITY;
        float s1 = (lane + 32 < nk) ? sS[i * C + lane + 32] : -INFINITY;
        const float mx = warp_max(fmaxf(s0, s1));
        const float p0 = (lane < nk) ? __expf(s0 - mx) : 0.f;
        const float p1 = (lane + 32 < nk) ? __expf(s1 - mx) : 0.f;
        sS[i * C + lane] = p0;
        sS[i * C + lane + 32] = p1;
        const float l = warp_sum(p0 + p1);
        if (lane == 0 && nk > 0) {
          float* ml = ap.part_ml + ((((size_t)(row0 + i)) * ap.n_heads + head) * ap.n_chunks + c) * 2;
          ml[0] = mx;
          ml[1] = l;
        }
      }
    }
    __syncthreads();

    // o[i][d] = Σ_key p[i][key] · V[key][d], keys in order
    for (int d = tid; d < HD; d += kAttnThreads) {
      float o[kAttnMaxR];
#pragma unroll
      for (int i = 0; i < kAttnMaxR; ++i) o[i] = 0.f;
      for (int key = 0; key < nk_all; ++key) {
        const float v = to_f32(sV[key * KV_LD + d]);
#pragma unroll
        for (int i = 0; i < kAttnMaxR; ++i)
          if (i < R) o[i] = fmaf(sS[i * C + key], v, o[i]);   // p is exactly 0 beyond the row's keys
      }
#pragma unroll
      for (int i = 0; i < kAttnMaxR; ++i) {
        if (i < R && s_pos[i] >= key0)
          ap.part_o[((((size_t)(row0 + i)) * ap.n_heads + head) * ap.n_chunks + c) * HD + d] = o[i];
      }
    }
  }

  // last CTA of this (sequence, head) folds the chunks
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int prev = atomicAdd(&ap.counters[b * ap.n_heads + head], 1);
    s_last = (prev == (int)gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid == 0) ap.counters[b * ap.n_heads + head] = 0;
  for (int i = 0; i < R; ++i) {
    const int pos = s_pos[i];
    float* dst = ap.out + (size_t)(row0 + i) * d_model;
    if (pos < 0) {
      for (int d = tid; d < HD; d += kAttnThreads) attn_store(ap, dst, row0 + i, head * HD + d, 0.f);
      continue;
    }
    const int nc = pos / C + 1;
    const float* ml = ap.part_ml + (((size_t)(row0 + i)) * ap.n_heads + head) * ap.n_chunks * 2;
    const float* po = ap.part_o + (((size_t)(row0 + i)) * ap.n_heads + head) * ap.n_chunks * HD;
    float mx = -INFINITY;
    for (int cc = 0; cc < nc; ++cc) mx = fmaxf(mx, __ldcg(ml + cc * 2));
    float l = 0.f;
    for (int cc = 0; cc < nc; ++cc) l = fmaf(__ldcg(ml + cc * 2 + 1), __expf(__ldcg(ml + cc * 2) - mx), l);
    const float inv_l = 1.0f / l;
    for (int d = tid; d < HD; d += kAttnThreads) {
      float o = 0.f;
      for (int cc = 0; cc < nc; ++cc)
        o = fmaf(__ldcg(po + (size_t)cc * HD + d), __expf(__ldcg(ml + cc * 2) - mx), o);
      attn_store(ap, dst, row0 + i, head * HD + d, o * inv_l);
    }
  }
}

template <typename KT, int HD>
constexpr size_t attention_smem_bytes() {
  return (size_t)2 * kAttnChunk * (HD + 8) * sizeof(KT) + (size_t)kAttnMaxR * HD * sizeof(float) +
         (size_t)kAttnMaxR * kAttnChunk * sizeof(float);
}

}  // namespace sdfp
