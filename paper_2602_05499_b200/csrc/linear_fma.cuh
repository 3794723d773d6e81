// CUDA-core weight-streaming linear kernel: Y = [RMSNorm](X) · Wᵀ with a fused epilogue.
//
// Used for fp32 models (the tiny configuration) and, on request, for bf16 models as
// the comparison path of the tensor-core kernel.  Weights are stored pair-major,
// W[pair][2][K] (see EpiMode in common.cuh for what a pair is).  One warp owns one
// pair at a time and sweeps K with 128-bit loads; lanes reduce with a fixed xor
// tree.  A row's result does not depend on how many rows the launch carries:
// every row runs the same instruction sequence on its own accumulators.
#pragma once

#include "common.cuh"

namespace sdfp {

constexpr int kFmaThreads = 256;

// inv_rms[m] = 1/sqrt(mean_k x[m,k]^2 + eps), computed redundantly by every CTA in a
// fixed order: lane-strided sequential sums, then the xor tree.
__device__ __forceinline__ void cta_inv_rms(const float* X, int ldx, int M, int K, float eps, float* inv_rms) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  for (int m = warp; m < M; m += nwarps) {
    const float* x = X + (size_t)m * ldx;
    float s = 0.f;
    for (int k = lane * 4; k < K; k += 128) {
      const float4 v = ld_act4(x + k);
      s = fmaf(v.x, v.x, s);
      s = fmaf(v.y, v.y, s);
      s = fmaf(v.z, v.z, s);
      s = fmaf(v.w, v.w, s);
    }
    s = warp_sum(s);
    if (lane == 0) inv_rms[m] = rsqrtf(s / (float)K + eps);
  }
}

template <typename WT, typename KT>
__global__ void __launch_bounds__(kFmaThreads)
linear_fma_kernel(const WT* __restrict__ W, const float* __restrict__ X, int ldx, int M, int K, int n_pairs,
                  const float* __restrict__ gain, float eps, EpiParams ep) {
  __shared__ float inv_rms[kMaxRows];
  pdl_wait();
  pdl_launch_dependents();
  if (gain != nullptr) {
    cta_inv_rms(X, ldx, M, K, eps, inv_rms);
    __syncthreads();
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int p = blockIdx.x * (kFmaThreads / 32) + warp; p < n_pairs; p += gridDim.x * (kFmaThreads / 32)) {
    const WT* w0p = W + (size_t)p * 2 * K;
    const WT* w1p = w0p + K;
    for (int m0 = 0; m0 < M; m0 += 8) {
      float a0[8], a1[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) a0[i] = a1[i] = 0.f;
      for (int k = lane * 4; k < K; k += 128) {
        const float4 w0 = load4(w0p + k);
        const float4 w1 = load4(w1p + k);
        float4 g = make_float4(1.f, 1.f, 1.f, 1.f);
        if (gain != nullptr) g = load4(gain + k);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int m = m0 + i;
          if (m < M) {
            float4 x = ld_act4(X + (size_t)m * ldx + k);
            if (gain != nullptr) {
              const float r = inv_rms[m];
              x.x = x.x * r * g.x;
              x.y = x.y * r * g.y;
              x.z = x.z * r * g.z;
              x.w = x.w * r * g.w;
            }
            a0[i] = fmaf(w0.x, x.x, a0[i]);
            a0[i] = fmaf(w0.y, x.y, a0[i]);
            a0[i] = fmaf(w0.z, x.z, a0[i]);
            a0[i] = fmaf(w0.w, x.w, a0[i]);
            a1[i] = fmaf(w1.x, x.x, a1[i]);
            a1[i] = fmaf(w1.y, x.y, a1[i]);
            a1[i] = fmaf(w1.z, x.z, a1[i]);
            a1[i] = fmaf(w1.w, x.w, a1[i]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float s0 = warp_sum(a0[i]);
        const float s1 = warp_sum(a1[i]);
        if (lane == i && m0 + i < M) apply_epilogue<KT>(ep, p, m0 + i, s0, s1);
      }
    }
  }
}

// ---- packing: caller's row-major [out, in] matrices -> pair-major ----------------
// src row of (pair p, half r):
//   kind 0 (QKV)    three sources q, k, v of [d, d]
//   kind 1 (GATEUP) two sources gate, up of [f, d]: pair j = (gate_j, up_j)
//   kind 2 (PLAIN)  one source: rows 16*(p/8) + p%8 (+8)
struct PackSrc {
  const void* s0;
  const void* s1;
  const void* s2;
  int kind;
  int n_heads, head_dim;
};

template <typename WT>
__device__ __forceinline__ const WT* pack_src_row(const PackSrc& ps, int p, int r, int K) {
  if (ps.kind == 0) {
    const int hp = ps.head_dim >> 1;
    const int per_tensor = ps.n_heads * hp;
    const int t = p / per_tensor;
    const int rem = p - t * per_tensor;
    const int head = rem / hp;
    const int i = rem - head * hp;
    const WT* base = reinterpret_cast<const WT*>(t == 0 ? ps.s0 : (t == 1 ? ps.s1 : ps.s2));
    return base + (size_t)(head * ps.head_dim + i + r * hp) * K;
  } else if (ps.kind == 1) {
    const WT* base = reinterpret_cast<const WT*>(r == 0 ? ps.s0 : ps.s1);
    return base + (size_t)p * K;
  }
  return reinterpret_cast<const WT*>(ps.s0) + (size_t)(((p >> 3) << 4) + (p & 7) + 8 * r) * K;
}

template <typename WT>
__global__ void pack_pairs_kernel(WT* __restrict__ dst, PackSrc ps, int n_pairs, int K) {
  const size_t total = (size_t)n_pairs * 2 * K;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int k = (int)(idx % K);
    const size_t pr = idx / K;
    const int r = (int)(pr & 1);
    const int p = (int)(pr >> 1);
    dst[idx] = pack_src_row<WT>(ps, p, r, K)[k];
  }
}

template <typename WT>
__global__ void widen_vector_kernel(float* __restrict__ dst, const WT* __restrict__ src, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = to_f32(src[i]);
}

}  // namespace sdfp
