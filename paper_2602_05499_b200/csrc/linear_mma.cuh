// Tensor-core weight-streaming linear kernel for bf16 models:
//   Y[m, n] = Σ_k W[n, k] · X'[m, k]   with X' = X or g ⊙ X / rms(X)   (+ fused epilogue).
//
// The work is bound by the bytes of W (each weight is used for at most 80 rows), so the
// kernel is organised around the weight stream, not around the MMA:
//   * W is re-packed once into 16x16 tiles in the register order of the A operand of
//     mma.sync.m16n8k16 (out-features on the 16-row side), 512 contiguous bytes per tile,
//     tiles ordered [row tile / 8][k tile][row tile % 8] (the unit layout of pass_kernel.cuh,
//     which both kernels share).  A warp loads a tile with ONE 128-bit load per lane, fully
//     coalesced, straight into MMA registers: no shared-memory staging, no ldmatrix.
//   * A CTA owns R row tiles (16·R out-features) over the whole K; its 8 warps split K into 8
//     contiguous ranges, so every warp reads R sequential streams.  Loads are issued two
//     batches ahead (register double buffer), the first batch BEFORE griddepcontrol.wait so
//     that the weight stream of a kernel starts while its predecessor is still running.
//   * Activations are the B operand (tokens on the 8-column side).  An fp32 activation is split
//     x = hi + lo into two bf16 values and fed to two MMAs, which keeps ~16 mantissa bits;
//     products with bf16 weights are exact in the fp32 accumulator.
//   * RMSNorm is folded in: B carries g ⊙ x, each lane accumulates Σx² of what it loads, and
//     the per-row 1/rms is applied to the accumulators in the epilogue.
//   * The 8 per-warp partial sums are added in warp order through shared memory: fixed order,
//     no atomics.
// Batch invariance: an output element depends on its A row and its B column only, every
// column runs the same MMA sequence, so a row's result is the same whatever else (and however
// much) is in the launch.
#pragma once

#include "common.cuh"
#include "linear_fma.cuh"

namespace sdfp {

constexpr int kMmaThreads = 256;
constexpr int kMmaWarps = 8;

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

// x = hi + lo with hi = bf16(x), lo = bf16(x - hi); returns the two packed pairs.
__device__ __forceinline__ void split_pack(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
  const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0));
  const __nv_bfloat16 l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
  hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
}

struct XFrag {
  float2 lo8, hi8;  // x[m][16kt + 2q .. +1] and x[m][16kt + 2q + 8 .. +9]
};

// R row tiles per CTA, CG column groups of 8 rows (tokens), U k-tiles per load batch.
template <int R, int CG, int U>
__global__ void __launch_bounds__(kMmaThreads)
linear_mma_kernel(const uint4* __restrict__ W, const float* __restrict__ X, int ldx, int M, int K, int NT,
                  const float* __restrict__ gain, float eps, EpiParams ep) {
  extern __shared__ __align__(16) float s_red[];  // [warp][R][CG][lane][4]
  __shared__ float s_ss[kMmaWarps][CG * 8];
  __shared__ float s_inv[CG * 8];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, q = lane & 3;
  const int KT = K >> 4;
  const int ktw = (KT + kMmaWarps - 1) / kMmaWarps;
  const int kt0 = warp * ktw;
  const int kt1 = min(KT, kt0 + ktw);
  const int rt0 = blockIdx.x * R;

  pdl_launch_dependents();

  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  auto load_a = [&](uint4(&dst)[U][R], int ktb) {
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int kt = ktb + u, rt = rt0 + r;
        dst[u][r] = (kt < kt1 && rt < NT) ? __ldcs(W + (((size_t)(rt >> 3) * KT + kt) * 8 + (rt & 7)) * 32 + lane) : zero4;
      }
  };
  auto load_x = [&](XFrag(&dst)[U][CG], int ktb) {
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int cg = 0; cg < CG; ++cg) {
        const int kt = ktb + u, m = cg * 8 + g;
        XFrag f;
        f.lo8 = make_float2(0.f, 0.f);
        f.hi8 = make_float2(0.f, 0.f);
        if (kt < kt1 && m < M) {
          const float* xp = X + (size_t)m * ldx + kt * 16 + 2 * q;
          f.lo8 = ld_act2(xp);
          f.hi8 = ld_act2(xp + 8);
        }
        dst[u][cg] = f;
      }
  };

  uint4 a[U][R];
  load_a(a, kt0);  // weights do not depend on the preceding kernel

  pdl_wait();

  XFrag x[U][CG];
  load_x(x, kt0);

  float acc[R][CG][4];
  float ss[CG];
#pragma unroll
  for (int cg = 0; cg < CG; ++cg) {
    ss[cg] = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[r][cg][i] = 0.f;
  }

  for (int ktb = kt0; ktb < kt1; ktb += U) {
    uint4 an[U][R];
    XFrag xn[U][CG];
    load_a(an, ktb + U);
    load_x(xn, ktb + U);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float2 g0 = make_float2(1.f, 1.f), g1 = make_float2(1.f, 1.f);
      if (gain != nullptr && ktb + u < kt1) {
        const float* gp = gain + (ktb + u) * 16 + 2 * q;
        g0 = *reinterpret_cast<const float2*>(gp);
        g1 = *reinterpret_cast<const float2*>(gp + 8);
      }
#pragma unroll
      for (int cg = 0; cg < CG; ++cg) {
        const XFrag f = x[u][cg];
        ss[cg] = fmaf(f.lo8.x, f.lo8.x, ss[cg]);
        ss[cg] = fmaf(f.lo8.y, f.lo8.y, ss[cg]);
        ss[cg] = fmaf(f.hi8.x, f.hi8.x, ss[cg]);
        ss[cg] = fmaf(f.hi8.y, f.hi8.y, ss[cg]);
        uint32_t bh0, bl0, bh1, bl1;
        split_pack(f.lo8.x * g0.x, f.lo8.y * g0.y, bh0, bl0);
        split_pack(f.hi8.x * g1.x, f.hi8.y * g1.y, bh1, bl1);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          mma_bf16_16816(acc[r][cg], a[u][r], bh0, bh1);
          mma_bf16_16816(acc[r][cg], a[u][r], bl0, bl1);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
#pragma unroll
      for (int r = 0; r < R; ++r) a[u][r] = an[u][r];
#pragma unroll
      for (int cg = 0; cg < CG; ++cg) x[u][cg] = xn[u][cg];
    }
  }

  // per-warp partials -> shared memory
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int cg = 0; cg < CG; ++cg)
      *reinterpret_cast<float4*>(s_red + ((((size_t)warp * R + r) * CG + cg) * 32 + lane) * 4) =
          make_float4(acc[r][cg][0], acc[r][cg][1], acc[r][cg][2], acc[r][cg][3]);
#pragma unroll
  for (int cg = 0; cg < CG; ++cg) {
    float s = ss[cg];
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    if (q == 0) s_ss[warp][cg * 8 + g] = s;
  }
  __syncthreads();
  if (threadIdx.x < CG * 8) {
    float inv = 1.f;
    if (gain != nullptr) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kMmaWarps; ++w) s += s_ss[w][threadIdx.x];
      inv = rsqrtf(s / (float)K + eps);
    }
    s_inv[threadIdx.x] = inv;
  }
  __syncthreads();

  // add the 8 partials in warp order, apply the epilogue
  for (int it = threadIdx.x; it < R * CG * 64; it += kMmaThreads) {
    const int ch = it & 1;
    const int ln = (it >> 1) & 31;
    const int rc = it >> 6;
    const int cg = rc % CG, r = rc / CG;
    float v0 = 0.f, v1 = 0.f;
#pragma unroll
    for (int w = 0; w < kMmaWarps; ++w) {
      const float* p = s_red + ((((size_t)w * R + r) * CG + cg) * 32 + ln) * 4;
      v0 += p[ch];
      v1 += p[ch + 2];
    }
    const int m = cg * 8 + 2 * (ln & 3) + ch;
    const int rt = rt0 + r;
    if (m < M && rt < NT) {
      const float inv = s_inv[m];
      apply_epilogue<__nv_bfloat16>(ep, 8 * rt + (ln >> 2), m, v0 * inv, v1 * inv);
    }
  }
}

template <int R, int CG, int U>
inline cudaError_t launch_mma_t(const Launcher& L, const void* W, const float* X, int ldx, int M, int K, int NT,
                                const float* gain, float eps, const EpiParams& ep) {
  const size_t smem = (size_t)kMmaWarps * R * CG * 32 * 4 * sizeof(float);
  const int grid = (NT + R - 1) / R;
  return launch_kernel(L, linear_mma_kernel<R, CG, U>, dim3(grid), dim3(kMmaThreads), smem,
                       reinterpret_cast<const uint4*>(W), X, ldx, M, K, NT, gain, eps, ep);
}

// n_pairs = out_features / 2; W in the tile order written by pack_mma.
inline cudaError_t launch_linear_mma(const Launcher& L, int num_sms, const void* W, const float* X, int ldx, int M, int K,
                                     int n_pairs, const float* gain, float eps, const EpiParams& ep) {
  const int NT = n_pairs / 8;
  const int want = 2 * num_sms;  // CTAs needed to fill the machine at 2 per SM
  if (M <= 8) {
    if ((NT + 3) / 4 >= want) return launch_mma_t<4, 1, 2>(L, W, X, ldx, M, K, NT, gain, eps, ep);
    if ((NT + 1) / 2 >= want) return launch_mma_t<2, 1, 4>(L, W, X, ldx, M, K, NT, gain, eps, ep);
    return launch_mma_t<1, 1, 8>(L, W, X, ldx, M, K, NT, gain, eps, ep);
  }
  if (M <= 16) {
    if ((NT + 1) / 2 >= want) return launch_mma_t<2, 2, 2>(L, W, X, ldx, M, K, NT, gain, eps, ep);
    return launch_mma_t<1, 2, 4>(L, W, X, ldx, M, K, NT, gain, eps, ep);
  }
  if (M <= 32) {
    if ((NT + 1) / 2 >= want) return launch_mma_t<2, 4, 1>(L, W, X, ldx, M, K, NT, gain, eps, ep);
    return launch_mma_t<1, 4, 2>(L, W, X, ldx, M, K, NT, gain, eps, ep);
  }
  if (M <= 64) return launch_mma_t<1, 8, 1>(L, W, X, ldx, M, K, NT, gain, eps, ep);
  return launch_mma_t<1, 10, 1>(L, W, X, ldx, M, K, NT, gain, eps, ep);
}

}  // namespace sdfp
