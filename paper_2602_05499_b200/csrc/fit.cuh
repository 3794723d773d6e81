// Stage A of Algorithm 1 on the GPU: the per-layer empirical-Fisher trace
//   T_l = (1/N) sum_i || grad_{theta_l} f(z_i, theta) ||^2                     (Eq. 11; Eq. 8-9)
// and the layer-wise FIT form  FIT_l = sum_{tensors t of layer l} T_t * mean(theta_t^2)   (Eq. 7,
// with the perturbation of removing the layer read as delta theta = -theta).
//
// f(z_i, theta) is the mean next-token cross-entropy of one calibration sequence: one forward pass
// that keeps the activations, one backward pass that carries the gradient with respect to the
// ACTIVATIONS only.  The gradient of a weight matrix is never formed: for y = x W^T over T rows,
// dW = dY^T X, so
//   ||dW||_F^2 = sum_{t,t'} (dY dY^T)[t,t'] * (X X^T)[t,t']
// - two T x T Gram matrices and their elementwise dot product (T is a calibration sequence's
// length, tens of tokens), instead of an [out, in] matrix per weight.  A norm gain's gradient is a
// vector and is summed directly.
//
// Everything is fp32 on CUDA cores with fp64 accumulation of the squared norms; weights are read in
// their storage type (fp32 or bf16) from the caller's row-major [out, in] matrices.  This is the
// offline, one-shot stage of the method: the kernels are plain (register-tiled GEMMs through shared memory,
// one block per (row, head) in attention) and every reduction runs in a fixed order, so the scores
// are reproducible bit for bit.
#pragma once

#include <algorithm>
#include <cmath>
#include <vector>

#include "../../include/sdfp.h"
#include "common.cuh"

namespace sdfp {
namespace fit {


__device__ __forceinline__ float wload(const float* p) { return *p; }
__device__ __forceinline__ float wload(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// Tiled fp32 GEMMs: a 64 x 64 output tile per block of 256 threads, 4 x 4 outputs per thread, the
// contraction in steps of 16 through shared memory.  Rows (tokens) are few (a calibration sequence),
// so every weight is read once per GEMM.
constexpr int kGT = 64, kGK = 16;

// C[T, N] = A[T, K] * W[N, K]^T
template <typename WT>
__global__ void __launch_bounds__(256) gemm_nt_kernel(const float* __restrict__ A, const WT* __restrict__ W, float* __restrict__ C,
                                                       int T, int N, int K) {
  __shared__ __align__(16) float sA[kGK][kGT + 4], sW[kGK][kGT + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int t0 = blockIdx.y * kGT, n0 = blockIdx.x * kGT;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += kGK) {
    for (int e = tid; e < kGT * kGK; e += 256) {  // element (row r, column kk): consecutive threads along k
      const int r = e >> 4, kk = e & 15;
      sA[kk][r] = (t0 + r < T && k0 + kk < K) ? A[(size_t)(t0 + r) * K + k0 + kk] : 0.f;
      sW[kk][r] = (n0 + r < N && k0 + kk < K) ? wload(W + (size_t)(n0 + r) * K + k0 + kk) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kGK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&sA[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&sW[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j2 = 0; j2 < 4; ++j2) acc[i][j2] = fmaf(av[i], bv[j2], acc[i][j2]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j2 = 0; j2 < 4; ++j2) {
      const int t = t0 + ty * 4 + i, n = n0 + tx * 4 + j2;
      if (t < T && n < N) C[(size_t)t * N + n] = acc[i][j2];
    }
}

// C[T, K] (+)= A[T, N] * W[N, K]     (the gradient of a linear layer's input)
template <typename WT>
__global__ void __launch_bounds__(256) gemm_nn_kernel(const float* __restrict__ A, const WT* __restrict__ W, float* __restrict__ C,
                                                       int T, int N, int K, int accumulate) {
  __shared__ __align__(16) float sA[kGK][kGT + 4], sW[kGK][kGT + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int t0 = blockIdx.y * kGT, c0 = blockIdx.x * kGT;
  float acc[4][4] = {};
  for (int n0 = 0; n0 < N; n0 += kGK) {
    for (int e = tid; e < kGT * kGK; e += 256) {
      const int r = e >> 4, nn = e & 15;  // A: (row r, contraction index nn), consecutive threads along n
      sA[nn][r] = (t0 + r < T && n0 + nn < N) ? A[(size_t)(t0 + r) * N + n0 + nn] : 0.f;
      const int wn = e >> 6, wc = e & 63;  // W: (contraction index wn, column wc), consecutive threads along the row
      sW[wn][wc] = (n0 + wn < N && c0 + wc < K) ? wload(W + (size_t)(n0 + wn) * K + c0 + wc) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int nn = 0; nn < kGK; ++nn) {
      const float4 a = *reinterpret_cast<const float4*>(&sA[nn][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&sW[nn][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j2 = 0; j2 < 4; ++j2) acc[i][j2] = fmaf(av[i], bv[j2], acc[i][j2]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j2 = 0; j2 < 4; ++j2) {
      const int t = t0 + ty * 4 + i, c = c0 + tx * 4 + j2;
      if (t < T && c < K) C[(size_t)t * K + c] = (accumulate ? C[(size_t)t * K + c] : 0.f) + acc[i][j2];
    }
}

// fixed-order block sum (blockDim.x a multiple of 32, at most 1024); every thread gets the result
__device__ __forceinline__ double block_sum_d(double v, double* s_red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  double r = 0.0;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r += s_red[w];
  return r;
}

// h[t, :] = E[token_t, :]
template <typename WT>
__global__ void embed_kernel(const int* __restrict__ tok, const WT* __restrict__ E, float* __restrict__ h, int d) {
  const int t = blockIdx.x;
  for (int k = threadIdx.x; k < d; k += blockDim.x) h[(size_t)t * d + k] = wload(E + (size_t)tok[t] * d + k);
}

// y = x * r * g with r = 1/sqrt(mean(x^2) + eps); keeps r per row
template <typename WT>
__global__ void __launch_bounds__(256) rmsnorm_fwd_kernel(const float* __restrict__ x, const WT* __restrict__ g, float* __restrict__ y,
                                                           float* __restrict__ inv, int d, float eps) {
  __shared__ double s_red[8];
  const int t = blockIdx.x;
  double s = 0.0;
  for (int k = threadIdx.x; k < d; k += blockDim.x) {
    const double v = x[(size_t)t * d + k];
    s += v * v;
  }
  const double tot = block_sum_d(s, s_red);
  const float r = (float)(1.0 / sqrt(tot / d + (double)eps));
  if (threadIdx.x == 0) inv[t] = r;
  for (int k = threadIdx.x; k < d; k += blockDim.x) y[(size_t)t * d + k] = x[(size_t)t * d + k] * r * wload(g + k);
}

// Given dy: dx (+)= r z - x r^3 mean(z x) with z = g * dy; dgain[k] += sum_t dy[t,k] x[t,k] r[t] is
// taken by gain_grad_sq_kernel below.
template <typename WT>
__global__ void __launch_bounds__(256) rmsnorm_bwd_kernel(const float* __restrict__ dy, const float* __restrict__ x,
                                                           const WT* __restrict__ g, const float* __restrict__ inv,
                                                           float* __restrict__ dx, int d, int accumulate) {
  __shared__ double s_red[8];
  const int t = blockIdx.x;
  const float r = inv[t];
  double s = 0.0;
  for (int k = threadIdx.x; k < d; k += blockDim.x)
    s += (double)(wload(g + k) * dy[(size_t)t * d + k]) * (double)x[(size_t)t * d + k];
  const float mzx = (float)(block_sum_d(s, s_red) / d);
  for (int k = threadIdx.x; k < d; k += blockDim.x) {
    const size_t i = (size_t)t * d + k;
    const float v = r * wload(g + k) * dy[i] - x[i] * r * r * r * mzx;
    dx[i] = (accumulate ? dx[i] : 0.f) + v;
  }
}

// out += || sum_t dy[t,:] * x[t,:] * r[t] ||^2   (squared norm of a gain's gradient); one block
__global__ void __launch_bounds__(256) gain_grad_sq_kernel(const float* __restrict__ dy, const float* __restrict__ x,
                                                            const float* __restrict__ inv, int T, int d, double* out) {
  __shared__ double s_red[8];
  double s = 0.0;
  for (int k = threadIdx.x; k < d; k += blockDim.x) {
    double gk = 0.0;
    for (int t = 0; t < T; ++t) gk += (double)dy[(size_t)t * d + k] * (double)x[(size_t)t * d + k] * (double)inv[t];
    s += gk * gk;
  }
  const double tot = block_sum_d(s, s_red);
  if (threadIdx.x == 0) *out += tot;
}

// Rotary embedding of q or k in place, pairs (i, i + hd/2) of every head; dir = +1 forward, -1 the
// transpose (the backward pass: the rotation is orthogonal).  cs, sn: [T][hd/2], positions 0..T-1.
__global__ void rope_kernel(float* __restrict__ x, const float* __restrict__ cs, const float* __restrict__ sn, int n_heads, int hd,
                            float dir) {
  const int t = blockIdx.x, hp = hd >> 1;
  for (int e = threadIdx.x; e < n_heads * hp; e += blockDim.x) {
    const int h = e / hp, i = e - h * hp;
    float* p = x + (size_t)t * n_heads * hd + h * hd;
    const float c = cs[t * hp + i], s = dir * sn[t * hp + i];
    const float a = p[i], b = p[i + hp];
    p[i] = a * c - b * s;
    p[i + hp] = b * c + a * s;
  }
}

// Causal attention forward, one block per (row t, head): P[h, t, 0..t] = softmax(q_t K^T / sqrt(hd)),
// a[t, head] = P V.  P is kept for the backward pass.  Dynamic shared memory: T floats.
__global__ void __launch_bounds__(128) attn_fwd_kernel(const float* __restrict__ q, const float* __restrict__ k,
                                                        const float* __restrict__ v, float* __restrict__ P, float* __restrict__ a,
                                                        int T, int n_heads, int hd, float scale) {
  extern __shared__ float s_p[];
  __shared__ double s_red[4];
  const int t = blockIdx.x, h = blockIdx.y, d_model = n_heads * hd;
  const float* qt = q + (size_t)t * d_model + h * hd;
  float mx = -INFINITY;
  for (int j = threadIdx.x; j <= t; j += blockDim.x) {
    const float* kj = k + (size_t)j * d_model + h * hd;
    float s = 0.f;
    for (int d = 0; d < hd; ++d) s = fmaf(qt[d], kj[d], s);
    s *= scale;
    s_p[j] = s;
    mx = fmaxf(mx, s);
  }
  mx = warp_max(mx);
  __shared__ float s_mx[4];
  if ((threadIdx.x & 31) == 0) s_mx[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = fmaxf(fmaxf(s_mx[0], s_mx[1]), fmaxf(s_mx[2], s_mx[3]));
  double part = 0.0;
  for (int j = threadIdx.x; j <= t; j += blockDim.x) {
    const float e = expf(s_p[j] - mx);
    s_p[j] = e;
    part += e;
  }
  const float inv = (float)(1.0 / block_sum_d(part, s_red));
  float* Pt = P + ((size_t)h * T + t) * T;
  for (int j = threadIdx.x; j < T; j += blockDim.x) {
    const float pj = j <= t ? s_p[j] * inv : 0.f;
    Pt[j] = pj;
    if (j <= t) s_p[j] = pj;
  }
  __syncthreads();
  for (int d = threadIdx.x; d < hd; d += blockDim.x) {
    float o = 0.f;
    for (int j = 0; j <= t; ++j) o = fmaf(s_p[j], v[(size_t)j * d_model + h * hd + d], o);
    a[(size_t)t * d_model + h * hd + d] = o;
  }
}

// Backward, step 1, one block per (row t, head): dS[h,t,j] = P (dP - sum_j P dP) with dP = da V^T,
// and dq[t, head] = dS K * scale.  Dynamic shared memory: T floats.
__global__ void __launch_bounds__(128) attn_bwd_q_kernel(const float* __restrict__ da, const float* __restrict__ k,
                                                          const float* __restrict__ v, const float* __restrict__ P,
                                                          float* __restrict__ dS, float* __restrict__ dq, int T, int n_heads, int hd,
                                                          float scale) {
  extern __shared__ float s_ds[];
  __shared__ double s_red[4];
  const int t = blockIdx.x, h = blockIdx.y, d_model = n_heads * hd;
  const float* dat = da + (size_t)t * d_model + h * hd;
  const float* Pt = P + ((size_t)h * T + t) * T;
  double part = 0.0;
  for (int j = threadIdx.x; j <= t; j += blockDim.x) {
    const float* vj = v + (size_t)j * d_model + h * hd;
    float dp = 0.f;
    for (int d = 0; d < hd; ++d) dp = fmaf(dat[d], vj[d], dp);
    s_ds[j] = dp;
    part += (double)Pt[j] * dp;
  }
  const float rs = (float)block_sum_d(part, s_red);
  float* dSt = dS + ((size_t)h * T + t) * T;
  for (int j = threadIdx.x; j < T; j += blockDim.x) {
    const float x = j <= t ? Pt[j] * (s_ds[j] - rs) : 0.f;
    dSt[j] = x;
    if (j <= t) s_ds[j] = x;
  }
  __syncthreads();
  for (int d = threadIdx.x; d < hd; d += blockDim.x) {
    float o = 0.f;
    for (int j = 0; j <= t; ++j) o = fmaf(s_ds[j], k[(size_t)j * d_model + h * hd + d], o);
    dq[(size_t)t * d_model + h * hd + d] = o * scale;
  }
}

// Backward, step 2, one block per (key j, head): dk[j] = sum_{t>=j} dS[t,j] q[t] * scale, dv[j] = sum_{t>=j} P[t,j] da[t]
__global__ void __launch_bounds__(128) attn_bwd_kv_kernel(const float* __restrict__ da, const float* __restrict__ q,
                                                           const float* __restrict__ P, const float* __restrict__ dS,
                                                           float* __restrict__ dk, float* __restrict__ dv, int T, int n_heads, int hd,
                                                           float scale) {
  const int j = blockIdx.x, h = blockIdx.y, d_model = n_heads * hd;
  for (int d = threadIdx.x; d < hd; d += blockDim.x) {
    float ak = 0.f, av = 0.f;
    for (int t = j; t < T; ++t) {
      const size_t pi = ((size_t)h * T + t) * T + j;
      ak = fmaf(dS[pi], q[(size_t)t * d_model + h * hd + d], ak);
      av = fmaf(P[pi], da[(size_t)t * d_model + h * hd + d], av);
    }
    dk[(size_t)j * d_model + h * hd + d] = ak * scale;
    dv[(size_t)j * d_model + h * hd + d] = av;
  }
}

// u = silu(gate) * up
__global__ void swiglu_fwd_kernel(const float* __restrict__ gt, const float* __restrict__ up, float* __restrict__ u, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const float g = gt[i];
    u[i] = g / (1.0f + expf(-g)) * up[i];
  }
}
// dgate = du * up * silu'(gate), dup = du * silu(gate)
__global__ void swiglu_bwd_kernel(const float* __restrict__ du, const float* __restrict__ gt, const float* __restrict__ up,
                                  float* __restrict__ dgt, float* __restrict__ dup, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const float g = gt[i], sg = 1.0f / (1.0f + expf(-g));
    dgt[i] = du[i] * up[i] * sg * (1.0f + g * (1.0f - sg));
    dup[i] = du[i] * g * sg;
  }
}
__global__ void add_kernel(float* __restrict__ dst, const float* __restrict__ a, const float* __restrict__ b, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) dst[i] = a[i] + b[i];
}

// Mean next-token cross-entropy: dlogits[t,:] = (softmax(logits[t,:]) - onehot(target_t)) / T, in place; loss[t] kept
__global__ void __launch_bounds__(256) ce_bwd_kernel(float* __restrict__ logits, const int* __restrict__ target, int V, int T,
                                                      float* __restrict__ loss) {
  __shared__ double s_red[8];
  __shared__ float s_mx[8];
  const int t = blockIdx.x;
  float* l = logits + (size_t)t * V;
  float mx = -INFINITY;
  for (int v = threadIdx.x; v < V; v += blockDim.x) mx = fmaxf(mx, l[v]);
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0) s_mx[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = s_mx[0];
  for (int w = 1; w < 8; ++w) mx = fmaxf(mx, s_mx[w]);
  double part = 0.0;
  for (int v = threadIdx.x; v < V; v += blockDim.x) part += exp((double)l[v] - (double)mx);
  const double tot = block_sum_d(part, s_red);
  const int y = target[t];
  if (threadIdx.x == 0) loss[t] = (float)(log(tot) + (double)mx - (double)l[y]);
  __syncthreads();
  for (int v = threadIdx.x; v < V; v += blockDim.x) {
    const double pv = exp((double)l[v] - (double)mx) / tot;
    l[v] = (float)((pv - (v == y ? 1.0 : 0.0)) / T);
  }
}

// G[t, t'] = A[t,:] . A[t',:]  (fp64), one block per pair
__global__ void __launch_bounds__(128) gram_kernel(const float* __restrict__ A, int n, int T, double* __restrict__ G) {
  __shared__ double s_red[4];
  const int t = blockIdx.x, u = blockIdx.y;
  if (u > t) return;  // symmetric: the lower triangle is computed and mirrored
  const float* a = A + (size_t)t * n;
  const float* b = A + (size_t)u * n;
  double s = 0.0;
  for (int k = threadIdx.x; k < n; k += blockDim.x) s += (double)a[k] * (double)b[k];
  const double tot = block_sum_d(s, s_red);
  if (threadIdx.x == 0) {
    G[(size_t)t * T + u] = tot;
    G[(size_t)u * T + t] = tot;
  }
}
// out += sum_i G1[i] * G2[i]; one block
__global__ void __launch_bounds__(256) gram_dot_kernel(const double* __restrict__ G1, const double* __restrict__ G2, int n,
                                                        double* out) {
  __shared__ double s_red[8];
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) s += G1[i] * G2[i];
  const double tot = block_sum_d(s, s_red);
  if (threadIdx.x == 0) *out += tot;
}
// mean of w^2 over n elements in two fixed-order steps: per-block partial sums, then one block adds them
constexpr int kMsBlocks = 592;
template <typename WT>
__global__ void __launch_bounds__(256) sum_sq_partial_kernel(const WT* __restrict__ w, size_t n, double* __restrict__ partial) {
  __shared__ double s_red[8];
  double s = 0.0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const double v = wload(w + i);
    s += v * v;
  }
  const double tot = block_sum_d(s, s_red);
  if (threadIdx.x == 0) partial[blockIdx.x] = tot;
}
__global__ void __launch_bounds__(256) mean_finish_kernel(const double* __restrict__ partial, int n_part, double n, double* out) {
  __shared__ double s_red[8];
  double s = 0.0;
  for (int i = threadIdx.x; i < n_part; i += blockDim.x) s += partial[i];
  const double tot = block_sum_d(s, s_red);
  if (threadIdx.x == 0) *out = tot / n;
}

// ---- host side --------------------------------------------------------------------------------------
enum Tensor { T_WQ = 0, T_WK, T_WV, T_WO, T_GATE, T_UP, T_DOWN, T_ATTN_NORM, T_FFN_NORM, kTensors };

struct Arena {  // device buffers of one call, freed together
  std::vector<void*> ptrs;
  cudaError_t err = cudaSuccess;
  template <typename T>
  T* get(size_t n) {
    void* p = nullptr;
    if (err == cudaSuccess) err = cudaMalloc(&p, std::max<size_t>(n * sizeof(T), 16));
    if (err != cudaSuccess) return nullptr;
    ptrs.push_back(p);
    return reinterpret_cast<T*>(p);
  }
  ~Arena() {
    for (void* p : ptrs) cudaFree(p);
  }
};

#define FIT_OK(call)                      \
  do {                                    \
    cudaError_t e_ = (call);              \
    if (e_ != cudaSuccess) return e_;     \
  } while (0)

template <typename WT>
cudaError_t run(const sdfp_config& g, const sdfp_weights* w, cudaStream_t st, const int32_t* tokens, int n_seq, int seq_len,
                double* out_trace, double* out_fit) {
  const int L = g.n_layers, d = g.d_model, f = g.d_ffn, V = g.vocab, H = g.n_heads, hd = g.head_dim, T = seq_len - 1;
  const float scale = 1.0f / std::sqrt((float)hd);
  Arena A;
  const size_t Td = (size_t)T * d, Tf = (size_t)T * f;
  // activations kept for the backward pass
  std::vector<float*> Hs(L + 1), Hmid(L), x1(L), q(L), k(L), v(L), P(L), a(L), x2(L), gt(L), up(L), u(L), inv1(L), inv2(L);
  for (int l = 0; l <= L; ++l) Hs[l] = A.get<float>(Td);
  for (int l = 0; l < L; ++l) {
    Hmid[l] = A.get<float>(Td); x1[l] = A.get<float>(Td); q[l] = A.get<float>(Td); k[l] = A.get<float>(Td); v[l] = A.get<float>(Td);
    P[l] = A.get<float>((size_t)H * T * T); a[l] = A.get<float>(Td); x2[l] = A.get<float>(Td);
    gt[l] = A.get<float>(Tf); up[l] = A.get<float>(Tf); u[l] = A.get<float>(Tf);
    inv1[l] = A.get<float>(T); inv2[l] = A.get<float>(T);
  }
  float *xf = A.get<float>(Td), *invf = A.get<float>(T), *logits = A.get<float>((size_t)T * V), *loss = A.get<float>(T);
  float *tmp = A.get<float>(Td), *dH = A.get<float>(Td), *dx = A.get<float>(Td), *da = A.get<float>(Td);
  float *dq = A.get<float>(Td), *dk = A.get<float>(Td), *dv = A.get<float>(Td), *dS = A.get<float>((size_t)H * T * T);
  float *du = A.get<float>(Tf), *dgt = A.get<float>(Tf), *dup = A.get<float>(Tf);
  double *G1 = A.get<double>((size_t)T * T), *G2 = A.get<double>((size_t)T * T);
  double *sq = A.get<double>((size_t)L * kTensors), *msq = A.get<double>((size_t)L * kTensors);
  double* ms_part = A.get<double>(kMsBlocks);
  int* tok = A.get<int>(seq_len);
  float *cs = A.get<float>((size_t)T * (hd / 2)), *sn = A.get<float>((size_t)T * (hd / 2));
  if (A.err != cudaSuccess) return A.err;
  FIT_OK(cudaMemsetAsync(sq, 0, (size_t)L * kTensors * sizeof(double), st));
  {
    const int hp = hd / 2;
    std::vector<float> hc((size_t)T * hp), hs((size_t)T * hp);
    for (int i = 0; i < hp; ++i) {
      const double inv = std::pow((double)g.rope_theta, -2.0 * i / hd);
      for (int t = 0; t < T; ++t) {
        hc[(size_t)t * hp + i] = (float)std::cos(t * inv);
        hs[(size_t)t * hp + i] = (float)std::sin(t * inv);
      }
    }
    FIT_OK(cudaMemcpyAsync(cs, hc.data(), hc.size() * 4, cudaMemcpyHostToDevice, st));
    FIT_OK(cudaMemcpyAsync(sn, hs.data(), hs.size() * 4, cudaMemcpyHostToDevice, st));
    FIT_OK(cudaStreamSynchronize(st));
  }
  auto W = [&](const void* const* arr, int l) { return reinterpret_cast<const WT*>(arr[l]); };
  auto nt = [&](const float* Ain, const WT* Wm, float* C, int N, int K) {  // C[T,N] = A[T,K] W[N,K]^T
    gemm_nt_kernel<WT><<<dim3((N + kGT - 1) / kGT, (T + kGT - 1) / kGT), 256, 0, st>>>(Ain, Wm, C, T, N, K);
  };
  auto nn = [&](const float* Ain, const WT* Wm, float* C, int N, int K, int acc) {  // C[T,K] (+)= A[T,N] W[N,K]
    gemm_nn_kernel<WT><<<dim3((K + kGT - 1) / kGT, (T + kGT - 1) / kGT), 256, 0, st>>>(Ain, Wm, C, T, N, K, acc);
  };
  auto gram = [&](const float* Ain, int n, double* G) { gram_kernel<<<dim3(T, T), 128, 0, st>>>(Ain, n, T, G); };
  auto gdot = [&](int l, int tensor) { gram_dot_kernel<<<1, 256, 0, st>>>(G1, G2, T * T, sq + (size_t)l * kTensors + tensor); };
  const int eb = 592;  // blocks of the elementwise kernels

  for (int s = 0; s < n_seq; ++s) {
    FIT_OK(cudaMemcpyAsync(tok, tokens + (size_t)s * seq_len, (size_t)seq_len * 4, cudaMemcpyHostToDevice, st));
    // ---- forward ----
    embed_kernel<WT><<<T, 256, 0, st>>>(tok, reinterpret_cast<const WT*>(w->tok_embed), Hs[0], d);
    for (int l = 0; l < L; ++l) {
      rmsnorm_fwd_kernel<WT><<<T, 256, 0, st>>>(Hs[l], W(w->attn_norm, l), x1[l], inv1[l], d, g.rms_eps);
      nt(x1[l], W(w->wq, l), q[l], d, d);
      nt(x1[l], W(w->wk, l), k[l], d, d);
      nt(x1[l], W(w->wv, l), v[l], d, d);
      rope_kernel<<<T, 128, 0, st>>>(q[l], cs, sn, H, hd, 1.f);
      rope_kernel<<<T, 128, 0, st>>>(k[l], cs, sn, H, hd, 1.f);
      attn_fwd_kernel<<<dim3(T, H), 128, T * sizeof(float), st>>>(q[l], k[l], v[l], P[l], a[l], T, H, hd, scale);
      nt(a[l], W(w->wo, l), tmp, d, d);
      add_kernel<<<eb, 256, 0, st>>>(Hmid[l], Hs[l], tmp, Td);
      rmsnorm_fwd_kernel<WT><<<T, 256, 0, st>>>(Hmid[l], W(w->ffn_norm, l), x2[l], inv2[l], d, g.rms_eps);
      nt(x2[l], W(w->w_gate, l), gt[l], f, d);
      nt(x2[l], W(w->w_up, l), up[l], f, d);
      swiglu_fwd_kernel<<<eb, 256, 0, st>>>(gt[l], up[l], u[l], Tf);
      nt(u[l], W(w->w_down, l), tmp, d, f);
      add_kernel<<<eb, 256, 0, st>>>(Hs[l + 1], Hmid[l], tmp, Td);
    }
    rmsnorm_fwd_kernel<WT><<<T, 256, 0, st>>>(Hs[L], reinterpret_cast<const WT*>(w->final_norm), xf, invf, d, g.rms_eps);
    nt(xf, reinterpret_cast<const WT*>(w->lm_head), logits, V, d);
    ce_bwd_kernel<<<T, 256, 0, st>>>(logits, tok + 1, V, T, loss);  // logits now hold d f / d logits
    // ---- backward: gradients with respect to activations, squared norms of the weight gradients by Gram matrices ----
    nn(logits, reinterpret_cast<const WT*>(w->lm_head), dx, V, d, 0);
    rmsnorm_bwd_kernel<WT><<<T, 256, 0, st>>>(dx, Hs[L], reinterpret_cast<const WT*>(w->final_norm), invf, dH, d, 0);
    for (int l = L - 1; l >= 0; --l) {
      // FFN block: H[l+1] = Hmid + u Wd^T
      gram(dH, d, G1);
      gram(u[l], f, G2);
      gdot(l, T_DOWN);
      nn(dH, W(w->w_down, l), du, d, f, 0);
      swiglu_bwd_kernel<<<eb, 256, 0, st>>>(du, gt[l], up[l], dgt, dup, Tf);
      gram(x2[l], d, G2);
      gram(dgt, f, G1);
      gdot(l, T_GATE);
      gram(dup, f, G1);
      gdot(l, T_UP);
      nn(dgt, W(w->w_gate, l), dx, f, d, 0);
      nn(dup, W(w->w_up, l), dx, f, d, 1);
      gain_grad_sq_kernel<<<1, 256, 0, st>>>(dx, Hmid[l], inv2[l], T, d, sq + (size_t)l * kTensors + T_FFN_NORM);
      rmsnorm_bwd_kernel<WT><<<T, 256, 0, st>>>(dx, Hmid[l], W(w->ffn_norm, l), inv2[l], dH, d, 1);  // dH is now d f / d Hmid
      // attention block: Hmid = H[l] + a Wo^T
      gram(dH, d, G1);
      gram(a[l], d, G2);
      gdot(l, T_WO);
      nn(dH, W(w->wo, l), da, d, d, 0);
      attn_bwd_q_kernel<<<dim3(T, H), 128, T * sizeof(float), st>>>(da, k[l], v[l], P[l], dS, dq, T, H, hd, scale);
      attn_bwd_kv_kernel<<<dim3(T, H), 128, 0, st>>>(da, q[l], P[l], dS, dk, dv, T, H, hd, scale);
      rope_kernel<<<T, 128, 0, st>>>(dq, cs, sn, H, hd, -1.f);
      rope_kernel<<<T, 128, 0, st>>>(dk, cs, sn, H, hd, -1.f);
      gram(x1[l], d, G2);
      gram(dq, d, G1);
      gdot(l, T_WQ);
      gram(dk, d, G1);
      gdot(l, T_WK);
      gram(dv, d, G1);
      gdot(l, T_WV);
      nn(dq, W(w->wq, l), dx, d, d, 0);
      nn(dk, W(w->wk, l), dx, d, d, 1);
      nn(dv, W(w->wv, l), dx, d, d, 1);
      gain_grad_sq_kernel<<<1, 256, 0, st>>>(dx, Hs[l], inv1[l], T, d, sq + (size_t)l * kTensors + T_ATTN_NORM);
      rmsnorm_bwd_kernel<WT><<<T, 256, 0, st>>>(dx, Hs[l], W(w->attn_norm, l), inv1[l], dH, d, 1);  // d f / d H[l]
    }
    FIT_OK(cudaGetLastError());
  }
  // mean(theta^2) per tensor
  for (int l = 0; l < L; ++l) {
    const void* ptr[kTensors] = {w->wq[l], w->wk[l], w->wv[l], w->wo[l], w->w_gate[l], w->w_up[l], w->w_down[l], w->attn_norm[l], w->ffn_norm[l]};
    const size_t n[kTensors] = {(size_t)d * d, (size_t)d * d, (size_t)d * d, (size_t)d * d, (size_t)f * d, (size_t)f * d, (size_t)d * f, (size_t)d, (size_t)d};
    for (int t = 0; t < kTensors; ++t) {
      sum_sq_partial_kernel<WT><<<kMsBlocks, 256, 0, st>>>(reinterpret_cast<const WT*>(ptr[t]), n[t], ms_part);
      mean_finish_kernel<<<1, 256, 0, st>>>(ms_part, kMsBlocks, (double)n[t], msq + (size_t)l * kTensors + t);
    }
  }
  FIT_OK(cudaGetLastError());
  std::vector<double> hsq((size_t)L * kTensors), hms((size_t)L * kTensors);
  FIT_OK(cudaMemcpyAsync(hsq.data(), sq, hsq.size() * sizeof(double), cudaMemcpyDeviceToHost, st));
  FIT_OK(cudaMemcpyAsync(hms.data(), msq, hms.size() * sizeof(double), cudaMemcpyDeviceToHost, st));
  FIT_OK(cudaStreamSynchronize(st));
  for (int l = 0; l < L; ++l) {
    double tr = 0.0, ft = 0.0;
    for (int t = 0; t < kTensors; ++t) {
      const double Tt = hsq[(size_t)l * kTensors + t] / n_seq;
      tr += Tt;
      ft += Tt * hms[(size_t)l * kTensors + t];
    }
    out_trace[l] = tr;
    if (out_fit) out_fit[l] = ft;
  }
  return cudaSuccess;
}
#undef FIT_OK

}  // namespace fit
}  // namespace sdfp
