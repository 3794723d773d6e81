// Causal attention over a whole prompt (the pass that fills the KV cache, Section II-A), one
// sequence at a time: row m (position m) attends keys 0..m of the cache the QKV epilogue of the
// same layer has just written.
//
// One CTA = (block of 64 query rows, head); its four warps own 16 query rows each and walk the key
// blocks 0..diagonal with the usual running max / running sum per row (exact softmax, rescaled as
// the maximum grows).  Both products run on mma.sync.m16n8k16 with fp32 accumulators:
//   S = Q K^T    Q is fp32: split q = hi + lo into bf16, two MMAs; K is bf16 in the cache
//   O += P V     P is fp32: split p = hi + lo, two MMAs; V is bf16 in the cache
// so nothing is rounded to 8 mantissa bits that the decode kernels keep in fp32.  K and V tiles are
// double-buffered in shared memory with 16-byte asynchronous copies; rows are padded by 16 bytes so
// that the 8 row addresses of an ldmatrix fall into different banks.
#pragma once

#include "common.cuh"
#include "linear_mma.cuh"
#include "pass_kernel.cuh"

namespace sdfp {

constexpr int kPfaThreads = 128;
constexpr int kPfaQ = 64;  // query rows per CTA
constexpr int kPfaK = 64;  // keys per block

template <int HD>
constexpr size_t prefill_attention_smem() {
  return (size_t)6 * kPfaQ * (HD + 8) * 2;  // Q hi, Q lo, 2 x K, 2 x V
}

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int HD>
__global__ void __launch_bounds__(kPfaThreads)
prefill_attention_kernel(const float* __restrict__ q, const __nv_bfloat16* __restrict__ kcache,
                         const __nv_bfloat16* __restrict__ vcache, float* __restrict__ out, int M, int n_heads, int max_seq,
                         int seq, float scale, unsigned char* __restrict__ img, int img_rb, int img_kb) {
  constexpr int LD = HD + 8;
  extern __shared__ __align__(16) unsigned char pfa_smem[];
  __nv_bfloat16* sQh = reinterpret_cast<__nv_bfloat16*>(pfa_smem);
  __nv_bfloat16* sQl = sQh + kPfaQ * LD;
  __nv_bfloat16* sK = sQl + kPfaQ * LD;   // [2][64][LD]
  __nv_bfloat16* sV = sK + 2 * kPfaK * LD;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, qd = lane & 3;
  // the longest blocks (most key blocks) first: they decide when the grid ends
  const int qb = (int)gridDim.x - 1 - (int)blockIdx.x, head = blockIdx.y;
  const int q0 = qb * kPfaQ;
  const size_t d_model = (size_t)n_heads * HD;
  const __nv_bfloat16* gK = kcache + ((size_t)seq * n_heads + head) * (size_t)max_seq * HD;
  const __nv_bfloat16* gV = vcache + ((size_t)seq * n_heads + head) * (size_t)max_seq * HD;

  pdl_wait();
  pdl_launch_dependents();

  auto load_kv = [&](int kb, int buf) {
    const int key0 = kb * kPfaK;
    constexpr int VPR = HD / 8;  // 16-byte vectors per row
    for (int v = tid; v < kPfaK * VPR; v += kPfaThreads) {
      const int key = v / VPR, j = v - key * VPR;
      __nv_bfloat16* dk = sK + ((size_t)buf * kPfaK + key) * LD + j * 8;
      __nv_bfloat16* dv = sV + ((size_t)buf * kPfaK + key) * LD + j * 8;
      if (key0 + key < M) {
        cp_async16(dk, gK + (size_t)(key0 + key) * HD + j * 8);
        cp_async16(dv, gV + (size_t)(key0 + key) * HD + j * 8);
      } else {  // beyond the prompt: never visible, but keep the tile finite
        *reinterpret_cast<uint4*>(dk) = make_uint4(0u, 0u, 0u, 0u);
        *reinterpret_cast<uint4*>(dv) = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    cp_async_commit();
  };
  load_kv(0, 0);

  // q rows of this block and head: fp32 -> bf16 hi + lo
  for (int e = tid; e < kPfaQ * (HD / 4); e += kPfaThreads) {
    const int i = e / (HD / 4), d = (e - i * (HD / 4)) * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q0 + i < M) v = ld_act4(q + (size_t)(q0 + i) * d_model + head * HD + d);
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
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // rows g and g + 8 of this warp
  const int row_a = q0 + warp * 16 + g, row_b = row_a + 8;

  for (int kb = 0; kb <= qb; ++kb) {
    const int buf = kb & 1;
    if (kb < qb) load_kv(kb + 1, buf ^ 1);
    if (kb < qb)
      cp_async_wait_group<1>();
    else
      cp_async_wait_group<0>();
    __syncthreads();  // tile kb (and, the first time, q) is visible to everyone

    // ---- S = Q K^T for 16 rows x 64 keys ----
    float s[kPfaK / 8][4];
#pragma unroll
    for (int j = 0; j < kPfaK / 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[j][e] = 0.f;
    const __nv_bfloat16* tK = sK + (size_t)buf * kPfaK * LD;
    const __nv_bfloat16* tV = sV + (size_t)buf * kPfaK * LD;
#pragma unroll
    for (int k16 = 0; k16 < HD / 16; ++k16) {
      uint32_t ah[4], al[4];
      const int arow = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, acol = k16 * 16 + (lane >> 4) * 8;
      ldsm_x4(ah, sQh + arow * LD + acol);
      ldsm_x4(al, sQl + arow * LD + acol);
#pragma unroll
      for (int j2 = 0; j2 < kPfaK / 16; ++j2) {  // two key groups of 8 per ldmatrix
        uint32_t b[4];
        const int key = j2 * 16 + (lane & 7) + (lane >> 4) * 8, dim = k16 * 16 + ((lane >> 3) & 1) * 8;
        ldsm_x4(b, tK + key * LD + dim);
        mma_16816(s[2 * j2], ah, b[0], b[1]);
        mma_16816(s[2 * j2], al, b[0], b[1]);
        mma_16816(s[2 * j2 + 1], ah, b[2], b[3]);
        mma_16816(s[2 * j2 + 1], al, b[2], b[3]);
      }
    }
    // ---- scale, causal mask, running max and sum ----
    const int key0 = kb * kPfaK;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < kPfaK / 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = key0 + j * 8 + 2 * qd + (e & 1);
        const int row = (e < 2) ? row_a : row_b;
        const float v = (key <= row) ? s[j][e] * scale : -INFINITY;
        s[j][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    float alpha[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r]);  // finite from the first block on: key 0 is visible to every row
      alpha[r] = __expf(m_run[r] - m_new);         // exp(-inf) = 0 the first time
      m_run[r] = m_new;
    }
    float ps[2] = {0.f, 0.f};
#pragma unroll
    for (int j = 0; j < kPfaK / 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float pv = __expf(s[j][e] - m_run[e >> 1]);  // masked entries: exp(-inf) = 0
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
#pragma unroll
    for (int k16 = 0; k16 < kPfaK / 16; ++k16) {
      uint32_t ph[4], pl[4];
      split_pack(s[2 * k16][0], s[2 * k16][1], ph[0], pl[0]);
      split_pack(s[2 * k16][2], s[2 * k16][3], ph[1], pl[1]);
      split_pack(s[2 * k16 + 1][0], s[2 * k16 + 1][1], ph[2], pl[2]);
      split_pack(s[2 * k16 + 1][2], s[2 * k16 + 1][3], ph[3], pl[3]);
#pragma unroll
      for (int d2 = 0; d2 < HD / 16; ++d2) {  // two dimension groups of 8 per ldmatrix
        uint32_t b[4];
        const int key = k16 * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, dim = d2 * 16 + (lane >> 4) * 8;
        ldsm_x4_trans(b, tV + key * LD + dim);
        mma_16816(o[2 * d2], ph, b[0], b[1]);
        mma_16816(o[2 * d2], pl, b[0], b[1]);
        mma_16816(o[2 * d2 + 1], ph, b[2], b[3]);
        mma_16816(o[2 * d2 + 1], pl, b[2], b[3]);
      }
    }
    __syncthreads();  // the tile may be overwritten by the copy issued at the top of the next round
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  const float inv_a = 1.0f / l_run[0], inv_b = 1.0f / l_run[1];
  // The result goes out as fp32 rows, or (img non-null) straight into the activation image of the
  // O-projection on the dense path: bf16 hi + lo, two neighbouring columns per 4-byte store (layout
  // as in attn_store of attention.cuh: row block img_rb, img_kb k blocks of 64).
  auto put = [&](int m, int col, float x0, float x1) {
    if (img == nullptr) {
      *reinterpret_cast<float2*>(out + (size_t)m * d_model + col) = make_float2(x0, x1);
      return;
    }
    const int rb = m / img_rb, tm = m - rb * img_rb, kg = col >> 3;
    unsigned char* p = img + ((size_t)rb * img_kb + (kg >> 3)) * ((size_t)img_rb * 256) + (size_t)(kg & 7) * (img_rb * 32) +
                       (size_t)(tm >> 3) * 128 + (tm & 7) * 16 + (col & 7) * 2;
    uint32_t hi, lo;
    split_pack(x0, x1, hi, lo);
    *reinterpret_cast<uint32_t*>(p) = hi;
    *reinterpret_cast<uint32_t*>(p + (size_t)img_rb * 16) = lo;
  };
#pragma unroll
  for (int j = 0; j < HD / 8; ++j) {
    const int d = j * 8 + 2 * qd;
    if (row_a < M) put(row_a, head * HD + d, o[j][0] * inv_a, o[j][1] * inv_a);
    if (row_b < M) put(row_b, head * HD + d, o[j][2] * inv_b, o[j][3] * inv_b);
  }
}

}  // namespace sdfp
