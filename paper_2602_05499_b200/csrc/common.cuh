// Shared device helpers of the SDFP speculative-decode library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sdfp {

constexpr int kMaxRows = 80;    // rows (tokens) one pass may carry: 8 sequences x (k = 8 drafts + 1) = 72, in column groups of 8
constexpr int kAttnChunk = 64;  // keys per attention work unit; fixed so that a
                                // row's result never depends on the context length
                                // of other rows or on how many rows share the sweep

// ---- programmatic dependent launch -------------------------------------------------
// Every kernel of a pass is launched with the programmatic-stream-serialization
// attribute.  A kernel may touch weights (constant for the life of the context)
// before pdl_wait(); it must not touch anything another kernel writes until
// pdl_wait() has returned, which happens once all preceding kernels in the stream
// have completed and flushed their writes.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---- host-side launch with the programmatic-dependent-launch attribute ---------
struct Launcher {
  cudaStream_t stream = nullptr;
  bool pdl = true;
  long long* count = nullptr;  // kernels launched (or captured) so far
};

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(const Launcher& L, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 Args&&... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = L.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = L.pdl ? 1 : 0;
  if (L.count) *L.count += 1;
  return cudaLaunchKernelEx(&lc, kernel, KArgs(static_cast<Args&&>(args))...);
}

// ---- loads of data another kernel of the same stream wrote ------------------------
// With programmatic dependent launch a kernel starts (and its SM's L1 is invalidated)
// while its predecessors are still running, so a line of an activation buffer can enter
// L1 after that invalidation and before the predecessor's final write.  Everything that
// is not constant for the life of the context is therefore read through L2 (ld.global.cg).
__device__ __forceinline__ float ld_act(const float* p) { return __ldcg(p); }
__device__ __forceinline__ int ld_act(const int* p) { return __ldcg(p); }
__device__ __forceinline__ double ld_act(const double* p) { return __ldcg(p); }
__device__ __forceinline__ float2 ld_act2(const float* p) { return __ldcg(reinterpret_cast<const float2*>(p)); }
__device__ __forceinline__ float4 ld_act4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

// ---- storage-type helpers -----------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void store_as(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_as(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  uint2 r = *reinterpret_cast<const uint2*>(p);
  float4 o;
  o.x = __uint_as_float(r.x << 16);
  o.y = __uint_as_float(r.x & 0xffff0000u);
  o.z = __uint_as_float(r.y << 16);
  o.w = __uint_as_float(r.y & 0xffff0000u);
  return o;
}

// ---- fixed-order warp reductions ---------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ---- what a linear kernel does with a finished pair of output features ------------
// Output features are handled in PAIRS (a, b) that one thread owns for one row:
//   QKV      pair = (dim i, dim i + head_dim/2) of one head of q, k or v: the two
//            elements a rotary embedding mixes
//   SWIGLU   pair = (gate_j, up_j)
//   others   pair p = features (16*(p/8) + p%8, the same + 8)
enum EpiMode { EPI_QKV = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_LOGITS = 3 };

struct EpiParams {
  int mode;
  float* out;  // QKV: q buffer [rows, d_model]; RESID: h [rows, d_model] (accumulated into);
               // SWIGLU: u [rows, d_ffn]; LOGITS: logits [rows, vocab]
  int out_ld;
  void* kcache;  // QKV: this layer's K cache [seq][head][max_seq][head_dim]
  void* vcache;
  const float* rope_cos;  // [max_seq][head_dim/2]
  const float* rope_sin;
  const int* row_pos;  // [rows] absolute position, < 0 = the row carries nothing
  const int* row_seq;  // [rows] sequence slot
  int n_heads, head_dim, max_seq;
};

template <typename KT>
__device__ __forceinline__ void apply_epilogue(const EpiParams& ep, int p, int m, float v0, float v1) {
  if (ep.mode == EPI_QKV) {
    const int pos = ld_act(ep.row_pos + m);
    if (pos < 0) return;
    const int hp = ep.head_dim >> 1;
    const int per_tensor = ep.n_heads * hp;
    const int t = p / per_tensor;
    const int rem = p - t * per_tensor;
    const int head = rem / hp;
    const int i = rem - head * hp;
    if (t < 2) {
      const float c = ep.rope_cos[(size_t)pos * hp + i];
      const float s = ep.rope_sin[(size_t)pos * hp + i];
      const float r0 = v0 * c - v1 * s;
      const float r1 = v1 * c + v0 * s;
      v0 = r0;
      v1 = r1;
    }
    if (t == 0) {
      float* q = ep.out + (size_t)m * ep.out_ld + head * ep.head_dim;
      q[i] = v0;
      q[i + hp] = v1;
    } else {
      KT* base = reinterpret_cast<KT*>(t == 1 ? ep.kcache : ep.vcache);
      KT* dst = base + (((size_t)ld_act(ep.row_seq + m) * ep.n_heads + head) * ep.max_seq + pos) * ep.head_dim;
      store_as(dst + i, v0);
      store_as(dst + i + hp, v1);
    }
  } else if (ep.mode == EPI_RESID) {
    const int r0 = ((p >> 3) << 4) + (p & 7);
    float* h = ep.out + (size_t)m * ep.out_ld;
    h[r0] = ld_act(h + r0) + v0;
    h[r0 + 8] = ld_act(h + r0 + 8) + v1;
  } else if (ep.mode == EPI_SWIGLU) {
    const float g = v0 / (1.0f + __expf(-v0));
    ep.out[(size_t)m * ep.out_ld + p] = g * v1;
  } else {
    const int r0 = ((p >> 3) << 4) + (p & 7);
    float* o = ep.out + (size_t)m * ep.out_ld;
    o[r0] = v0;
    o[r0 + 8] = v1;
  }
}

}  // namespace sdfp
