// Decode / verify attention for the passes of a batch on the dense path: the rows a sequence
// carries in a pass attend the keys of its cache up to their own positions; the result goes out as
// bf16 hi + lo into the activation image of the O-projection (or as fp32 rows).
//
// The K/V stream is decoupled from the arithmetic: one CTA = (split j of
// n_splits, head, sequence [, group of RM rows]); a producer thread brings the 64-key chunks j,
// j + n_splits, ... of the head (K and V, 2 x 64 x HD x 2 bytes) into a ring of shared-memory stages
// with bulk copies that complete on an mbarrier, as far ahead as the ring allows, so that the bytes
// in flight do not depend on how far the arithmetic has come.  Eight consumer warps share every
// stage: a group of HD / VEC lanes owns one key per step (VEC dimensions per lane: one 16- or 8-byte
// shared-memory load for K, one for V), so a warp step covers 32 * VEC / HD keys and a stage takes
// 64 * HD / (256 * VEC) steps.  (Every instantiation a context launches uses the same VEC: the
// grouping of the dimensions and of the keys is part of a row's arithmetic.)  Every lane group keeps its own running maximum, sum and
// un-normalised output per row for the keys it has seen (a masked key is skipped, which changes
// nothing), and never waits for another group until the end, where the groups' partial results are
// combined in group order through the ring's memory.  Which group sees which key depends on the
// key's index alone, so a row's numbers depend on its position alone: a verify row equals the same
// token decoded alone, whatever else is in the batch.  With more than one split the CTA that
// arrives last for its (sequence, row group, head) folds the splits in split order.
#pragma once

#include "attention.cuh"
#include "pass_kernel.cuh"
#include "umma_linear.cuh"

namespace sdfp {

constexpr int kAsWarps = 8;
constexpr int kAsConsumers = 32 * kAsWarps;
constexpr int kAsThreads = kAsConsumers + 32;  // + the producer's warp
constexpr int kAsKeys = 64;                    // keys per stage
constexpr int kAsMaxStages = 6;

enum { ATTN_ERR_STAGE_FULL = 6, ATTN_ERR_STAGE_EMPTY = 7 };  // continues UmmaError: one error word for the dense path

// CTAs per SM: two for the narrow passes; from five rows on the per-row registers (q and the output,
// 2 * VEC * RM) no longer fit twice, and one CTA with a ring twice as deep measured faster than two that spill
template <int RM>
__host__ __device__ constexpr int as_ctas() { return RM <= 2 ? 2 : 1; }
template <int RM>
__host__ __device__ constexpr int as_stages() { return as_ctas<RM>() == 2 ? 3 : 6; }
template <int HD, int RM>
__host__ __device__ constexpr size_t attention_stream_smem() { return (size_t)as_stages<RM>() * 2 * kAsKeys * HD * 2; }

struct AsShared {
  uint64_t full[kAsMaxStages], empty[kAsMaxStages];
  int row_pos[8];
  int seq, abort, last;
};

__device__ __forceinline__ void as_consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kAsConsumers) : "memory"); }

// VEC bf16 values from shared memory as floats; returns a word that depends on every bit read
template <int VEC>
__device__ __forceinline__ unsigned as_load(const __nv_bfloat16* p, float (&f)[VEC]) {
  if constexpr (VEC == 8) {
    const uint4 w = *reinterpret_cast<const uint4*>(p);
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      f[2 * e] = __uint_as_float(u[e] << 16);
      f[2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u);
    }
    return w.x ^ w.y ^ w.z ^ w.w;
  } else {
    const uint2 w = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(w.x << 16);
    f[1] = __uint_as_float(w.x & 0xffff0000u);
    f[2] = __uint_as_float(w.y << 16);
    f[3] = __uint_as_float(w.y & 0xffff0000u);
    return w.x ^ w.y;
  }
}

template <int HD, int RM, int VEC>
__global__ void __launch_bounds__(kAsThreads, as_ctas<RM>()) attention_stream_kernel(AttnParams ap, int M) {
  constexpr int LPK = HD / VEC;                       // lanes that share a key
  constexpr int KPS = 32 / LPK;                       // keys per warp step
  constexpr int STEPS = kAsKeys / (kAsWarps * KPS);   // steps per stage
  constexpr int G = kAsWarps * KPS;                   // independent partial results per CTA
  constexpr int ST = as_stages<RM>();
  constexpr int KV_ELEMS = kAsKeys * HD;              // K (or V) of one stage
  static_assert(LPK <= 32 && STEPS >= 1 && (size_t)G * RM * (HD + 2) * 4 <= attention_stream_smem<HD, RM>(), "shape");
  extern __shared__ __align__(128) unsigned char as_smem[];
  __shared__ AsShared sh;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, head = blockIdx.y, n_splits = ap.n_splits;
  const int R = ap.rows_per_seq, n_rg = (R + RM - 1) / RM;
  const int b = blockIdx.z / n_rg, rg = blockIdx.z - b * n_rg;
  const int row0 = b * R + rg * RM;
  const int nr = min(RM, R - rg * RM);

  pdl_wait();  // q and the newest K/V rows are the preceding kernel's output
  pdl_launch_dependents();

  if (tid < RM) {
    const bool live = tid < nr && row0 + tid < M;
    sh.row_pos[tid] = live ? ld_act(ap.row_pos + row0 + tid) : -1;
  }
  if (tid == 0) {
    for (int s = 0; s < ST; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], kAsWarps);
    }
    sh.seq = ld_act(ap.row_seq + b * R);
    sh.abort = *reinterpret_cast<volatile int*>(ap.error) != 0 ? 1 : 0;  // an earlier kernel gave up: move nothing
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int* s_abort = &sh.abort;
  int pos[RM], max_pos = -1;
#pragma unroll
  for (int r = 0; r < RM; ++r) {
    pos[r] = sh.row_pos[r];
    max_pos = max(max_pos, pos[r]);
  }
  const int nc = (max_pos + kAsKeys) / kAsKeys;  // chunks that hold a visible key
  const int n_my = nc > split ? (nc - split + n_splits - 1) / n_splits : 0;
  __nv_bfloat16* ring = reinterpret_cast<__nv_bfloat16*>(as_smem);

  if (warp == kAsWarps) {
    // ================= producer =================
    if (lane == 0 && !*s_abort) {
      const size_t base = ((size_t)sh.seq * ap.n_heads + head) * (size_t)ap.max_seq * HD;
      const __nv_bfloat16* gK = reinterpret_cast<const __nv_bfloat16*>(ap.kcache) + base;
      const __nv_bfloat16* gV = reinterpret_cast<const __nv_bfloat16*>(ap.vcache) + base;
      const uint64_t pol = l2_policy_evict_first();
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < n_my; ++i) {
        const int stage = i % ST;
        if (i >= ST) {
          const unsigned par = (unsigned)((i / ST) - 1) & 1u;
          ok = um_wait([&] { return mbar_try_wait(&sh.empty[stage], par); }, ap.error, s_abort, ATTN_ERR_STAGE_EMPTY);
          if (!ok) break;
        }
        const int key0 = (split + i * n_splits) * kAsKeys;
        const unsigned bytes = (unsigned)min(kAsKeys, ap.max_seq - key0) * HD * 2;  // the cache ends at max_seq
        __nv_bfloat16* dst = ring + (size_t)stage * 2 * KV_ELEMS;
        mbar_arrive_expect_tx(&sh.full[stage], 2 * bytes);
        bulk_load(dst, gK + (size_t)key0 * HD, bytes, &sh.full[stage], pol);
        bulk_load(dst + KV_ELEMS, gV + (size_t)key0 * HD, bytes, &sh.full[stage], pol);
        ++issued;
      }
      if (!ok || *s_abort) {  // nothing may still be landing in shared memory when the CTA exits
        for (int j = max(0, issued - ST); j < issued; ++j) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&sh.full[j % ST], (unsigned)(j / ST) & 1u))
            if (global_ns() - t0 > kWaitLimitNs) break;
        }
      }
    }
    return;
  }

  // ================= consumers =================
  const int grp = lane / LPK, d0 = (lane - grp * LPK) * VEC;
  const size_t d_model = (size_t)ap.n_heads * HD;
  float q[RM][VEC], acc[RM][VEC], mrun[RM], lrun[RM];
#pragma unroll
  for (int r = 0; r < RM; ++r) {
    mrun[r] = -INFINITY;
    lrun[r] = 0.f;
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[r][e] = 0.f, q[r][e] = 0.f;
    if (pos[r] >= 0) {
      const float* qp = ap.q + (size_t)(row0 + r) * d_model + head * HD + d0;
#pragma unroll
      for (int e = 0; e < VEC; e += 4) {
        const float4 v = ld_act4(qp + e);
        q[r][e] = v.x * ap.scale, q[r][e + 1] = v.y * ap.scale, q[r][e + 2] = v.z * ap.scale, q[r][e + 3] = v.w * ap.scale;
      }
    }
  }
  bool ok = !*s_abort;
  for (int i = 0; i < n_my && ok; ++i) {
    const int stage = i % ST;
    const unsigned par = (unsigned)(i / ST) & 1u;
    ok = um_wait([&] { return mbar_try_wait(&sh.full[stage], par); }, ap.error, s_abort, ATTN_ERR_STAGE_FULL);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    const __nv_bfloat16* sK = ring + (size_t)stage * 2 * KV_ELEMS;
    const __nv_bfloat16* sV = sK + KV_ELEMS;
    const int key0 = (split + i * n_splits) * kAsKeys;
    unsigned dep = 0;
#pragma unroll
    for (int t = 0; t < STEPS; ++t) {
      const int kk = (t * kAsWarps + warp) * KPS + grp;
      const int key = key0 + kk;
      float kf[VEC], vf[VEC];
      dep ^= as_load<VEC>(sK + kk * HD + d0, kf);
      dep ^= as_load<VEC>(sV + kk * HD + d0, vf);
#pragma unroll
      for (int r = 0; r < RM; ++r) {
        float sc = 0.f;
#pragma unroll
        for (int e = 0; e < VEC; ++e) sc = fmaf(q[r][e], kf[e], sc);
#pragma unroll
        for (int o = LPK / 2; o > 0; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
        if (key <= pos[r]) {  // the same for all lanes of the group; a key a row cannot see changes nothing
          const float m_new = fmaxf(mrun[r], sc);
          if (m_new > mrun[r]) {
            const float a = __expf(mrun[r] - m_new);  // exp(-inf) = 0 the first time
            lrun[r] *= a;
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[r][e] *= a;
            mrun[r] = m_new;
          }
          const float pr = __expf(sc - m_new);
          lrun[r] += pr;
#pragma unroll
          for (int e = 0; e < VEC; ++e) acc[r][e] = fmaf(pr, vf[e], acc[r][e]);
        }
      }
    }
    // The stage goes back once this warp's reads of it have RETURNED: the arrival's address depends
    // on every word read (masked to zero at run time), see mbar_arrive_relaxed_after.
    asm volatile("" : "+r"(dep)::"memory");
    dep &= ap.zero;
    __syncwarp();
    if (lane == 0) mbar_arrive_relaxed_after(&sh.empty[stage], dep);
  }

  // ---- the lane groups' partial results, combined in group order ----
  as_consumer_sync();  // every warp has left the ring
  float* mo = reinterpret_cast<float*>(as_smem);  // [G][RM][HD]
  float* mml = mo + (size_t)G * RM * HD;          // [G][RM][2]
  {
    const int g = warp * KPS + grp;
#pragma unroll
    for (int r = 0; r < RM; ++r) {
#pragma unroll
      for (int e = 0; e < VEC; e += 4)
        *reinterpret_cast<float4*>(mo + ((size_t)g * RM + r) * HD + d0 + e) = make_float4(acc[r][e], acc[r][e + 1], acc[r][e + 2], acc[r][e + 3]);
      if (d0 == 0) {
        mml[((size_t)g * RM + r) * 2] = mrun[r];
        mml[((size_t)g * RM + r) * 2 + 1] = lrun[r];
      }
    }
  }
  as_consumer_sync();
  for (int e = tid; e < nr * HD; e += kAsConsumers) {
    const int r = e / HD, d = e - r * HD;
    const int m = row0 + r;
    if (m >= M) continue;
    float mx = -INFINITY;
    for (int g = 0; g < G; ++g)
      if (mml[((size_t)g * RM + r) * 2 + 1] > 0.f) mx = fmaxf(mx, mml[((size_t)g * RM + r) * 2]);
    float l = 0.f, o = 0.f;
    for (int g = 0; g < G; ++g) {
      const float lg = mml[((size_t)g * RM + r) * 2 + 1];
      const float w = lg > 0.f ? __expf(mml[((size_t)g * RM + r) * 2] - mx) : 0.f;
      l = fmaf(lg, w, l);
      o = fmaf(w, mo[((size_t)g * RM + r) * HD + d], o);
    }
    if (n_splits == 1) {
      attn_store(ap, ap.out + (size_t)m * d_model, m, head * HD + d, l > 0.f ? o / l : 0.f);  // no visible key: zero
    } else {
      const size_t slot = ((size_t)m * ap.n_heads + head) * kAttnSplits + split;
      ap.part_o[slot * HD + d] = o;
      if (d == 0) {
        ap.part_ml[slot * 2] = mx;
        ap.part_ml[slot * 2 + 1] = l;
      }
    }
  }
  if (n_splits == 1) return;

  // ---- the last CTA of this (sequence, row group, head) folds the splits ----
  __threadfence();
  as_consumer_sync();
  if (tid == 0) {
    const int prev = atomicAdd(&ap.counters[blockIdx.z * ap.n_heads + head], 1);
    sh.last = (prev == n_splits - 1);
  }
  as_consumer_sync();
  if (!sh.last) return;
  __threadfence();
  if (tid == 0) ap.counters[blockIdx.z * ap.n_heads + head] = 0;
  for (int e = tid; e < nr * HD; e += kAsConsumers) {
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
    float l = 0.f, o = 0.f;
#pragma unroll
    for (int j = 0; j < kAttnSplits; ++j) {
      const float w = lj[j] > 0.f ? __expf(mj[j] - mx) : 0.f;
      l = fmaf(lj[j], w, l);
      o = fmaf(w, oj[j], o);
    }
    attn_store(ap, ap.out + (size_t)m * d_model, m, head * HD + d, l > 0.f ? o / l : 0.f);
  }
}

}  // namespace sdfp
