// Dense linear kernel on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
// memory) for passes of many rows: the prompt pass (hundreds to thousands of rows, Section II-A:
// "computed efficiently via KV caching" presupposes the cache of the prompt) and the passes of a
// batch of sequences (up to 80 rows).
//
//   Y[m, n] = sum_k W[n, k] * X'[m, k],   X' given as bf16 pairs hi + lo   (+ fused epilogue)
//
// Operands.  The weight matrix is the A operand: a tile of 128 output features sits on the 128
// lanes of tensor memory.  The rows (tokens) are the N side: a block of RB rows enters as 2*RB
// columns, the bf16 high parts first, the bf16 low parts behind them, so ONE instruction per 16
// columns of K multiplies the weight tile with both parts, and the epilogue adds the two halves
// of the accumulator: x = hi + lo keeps 16 mantissa bits and products with bf16 weights are exact
// in the fp32 accumulator.
//
// Memory images.  Both operands live in global memory exactly as the instruction wants them in
// shared memory (canonical K-major layout without swizzle: 8 x 16-byte core matrices, 128
// contiguous bytes each), so a pipeline stage is filled by two plain bulk copies:
//   weights      [feature tile][k block of 64][k group of 8][16 row groups][8 rows][8 elements]
//   activations  [row block][k block of 64][k group of 8][2*RB/8 row groups][8 rows][8 elements]
// A k block is four MMA steps (K = 16 each = two k groups).  Inside a feature tile, rows 32w..32w+15
// are the first features of output pairs 64*tile + 16w .. +15 and rows 32w+16..32w+31 their second
// features (see EpiMode), so the two values a fused epilogue combines (rotary pair, gate/up) sit 16
// lanes apart in the warp that reads that quarter of tensor memory: one shuffle, no barrier.
//
// Work split (stream-K).  Tiles (feature tile, row block) times k blocks form one list of units,
// cut into equal contiguous ranges, one per CTA (one CTA per SM): every SM streams the same number
// of bytes whatever the matrix shape.  A tile whose k range is cut is finished by the CTA that holds
// its beginning (it reaches that piece last); the CTAs holding the rest post their partial
// accumulators to global scratch and raise a flag; the finisher adds them in CTA order, so the
// result does not depend on timing.  A row's result depends on its own column only.
//
// Roles: warp 0 = producer (bulk copies into a ring of stages, mbarrier transaction counts),
// warp 1 = MMA issue (one thread) and owner of the tensor-memory allocation, warps 2..9 = epilogue
// (two per quarter of tensor memory, one for the even and one for the odd 16-row chunks: tcgen05.ld,
// pair partner by a shuffle, the same fused epilogues as the other linear kernels).  Two accumulators alternate, so the epilogue of one piece overlaps the MMAs of the next.
// Every wait is bounded: a wait that runs out records an error word and the CTA winds down.
#pragma once

#include "common.cuh"
#include "linear_fma.cuh"
#include "pass_kernel.cuh"

namespace sdfp {

constexpr int kUmBK = 64;                          // k elements per pipeline stage
constexpr int kUmFeat = 128;                       // output features per tile = tensor-memory lanes
constexpr int kUmABytes = kUmFeat * kUmBK * 2;     // weight bytes per stage
constexpr int kUmMaxRB = 128;                      // rows per row block (N = 2 * RB <= 256)
constexpr int kUmEpiWarps = 8;                     // two per quarter of tensor memory: even and odd chunks of rows
constexpr int kUmEpiThreads = kUmEpiWarps * 32;
constexpr int kUmThreads = 64 + kUmEpiThreads;
constexpr int kUmChunk = 16;                       // rows the epilogue handles at a time
constexpr int kUmExLd = kUmChunk + 1;
constexpr int kUmMaxStages = 8;
constexpr int kUmTmemCols = 512;

enum UmmaError { UMMA_OK = 0, UMMA_ERR_STAGE_EMPTY = 1, UMMA_ERR_STAGE_FULL = 2, UMMA_ERR_ACC_EMPTY = 3,
                 UMMA_ERR_ACC_FULL = 4, UMMA_ERR_POST = 5 };

__host__ __device__ constexpr int um_b_stage_bytes(int RB) { return RB * 256; }  // 2*RB rows x 64 k x 2 bytes
__host__ __device__ constexpr int um_stage_bytes(int RB) { return kUmABytes + um_b_stage_bytes(RB); }

struct UmmaShared {
  uint64_t full[kUmMaxStages], empty[kUmMaxStages];
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort;     // set by whichever thread gives up a wait
  int decision;  // abort as sampled by one epilogue thread between two barriers
  int n_posts;
  int posts[160];
  float inv[kUmMaxRB];  // 1/rms of the rows of the running tile
};

inline size_t umma_smem_bytes(int RB, int n_stages) {
  return (size_t)n_stages * um_stage_bytes(RB) + (size_t)kUmEpiWarps * 32 * kUmExLd * 4 + sizeof(UmmaShared) + 1024;
}
inline int umma_stages_for(int RB, int max_smem_optin) {
  int s = kUmMaxStages;
  while (s > 2 && umma_smem_bytes(RB, s) > (size_t)max_smem_optin) --s;
  return s;
}

struct UmmaParams {
  const unsigned char* W;  // weight image
  const unsigned char* X;  // activation image
  int n_ft, n_rb, KB, RB;  // feature tiles, row blocks, k blocks, rows per row block (multiple of 16)
  int M;                   // valid rows (<= n_rb * RB)
  int n_pairs;             // valid output pairs (<= 64 * n_ft)
  int n_stages;
  float* partial;          // [grid][RB * 128] partial accumulators of cut tiles
  int* flags;              // [grid], zero between launches: "CTA c has posted its partial accumulator"
  int* flags_post;         // where a CTA raises its flag: flags, except under the failure-path test hook
  int* error;              // first UmmaError seen, sticky
  unsigned long long wait_limit_ns;  // after this long a wait gives up (kWaitLimitNs unless the test hook shortens it)
  // RMSNorm folded in: the activation image carries gain * h; 1/rms of row m comes from ssq_groups
  // partial sums of squares ssq_in[g * ssq_ld + m] left by whoever wrote h (null: no norm)
  const float* ssq_in;
  int ssq_groups, ssq_ld;
  float inv_k, eps;
  // The epilogue can leave its result as the activation image of the NEXT linear layer (row block
  // size RB, k blocks img_KB), so that no conversion kernel runs between the two:
  //   EPI_SWIGLU  image of u (img_out non-null); the fp32 copy is written only if ep.out is non-null
  //   EPI_RESID   image of gain_out * h_new, and this tile's sum of squares of h_new per row in
  //               ssq_out[tile * ssq_ld + m]
  unsigned char* img_out;
  int img_KB;
  const float* gain_out;
  float* ssq_out;
  EpiParams ep;
};

// byte offset of the 16-byte piece (row m, k group kg = k / 8) of the high parts in an activation image
__host__ __device__ __forceinline__ size_t um_img_offset(int RB, int KB, int m, int kg) {
  const int rb = m / RB, tm = m - rb * RB;
  return ((size_t)rb * KB + (kg >> 3)) * (size_t)um_b_stage_bytes(RB) + (size_t)(kg & 7) * (RB * 32) + (size_t)(tm >> 3) * 128 + (tm & 7) * 16;
}
// ... and from there to the piece of the low parts
__host__ __device__ __forceinline__ size_t um_img_lo(int RB) { return (size_t)(RB / 8) * 128; }

// ---- tcgen05 / descriptor helpers ----------------------------------------------------------------
// Shared-memory matrix descriptor, K-major, no swizzle: start address, leading-dimension byte offset
// (between the two k groups of one MMA step), stride-dimension byte offset (between 8-row groups),
// all in units of 16 bytes; bits 46..47 = 1 (descriptor version of this architecture).
__device__ __forceinline__ uint64_t um_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = (uint64_t)((saddr & 0x3ffffu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= 1ull << 46;
  return d;
}
// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t um_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kUmFeat >> 4) << 24);
}
__device__ __forceinline__ void um_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on an mbarrier once every MMA issued so far by this thread has completed
__device__ __forceinline__ void um_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void um_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void um_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 16 consecutive columns of this warp's 32 lanes: thread t gets lane (lane field of taddr) + t
__device__ __forceinline__ void um_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void um_epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kUmEpiThreads) : "memory"); }
__device__ __forceinline__ void st_release(int* p, int v) { asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory"); }
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// apply_epilogue's EPI_QKV case with the pair already located (tensor t = q, k or v; head; index i
// inside the half head): rotary embedding of q and k at the row's position, q to its buffer, k and v
// into the cache.  Same operations in the same order.
__device__ __forceinline__ void um_qkv_epilogue(const EpiParams& ep, int t, int head, int i, int m, float v0, float v1) {
  const int pos = ld_act(ep.row_pos + m);
  if (pos < 0) return;
  const int hp = ep.head_dim >> 1;
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
    __nv_bfloat16* base = reinterpret_cast<__nv_bfloat16*>(t == 1 ? ep.kcache : ep.vcache);
    __nv_bfloat16* dst = base + (((size_t)ld_act(ep.row_seq + m) * ep.n_heads + head) * ep.max_seq + pos) * ep.head_dim;
    dst[i] = __float2bfloat16_rn(v0);
    dst[i + hp] = __float2bfloat16_rn(v1);
  }
}

template <typename Pred>
__device__ __forceinline__ bool um_wait(Pred pred, int* error, volatile int* s_abort, int code, unsigned long long limit_ns) {
  if (pred()) return true;
  const unsigned long long t0 = global_ns();
  unsigned spins = 0;
  for (;;) {
    if (pred()) return true;
    if (((++spins) & 63u) == 0) {
      if (*s_abort) return false;
      if (global_ns() - t0 > limit_ns) {
        atomicCAS(error, 0, code);
        *s_abort = 1;
        return false;
      }
    }
  }
}

// position of a unit range in the tile list
struct UmSeg {
  int tile, kb0, kb1;
};

__global__ void __launch_bounds__(kUmThreads, 1) umma_linear_kernel(UmmaParams p) {
  extern __shared__ unsigned char um_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(um_smem_raw) + 1023) & ~(uintptr_t)1023);
  const int stage_bytes = um_stage_bytes(p.RB);
  float* ex = reinterpret_cast<float*>(smem + (size_t)p.n_stages * stage_bytes);
  UmmaShared* sh = reinterpret_cast<UmmaShared*>(ex + kUmEpiWarps * 32 * kUmExLd);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const int KB = p.KB;
  const long long n_units = (long long)p.n_ft * p.n_rb * KB;
  long long ub, ue;
  unit_range(n_units, cta, n_cta, ub, ue);

  if (tid == 0) {
    for (int s = 0; s < p.n_stages; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sh->acc_full[b], 1);
      mbar_init(&sh->acc_empty[b], kUmEpiWarps);
    }
    sh->abort = *reinterpret_cast<volatile int*>(p.error) != 0 ? 1 : 0;  // an earlier kernel gave up: do nothing
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // tensor memory: all 512 columns (one CTA per SM), two accumulators of 2*RB columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"((uint32_t)kUmTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  um_fence_before();
  __syncthreads();
  um_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  volatile int* s_abort = &sh->abort;
  // The next kernel of the stream may be scheduled from here on: its CTAs find room only where a
  // CTA of this kernel has exited (shared memory), and they wait for this whole grid before they
  // touch anything it writes.
  pdl_launch_dependents();

  auto next_seg = [&](long long u) {
    UmSeg s;
    s.tile = (int)(u / KB);
    s.kb0 = (int)(u - (long long)s.tile * KB);
    const long long left = ue - u;
    s.kb1 = (int)(left < (long long)(KB - s.kb0) ? s.kb0 + left : KB);
    return s;
  };

  if (warp == 0) {
    // ================= producer =================
    if (lane == 0 && !*s_abort) {
      const uint64_t pol = l2_policy_evict_first();  // a weight is read once per launch
      uint64_t pol_x;                                  // the activation image is read by every CTA
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_x));
      int stage = 0;
      unsigned phase = 0, issued = 0;
      bool ok = true;
      // Weights do not depend on the kernels before this one: the first ring's worth of weight
      // blocks is requested before the wait on the preceding kernel, the activation blocks of the
      // same stages right after it.
      for (int pass = 0; pass < 2 && ok; ++pass) {
        unsigned i = 0;  // k blocks of this CTA in order
        stage = 0;
        phase = 0;
        for (long long u = ub; u < ue && ok;) {
          const UmSeg s = next_seg(u);
          const int ft = s.tile / p.n_rb, rb = s.tile - ft * p.n_rb;
          const unsigned char* wsrc = p.W + ((size_t)ft * KB + s.kb0) * kUmABytes;
          const unsigned char* xsrc = p.X + ((size_t)rb * KB + s.kb0) * um_b_stage_bytes(p.RB);
          for (int kb = s.kb0; kb < s.kb1; ++kb, ++i) {
            const bool early = i < (unsigned)p.n_stages;  // first use of its stage: nothing to wait for
            if (pass == 0 && !early) break;
            unsigned char* dst = smem + (size_t)stage * stage_bytes;
            if (pass == 0) {
              mbar_arrive_expect_tx(&sh->full[stage], (unsigned)stage_bytes);
              bulk_load(dst, wsrc, kUmABytes, &sh->full[stage], pol);
              ++issued;
            } else if (early) {
              bulk_load(dst + kUmABytes, xsrc, (unsigned)um_b_stage_bytes(p.RB), &sh->full[stage], pol_x);
            } else {
              ok = um_wait([&] { return mbar_try_wait(&sh->empty[stage], phase ^ 1u); }, p.error, s_abort, UMMA_ERR_STAGE_EMPTY, p.wait_limit_ns);
              if (!ok) break;
              mbar_arrive_expect_tx(&sh->full[stage], (unsigned)stage_bytes);
              bulk_load(dst, wsrc, kUmABytes, &sh->full[stage], pol);
              bulk_load(dst + kUmABytes, xsrc, (unsigned)um_b_stage_bytes(p.RB), &sh->full[stage], pol_x);
              ++issued;
            }
            wsrc += kUmABytes;
            xsrc += um_b_stage_bytes(p.RB);
            if (++stage == p.n_stages) {
              stage = 0;
              phase ^= 1u;
            }
          }
          if (pass == 0 && i >= (unsigned)p.n_stages) break;
          u += s.kb1 - s.kb0;
        }
        if (pass == 0) pdl_wait();  // the activation image is the preceding kernel's output
      }
      if (!ok) {
        // nothing may still be landing in shared memory when the CTA exits
        const unsigned first = issued > (unsigned)p.n_stages ? issued - (unsigned)p.n_stages : 0u;
        for (unsigned j = first; j < issued; ++j) {
          const unsigned sl = j % (unsigned)p.n_stages, par = (j / (unsigned)p.n_stages) & 1u;
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&sh->full[sl], par))
            if (global_ns() - t0 > p.wait_limit_ns) break;
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issue =================
    if (lane == 0 && !*s_abort) {
      const uint32_t idesc = um_idesc(2 * p.RB);
      const uint32_t lbo_b = (uint32_t)p.RB * 32u;  // 2*RB/8 row groups of 128 bytes between the k groups
      int stage = 0, buf = 0;
      unsigned phase = 0, acc_phase = 0;
      bool ok = true;
      for (long long u = ub; u < ue && ok;) {
        const UmSeg s = next_seg(u);
        ok = um_wait([&] { return mbar_try_wait(&sh->acc_empty[buf], acc_phase ^ 1u); }, p.error, s_abort, UMMA_ERR_ACC_EMPTY, p.wait_limit_ns);
        if (!ok) break;
        um_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(buf * 2 * p.RB);
        for (int kb = s.kb0; kb < s.kb1; ++kb) {
          ok = um_wait([&] { return mbar_try_wait(&sh->full[stage], phase); }, p.error, s_abort, UMMA_ERR_STAGE_FULL, p.wait_limit_ns);
          if (!ok) break;
          um_fence_after();
          const uint32_t a0 = smem_u32(smem + (size_t)stage * stage_bytes);
          const uint32_t b0 = a0 + kUmABytes;
#pragma unroll
          for (int st = 0; st < kUmBK / 16; ++st) {
            const uint64_t ad = um_desc(a0 + st * 4096u, 2048u, 128u);
            const uint64_t bd = um_desc(b0 + st * 2u * lbo_b, lbo_b, 128u);
            um_mma(tmem_d, ad, bd, idesc, (kb > s.kb0 || st > 0) ? 1u : 0u);
          }
          um_commit(&sh->empty[stage]);  // the stage is free once these MMAs have read it
          if (++stage == p.n_stages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        um_commit(&sh->acc_full[buf]);
        if ((buf ^= 1) == 0) acc_phase ^= 1u;
        u += s.kb1 - s.kb0;
      }
    }
  } else {
    // ================= epilogue: 4 warps, warp w reads lanes 32*(w%4).. of tensor memory =================
    const int et = tid - 64;                 // 0..255
    const int ew = warp - 2;                 // epilogue warp 0..7
    const int quarter = warp & 3;            // the quarter of tensor memory this warp may read (warp index mod 4)
    const int chalf = ew >> 2;               // it takes the chunks of rows c = chalf, chalf + 2, ...
    const int R = quarter * 32 + lane;       // tile row (tensor-memory lane) of this thread
    const int pl = quarter * 16 + (lane & 15), half = lane >> 4;  // the output pair it finishes and which 8 rows of a chunk
    int buf = 0;
    unsigned acc_phase = 0;
    const int RB = p.RB;
    pdl_wait();  // everything this role reads or writes in global memory belongs to the stream's order
    // 1/rms of a row block's rows, from the partial sums of squares whoever wrote h left behind:
    // computed when the role starts (under the MMAs of the first piece) and again only if the row
    // block changes.  A row's partial sums are asked for 16 at a time and added in group order.
    int inv_rb = -1;
    auto ensure_inv = [&](int rb_) {
      if (p.ssq_in == nullptr || rb_ == inv_rb) return;  // uniform over the role
      if (inv_rb >= 0) um_epi_sync();                    // the previous block's values are no longer read
      const int m = rb_ * RB + et;
      if (et < RB && m < p.M) {
        float ssum = 0.f;
        for (int g0 = 0; g0 < p.ssq_groups; g0 += 16) {
          float part[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) part[j] = g0 + j < p.ssq_groups ? __ldcg(p.ssq_in + (size_t)(g0 + j) * p.ssq_ld + m) : 0.f;
#pragma unroll
          for (int j = 0; j < 16; ++j) ssum += part[j];
        }
        sh->inv[et] = rsqrtf(ssum * p.inv_k + p.eps);
      }
      um_epi_sync();
      inv_rb = rb_;
    };
    if (ub < ue) ensure_inv(next_seg(ub).tile % p.n_rb);
    for (long long u = ub; u < ue;) {
      const UmSeg s = next_seg(u);
      const int ft = s.tile / p.n_rb, rb = s.tile - ft * p.n_rb;
      const bool starts = s.kb0 == 0, whole = starts && s.kb1 == KB;
      const bool owner = starts && !whole;
      const bool okw = um_wait([&] { return mbar_try_wait(&sh->acc_full[buf], acc_phase); }, p.error, s_abort, UMMA_ERR_ACC_FULL, p.wait_limit_ns);
      (void)okw;
      if (owner && et == 0) {
        // the rest of the tile lies at the start of the ranges of the CTAs that follow
        const long long tile_end = (long long)(s.tile + 1) * KB;
        int n = 0;
        for (int c2 = cta + 1; c2 < n_cta; ++c2) {
          long long b2, e2;
          unit_range(n_units, c2, n_cta, b2, e2);
          if (b2 >= tile_end) break;
          if (e2 > b2) {
            um_wait([&] { return ld_acquire(p.flags + c2) != 0; }, p.error, s_abort, UMMA_ERR_POST, p.wait_limit_ns);
            sh->posts[n++] = c2;
          }
        }
        sh->n_posts = n;
      }
      um_epi_sync();
      if (et == 0) sh->decision = sh->abort;
      um_epi_sync();
      if (sh->decision) break;
      um_fence_after();
      const int n_posts = owner ? sh->n_posts : 0;
      const int row0 = rb * RB;
      ensure_inv(rb);
      float* my_post = p.partial + (size_t)cta * (RB * kUmFeat);
      // the output pair this thread finishes, located once per piece (not once per row)
      const int pg = ft * 64 + pl;
      int q_t = 0, q_head = 0, q_i = 0;
      if (p.ep.mode == EPI_QKV) {
        const int hp = p.ep.head_dim >> 1, per_tensor = p.ep.n_heads * hp;
        q_t = pg / per_tensor;
        const int rem = pg - q_t * per_tensor;
        q_head = rem / hp;
        q_i = rem - q_head * hp;
      }
      for (int c = chalf; c < RB / kUmChunk; c += 2) {
        if (row0 + c * kUmChunk >= p.M) break;  // rows that carry nothing (uniform over the warp)
        float hi[16], lo[16];
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * 2 * RB + c * kUmChunk);
        um_ld16(taddr, hi);
        um_ld16(taddr + (uint32_t)RB, lo);
#pragma unroll
        for (int t = 0; t < 16; ++t) hi[t] += lo[t];
        if (!starts) {  // a piece from the middle or the end of a tile: post it
#pragma unroll
          for (int t = 0; t < 16; ++t) my_post[(size_t)(c * kUmChunk + t) * kUmFeat + R] = hi[t];
          continue;
        }
        for (int k2 = 0; k2 < n_posts; ++k2) {
          const float* src = p.partial + (size_t)sh->posts[k2] * (RB * kUmFeat) + (size_t)(c * kUmChunk) * kUmFeat + R;
#pragma unroll
          for (int t = 0; t < 16; ++t) hi[t] += __ldcg(src + t * kUmFeat);
        }
        // The two features of an output pair sit 16 lanes apart in the same warp: one shuffle per
        // row brings them together, and thread (pair, half) finishes rows half*8 .. half*8+7.
        const bool want_img = p.img_out != nullptr;
        float keep0[8], keep1[8];  // results this thread owes the output image
#pragma unroll
        for (int t8 = 0; t8 < 8; ++t8) {
          const float own_lo = hi[t8], own_hi = hi[8 + t8];  // rows 0..7 and 8..15 of the chunk, this lane's feature
          const float oth_lo = __shfl_xor_sync(0xffffffffu, own_lo, 16), oth_hi = __shfl_xor_sync(0xffffffffu, own_hi, 16);
          float v0 = half ? oth_hi : own_lo, v1 = half ? own_hi : oth_lo;
          const int t = half * 8 + t8;
          const int m = row0 + c * kUmChunk + t;
          keep0[t8] = 0.f;
          keep1[t8] = 0.f;
          if (m < p.M && pg < p.n_pairs) {
            if (p.ssq_in != nullptr) {
              const float inv = sh->inv[c * kUmChunk + t];
              v0 *= inv;
              v1 *= inv;
            }
            if (p.ep.mode == EPI_RESID && want_img) {
              const int r0 = ((pg >> 3) << 4) + (pg & 7);
              float* hp = p.ep.out + (size_t)m * p.ep.out_ld;
              keep0[t8] = ld_act(hp + r0) + v0;
              keep1[t8] = ld_act(hp + r0 + 8) + v1;
              hp[r0] = keep0[t8];
              hp[r0 + 8] = keep1[t8];
            } else if (p.ep.mode == EPI_SWIGLU && want_img) {
              keep0[t8] = (v0 / (1.0f + __expf(-v0))) * v1;
              if (p.ep.out != nullptr) p.ep.out[(size_t)m * p.ep.out_ld + pg] = keep0[t8];
            } else if (p.ep.mode == EPI_QKV) {
              um_qkv_epilogue(p.ep, q_t, q_head, q_i, m, v0, v1);
            } else {
              apply_epilogue<__nv_bfloat16>(p.ep, pg, m, v0, v1);
            }
          }
        }
        if (want_img) {
          // Results into this warp's own piece of shared memory as [feature][row], then out as 16-byte
          // pieces of the image (8 consecutive features of one row, high parts and low parts).  A warp
          // covers 32 consecutive features of the residual stream, or 16 consecutive columns of u.
          const bool resid = p.ep.mode == EPI_RESID;
          float* exw = ex + ew * (32 * kUmExLd);
          const int li = lane & 15;
          const int f0 = resid ? ((li >> 3) << 4) + (li & 7) : li;
          __syncwarp();
#pragma unroll
          for (int t8 = 0; t8 < 8; ++t8) {
            exw[f0 * kUmExLd + half * 8 + t8] = keep0[t8];
            if (resid) exw[(f0 + 8) * kUmExLd + half * 8 + t8] = keep1[t8];
          }
          __syncwarp();
          const int t = lane & 15, m = row0 + c * kUmChunk + t;
          const int n_kg = resid ? 4 : 2, feat0 = resid ? ft * 128 + quarter * 32 : ft * 64 + quarter * 16;
          if (m < p.M) {
            for (int kgl = lane >> 4; kgl < n_kg; kgl += 2) {
              float v[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) v[e] = exw[(kgl * 8 + e) * kUmExLd + t];
              const int k0 = feat0 + kgl * 8;  // first feature of the piece = column of the next layer's input
              if (k0 >= p.img_KB * kUmBK) continue;
              if (p.gain_out != nullptr) {
                const float4 g0 = __ldg(reinterpret_cast<const float4*>(p.gain_out + k0)), g1 = __ldg(reinterpret_cast<const float4*>(p.gain_out + k0 + 4));
                v[0] *= g0.x; v[1] *= g0.y; v[2] *= g0.z; v[3] *= g0.w;
                v[4] *= g1.x; v[5] *= g1.y; v[6] *= g1.z; v[7] *= g1.w;
              }
              uint4 h4, l4;
              split_pack(v[0], v[1], h4.x, l4.x);
              split_pack(v[2], v[3], h4.y, l4.y);
              split_pack(v[4], v[5], h4.z, l4.z);
              split_pack(v[6], v[7], h4.w, l4.w);
              unsigned char* dst = p.img_out + um_img_offset(RB, p.img_KB, m, k0 >> 3);
              *reinterpret_cast<uint4*>(dst) = h4;
              *reinterpret_cast<uint4*>(dst + um_img_lo(RB)) = l4;
            }
          }
          if (resid && p.ssq_out != nullptr && lane < 16 && m < p.M) {
            float ssum = 0.f;  // this warp's 32 features of row `lane`, in feature order
            for (int fl = 0; fl < 32; ++fl) {
              const float x = exw[fl * kUmExLd + lane];
              ssum = fmaf(x, x, ssum);
            }
            p.ssq_out[(size_t)(ft * 4 + quarter) * p.ssq_ld + m] = ssum;
          }
        }
      }
      // tensor memory of this accumulator has been read: hand it back to the MMA warp
      um_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->acc_empty[buf]);
      if (!starts) {
        __threadfence();
        um_epi_sync();
        if (et == 0) st_release(p.flags_post + cta, 1);
      } else if (owner) {
        um_epi_sync();  // every thread has read the posts
        if (et < n_posts) p.flags[sh->posts[et]] = 0;
      }
      if ((buf ^= 1) == 0) acc_phase ^= 1u;
      u += s.kb1 - s.kb0;
    }
  }
  um_fence_before();
  __syncthreads();
  if (warp == 1) {
    um_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kUmTmemCols) : "memory");
  }
}

// ---- operand images ---------------------------------------------------------------------------------
// Weight image: element e of tile (ft, kb): k group j = e / 1024, row group i = (e % 1024) / 64, row
// r8 = (e % 64) / 8, element e8 = e % 8; tile row R = 8 i + r8 is the first (R % 32 < 16) or second
// feature of pair 64 ft + 16 (R / 32) + R % 16; column k = 64 kb + 8 j + e8.  Rows and columns beyond the matrix
// are zero.
__global__ void pack_umma_kernel(__nv_bfloat16* __restrict__ dst, PackSrc ps, int n_pairs, int K, int n_ft, int KB) {
  const size_t total = (size_t)n_ft * KB * (kUmABytes / 2);
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const size_t blk = e >> 13;  // 8192 elements per (ft, kb)
    const int w = (int)(e & 8191);
    const int ft = (int)(blk / KB), kb = (int)(blk % KB);
    const int j = w >> 10, i = (w >> 6) & 15, r8 = (w >> 3) & 7, e8 = w & 7;
    const int R = 8 * i + r8;
    const int pr = ft * 64 + 16 * (R >> 5) + (R & 15), second = (R >> 4) & 1;
    const int k = kb * kUmBK + 8 * j + e8;
    dst[e] = (pr < n_pairs && k < K) ? pack_src_row<__nv_bfloat16>(ps, pr, second, K)[k] : __float2bfloat16_rn(0.f);
  }
}

// Activation image of fp32 rows X[M, K]: x' = X (gain == null) or gain * X / rms(X), split
// x' = hi + lo into bf16.  One CTA per 8 rows (one row group of the image): a thread converts 8
// consecutive columns of one row, and the 8 rows' 16-byte pieces of a k group form 128
// contiguous bytes.  Columns K .. 64*KB-1 of a valid row are written as zeros; rows >= M are not
// written (their accumulator columns are never read).
constexpr int kPrepThreads = 256;
__global__ void __launch_bounds__(kPrepThreads)
prep_rows_kernel(const float* __restrict__ X, int ldx, int M, int K, const float* __restrict__ gain, float eps,
                 unsigned char* __restrict__ img, int RB, int KB) {
  __shared__ float s_part[kPrepThreads];
  __shared__ float s_inv[8];
  const int tid = threadIdx.x;
  const int r = tid & 7, m = blockIdx.x * 8 + r;
  const int c0 = tid >> 3;  // first k group of this thread, then every 32nd
  const int KG = K >> 3;
  const float* x = X + (size_t)m * ldx;
  pdl_wait();
  pdl_launch_dependents();
  if (gain != nullptr) {
    float s = 0.f;
    if (m < M)
      for (int kg = c0; kg < KG; kg += kPrepThreads / 8) {
        const float4 a = ld_act4(x + kg * 8), b = ld_act4(x + kg * 8 + 4);
        s = fmaf(a.x, a.x, s); s = fmaf(a.y, a.y, s); s = fmaf(a.z, a.z, s); s = fmaf(a.w, a.w, s);
        s = fmaf(b.x, b.x, s); s = fmaf(b.y, b.y, s); s = fmaf(b.z, b.z, s); s = fmaf(b.w, b.w, s);
      }
    s_part[tid] = s;
    __syncthreads();
    if (tid < 8) {
      float t = 0.f;
      for (int j = 0; j < kPrepThreads / 8; ++j) t += s_part[j * 8 + tid];  // fixed order
      s_inv[tid] = rsqrtf(t / (float)K + eps);
    }
    __syncthreads();
  }
  if (m >= M) return;
  const float inv = gain != nullptr ? s_inv[r] : 1.f;
  const int rb = m / RB, tm = m - rb * RB;
  const int n_rg = 2 * RB / 8;  // row groups per k group: RB/8 of high parts, then RB/8 of low parts
  for (int kg = c0; kg < KB * 8; kg += kPrepThreads / 8) {
    float v[8];
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (kg < KG) {
      a = ld_act4(x + kg * 8);
      b = ld_act4(x + kg * 8 + 4);
    }
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    if (gain != nullptr && kg < KG) {
      const float4 g0 = __ldg(reinterpret_cast<const float4*>(gain + kg * 8)), g1 = __ldg(reinterpret_cast<const float4*>(gain + kg * 8 + 4));
      v[0] = v[0] * inv * g0.x; v[1] = v[1] * inv * g0.y; v[2] = v[2] * inv * g0.z; v[3] = v[3] * inv * g0.w;
      v[4] = v[4] * inv * g1.x; v[5] = v[5] * inv * g1.y; v[6] = v[6] * inv * g1.z; v[7] = v[7] * inv * g1.w;
    }
    uint4 hi, lo;
    split_pack(v[0], v[1], hi.x, lo.x);
    split_pack(v[2], v[3], hi.y, lo.y);
    split_pack(v[4], v[5], hi.z, lo.z);
    split_pack(v[6], v[7], hi.w, lo.w);
    const int kb = kg >> 3, j = kg & 7;
    unsigned char* base = img + ((size_t)rb * KB + kb) * um_b_stage_bytes(RB) + (size_t)j * n_rg * 128;
    *reinterpret_cast<uint4*>(base + (size_t)(tm >> 3) * 128 + (tm & 7) * 16) = hi;
    *reinterpret_cast<uint4*>(base + (size_t)(RB / 8 + (tm >> 3)) * 128 + (tm & 7) * 16) = lo;
  }
}

}  // namespace sdfp
