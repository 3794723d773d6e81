// Persistent forward-pass kernel for bf16 models (sm_100a): every stage of one pass
//   per layer [RMSNorm + QKV + RoPE + KV append] [split-KV attention] [O-proj + residual]
//             [RMSNorm + gate/up + SwiGLU] [down-proj + residual],  then [final RMSNorm + lm-head]
// runs inside ONE cooperative launch of one CTA per SM.
//
// Why one kernel: a decode pass is bound by the bytes of the weights (each is used for at most
// 16 rows), and a 7B layer is four weight sweeps of 5..28 us each.  As separate launches every
// sweep pays a ramp-up and a tail; here the weight stream never stops:
//   * One producer warp per CTA walks the whole stage list and copies this CTA's share of every
//     weight matrix into a ring of 32 KB shared-memory slots with bulk asynchronous copies
//     (cp.async.bulk + mbarrier transaction counts).  Weights do not depend on activations, so the
//     producer runs ahead of the consumers across stage boundaries, through the grid barriers,
//     as far as the ring allows (three slots, 96 KB per SM, ~14 MB over the GPU; two slots when a
//     pass carries more than 8 rows and the work area is larger).
//   * Sixteen consumer warps take the slots in order, feed the tiles to mma.sync.m16n8k16 (weights
//     are the A operand, tokens the 8-wide B operand) and run the fused epilogues.
//   * Stages are separated by a grid barrier (arrival counter in global memory, bounded spin).
//
// Weight layout ("unit" layout, written by pack_units_kernel): a matrix with NT 16-row tiles and
// KT 16-column tiles is stored as units of 8 row tiles at one k-tile, 4096 contiguous bytes,
// unit index = group * KT + kt with group = row tile / 8; inside a unit tile r at r*512 bytes in
// the register order of the MMA A fragment.  The units of a matrix are split evenly over the
// CTAs as contiguous ranges, so every CTA streams one contiguous byte range per stage and the
// shares differ by at most one unit (4 KB).  A range cuts groups at arbitrary k: a group that
// spans several CTAs is finished by the CTA that holds its beginning (which reaches it last),
// after the others have posted their partial sums to global scratch; partials are added in CTA
// order, so the result does not depend on timing.  A post is written as 64-bit words that hold a
// value and the stage's serial number side by side: the owner sees a value as soon as its word
// has arrived and no fence or flag stands between the poster's stores and the owner's loads (a
// fence issued under the weight stream takes 1-5 us).
//
// Inside a CTA the 16 consumer warps are 8 k-classes x 2 tile halves: the unit with index
// (range start + c + 8i) belongs to class c, and warp (c, t) multiplies its tiles 4t..4t+3.  The
// eight class partials are added in class order through shared memory.  All of this is fixed by
// the matrix shape and the grid size alone, never by the number of rows, so a row's result is
// bit-identical whether it is computed alone (autoregressive step) or among k+1 rows (verify).
#pragma once

#include "attention.cuh"
#include "common.cuh"
#include "linear_mma.cuh"

namespace sdfp {

constexpr int kClasses = 8;  // k-classes: units of a CTA's range are dealt round-robin to them
constexpr int kPassConsumerWarps = 2 * kClasses;
constexpr int kPassConsumerThreads = kPassConsumerWarps * 32;
// Consumers are four warpgroups; the producer warp sits in a fifth whose other three warps only
// give their registers away.  The kernel is launched with kPassLaunchRegs registers per thread (20
// warps put five on every scheduler, which caps it there); the producer's group then shrinks to
// kPassProducerRegs and every consumer grows to kPassConsumerRegs:
// 128 * (96 - 32) = 512 * (112 - 96) registers change hands.
constexpr int kPassThreads = kPassConsumerThreads + 128;
constexpr int kPassLaunchRegs = 96, kPassProducerRegs = 32, kPassConsumerRegs = 112;
static_assert(128 * (kPassLaunchRegs - kPassProducerRegs) >= kPassConsumerThreads * (kPassConsumerRegs - kPassLaunchRegs),
              "the consumers would wait for registers nobody gives back");
constexpr int kHalfThreads = kPassConsumerThreads / 2;   // an attention item is run by half the consumers
constexpr int kUnitTiles = 8;                            // row tiles per unit
constexpr int kUnitBytes = kUnitTiles * 512;
constexpr int kChunkUnits = kClasses;  // units per ring slot
constexpr int kSlotBytes = kChunkUnits * kUnitBytes;
constexpr int kPassMaxRows = 16;    // rows one launch may carry (two column groups of 8)
constexpr int kPassAttnR = 16;      // rows of one sequence per attention item
constexpr int kAttnSplits = 8;      // a head's 64-key chunks are dealt round-robin to this many items
constexpr int kPassMaxHeads = 48;
constexpr int kSsqMaxGroups = 256;  // groups of 128 features of the residual stream (d_model <= 32768)

enum StageKind { ST_LINEAR = 0, ST_ATTN = 1 };
// How a linear stage reads its activations.  X_ATTN_FOLD: they are the attention output, which
// exists only as kAttnSplits partial sums per (row, head), and every fragment load folds them.
// X_STAGED (chosen by the kernel, never in a stage descriptor): the CTA has folded the columns
// its units need into shared memory before its first unit.
enum XMode { X_PLAIN = 0, X_ATTN_FOLD = 1, X_STAGED = 2 };
enum RmsMode { RMS_NONE = 0, RMS_DIRECT = 1, RMS_FROM_PARTS = 2 };

struct StageDesc {
  int kind;
  int K, KT, NT, n_groups;  // linear: in-features, k-tiles, row tiles, groups of 8 row tiles
  int ldx;
  int x_mode, rms_mode;
  int write_ssq;      // EPI_RESID stages: leave per-group sums of squares of the new residual rows
  int ssq_groups;     // RMS_FROM_PARTS: how many group sums make a row's sum
  const uint4* W;     // unit layout
  const float* X;     // linear: activations [rows, K]; attention: q [rows, d_model]
  const float* gain;  // linear: RMSNorm gain or null
  EpiParams ep;       // linear epilogue; attention: kcache, vcache, n_heads, max_seq
};

// what a wait that gave up leaves in PassSync::error
enum PassError { PASS_OK = 0, PASS_ERR_GRID_BARRIER = 1, PASS_ERR_SLOT_FULL = 2, PASS_ERR_SLOT_EMPTY = 3, PASS_ERR_SPLIT_FLAG = 4 };

struct PassSync {                // one per context, in global memory, zero-initialised
  unsigned long long bar_count;  // grid-barrier arrivals of all launches so far: serial * grid when barrier `serial` is complete
  unsigned pad0[30];
  int error;           // first PassError seen, sticky
  unsigned pad1[31];
  // Failure-path test hook, both zero in normal operation: every grid barrier expects this many
  // arrivals more than the grid provides (so its wait can only run out), and waits give up after
  // wait_limit_ns nanoseconds instead of the default (0 = default).
  unsigned long long bar_extra;
  unsigned long long wait_limit_ns;
  unsigned pad2[28];
};

struct PassParams {
  const StageDesc* prog;
  int n_stages;
  int M;             // rows in this pass (<= kPassMaxRows); rows beyond carry nothing
  int rows_per_seq;  // attention: rows m0..m0+R-1 of a group belong to one sequence
  const int* row_pos;
  const int* row_seq;
  float eps;
  float attn_scale;
  unsigned zero;  // always 0: lets code build values the compiler cannot fold away
  int pf_chunks;  // how many chunks ahead of the ring the producer prefetches weights into L2
  // scratch
  float* part_o;          // attention partials [rows][head][kAttnSplits][head_dim], not normalised
  float* part_ml;         // [rows][head][kAttnSplits][2] running max and sum
  ulonglong2* split_partials;  // [grid][kUnitTiles * CG * 64] packets of two (value, stage serial) words
  float* ssq_part;        // [kSsqMaxGroups][kPassMaxRows]
  // Greedy decision fused into the lm-head: non-null = the EPI_LOGITS stage writes no logits but,
  // per (128-feature group, row), the largest logit and its index (ties: lowest index); whoever
  // needs the token takes the maximum over the groups (amax_finish in misc_kernels.cuh).
  int2* amax_part;        // [groups of the vocabulary][kPassMaxRows]
  PassSync* sync;
};

// ---- PTX helpers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(smem_u32(bar)) : "memory");
}
// Arrival without ordering semantics of its own, at an address that depends on `dep`.  A
// releasing arrival would first wait for every earlier memory operation of the thread, including
// activation loads still on their way from L2, and the consumer loop then runs at one L2 round
// trip per unit.  The only accesses that must be over before a slot is handed back are the
// shared-memory reads of its tiles: the caller passes a value computed from the registers those
// reads filled (and masked to zero), so the arrival cannot issue before they have returned.
__device__ __forceinline__ void mbar_arrive_relaxed_after(uint64_t* bar, unsigned dep) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.relaxed.cta.shared::cta.b64 st, [%0];\n}" ::"r"(smem_u32(bar) + dep) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// Bulk asynchronous copy global -> shared, completion counted in bytes on an mbarrier; `pol` says
// how long L2 should keep the lines.  Both addresses and the size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
               : "memory");
}
// Ask for a range of global memory to be brought into L2 (nothing waits for it).  Address and size
// are multiples of 16 bytes.
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, unsigned bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
// 16-byte asynchronous copy global -> shared through L2 only (attention's V tiles)
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// (value, serial) packets of the split-group posts: a 64-bit word is written and read whole, so a
// reader that finds the stage's serial number in a word has the value that came with it
__device__ __forceinline__ void st_packet(ulonglong2* p, float v0, float v1, unsigned serial) {
  const unsigned long long hi = (unsigned long long)serial << 32;
  asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(hi | __float_as_uint(v0)), "l"(hi | __float_as_uint(v1))
               : "memory");
}
__device__ __forceinline__ ulonglong2 ld_packet(const ulonglong2* p) {
  ulonglong2 v;
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ bool packet_is(const ulonglong2& v, unsigned serial) {
  return (unsigned)(v.x >> 32) == serial && (unsigned)(v.y >> 32) == serial;
}
__device__ __forceinline__ unsigned long long ld_relaxed(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_add_relaxed(unsigned long long* p, unsigned long long v) {
  asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kPassConsumerThreads) : "memory"); }
__device__ __forceinline__ void half_sync(int half) { asm volatile("bar.sync %0, %1;" ::"r"(2 + half), "n"(kHalfThreads) : "memory"); }

// Every wait in this kernel gives up after this long, records why, and the kernel winds down.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct PassShared {
  uint64_t full[8];
  uint64_t empty[8];
  StageDesc st;       // the running stage
  StageDesc st_next;  // the next one, fetched while the running stage works
  float inv_rms[kPassMaxRows];
  int row_pos[kPassMaxRows], row_seq[kPassMaxRows];  // fixed for the whole pass
  unsigned long long bar_base;
  unsigned long long bar_extra;  // PassSync::bar_extra as found at launch
  int abort;     // set by whichever thread gives up a wait
  int decision;  // abort as sampled by thread 0 between two consumer barriers: uniform for all
  float attn_m[2][kPassAttnR], attn_l[2][kPassAttnR], attn_a[2][kPassAttnR];
  int n_parts;
  int parts[160];  // CTAs that post a partial for the group this CTA finishes
};

// All consumer threads learn the same answer to "has anything failed": thread 0 samples the
// flag between two barriers, so warps never disagree about leaving a loop that contains barriers.
__device__ __forceinline__ bool consumers_agree_ok(PassShared* sh) {
  consumer_sync();
  if (threadIdx.x == 0) sh->decision = sh->abort;
  consumer_sync();
  return sh->decision == 0;
}

// Spin until pred() holds; false (and the error recorded) if the limit passes or another CTA
// has already failed.
template <typename Pred>
__device__ __forceinline__ bool bounded_wait(Pred pred, PassSync* sync, volatile int* s_abort, int code) {
  if (pred()) return true;
  const unsigned long long t0 = global_ns();
  unsigned spins = 0;
  for (;;) {
    if (pred()) return true;
    if (((++spins) & 255u) == 0) {
      if (*s_abort) return false;
      if (*reinterpret_cast<volatile int*>(&sync->error) != 0) {
        *s_abort = 1;
        return false;
      }
      const unsigned long long set = *reinterpret_cast<volatile unsigned long long*>(&sync->wait_limit_ns);
      if (global_ns() - t0 > (set ? set : kWaitLimitNs)) {
        atomicCAS(&sync->error, 0, code);
        *s_abort = 1;
        return false;
      }
    }
  }
}

// Wait for one packet of a post, polls a little apart.  Out of line: the common case (the packet
// is there at the first look) should not pay registers for this loop.
__device__ __noinline__ ulonglong2 wait_packet(const ulonglong2* src, unsigned serial, PassSync* sync, volatile int* s_abort) {
  ulonglong2 pk = make_ulonglong2(0ull, 0ull);
  bounded_wait(
      [&] {
        pk = ld_packet(src);
        if (packet_is(pk, serial)) return true;
        __nanosleep(50);
        return false;
      },
      sync, s_abort, PASS_ERR_SPLIT_FLAG);
  return pk;
}

// ---- grid barrier (consumer threads of every CTA) ------------------------------------------------
// Everything the consumer threads of this CTA wrote before is visible to every CTA after.  One
// 64-bit counter in global memory only ever grows: barrier number `serial` (counted over all
// launches of the context) is complete when it reads serial * grid.  A CTA arrives with
// a reduction that returns nothing and then polls the counter with relaxed loads; the fences
// before the arrival and after the last poll carry the ordering.  The critical path after the last
// arrival is one trip of the reduction to L2 and one poll, where a scheme in which the last
// arriver publishes a flag adds the return of its atomic, another fence and a store.
__device__ __forceinline__ bool grid_barrier(PassSync* sync, unsigned long long serial, PassShared* sh) {
  consumer_sync();
  if (threadIdx.x == 0) {
    const unsigned long long target = serial * gridDim.x + sh->bar_extra;
    __threadfence();
    red_add_relaxed(&sync->bar_count, 1ull);
    bounded_wait([&] { return ld_relaxed(&sync->bar_count) >= target; }, sync, &sh->abort, PASS_ERR_GRID_BARRIER);
    __threadfence();
    sh->decision = sh->abort;
  }
  consumer_sync();
  return sh->decision == 0;
}

__device__ __forceinline__ void unit_range(long long n_units, int cta, int n_cta, long long& ub, long long& ue) {
  ub = n_units * cta / n_cta;
  ue = n_units * (cta + 1) / n_cta;
}

// ---- one linear stage, consumer side -------------------------------------------------------------
template <int CG>
struct XRegs {
  float2 lo8[CG], hi8[CG];  // x[m][16kt + 2q .. +1] and x[m][16kt + 2q + 8 .. +9], m = 8 cg + g
  float2 g0, g1;            // the RMSNorm gain at the same columns (1 when the stage has no norm)
};

struct XSource {  // the fields of the stage an activation load needs, kept in registers
  const float* X;  // X_STAGED: shared memory, column 0 = first column of k-tile kt0
  const float* gain;
  const float* part_o;
  int ldx, n_heads;
  int kt0, KT;  // X_STAGED only
};

// Activation fragment of k-tile kt for every column group.  X_ATTN_FOLD: the activation is the
// attention output, which exists only as kAttnSplits partial sums per (row, head); sc[m][head][j]
// holds exp(m_j - max)/sum, and the fragment is the weighted sum of the partials in split order.
template <int CG, int HD, int XM>
__device__ __forceinline__ void load_xregs(XRegs<CG>& x, const XSource& xs, const float* sc, int M, int kt, int g, int q,
                                           bool valid) {
  x.g0 = make_float2(1.f, 1.f);
  x.g1 = make_float2(1.f, 1.f);
  if (valid && xs.gain != nullptr) {  // asked for together with the activations: a first touch misses L1
    const float* gp = xs.gain + kt * 16 + 2 * q;
    x.g0 = __ldg(reinterpret_cast<const float2*>(gp));
    x.g1 = __ldg(reinterpret_cast<const float2*>(gp + 8));
  }
#pragma unroll
  for (int cg = 0; cg < CG; ++cg) {
    const int m = cg * 8 + g;
    x.lo8[cg] = make_float2(0.f, 0.f);
    x.hi8[cg] = make_float2(0.f, 0.f);
    if (valid && m < M) {
      if (XM == X_PLAIN) {
        const float* xp = xs.X + (size_t)m * xs.ldx + kt * 16 + 2 * q;
        x.lo8[cg] = ld_act2(xp);
        x.hi8[cg] = ld_act2(xp + 8);
      } else if (XM == X_STAGED) {
        int dk = kt - xs.kt0;
        if (dk < 0) dk += xs.KT;
        const float* xp = xs.X + m * xs.ldx + dk * 16 + 2 * q;
        x.lo8[cg] = *reinterpret_cast<const float2*>(xp);
        x.hi8[cg] = *reinterpret_cast<const float2*>(xp + 8);
      } else {
        const int k = kt * 16 + 2 * q;
        const int head = k / HD, d = k - head * HD;
        const float* po = xs.part_o + (((size_t)m * xs.n_heads + head) * kAttnSplits) * HD + d;
        const float* s8 = sc + ((size_t)m * xs.n_heads + head) * kAttnSplits;
        float2 lo = make_float2(0.f, 0.f), hi = make_float2(0.f, 0.f);
#pragma unroll
        for (int j = 0; j < kAttnSplits; ++j) {
          const float w = s8[j];
          const float2 a = ld_act2(po + (size_t)j * HD);
          const float2 b = ld_act2(po + (size_t)j * HD + 8);
          lo.x = fmaf(w, a.x, lo.x);
          lo.y = fmaf(w, a.y, lo.y);
          hi.x = fmaf(w, b.x, hi.x);
          hi.y = fmaf(w, b.y, hi.y);
        }
        x.lo8[cg] = lo;
        x.hi8[cg] = hi;
      }
    }
  }
}

// work-area layout of a linear stage (bytes from the start of the area)
template <int CG>
__host__ __device__ constexpr int work_red_bytes() { return kClasses * kUnitTiles * CG * 32 * 16; }  // class partials
template <int CG>
__host__ __device__ constexpr int work_sq_off() { return work_red_bytes<CG>(); }  // squares of new residual values [it]
template <int CG>
__host__ __device__ constexpr int work_sc_off() { return work_sq_off<CG>() + kUnitTiles * CG * 64 * 4; }  // attention fold weights
constexpr int kWorkScBytes = kPassMaxRows * kPassMaxHeads * kAttnSplits * 4;

template <int CG, int HD, int XM>
__device__ void linear_stage(const PassParams& pp, PassShared* sh, const unsigned char* ring, int n_slots, unsigned char* work,
                             unsigned& chunk_base, unsigned epoch) {
  const StageDesc& st = sh->st;
  float4* red = reinterpret_cast<float4*>(work);
  float* sq_buf = reinterpret_cast<float*>(work + work_sq_off<CG>());
  float* sc = reinterpret_cast<float*>(work + work_sc_off<CG>());
  const bool fused_argmax = st.ep.mode == EPI_LOGITS && pp.amax_part != nullptr;
  int* idx_buf = reinterpret_cast<int*>(sc);  // the lm-head reads plain activations: the fold area is free
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, q = lane & 3;
  const int cls = warp & (kClasses - 1), th = warp / kClasses;
  const int KT = st.KT, M = pp.M, NT = st.NT;
  const int epi_mode = st.ep.mode;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const long long n_units = (long long)st.n_groups * KT;
  long long ub64, ue64;
  unit_range(n_units, cta, n_cta, ub64, ue64);
  const int nun = (int)(ue64 - ub64);  // units of this CTA; below, units are numbered from ub64
  const int n_chunks = (nun + kChunkUnits - 1) / kChunkUnits;
  const int my_n = nun > cls ? (nun - cls + kChunkUnits - 1) / kChunkUnits : 0;
  const int grp0 = (int)(ub64 / KT);
  const int kt_first = (int)(ub64 - (long long)grp0 * KT);  // k-tile of unit 0
  // ring position of this stage's first chunk; advanced by one slot per unit of this warp
  unsigned slot = chunk_base % (unsigned)n_slots, parity = (chunk_base / (unsigned)n_slots) & 1u;

  // ---- 1/rms of every row (needed only by the epilogue) ----
  if (st.rms_mode == RMS_DIRECT) {
    float* s_part = reinterpret_cast<float*>(red);  // [warp][row]
    for (int m = 0; m < M; ++m) {
      const float* x = st.X + (size_t)m * st.ldx;
      float s = 0.f;
      for (int k = tid * 4; k < st.K; k += kPassConsumerThreads * 4) {
        const float4 v = ld_act4(x + k);
        s = fmaf(v.x, v.x, s);
        s = fmaf(v.y, v.y, s);
        s = fmaf(v.z, v.z, s);
        s = fmaf(v.w, v.w, s);
      }
      s = warp_sum(s);
      if (lane == 0) s_part[warp * kPassMaxRows + m] = s;
    }
    consumer_sync();
    if (tid < M) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kPassConsumerWarps; ++w) s += s_part[w * kPassMaxRows + tid];
      sh->inv_rms[tid] = rsqrtf(s / (float)st.K + pp.eps);
    }
    consumer_sync();
  } else if (st.rms_mode == RMS_NONE && tid < kPassMaxRows) {
    sh->inv_rms[tid] = 1.f;
  }

  // ---- attention fold weights: per (row, head) the factor of each split's partial ----
  if (XM == X_ATTN_FOLD) {
    const int n_heads = st.ep.n_heads;
    for (int e = tid; e < M * n_heads; e += kPassConsumerThreads) {
      const float* ml = pp.part_ml + (size_t)e * kAttnSplits * 2;  // e = m * n_heads + head
      float mj[kAttnSplits], lj[kAttnSplits];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < kAttnSplits; ++j) {
        const float2 v = ld_act2(ml + 2 * j);
        mj[j] = v.x;
        lj[j] = v.y;
        if (v.y > 0.f) mx = fmaxf(mx, v.x);
      }
      float l = 0.f, wj[kAttnSplits];
#pragma unroll
      for (int j = 0; j < kAttnSplits; ++j) {
        wj[j] = lj[j] > 0.f ? __expf(mj[j] - mx) : 0.f;
        l = fmaf(lj[j], wj[j], l);
      }
      const float inv_l = l > 0.f ? 1.0f / l : 0.f;
#pragma unroll
      for (int j = 0; j < kAttnSplits; ++j) sc[(size_t)e * kAttnSplits + j] = wj[j] * inv_l;
    }
    consumer_sync();
  }

  // ---- or the folded activations themselves, for the k-tiles this CTA's units use ----
  // Every element asks for its 8 (max, sum) pairs and its 8 partial values at once, so the whole
  // fold costs one round trip to L2, where folding inside the fragment loads costs one for the
  // weights and one more for each of the first three fragments.  Same operations in the same
  // order as above: the result is bit-identical whichever way a CTA takes.
  float* const x_staged = sc;  // same place: a stage uses one or the other
  const int staged_kts = min(nun, KT), staged_ld = staged_kts * 16 + 8;  // +8: rows start 8 banks apart
  if (XM == X_STAGED) {
    const int n_heads = st.ep.n_heads;
    const int pairs_per_row = staged_kts * 8;
#pragma unroll 2
    for (int e = tid; e < M * pairs_per_row; e += kPassConsumerThreads) {
      const int m = e / pairs_per_row, c = (e - m * pairs_per_row) * 2;
      int kt = kt_first + (c >> 4);
      if (kt >= KT) kt -= KT;
      const int k = kt * 16 + (c & 15);
      const int head = k / HD, d = k - head * HD;
      const size_t rh = (size_t)m * n_heads + head;
      const float* ml = pp.part_ml + rh * kAttnSplits * 2;
      const float* po = pp.part_o + rh * kAttnSplits * HD + d;
      float mj[kAttnSplits], lj[kAttnSplits];
      float2 oj[kAttnSplits];
#pragma unroll
      for (int j = 0; j < kAttnSplits; ++j) {
        const float2 v = ld_act2(ml + 2 * j);
        mj[j] = v.x;
        lj[j] = v.y;
        oj[j] = ld_act2(po + (size_t)j * HD);
      }
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < kAttnSplits; ++j)
        if (lj[j] > 0.f) mx = fmaxf(mx, mj[j]);
      float l = 0.f, wj[kAttnSplits];
#pragma unroll
      for (int j = 0; j < kAttnSplits; ++j) {
        wj[j] = lj[j] > 0.f ? __expf(mj[j] - mx) : 0.f;
        l = fmaf(lj[j], wj[j], l);
      }
      const float inv_l = l > 0.f ? 1.0f / l : 0.f;
      float2 xv = make_float2(0.f, 0.f);
#pragma unroll
      for (int j = 0; j < kAttnSplits; ++j) {
        const float w = wj[j] * inv_l;
        xv.x = fmaf(w, oj[j].x, xv.x);
        xv.y = fmaf(w, oj[j].y, xv.y);
      }
      *reinterpret_cast<float2*>(x_staged + m * staged_ld + c) = xv;
    }
    consumer_sync();
  }

  // activation fragments of my next three units; kt_pref = k-tile of the next unit to prefetch
  const XSource xs{XM == X_STAGED ? x_staged : st.X, st.gain, pp.part_o, XM == X_STAGED ? staged_ld : st.ldx, st.ep.n_heads, kt_first, KT};
  XRegs<CG> x0, x1, x2;
  int kt_pref = (kt_first + cls) % KT;
  auto prefetch = [&](XRegs<CG>& x, int i) {
    load_xregs<CG, HD, XM>(x, xs, sc, M, kt_pref, g, q, i < my_n);
    kt_pref += kChunkUnits;
    if (kt_pref >= KT) kt_pref -= KT;
  };
  prefetch(x0, 0);
  prefetch(x1, 1);
  prefetch(x2, 2);
  if (st.rms_mode == RMS_FROM_PARTS && warp == kPassConsumerWarps - 1) {
    // The stage that produced the residual stream left one sum of squares per 128-feature group.
    // One warp adds them: every lane asks for all its terms at once (a serial chain of loads
    // would hold this warp, and with it the ring, for dozens of L2 round trips); per lane the
    // terms are added in group order, across lanes with the fixed xor tree.
    float part[kPassMaxRows];
#pragma unroll
    for (int m = 0; m < kPassMaxRows; ++m) part[m] = 0.f;
    for (int gi = lane; gi < st.ssq_groups; gi += 32) {
#pragma unroll
      for (int m = 0; m < kPassMaxRows; ++m)
        if (m < M) part[m] += ld_act(pp.ssq_part + gi * kPassMaxRows + m);
    }
#pragma unroll
    for (int m = 0; m < kPassMaxRows; ++m) {
      if (m < M) {
        const float s = warp_sum(part[m]);
        if (lane == 0) sh->inv_rms[m] = rsqrtf(s / (float)st.K + pp.eps);
      }
    }
  }

  int i = 0;          // my next unit is number cls + kChunkUnits * i
  int seg_begin = 0;  // in units from ub64
  int grp = grp0;
  int seg_kt0 = kt_first;  // k-tile at seg_begin
  while (seg_begin < nun) {
    const int seg_len = min(nun - seg_begin, KT - seg_kt0);
    const int seg_end = seg_begin + seg_len;
    const bool starts_group = (seg_kt0 == 0);
    const bool whole = starts_group && (seg_len == KT);
    const bool owner = starts_group && !whole;

    // the old residual values this thread will add to, fetched now so that they are there at the end
    float2 hold[CG];
#pragma unroll
    for (int j = 0; j < CG; ++j) hold[j] = make_float2(0.f, 0.f);
    if (starts_group && epi_mode == EPI_RESID) {
#pragma unroll
      for (int j = 0; j < CG; ++j) {
        const int it = tid + j * kPassConsumerThreads;
        const int ch = it & 1, ln = (it >> 1) & 31, rc = it >> 6;
        const int cg = rc % CG, tile = rc / CG;
        const int m = cg * 8 + 2 * (ln & 3) + ch;
        const int rt = grp * kUnitTiles + tile;
        if (m < M && rt < NT) {
          const float* hp = st.ep.out + (size_t)m * st.ep.out_ld + 16 * rt + (ln >> 2);
          hold[j] = make_float2(ld_act(hp), ld_act(hp + 8));
        }
      }
    }

    float acc[4][CG][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int cg = 0; cg < CG; ++cg)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[r][cg][e] = 0.f;

    bool warp_ok = true;
    int kt = seg_kt0 + (cls + kChunkUnits * i - seg_begin);  // k-tile of my next unit while it lies in this segment
    while (warp_ok && i < my_n && cls + kChunkUnits * i < seg_end) {
      // Lanes leave the polling loop at different times.  mma.sync needs the whole warp
      // converged, so the vote below is both the warp-uniform outcome and the reconvergence point.
      warp_ok = __all_sync(0xffffffffu, bounded_wait([&] { return mbar_try_wait(&sh->full[slot], parity); }, pp.sync,
                                                     &sh->abort, PASS_ERR_SLOT_FULL));
      if (!warp_ok) break;
      const uint4* tiles = reinterpret_cast<const uint4*>(ring + (size_t)slot * kSlotBytes + cls * kUnitBytes + th * 4 * 512);
      uint4 a[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) a[r] = tiles[r * 32 + lane];
      const float2 g0 = x0.g0, g1 = x0.g1;
#pragma unroll
      for (int cg = 0; cg < CG; ++cg) {
        uint32_t bh0, bl0, bh1, bl1;
        split_pack(x0.lo8[cg].x * g0.x, x0.lo8[cg].y * g0.y, bh0, bl0);
        split_pack(x0.hi8[cg].x * g1.x, x0.hi8[cg].y * g1.y, bh1, bl1);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          mma_bf16_16816(acc[r][cg], a[r], bh0, bh1);
          mma_bf16_16816(acc[r][cg], a[r], bl0, bl1);
        }
      }
      // Hand the slot back once the tile reads above have returned: the producer's next bulk
      // copy overwrites it through the async proxy, and an arrival that overtook pending reads
      // let a refill replace 64-byte pieces of a tile under them (rare wrong rows at full speed).
      {
        unsigned dep = a[0].x ^ a[1].y ^ a[2].z ^ a[3].w;
        asm volatile("" : "+r"(dep)::"memory");
        dep &= pp.zero;  // zero at run time, unknown to the compiler
        __syncwarp();
        if (lane == 0) mbar_arrive_relaxed_after(&sh->empty[slot], dep);
      }
      if (++slot == (unsigned)n_slots) {
        slot = 0;
        parity ^= 1u;
      }
      x0 = x1;
      x1 = x2;
      prefetch(x2, i + 3);
      ++i;
      kt += kChunkUnits;
    }

    // ---- end of the segment: add the class partials, then finish the group or post ----
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int cg = 0; cg < CG; ++cg)
        red[((cls * kUnitTiles + th * 4 + r) * CG + cg) * 32 + lane] =
            make_float4(acc[r][cg][0], acc[r][cg][1], acc[r][cg][2], acc[r][cg][3]);
    if (owner && warp == 0) {
      // The rest of the group sits at the beginning of the ranges of the CTAs that follow; every
      // lane looks at one candidate and waits for that CTA's flag, so the waits overlap.
      const long long grp_end = (long long)(grp + 1) * KT;
      int n = 0;
      bool more = true;
      for (int base = cta + 1; more; base += 32) {
        const int c2 = base + lane;
        long long b2 = grp_end, e2 = grp_end;
        if (c2 < n_cta) unit_range(n_units, c2, n_cta, b2, e2);
        const bool beyond = (c2 >= n_cta) || (b2 >= grp_end);
        const bool part = !beyond && e2 > b2;  // an empty range posts nothing
        // one lane per posting CTA waits for the packet that CTA's last thread writes; the others
        // are then there too or about to be, and every reader checks its own packets anyway
        if (part) wait_packet(pp.split_partials + (size_t)c2 * (kUnitTiles * CG * 64) + (kPassConsumerThreads * CG - 1), epoch, pp.sync, &sh->abort);
        const unsigned mask = __ballot_sync(0xffffffffu, part);
        if (part) sh->parts[n + __popc(mask & ((1u << lane) - 1u))] = c2;
        n += __popc(mask);
        more = !__any_sync(0xffffffffu, beyond);
      }
      if (lane == 0) sh->n_parts = n;
    }
    if (!consumers_agree_ok(sh)) return;

    {
      ulonglong2* my_post = pp.split_partials + (size_t)cta * (kUnitTiles * CG * 64);
      const int n_parts = owner ? sh->n_parts : 0;
#pragma unroll
      for (int j = 0; j < CG; ++j) {
        const int it = tid + j * kPassConsumerThreads;
        const int ch = it & 1;
        const int ln = (it >> 1) & 31;
        const int rc = it >> 6;
        const int cg = rc % CG, tile = rc / CG;
        float v0 = 0.f, v1 = 0.f;
#pragma unroll
        for (int c8 = 0; c8 < kClasses; ++c8) {
          const float* p = reinterpret_cast<const float*>(red + ((c8 * kUnitTiles + tile) * CG + cg) * 32 + ln);
          v0 += p[ch];
          v1 += p[ch + 2];
        }
        if (!starts_group) {
          st_packet(my_post + it, v0, v1, epoch);
          continue;
        }
        for (int k2 = 0; k2 < n_parts; ++k2) {
          const ulonglong2* src = pp.split_partials + (size_t)sh->parts[k2] * (kUnitTiles * CG * 64) + it;
          ulonglong2 pk = ld_packet(src);
          if (!packet_is(pk, epoch)) pk = wait_packet(src, epoch, pp.sync, &sh->abort);
          v0 += __uint_as_float((unsigned)pk.x);
          v1 += __uint_as_float((unsigned)pk.y);
        }
        const int m = cg * 8 + 2 * (ln & 3) + ch;
        const int rt = grp * kUnitTiles + tile;
        float sq = 0.f;
        if (m < M && rt < NT) {
          const float inv = sh->inv_rms[m];
          if (epi_mode == EPI_RESID) {
            float* hp = st.ep.out + (size_t)m * st.ep.out_ld + 16 * rt + (ln >> 2);
            const float n0 = hold[j].x + v0 * inv, n1 = hold[j].y + v1 * inv;
            hp[0] = n0;
            hp[8] = n1;
            sq = fmaf(n0, n0, n1 * n1);
          } else if (fused_argmax) {
            const float a = v0 * inv, b2 = v1 * inv;  // logits of features 16 rt + ln/4 and + 8
            const int f0 = 16 * rt + (ln >> 2);
            sq = b2 > a ? b2 : a;
            idx_buf[it] = b2 > a ? f0 + 8 : f0;
          } else {
            apply_epilogue<__nv_bfloat16>(st.ep, 8 * rt + (ln >> 2), m, v0 * inv, v1 * inv);
          }
        } else if (fused_argmax) {
          sq = -INFINITY;
          idx_buf[it] = 0x7fffffff;
        }
        if (st.write_ssq || fused_argmax) sq_buf[it] = sq;
      }
    }
    if (starts_group && st.write_ssq) {
      // one sum of squares per row over this group's 128 features, in tile-then-row order
      consumer_sync();
      if (tid < M) {
        const int cg = tid >> 3, qq = (tid & 7) >> 1, ch = tid & 1;
        float s = 0.f;
        for (int tile = 0; tile < kUnitTiles; ++tile)
          for (int g8 = 0; g8 < 8; ++g8) s += sq_buf[(((tile * CG + cg) * 32) + g8 * 4 + qq) * 2 + ch];
        pp.ssq_part[grp * kPassMaxRows + tid] = s;
      }
    }
    if (starts_group && fused_argmax) {
      // the group's best logit per row, candidates in tile-then-row order, ties to the lowest index
      consumer_sync();
      if (tid < M) {
        const int cg = tid >> 3, qq = (tid & 7) >> 1, ch = tid & 1;
        float best = -INFINITY;
        int bi = 0x7fffffff;
        for (int tile = 0; tile < kUnitTiles; ++tile)
          for (int g8 = 0; g8 < 8; ++g8) {
            const int e = (((tile * CG + cg) * 32) + g8 * 4 + qq) * 2 + ch;
            const float x = sq_buf[e];
            const int xi = idx_buf[e];
            if (x > best || (x == best && xi < bi)) {
              best = x;
              bi = xi;
            }
          }
        pp.amax_part[grp * kPassMaxRows + tid] = make_int2(__float_as_int(best), bi);
      }
    }
    consumer_sync();  // red and parts may be rewritten
    seg_begin = seg_end;
    seg_kt0 = 0;
    ++grp;
  }
  // A class without a unit in the last, partial slot still has to hand that slot back, and only
  // once the slot has been filled: an earlier arrival would be counted for the slot's previous
  // use and let the producer overwrite tiles another warp is still reading.
  if (my_n < n_chunks) {
    if (bounded_wait([&] { return mbar_try_wait(&sh->full[slot], parity); }, pp.sync, &sh->abort, PASS_ERR_SLOT_FULL)) {
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->empty[slot]);
    }
  }
  chunk_base += (unsigned)n_chunks;
}

// ---- attention stage --------------------------------------------------------------------------
// One item = (head, split j, row group), handled by half the consumer threads.  Split j owns the
// 64-key chunks j, j + kAttnSplits, ... of the head (chunk grid fixed in absolute key index) and
// walks them in order with a running max and sum per row; it leaves an un-normalised partial
// (max, sum, o) per row.  The O-projection that follows combines the kAttnSplits partials in split
// order while it loads its activations, so nothing waits on another CTA inside this stage.  A
// row's numbers depend only on its own position: rows that cannot see a chunk skip it entirely.
// Thread t of the half: scores as (key t/4, quarter t%4 of the head dimension), output as
// (dimension t%HD, key half t/HD); the two key halves are added (first + second) at the end.
// RM = compile-time row capacity (the per-row registers are arrays of RM entries).
template <int HD, int RM>
__device__ void attention_item(const StageDesc& st, const PassParams& pp, PassShared* sh, unsigned char* smem, int half,
                               int htid, int head, int split, int b) {
  using KT = __nv_bfloat16;
  constexpr int C = kAttnChunk;
  static_assert(kHalfThreads == 4 * C, "one key per four threads");
  KT* sV = reinterpret_cast<KT*>(smem);               // [C][HD]; at the end the second key half's o [R][HD] fp32
  float* sQ = reinterpret_cast<float*>(sV + C * HD);  // [R][HD]
  float* sS = sQ + kPassAttnR * HD;                   // [R][C]
  float* s_m = sh->attn_m[half];
  float* s_l = sh->attn_l[half];
  float* s_a = sh->attn_a[half];
  const int R = pp.rows_per_seq;
  const int row0 = b * R;
  const int n_heads = st.ep.n_heads;
  const size_t d_model = (size_t)n_heads * HD;
  auto pos_of = [&](int i) { return (row0 + i < pp.M) ? sh->row_pos[row0 + i] : -1; };

  int max_pos = -1;
  for (int i = 0; i < R; ++i) max_pos = max(max_pos, pos_of(i));
  const int seq = sh->row_seq[row0];
  if (htid < R) {
    s_m[htid] = -INFINITY;
    s_l[htid] = 0.f;
  }
  // q rows of this head, 16 bytes at a time, straight into shared memory (rows that carry nothing:
  // zeros).  Inside quarter r of a row (QD dimensions) the dimensions are rotated by 8 r: the four
  // threads that work on one key read the same offset of the four quarters at once, and the
  // rotation puts those four addresses into different banks.
  constexpr int QD = HD / 4;  // dimensions of a key one thread multiplies
  auto fetch_q = [&]() {
    for (int e = htid; e < R * (HD / 4); e += kHalfThreads) {
      const int i = e / (HD / 4), d4 = e - i * (HD / 4);
      const int d = d4 * 4, r = d / QD, phys = r * QD + (d - r * QD + 8 * r) % QD;
      if (pos_of(i) >= 0)
        cp_async16(sQ + i * HD + phys, st.X + (size_t)(row0 + i) * d_model + head * HD + d);
      else
        *reinterpret_cast<float4*>(sQ + i * HD + phys) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };

  constexpr int KV4 = QD / 8;   // uint4 of bf16 per thread
  constexpr int VPR = HD / 8;   // uint4 per V row
  const int key = htid >> 2, qr = htid & 3;
  const int od = htid % HD, okh = htid / HD;        // output dimension and key half (HD = 128: 0/1; HD = 64: 0..3 -> use 2)
  constexpr int KH = (kHalfThreads / HD) >= 2 ? 2 : 1;  // key halves in the output phase
  const bool o_active = okh < KH;
  float o[RM];
#pragma unroll
  for (int i = 0; i < RM; ++i) o[i] = 0.f;

  for (int c = split; c * C <= max_pos; c += kAttnSplits) {
    const int key0 = c * C;
    const int nk_all = min(C, max_pos + 1 - key0);
    const size_t base = (((size_t)seq * n_heads + head) * st.ep.max_seq + key0) * HD;
    const KT* gK = reinterpret_cast<const KT*>(st.ep.kcache) + base;
    const KT* gV = reinterpret_cast<const KT*>(st.ep.vcache) + base;
    uint4 kreg[KV4];
#pragma unroll
    for (int j = 0; j < KV4; ++j) kreg[j] = make_uint4(0u, 0u, 0u, 0u);
    if (key < nk_all) {
      const uint4* kp = reinterpret_cast<const uint4*>(gK + (size_t)key * HD + qr * QD);
#pragma unroll
      for (int j = 0; j < KV4; ++j) kreg[j] = __ldcg(kp + j);
    }
    half_sync(half);  // the previous chunk's sV and sS are no longer read, the row state is written
    if (c == split) fetch_q();  // first chunk: all three requests (K, q, V) are in flight together
    for (int v = htid; v < nk_all * VPR; v += kHalfThreads) cp_async16(reinterpret_cast<uint4*>(sV) + v, reinterpret_cast<const uint4*>(gV) + v);
    if (c == split) {
      cp_async_wait_all();  // q (and V) have landed; make q visible to the whole half
      half_sync(half);
    }
    {
      float acc[RM];
#pragma unroll
      for (int i = 0; i < RM; ++i) acc[i] = 0.f;
#pragma unroll
      for (int j = 0; j < KV4; ++j) {
        const uint32_t w[4] = {kreg[j].x, kreg[j].y, kreg[j].z, kreg[j].w};
#pragma unroll
        for (int e = 0; e < 4; e += 2) {
          const float k0 = __uint_as_float(w[e] << 16), k1 = __uint_as_float(w[e] & 0xffff0000u);
          const float k2 = __uint_as_float(w[e + 1] << 16), k3 = __uint_as_float(w[e + 1] & 0xffff0000u);
          const int d = qr * QD + (j * 8 + e * 2 + 8 * qr) % QD;  // where fetch_q put these four dimensions
#pragma unroll
          for (int i = 0; i < RM; ++i) {
            if (i < R) {
              const float4 qv = *reinterpret_cast<const float4*>(sQ + i * HD + d);
              acc[i] = fmaf(k0, qv.x, acc[i]);
              acc[i] = fmaf(k1, qv.y, acc[i]);
              acc[i] = fmaf(k2, qv.z, acc[i]);
              acc[i] = fmaf(k3, qv.w, acc[i]);
            }
          }
        }
      }
#pragma unroll
      for (int i = 0; i < RM; ++i) {
        if (i < R) {
          float s = acc[i];
          s += __shfl_xor_sync(0xffffffffu, s, 1);  // quarters (0+1), (2+3)
          s += __shfl_xor_sync(0xffffffffu, s, 2);  // then the two pairs
          if (qr == 0) sS[i * C + key] = s * pp.attn_scale;
        }
      }
    }
    half_sync(half);
    {
      const int w8 = htid >> 5, lane = htid & 31;
      for (int i = w8; i < R; i += kHalfThreads / 32) {
        const int nk = min(C, pos_of(i) + 1 - key0);
        if (nk <= 0) {  // the row cannot see this chunk: leave its state alone
          if (lane == 0) s_a[i] = 1.f;
          sS[i * C + lane] = 0.f;
          sS[i * C + lane + 32] = 0.f;
          continue;
        }
        const float s0 = (lane < nk) ? sS[i * C + lane] : -INFINITY;
        const float s1 = (lane + 32 < nk) ? sS[i * C + lane + 32] : -INFINITY;
        const float m_old = s_m[i];
        const float m_new = fmaxf(m_old, warp_max(fmaxf(s0, s1)));
        const float p0 = (lane < nk) ? __expf(s0 - m_new) : 0.f;
        const float p1 = (lane + 32 < nk) ? __expf(s1 - m_new) : 0.f;
        sS[i * C + lane] = p0;
        sS[i * C + lane + 32] = p1;
        const float psum = warp_sum(p0 + p1);
        if (lane == 0) {
          const float alpha = __expf(m_old - m_new);  // exp(-inf) = 0 on the row's first chunk
          s_a[i] = alpha;
          s_m[i] = m_new;
          s_l[i] = fmaf(s_l[i], alpha, psum);
        }
      }
    }
    cp_async_wait_all();
    half_sync(half);
    if (o_active) {
#pragma unroll
      for (int i = 0; i < RM; ++i)
        if (i < R) o[i] *= s_a[i];
      const int k_lo = okh * (C / KH), k_hi = min(nk_all, k_lo + C / KH);
      int k2 = k_lo;
      for (; k2 + 4 <= k_hi; k2 += 4) {  // four keys per step, added in key order
        const float v0 = __bfloat162float(sV[(k2 + 0) * HD + od]), v1 = __bfloat162float(sV[(k2 + 1) * HD + od]);
        const float v2 = __bfloat162float(sV[(k2 + 2) * HD + od]), v3 = __bfloat162float(sV[(k2 + 3) * HD + od]);
#pragma unroll
        for (int i = 0; i < RM; ++i)
          if (i < R) {
            const float4 p4 = *reinterpret_cast<const float4*>(sS + i * C + k2);
            o[i] = fmaf(p4.x, v0, o[i]);
            o[i] = fmaf(p4.y, v1, o[i]);
            o[i] = fmaf(p4.z, v2, o[i]);
            o[i] = fmaf(p4.w, v3, o[i]);
          }
      }
      for (; k2 < k_hi; ++k2) {
        const float v = __bfloat162float(sV[k2 * HD + od]);
#pragma unroll
        for (int i = 0; i < RM; ++i)
          if (i < R) o[i] = fmaf(sS[i * C + k2], v, o[i]);
      }
    }
  }
  // add the two key halves (first + second) and leave the partial of every row of the group,
  // also of rows that saw nothing here (sum 0)
  half_sync(half);
  float* sO = reinterpret_cast<float*>(sV);
  if (KH == 2 && o_active && okh == 1) {
#pragma unroll
    for (int i = 0; i < RM; ++i)
      if (i < R) sO[i * HD + od] = o[i];
  }
  half_sync(half);
  if (o_active && okh == 0) {
#pragma unroll
    for (int i = 0; i < RM; ++i)
      if (i < R && row0 + i < pp.M) {
        const float v = (KH == 2) ? o[i] + sO[i * HD + od] : o[i];
        pp.part_o[((((size_t)(row0 + i)) * n_heads + head) * kAttnSplits + split) * HD + od] = v;
      }
  }
  if (htid < R && row0 + htid < pp.M) {
    float* ml = pp.part_ml + ((((size_t)(row0 + htid)) * n_heads + head) * kAttnSplits + split) * 2;
    ml[0] = s_m[htid];
    ml[1] = s_l[htid];
  }
  half_sync(half);  // smem and the per-row state are reused by the next item
}

template <int HD>
__host__ __device__ constexpr size_t pass_attn_smem_half() {
  return (size_t)kAttnChunk * HD * 2 + (size_t)kPassAttnR * HD * 4 + (size_t)kPassAttnR * kAttnChunk * 4;
}

template <int CG, int HD>
__host__ __device__ constexpr size_t pass_work_bytes() {
  return (size_t)(work_sc_off<CG>() + kWorkScBytes) > 2 * pass_attn_smem_half<HD>() ? (size_t)(work_sc_off<CG>() + kWorkScBytes)
                                                                                    : 2 * pass_attn_smem_half<HD>();
}

// Dynamic shared memory: [ring: n_slots * 32 KB][work area][PassShared]
template <int CG, int HD>
__global__ void __launch_bounds__(kPassThreads, 1) pass_kernel(PassParams pp, int n_slots) {
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* ring = smem;
  unsigned char* work = smem + (size_t)n_slots * kSlotBytes;
  PassShared* sh = reinterpret_cast<PassShared*>(work + pass_work_bytes<CG, HD>());
  const int tid = threadIdx.x;

  if (tid == 0) {
    for (int s = 0; s < n_slots; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], kPassConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Barriers completed by earlier launches: the counter is a multiple of the grid size when a
  // launch starts and stays below the next multiple until every CTA, this one included, has
  // arrived at the launch's first barrier.
  if (tid == 32) {
    sh->bar_base = ld_relaxed(&pp.sync->bar_count) / gridDim.x;
    sh->bar_extra = ld_relaxed(&pp.sync->bar_extra);
    // an earlier launch gave up a wait and the host has not cleared it yet: this launch's inputs
    // are not to be trusted, so it does nothing at all
    sh->abort = *reinterpret_cast<volatile int*>(&pp.sync->error) != 0 ? 1 : 0;
  }
  if (tid < kPassMaxRows) {  // where the rows sit does not change during the pass
    sh->row_pos[tid] = tid < pp.M ? pp.row_pos[tid] : -1;
    sh->row_seq[tid] = tid < pp.M ? pp.row_seq[tid] : 0;
  }
  __syncthreads();
  if (sh->abort) return;  // uniform over the CTA: nothing is in flight yet

  if (tid >= kPassConsumerThreads) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kPassProducerRegs));
    // ================= producer warp: stream this CTA's share of every weight matrix =================
    if (tid == kPassConsumerThreads) {
      // Two cursors walk the same list of chunks (a chunk = up to kChunkUnits units of one stage):
      // `ld` copies a chunk into the ring as soon as a slot is free, `pf` runs up to pf_chunks
      // chunks further ahead and only asks for them to be brought into L2.  The ring holds about
      // 2 us of weight traffic, a stage boundary (partial posts, epilogue, grid barrier, the next
      // stage's activations) costs the consumers several times that; with the prefetch the memory
      // keeps streaming through those gaps and the ring refills from L2 afterwards.  The copies
      // into the ring mark their lines evict-first, so what L2 keeps is what has not been used yet.
      struct Cursor {
        int s;
        const unsigned char* src;
        long long left;
      };
      auto advance = [&](Cursor& c) {  // to the next linear stage that has units for this CTA
        while (c.left == 0 && c.s < pp.n_stages) {
          if (++c.s == pp.n_stages) break;
          const StageDesc& st = pp.prog[c.s];
          if (st.kind != ST_LINEAR) continue;
          long long ub, ue;
          unit_range((long long)st.n_groups * st.KT, blockIdx.x, gridDim.x, ub, ue);
          c.src = reinterpret_cast<const unsigned char*>(st.W) + (size_t)ub * kUnitBytes;
          c.left = ue - ub;
        }
      };
      const uint64_t pol_first = l2_policy_evict_first();  // a weight is read once per pass
      Cursor ld{-1, nullptr, 0}, pf{-1, nullptr, 0};
      advance(ld);
      advance(pf);
      unsigned slot = 0, parity = 1u, issued = 0, ahead = 0;
      bool ok = true;
      while (ld.s < pp.n_stages) {
        while (ahead < (unsigned)pp.pf_chunks && pf.s < pp.n_stages) {
          const unsigned n = pf.left < kChunkUnits ? (unsigned)pf.left : (unsigned)kChunkUnits;
          if (ahead >= (unsigned)n_slots) bulk_prefetch_l2(pf.src, n * kUnitBytes);  // nearer chunks are copied at once anyway
          pf.src += (size_t)n * kUnitBytes;
          pf.left -= n;
          advance(pf);
          ++ahead;
        }
        ok = bounded_wait([&] { return mbar_try_wait(&sh->empty[slot], parity); }, pp.sync, &sh->abort, PASS_ERR_SLOT_EMPTY);
        if (!ok) break;
        const unsigned n = ld.left < kChunkUnits ? (unsigned)ld.left : (unsigned)kChunkUnits;
        mbar_arrive_expect_tx(&sh->full[slot], n * kUnitBytes);
        bulk_load(ring + (size_t)slot * kSlotBytes, ld.src, n * kUnitBytes, &sh->full[slot], pol_first);
        ld.src += (size_t)n * kUnitBytes;
        ld.left -= n;
        advance(ld);
        ++issued;
        if (ahead > 0) --ahead;
        if (++slot == (unsigned)n_slots) {
          slot = 0;
          parity ^= 1u;
        }
      }
      // nothing may still be landing in shared memory when the CTA exits: wait (bounded) for the
      // copies of the last n_slots slots that were issued
      const unsigned first = issued > (unsigned)n_slots ? issued - (unsigned)n_slots : 0u;
      for (unsigned j = first; j < issued; ++j) {
        const unsigned sl = j % (unsigned)n_slots, par = (j / (unsigned)n_slots) & 1u;
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(&sh->full[sl], par))
          if (global_ns() - t0 > kWaitLimitNs) break;
      }
    }
    return;
  }

  // ================= consumer warps =================
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kPassConsumerRegs));
  const unsigned long long bar_base = sh->bar_base;
  unsigned chunk_base = 0;
  bool ok = true;
  constexpr int kDescWords = (int)(sizeof(StageDesc) / sizeof(int));
  static_assert(kDescWords <= 64, "two warps fetch a stage descriptor");
  const int desc_w = tid - (kPassConsumerThreads - 64);  // the last two warps fetch descriptors, one word per thread
  for (int s = 0; s < pp.n_stages && ok; ++s) {
    if (s == 0) {
      if (desc_w >= 0 && desc_w < kDescWords)
        reinterpret_cast<int*>(&sh->st)[desc_w] = reinterpret_cast<const int*>(pp.prog)[desc_w];
    } else {
      if (desc_w >= 0 && desc_w < kDescWords) reinterpret_cast<int*>(&sh->st)[desc_w] = reinterpret_cast<const int*>(&sh->st_next)[desc_w];
    }
    consumer_sync();
    // the next stage's descriptor: asked for now, stored at the end of this stage, so that the
    // stage after a barrier starts without a round trip to global memory
    int next_word = 0;
    if (s + 1 < pp.n_stages && desc_w >= 0 && desc_w < kDescWords)
      next_word = reinterpret_cast<const int*>(pp.prog + s + 1)[desc_w];
    if (sh->st.kind == ST_LINEAR) {
      // The posts of split groups carry a number no stage of any launch shares.  Barrier serials
      // advance by n_stages - 1 per launch, so stage s gets (bar_base + s) * 2 + (1 if it is the
      // launch's first stage): only a launch's last stage and the next launch's first would
      // otherwise collide.
      const unsigned serial = 2u * ((unsigned)bar_base + (unsigned)s) + (s == 0 ? 1u : 0u) + 2u;
      if (sh->st.x_mode == X_PLAIN) {
        linear_stage<CG, HD, X_PLAIN>(pp, sh, ring, n_slots, work, chunk_base, serial);
      } else {
        // fold the attention partials into shared memory first if the columns this CTA's units
        // use fit beside the other work buffers (they do for passes of a few rows)
        long long ub, ue;
        unit_range((long long)sh->st.n_groups * sh->st.KT, blockIdx.x, gridDim.x, ub, ue);
        const long long kts = ue - ub < sh->st.KT ? ue - ub : sh->st.KT;
        const size_t need = (size_t)pp.M * (size_t)(kts * 16 + 8) * sizeof(float);
        if (need <= pass_work_bytes<CG, HD>() - (size_t)work_sc_off<CG>())
          linear_stage<CG, HD, X_STAGED>(pp, sh, ring, n_slots, work, chunk_base, serial);
        else
          linear_stage<CG, HD, X_ATTN_FOLD>(pp, sh, ring, n_slots, work, chunk_base, serial);
      }
    } else {
      const int half = tid / kHalfThreads, htid = tid % kHalfThreads;
      const int n_heads = sh->st.ep.n_heads;
      const int n_groups = (pp.M + pp.rows_per_seq - 1) / pp.rows_per_seq;
      const int items = kAttnSplits * n_heads * n_groups;
      unsigned char* my = work + (size_t)half * pass_attn_smem_half<HD>();
      for (int it = blockIdx.x * 2 + half; it < items; it += gridDim.x * 2) {
        const int split = it % kAttnSplits;
        const int hb = it / kAttnSplits;
        const int hd_ = hb % n_heads, b_ = hb / n_heads;
        if (pp.rows_per_seq <= 2)
          attention_item<HD, 2>(sh->st, pp, sh, my, half, htid, hd_, split, b_);
        else if (pp.rows_per_seq <= 8)
          attention_item<HD, 8>(sh->st, pp, sh, my, half, htid, hd_, split, b_);
        else
          attention_item<HD, 16>(sh->st, pp, sh, my, half, htid, hd_, split, b_);
      }
    }
    if (desc_w >= 0 && desc_w < kDescWords) reinterpret_cast<int*>(&sh->st_next)[desc_w] = next_word;
    // the barrier also tells every thread whether a wait of this CTA gave up (the CTA still arrives)
    ok = (s + 1 < pp.n_stages) ? grid_barrier(pp.sync, bar_base + (unsigned long long)(s + 1), sh) : consumers_agree_ok(sh);
  }
}

// ---- packing into the unit layout -----------------------------------------------------------------
// element e: unit = e / 2048 = group * KT + kt; tile r = (e % 2048) / 256; inside the tile the
// register order of the MMA A fragment: lane = (e % 256) / 8, j = e % 8,
//   j = 0,1: (row g,     k 2q + j)        j = 2,3: (row g + 8, k 2q + j - 2)
//   j = 4,5: (row g,     k 2q + 8 + j-4)  j = 6,7: (row g + 8, k 2q + 8 + j - 6)
// Row g of tile rt is the first feature of pair 8*rt + g, row g + 8 its second.  Row tiles
// beyond NT (a ragged last group) are zero.
__global__ void pack_units_kernel(__nv_bfloat16* __restrict__ dst, PackSrc ps, int n_pairs, int K, int n_groups) {
  const int KT = K >> 4, NT = n_pairs >> 3;
  const size_t total = (size_t)n_groups * KT * (kUnitBytes / 2);
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const size_t unit = e >> 11;
    const int within = (int)(e & 2047);
    const int r = within >> 8, lane = (within & 255) >> 3, j = within & 7;
    const int grp = (int)(unit / KT), kt = (int)(unit % KT);
    const int rt = grp * kUnitTiles + r;
    const int g = lane >> 2, q = lane & 3;
    const int second = (j >> 1) & 1;
    const int k = kt * 16 + 2 * q + (j & 1) + ((j >> 2) ? 8 : 0);
    dst[e] = rt < NT ? pack_src_row<__nv_bfloat16>(ps, 8 * rt + g, second, K)[k] : __float2bfloat16_rn(0.f);
  }
}

}  // namespace sdfp
