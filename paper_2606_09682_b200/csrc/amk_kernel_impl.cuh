// The decode step as one persistent cooperative kernel for sm_100a: one block per SM, each block walks
// its statically known queue of tasks -- wait for the inputs, compute, publish -- as in the paper's
// per-SM scheduler loop (Algorithm 1) and counter model (Section 4, "Synchronization model").
//
// What is different from the paper's kernel (written for sm_75..sm_120, where it found the per-tile
// cross-SM synchronisation to be the limiter, Section 7):
//   * Weights do not depend on activations, so a dedicated producer warp streams this block's packed
//     weight bytes through a shared-memory ring with bulk asynchronous copies (TMA) and mbarriers,
//     running ahead across dependencies: the HBM pipe keeps flowing while consumers wait for an input.
//   * Activations travel as {value, sequence number} pairs written with one 8-byte store, so a reader
//     that sees the task's sequence number has the value: producers need no fence and readers no separate
//     flag.  The paper's release-increment / acquire-spin counters are kept as an optional second layer
//     (sync_mode 0: one counter per join, every block signals each once, never reset: step e waits for
//     e * n_blocks) so the two can be measured against each other.
//   * The matrix-vector products run on the tensor cores (warp-level mma, fragments loaded with ldmatrix
//     straight from the ring): the activation vector occupies two (bf16: high and low halves) or three
//     (int8 / int4: base-256 digits) of the eight B columns, so nothing is converted per weight and the
//     result keeps fp32 / exact-integer accuracy.  A scalar loop needs ~2 instructions per weight; the
//     traced consumer was 3x slower than the HBM stream with it.
//   * RMSNorm is folded into the consuming GEMV's prologue, RoPE and the KV append into the attention
//     task, SiLU*up and the residual adds into GEMV epilogues, the split-K combine and the global argmax
//     into "last arriver finishes" steps, so no extra joins are needed.
//   * Every wait is bounded; on expiry the block records the failure and every block drains and exits.
//
// This file is compiled twice (amk_kernel.cu, amk_kernel_trace.cu): once without and once with the trace stamps
// (AMK_TRACE_BUILD).  Every task's code runs once per task, straight through, so the step is sensitive to the
// kernel's instruction footprint: with the stamps merely compiled in (and switched off at run time) a TinyLlama
// step measured 4-9 % slower.  AMK_KERNEL / AMK_LAUNCH / AMK_ATTRS name the build's kernel and entry points.
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "amk.h"
#include "amk_internal.h"
#include "amk_ptx.cuh"

#ifndef AMK_TRACE_BUILD
#error "include this file from amk_kernel.cu or amk_kernel_trace.cu"
#endif

namespace amk {

namespace {

constexpr int kBarCons = 1;                          // named barrier of the consumer warps
constexpr int kOutWarps = (kPassRows + 31) / 32;     // warps that hold a pass's output rows
constexpr int kBatch = 4;                            // 32-byte items (four activation elements) a thread gathers at a
                                                     // time (a normed input must fit one batch per thread)
// int8 / int4 activations: X = round(a / scale) as three signed base-256 digits, |X| <= kDigitScale.  Adding
// kDigitBias = 2^23 + 0x408080 in the same fused multiply-add rounds to the integer and leaves, in the low three
// bytes of the float's bit pattern, d0 + 128, d1 + 128 and d2 + 64 (needs -4227200 <= X < 4161408; the margin
// covers the few ulp of the approximate reciprocal behind the scale).
constexpr float kDigitScale = 4161000.0f;
constexpr float kDigitBias = 12615808.0f;

struct Ctx {
  const KParams& p;
  SmemHeader* sh;
  unsigned char* xs;     // activation area (bf16 hi/lo halves or int8 digits) / attention scratch
  unsigned char* ring;
  int tid, warp, lane, cta, nblk;
  int stage;             // ring stage of the next tile this warp walks
  unsigned parity;       // its phase parity
  int token;
  bool bad;              // this thread saw a failure; agreed on at the next consumer barrier
};

// Barrier of the consumer warps that also ORs a failure predicate, so that all of them leave together.
__device__ __forceinline__ bool cons_sync_or(bool bad) {
  unsigned r;
  asm volatile(
      "{ .reg .pred p, q; setp.ne.u32 q, %1, 0; bar.red.or.pred p, %2, %3, q; selp.u32 %0, 1, 0, p; }"
      : "=r"(r)
      : "r"((unsigned)bad), "r"(kBarCons), "r"(kConsumerThreads)
      : "memory");
  return r != 0;
}

__device__ __noinline__ void report_failure(const KParams& p, unsigned code, int phase, unsigned seen, unsigned want) {
  if (atomicCAS(&p.status->code, 0u, code) == 0u) {
    p.status->phase = phase;
    p.status->block = blockIdx.x;
    p.status->seen = seen;
    p.status->want = want;
  }
  __threadfence();
  atomicExch(&p.status->abort, 1u);
}

// Acquire-spin on a monotonic counter until it reaches `target` (wrap-safe), bounded in time.
__device__ __noinline__ bool poll_counter(const KParams& p, const unsigned* ctr, unsigned target, int phase) {
  unsigned v = ld_acquire_gpu(ctr);
  if ((int)(v - target) >= 0) return true;
  const unsigned long long t0 = globaltimer_ns();
  unsigned spins = 0;
  for (;;) {
    v = ld_acquire_gpu(ctr);
    if ((int)(v - target) >= 0) return true;
    if ((++spins & 15u) == 0u) {
      if (ld_relaxed_gpu(&p.status->abort)) return false;
      if (globaltimer_ns() - t0 > p.timeout_ns) {
        report_failure(p, (unsigned)AMK_ERR_TIMEOUT, phase, v, target);
        return false;
      }
    }
  }
}

// Bounded wait on a ring mbarrier.  kind -1: a consumer waiting for a tile; -2: the producer waiting for a slot.
__device__ __noinline__ bool wait_mbar_slow(const KParams& p, uint64_t* bar, unsigned parity, int kind) {
  const unsigned long long t0 = globaltimer_ns();
  unsigned spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63u) == 0u) {
      if (ld_relaxed_gpu(&p.status->abort)) return false;
      if (globaltimer_ns() - t0 > p.timeout_ns) {
        report_failure(p, (unsigned)AMK_ERR_TIMEOUT, kind, 0u, parity);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ bool wait_mbar(const KParams& p, uint64_t* bar, unsigned parity, int kind) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_mbar_slow(p, bar, parity, kind);
}

// A step at position 0 with data-carried dependencies has no attention task: the QKV projection's epilogue
// publishes the attention output and appends the cache rows itself (see gemv_op).
// Test hook of the bounded waits (diagnostic build): this block withholds what it would publish for `task`.
__device__ __forceinline__ bool dropped(const KParams& p, int task, int cta) {
#if AMK_TRACE_BUILD
  return task == p.drop_phase && cta == p.drop_block;
#else
  return false;
#endif
}

#if AMK_TRACE_BUILD
__device__ __forceinline__ bool counter_joins(const KParams& p) { return p.sync_mode == 0; }
#else
__device__ __forceinline__ bool counter_joins(const KParams&) { return false; }     // (the diagnostic build has them)
#endif
__device__ __forceinline__ bool single_pos(const KParams& p) { return p.pos == 0 && !counter_joins(p); }

// Sequence number carried by everything task `task` publishes in this step (never 0).  Task -1 is the embedding
// row, which every block publishes its share of at kernel start like any other activation.
__device__ __forceinline__ unsigned seq_of(const KParams& p, int task) {
  return p.epoch * (unsigned)(5 * p.L + 2) + (unsigned)(task + 2);
}

// Counter layer (sync_mode 0): all consumer threads wait until every block has signalled `phase`.
__device__ __forceinline__ bool wait_phase(Ctx& c, int phase) {
  if (!counter_joins(c.p)) return true;
  if (c.tid == 0) {
    if (!poll_counter(c.p, c.p.phase_ctr + phase, c.p.ctr_epoch * (unsigned)c.nblk, phase)) c.bad = true;
  }
  c.bad = cons_sync_or(c.bad);
  return !c.bad;
}
// Called after a consumer barrier that follows the task's last store: release-increment the counter.
__device__ __forceinline__ void signal_phase(Ctx& c, int phase) {
  if (!counter_joins(c.p)) return;
  if (c.tid == 0 && !dropped(c.p, phase, c.cta))
    red_release_gpu_add(c.p.phase_ctr + phase, 1u);
}

// One thread stamps the global timer for (task, event) of this block when tracing is on.
__device__ __forceinline__ void stamp(const KParams& p, int cta, int task, int ev) {
#if AMK_TRACE_BUILD
  if (p.trace)
    p.trace[((size_t)cta * (5 * p.L + 1) + task) * AMK_TRACE_EVENTS + ev] =
        (p.flags & AMK_FLAG_TRACE_CYCLES) ? (unsigned long long)clock64() : globaltimer_ns();
#endif
}

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
// The two reductions that sit between the arrival of an input and its first multiply, for values >= 0, with the
// warp-wide integer reduction instruction (one instruction each instead of five dependent shuffles):
// the maximum through the bit patterns (ordered like the values), exact; the sum in fixed point relative to the
// largest lane (that lane in [2^26, 2^27), so 32 lanes cannot overflow 32 bits): relative error below 2.5e-7,
// the same in every thread and every run.
__device__ __forceinline__ float warp_max_nonneg(float v) {
  return __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(v)));
}
__device__ __forceinline__ float warp_sum_nonneg(float v) {
  const unsigned m = __reduce_max_sync(0xffffffffu, __float_as_uint(v));
  int e = (int)(m >> 23) - 127;                        // floor(log2(largest lane))
  e = max(-90, min(90, e));
  if (m == 0u) return 0.f;
  const float up = __uint_as_float((unsigned)(127 + 26 - e) << 23);       // 2^(26 - e)
  const float down = __uint_as_float((unsigned)(127 - 26 + e) << 23);     // 2^(e - 26)
  const unsigned t = __reduce_add_sync(0xffffffffu, __float2uint_rn(fminf(v * up, 134217727.f)));
  return (float)t * down;
}

// Spin until the element at `addr` carries `seq`; bounded.  On failure the returned element does not carry `seq`
// (values are returned, not written through a pointer, so callers' arrays stay in registers).
__device__ __noinline__ uint2 poll_pair_slow(const KParams& p, const void* addr, unsigned seq, int task) {
  const unsigned long long t0 = globaltimer_ns();
  unsigned spins = 0;
  for (;;) {
    uint2 v = ld_pair(addr);
    if (v.y == seq) return v;
    if ((++spins & 15u) == 0u) {
      bool give_up = ld_relaxed_gpu(&p.status->abort) != 0u;
      if (!give_up && globaltimer_ns() - t0 > p.timeout_ns) {
        report_failure(p, (unsigned)AMK_ERR_TIMEOUT, task, v.y, seq);
        give_up = true;
      }
      if (give_up) { v.y = seq + 1u; return v; }
    }
  }
}
// One activation element written by `task` in this step.
__device__ __forceinline__ float read_act(const KParams& p, bool& bad, const ActPair* a, unsigned seq, int task) {
  uint2 v = ld_pair(a);
  if (v.y != seq) {
    v = poll_pair_slow(p, a, seq, task);
    if (v.y != seq) bad = true;
  }
  return __uint_as_float(v.x);
}

// fp8 e4m3 cache entries: round to nearest even, saturating at +-448 (the hardware's conversion), and back (exact).
__device__ __forceinline__ unsigned char f32_to_e4m3(float v) {
  return (unsigned char)__nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3);
}
__device__ __forceinline__ float e4m3_to_f32(unsigned char code) {
  return __half2float(__half(__nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)code, __NV_E4M3)));
}
// Eight consecutive cache elements as fp32: 16 bytes of bf16, or 8 bytes of e4m3.
template <bool FP8>
__device__ __forceinline__ void cache8(const unsigned char* p8, float (&f)[8]) {
  if (FP8) {
    const uint2 w = *reinterpret_cast<const uint2*>(p8);
    const unsigned v[2] = {w.x, w.y};
#pragma unroll
    for (int i = 0; i < 2; i++) {
      const float2 a = __half22float2(__half2(__nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(v[i] & 0xffffu), __NV_E4M3)));
      const float2 b = __half22float2(__half2(__nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(v[i] >> 16), __NV_E4M3)));
      f[4 * i] = a.x; f[4 * i + 1] = a.y; f[4 * i + 2] = b.x; f[4 * i + 3] = b.y;
    }
  } else {
    const uint4 w = *reinterpret_cast<const uint4*>(p8);
    f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
    f[4] = bf16_lo(w.z); f[5] = bf16_hi(w.z); f[6] = bf16_lo(w.w); f[7] = bf16_hi(w.w);
  }
}

// (on the gate/up -> down critical path: the hardware's exp2 and reciprocal, ~1e-6 relative)
__device__ __forceinline__ float silu_f(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

// ------------------------------------------------------------------------------------------------
// Prologue of a matrix-vector product: bring the input vector (K elements written by `src_task`, or the
// embedding row) into shared memory in the form the tensor cores take, with RMSNorm folded in.
//   bf16 weights: X0[K] = bf16(a), X1[K] = bf16(a - X0): two B columns whose sum is a to 2^-17.
//   int8 / int4 : a / scale as three signed base-256 digits D2, D1, D0 (three B columns), exact integers.
// ------------------------------------------------------------------------------------------------

// Four input elements (item `it` = elements 4 it .. 4 it + 3) -> their shared-memory form.
// (This runs between the arrival of the input and the first multiply, so every instruction counts: the
// hardware's paired fp32 -> bf16 conversion, byte permutes for the digits, 8-byte stores.)
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {      // {bf16(lo), bf16(hi)}, round to nearest even
  unsigned r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// (integer weights: called by whole warps -- the warp's 32 items are one group of 128 elements sharing a scale; the
//  lanes beyond the end of a vector whose length is not a multiple of 128 pass zeros.)
//  `n4`: items per column (integer weights: of the column length rounded up to whole groups, the tail zero).
template <int WD>
__device__ __forceinline__ void store_item(unsigned char* xs, int n4, int it, const float (&a)[4]) {
  if (WD == W_BF16) {
    // two B columns: bf16(a) and bf16(a - bf16(a)); their sum is a to 2^-17 (a third column would make it exact
    // and measured 1.3 % slower at the TinyLlama shape for an error far below the others')
    uint2* X0 = reinterpret_cast<uint2*>(xs);                        // columns of K bf16 = n4 items of 8 bytes
    const unsigned h0 = pack_bf16x2(a[0], a[1]), h1 = pack_bf16x2(a[2], a[3]);
    X0[it] = make_uint2(h0, h1);
    X0[n4 + it] = make_uint2(pack_bf16x2(a[0] - bf16_lo(h0), a[1] - bf16_hi(h0)),                 // (differences exact)
                             pack_bf16x2(a[2] - bf16_lo(h1), a[3] - bf16_hi(h1)));
  } else {
    // X = d2 * 65536 + d1 * 256 + d0 with every digit in [-128, 127] (see kDigitBias)
    unsigned* D2 = reinterpret_cast<unsigned*>(xs);                  // columns of K bytes = n4 items of 4 bytes
    // a scale of its own for every group of 128 elements, which is exactly a warp's 32 items (items are dealt out
    // warp by warp): one warp-wide maximum, no pass over the whole vector
    const float gmax = warp_max_nonneg(fmaxf(fmaxf(fabsf(a[0]), fabsf(a[1])), fmaxf(fabsf(a[2]), fabsf(a[3]))));
    const float inv = gmax > 0.f ? __fdividef(kDigitScale, gmax) : 0.f;
    unsigned t[4];
#pragma unroll
    for (int e = 0; e < 4; e++) t[e] = __float_as_uint(fmaf(a[e], inv, kDigitBias));
    const unsigned p01 = __byte_perm(t[0], t[1], 0x5140), p23 = __byte_perm(t[2], t[3], 0x5140);   // {b0, b0', b1, b1'}
    const unsigned w0 = __byte_perm(p01, p23, 0x5410) ^ 0x80808080u;
    const unsigned w1 = __byte_perm(p01, p23, 0x7632) ^ 0x80808080u;
    const unsigned w2 = (__byte_perm(__byte_perm(t[0], t[1], 0x0062), __byte_perm(t[2], t[3], 0x0062), 0x5410) + 0x40404040u) ^ 0x80808080u;
    D2[2 * n4 + it] = w0;
    D2[n4 + it] = w1;
    D2[it] = w2;
    {
      // The group's entry of the table behind the digit columns, laid out by accumulator column pair:
      // {A2, A1, scale, -} {A0, 0, scale, -}.  int4: the zero point of a weight group meets the sum of the input's
      // integers X over the group (see consume_pass): one warp-wide integer sum (below 2^29), split into signed
      // base-256 digits A like the elements themselves so that each meets the accumulator column of its weight.
      int s0 = 0, s1 = 0, s2 = 0;
      if (WD == W_INT4) {
        const int sx = (int)(__reduce_add_sync(0xffffffffu, (t[0] + t[1]) + (t[2] + t[3])) - 128u * 0x4B408080u);
        s0 = (sx << 24) >> 24;
        const int r1 = (sx - s0) >> 8;
        s1 = (r1 << 24) >> 24;
        s2 = (r1 - s1) >> 8;
      }
      const int lane = threadIdx.x & 31;
      if (lane < 2) {
        const int sc = __float_as_int(gmax * (1.0f / kDigitScale));
        reinterpret_cast<int4*>(xs + 12 * (size_t)n4)[2 * (it >> 5) + lane] =
            lane == 0 ? make_int4(s2, s1, sc, 0) : make_int4(s0, 0, sc, 0);
      }
    }
  }
}

// An item of four consecutive activation elements, {value, sequence number} each, fetched with one 32-byte
// request (four 64-bit accesses, each single-copy atomic like the store that wrote it).
struct Item {
  unsigned long long e[4];
  __device__ __forceinline__ float val(int j) const { return __uint_as_float((unsigned)e[j]); }
  __device__ __forceinline__ bool carries(unsigned seq) const {
    return (unsigned)(e[0] >> 32) == seq && (unsigned)(e[1] >> 32) == seq && (unsigned)(e[2] >> 32) == seq &&
           (unsigned)(e[3] >> 32) == seq;
  }
};
__device__ __forceinline__ Item ld_item(const ActPair* p4) {
  Item t;
  asm volatile("ld.relaxed.gpu.global.L2::cache_hint.v4.u64 {%0,%1,%2,%3}, [%4], %5;"
               : "=l"(t.e[0]), "=l"(t.e[1]), "=l"(t.e[2]), "=l"(t.e[3])
               : "l"(p4), "l"(policy_evict_last())
               : "memory");
  return t;
}

// Gather one batch of items (item0, item0 + T, ...): request them all, and if any has not arrived yet request
// the whole batch again until all carry `seq` (bounded).  Returns true on failure.
__device__ __forceinline__ bool gather_batch(const KParams& p, Item (&raw)[kBatch], int item0, int n4,
                                             const ActPair* src, unsigned seq, int src_task, int cta, int task) {
  unsigned long long t0 = 0;
  for (unsigned spins = 0;; spins++) {
    bool all = true;
#pragma unroll
    for (int i = 0; i < kBatch; i++) {
      const int it = item0 + i * kConsumerThreads;
      if (it < n4) raw[i] = ld_item(src + 4 * it);
    }
#pragma unroll
    for (int i = 0; i < kBatch; i++) {
      const int it = item0 + i * kConsumerThreads;
      if (it < n4) all = all && raw[i].carries(seq);
    }
    if (all) {
#if AMK_TRACE_BUILD
      if (p.trace && item0 == 0)     // (not a time) how many requests thread 0 needed for its first batch
        p.trace[((size_t)cta * (5 * p.L + 1) + task) * AMK_TRACE_EVENTS + AMK_TR_POLLS] = spins + 1u;
#endif
      return false;
    }
    if (spins == 0) t0 = globaltimer_ns();
    if ((spins & 15u) == 15u) {
      if (ld_relaxed_gpu(&p.status->abort)) return true;
      if (globaltimer_ns() - t0 > p.timeout_ns) {
        report_failure(p, (unsigned)AMK_ERR_TIMEOUT, src_task, 0u, seq);
        return true;
      }
    }
  }
}

struct LoadResult {
  float rnorm;       // normed input: 1/rms, to be applied to the outputs (1 otherwise)
  bool bad;
};

// Every item is converted as soon as it has arrived.  RMSNorm's 1/rms is one scalar for the
// whole vector, so W (r * x * g) = r * (W (x * g)): the items go to shared memory as x * g while the sum of squares
// is still being collected, and r is applied to the outputs in the epilogue -- no second pass over the input and no
// block-wide reduction between the arrival of the input and the first multiply.  (Integer weights: the digits' scale
// is per group of 128 elements and meets the group's integer sums in one multiply-add, see consume_pass.)
template <int WD>
__device__ __forceinline__ LoadResult load_input_1pass(const KParams& p, SmemHeader* sh, unsigned char* xs, int cta, int K,
                                                       const ActPair* src, unsigned seq, int src_task,
                                                       const unsigned short* normw, int task) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n4 = K >> 2;                               // items of four elements
  const int n4s = (WD == W_BF16) ? n4 : ((n4 + 31) & ~31);   // items per shared-memory column (whole groups)
  LoadResult res{1.0f, false};
  Item raw[kBatch];
  // norm weights of my items: requested before the gather, so that their latency (they come from HBM, being
  // read once per token) is not added to the join's (a normed input is one batch per thread)
  uint2 gwt[kBatch];
  if (normw) {
#pragma unroll
    for (int i = 0; i < kBatch; i++) {
      const int it = tid + i * kConsumerThreads;
      gwt[i] = (it < n4) ? __ldg(reinterpret_cast<const uint2*>(normw) + it) : make_uint2(0u, 0u);
    }
  }
  float ss = 0.f;
  // (integer weights: the conversion works warp-wide, so a warp stays together through a ragged last group)
  constexpr int kWhole = (WD == W_BF16) ? 0 : 31;
#pragma unroll 1
  for (int i0 = tid; i0 - (lane & kWhole) < n4; i0 += kBatch * kConsumerThreads) {
    res.bad |= gather_batch(p, raw, i0, n4, src, seq, src_task, cta, task);
#pragma unroll
    for (int i = 0; i < kBatch; i++) {
      const int it = i0 + i * kConsumerThreads;
      if (it - (lane & kWhole) < n4) {
        const bool valid = it < n4;
        float a[4] = {raw[i].val(0), raw[i].val(1), raw[i].val(2), raw[i].val(3)};
        if (WD != W_BF16 && !valid) a[0] = a[1] = a[2] = a[3] = 0.f;
        if (normw) {
          ss = fmaf(a[0], a[0], ss);
          ss = fmaf(a[1], a[1], ss);
          ss = fmaf(a[2], a[2], ss);
          ss = fmaf(a[3], a[3], ss);
          a[0] *= bf16_lo(gwt[i].x);
          a[1] *= bf16_hi(gwt[i].x);
          a[2] *= bf16_lo(gwt[i].y);
          a[3] *= bf16_hi(gwt[i].y);
        }
        store_item<WD>(xs, n4s, it, a);
      }
    }
  }
  if (normw) {
    ss = warp_sum_nonneg(ss);
    if (lane == 0) sh->warp_part[0][warp] = ss;
  }
  if (tid == 0) stamp(p, cta, task, AMK_TR_JOINED);
  res.bad = cons_sync_or(res.bad);
  if (normw) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; w++) tot += sh->warp_part[0][w];
    res.rnorm = rsqrtf(__fdividef(tot, (float)K) + p.eps);       // (2 ulp: the same factor on every output)
  }
  return res;
}

// ------------------------------------------------------------------------------------------------
// One pass on the tensor cores: this warp walks every ring tile of the pass, multiplies its row group
// (<= 16 rows, one m16 tile) by the input columns over its column blocks, and publishes per-row sums.
// ------------------------------------------------------------------------------------------------

template <int WD>
__device__ __forceinline__ void consume_pass(Ctx& c, const PassGeom& g, int kind, int gw, int K, float* red,
                                             int task) {
  const KParams& p = c.p;
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_PASS_BEGIN);
  const int wr = c.sh->wr_of[kind][gw][c.warp], wk = c.sh->wk_of[kind][gw][c.warp];
  const bool active = wk < g.Wk;
  const int urows = (wr == g.Wr - 1) ? g.g_last : g.G;
  const int gq = c.lane >> 2, q = c.lane & 3;                                  // fragment row / column-pair index
  const int mrow = min((c.lane & 7) + ((c.lane >> 3) & 1) * 8, urows - 1);     // ldmatrix: my row of my 8x8 matrix
  const unsigned lane_off = (unsigned)(((c.lane >> 4) * urows + mrow) * 16);   // chunk half h = lane / 16
  const unsigned step_stride = (unsigned)(2 * urows * 16);                     // two chunks per k step
  const int S = p.n_stages;
  constexpr int BC = block_cols(WD);
  // B columns in use: int8 / int4 three digits; bf16 high + low parts
  constexpr int NCOL = (WD == W_BF16) ? 2 : 3;
  const int Ks = (WD == W_BF16) ? 2 * K : ((K + 127) & ~127);       // bytes per input column in shared memory
  const unsigned char* xcol = c.xs + (size_t)min(gq, NCOL - 1) * Ks;

  // All fragments of a unit are loaded before its first MMA, and two accumulator sets are used in turn, so
  // that consecutive MMAs do not wait for each other.
  float facc[4] = {0.f, 0.f, 0.f, 0.f}, facc2[4] = {0.f, 0.f, 0.f, 0.f};
  constexpr int NA = (WD == W_INT4) ? 2 : 4;         // ldmatrix.x4 loads per unit
  unsigned fa[NA][4];                                // pending unit: weight fragments,
  uint4 fx0 = make_uint4(0u, 0u, 0u, 0u), fx1 = fx0; // input fragments,
  unsigned fsz0 = 0u, fsz1 = 0u;                     // int4: {scale, zero} of my two rows,
  int4 fsx = make_int4(0, 0, 0, 0);                  //       the input group's digit sums for my two columns, its scale
  auto flush = [&]() {
    if (WD == W_BF16) {
      mma_bf16(facc, fa[0], fx0.x, fx0.y);
      mma_bf16(facc2, fa[1], fx0.z, fx0.w);
      mma_bf16(facc, fa[2], fx1.x, fx1.y);
      mma_bf16(facc2, fa[3], fx1.z, fx1.w);
    } else if (WD == W_INT8 || WD == W_INT8G) {
      // one group of 128 columns: exact integer sums in two chains, then the input's group scale -- times the
      // weights' group scale for grouped int8; a per-row weight scale meets the finished sum in the epilogue --
      // in one multiply-add per accumulator
      int g4[4] = {0, 0, 0, 0}, h4[4] = {0, 0, 0, 0};
      mma_s8(g4, fa[0][0], fa[0][1], fa[0][2], fa[0][3], fx0.x, fx0.y);
      mma_s8(h4, fa[1][0], fa[1][1], fa[1][2], fa[1][3], fx0.z, fx0.w);
      mma_s8(g4, fa[2][0], fa[2][1], fa[2][2], fa[2][3], fx1.x, fx1.y);
      mma_s8(h4, fa[3][0], fa[3][1], fa[3][2], fa[3][3], fx1.z, fx1.w);
      const float xsc = __int_as_float(fsx.z);
      const float s0 = (WD == W_INT8) ? xsc : __half2float(__ushort_as_half((unsigned short)(fsz0 & 0xffffu))) * xsc;
      const float s1 = (WD == W_INT8) ? xsc : __half2float(__ushort_as_half((unsigned short)(fsz1 & 0xffffu))) * xsc;
      facc[0] = fmaf(s0, (float)(g4[0] + h4[0]), facc[0]);
      facc[1] = fmaf(s0, (float)(g4[1] + h4[1]), facc[1]);
      facc[2] = fmaf(s1, (float)(g4[2] + h4[2]), facc[2]);
      facc[3] = fmaf(s1, (float)(g4[3] + h4[3]), facc[3]);
    } else {
      // sum over k of s (q_k - z) x_k = s (sum q_k x_k - z sum x_k): the codes go to the tensor cores as unsigned
      // bytes, and the zero point meets the sum of the input's digits over the group, which the input's loader
      // left in a table (store_item).
      const float xsc = __int_as_float(fsx.z);
      const float s0 = __half2float(__ushort_as_half((unsigned short)(fsz0 & 0xffffu))) * xsc;
      const float s1 = __half2float(__ushort_as_half((unsigned short)(fsz1 & 0xffffu))) * xsc;
      const int z0 = (int)(fsz0 >> 16), z1 = (int)(fsz1 >> 16);      // (the packer stores the zero point as an integer)
      // The low nibbles go in as they are (one AND per four codes); the high nibbles stay where they are, as 16 x
      // code (unsigned bytes 0..240), in a chain of their own whose exact sum is divided by 16 at the end.
      constexpr unsigned M = 0x0F0F0F0Fu, MH = 0xF0F0F0F0u;
      int g4[4] = {0, 0, 0, 0}, h4[4] = {0, 0, 0, 0};
      mma_u8s8(g4, fa[0][0] & M, fa[0][1] & M, fa[0][2] & M, fa[0][3] & M, fx0.x, fx0.y);
      mma_u8s8(h4, fa[0][0] & MH, fa[0][1] & MH, fa[0][2] & MH, fa[0][3] & MH, fx0.z, fx0.w);
      mma_u8s8(g4, fa[1][0] & M, fa[1][1] & M, fa[1][2] & M, fa[1][3] & M, fx1.x, fx1.y);
      mma_u8s8(h4, fa[1][0] & MH, fa[1][1] & MH, fa[1][2] & MH, fa[1][3] & MH, fx1.z, fx1.w);
      // digit sums of this group for my two accumulator columns (2q, 2q + 1): {D2, D1} for q = 0, {D0, -} for q = 1
      // (the other quad positions' columns are not in use and weigh nothing in the end)
      const int sx0 = fsx.x, sx1 = fsx.y;
#pragma unroll
      for (int e = 0; e < 4; e++) g4[e] += h4[e] >> 4;
      facc[0] = fmaf(s0, (float)(g4[0] - z0 * sx0), facc[0]);
      facc[1] = fmaf(s0, (float)(g4[1] - z0 * sx1), facc[1]);
      facc[2] = fmaf(s1, (float)(g4[2] - z1 * sx0), facc[2]);
      facc[3] = fmaf(s1, (float)(g4[3] - z1 * sx1), facc[3]);
    }
  };
  int next_b = wk;                                   // my next column block
  const int my_off = wr * g.ub_full;
  // first unit of the current tile as (block, row-warp), and the step from one tile to the next
  int t_b = 0, t_r = 0;
  const int step_b = c.sh->step_b[kind][gw], step_r = c.sh->step_r[kind][gw];
  for (int t = 0; t < g.n_tiles; ++t) {
    const int tile_off = t_b * g.bb + t_r * g.ub_full;
    int n_b = t_b + step_b, n_r = t_r + step_r;      // first unit of the next tile
    if (n_r >= g.Wr) { n_r -= g.Wr; n_b++; }
    if (!c.bad && !wait_mbar(p, &c.sh->full[c.stage], c.parity, -1)) c.bad = true;
    if (c.tid == 0 && t == 0) stamp(p, c.cta, task, AMK_TR_FIRST_TILE);
    if (active && !c.bad) {
      const unsigned char* sbase = c.ring + (size_t)c.stage * p.stage_bytes;
      // my units in this tile: blocks next_b, next_b + Wk, ... while (b, wr) comes before (n_b, n_r)
      const int end_b = min(g.nblk, n_b + (wr < n_r ? 1 : 0));
      for (; next_b < end_b; next_b += g.Wk) {
        const unsigned char* u = sbase + (next_b * g.bb + my_off - tile_off);
        // (B columns beyond NCOL repeat the last one: their accumulator columns weigh nothing in the end)
        if (WD == W_BF16) {
          const uint4* xp = reinterpret_cast<const uint4*>(xcol + ((size_t)next_b * BC + 16 * q) * 2);
          fx0 = xp[0];
          fx1 = xp[1];
        } else {
          const uint4* xp = reinterpret_cast<const uint4*>(xcol + (size_t)next_b * BC + 32 * q);
          fx0 = xp[0];
          fx1 = xp[1];
          if (WD != W_INT8) {
            // {scale, zero} of my two fragment rows for this group (= this column block)
            const unsigned* szp = reinterpret_cast<const unsigned*>(u + urows * (WD == W_INT4 ? 64 : 128));
            fsz0 = szp[min(gq, urows - 1)];
            fsz1 = szp[min(gq + 8, urows - 1)];
          }
          fsx = *reinterpret_cast<const int4*>(c.xs + 3 * (size_t)Ks + 32 * next_b + 16 * (q & 1));
        }
#pragma unroll
        for (int j = 0; j < NA; j++) ldmatrix_x4(fa[j], u + lane_off + j * step_stride);
        flush();
      }
    }
    __syncwarp();
    if (c.lane == 0 && !c.bad) mbar_arrive(&c.sh->empty[c.stage]);
    if (++c.stage == S) { c.stage = 0; c.parity ^= 1u; }
    t_b = n_b;
    t_r = n_r;
  }
#pragma unroll
  for (int e = 0; e < 4; e++) facc[e] += facc2[e];
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_TILES_DONE);
  // per-row result: sum of the B columns in use, with the digit weights for integer inputs
  float y0, y1;
  if (WD == W_BF16) {
    y0 = (q == 0) ? facc[0] + facc[1] : 0.f;           // columns 0 and 1: the high and low parts
    y1 = (q == 0) ? facc[2] + facc[3] : 0.f;
  } else {
    // columns 2q and 2q+1 of this lane: digit weights 65536 (col 0), 256 (col 1), 1 (col 2), 0 otherwise
    const float w0 = (q == 0) ? 65536.f : (q == 1 ? 1.f : 0.f);
    const float w1 = (q == 0) ? 256.f : 0.f;
    y0 = w0 * facc[0] + w1 * facc[1];
    y1 = w0 * facc[2] + w1 * facc[3];
  }
  y0 += __shfl_xor_sync(0xffffffffu, y0, 1);
  y0 += __shfl_xor_sync(0xffffffffu, y0, 2);
  y1 += __shfl_xor_sync(0xffffffffu, y1, 1);
  y1 += __shfl_xor_sync(0xffffffffu, y1, 2);
  if (active && q == 0) {
    float* dst = red + wk * g.R + wr * g.G;
    if (gq < urows) dst[gq] = y0;
    if (gq + 8 < urows) dst[gq + 8] = y1;
  }
}

// ------------------------------------------------------------------------------------------------
// One matrix-vector product with its fused prologue (gather / RMSNorm) and epilogue.
// ------------------------------------------------------------------------------------------------
// LMH: the LM head (bf16 unless the configuration quantises it; compiled apart from the per-layer code so that a
// quantised model's layers carry neither its code nor its registers); otherwise `kind_rt` is one of the four
// per-layer products.  WDL is the dtype of the product's weights.
template <int WDL, bool LMH>
__device__ __forceinline__ bool gemv_op(Ctx& c, int kind_rt, int l) {
  const KParams& p = c.p;
  const int kind = LMH ? (int)OP_LMHEAD : kind_rt;
  constexpr int WD = WDL;
  const OpShape d = p.shape[kind];
  const int task = (kind == OP_LMHEAD) ? 5 * p.L : 5 * l + (kind == OP_QKV ? 0 : kind + 1);
  Slice sl;
  sl.row0 = c.sh->slice_row0[kind];
  sl.rows = c.sh->slice_rows[kind];
  const int K = d.K;
  const unsigned my_seq = seq_of(p, task);
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_ENTER);

  // input vector, the task that wrote it, and the norm weight of this op
  const ActPair* src = nullptr;
  const unsigned short* normw = nullptr;
  int src_task = -1;
  switch (kind) {
    case OP_QKV:       // (layer 0: task -1, the embedding row)
      src = p.x_a; src_task = 5 * (l - 1) + 4; normw = p.attn_norm + (size_t)l * p.H;
      break;
    case OP_O: src = p.o; src_task = 5 * l + 1; break;
    case OP_GATEUP: src = p.x_b; src_task = 5 * l + 2; normw = p.mlp_norm + (size_t)l * p.H; break;
    case OP_DOWN: src = p.m; src_task = 5 * l + 3; break;
    default: src = p.x_a; src_task = 5 * (p.L - 1) + 4; normw = p.final_norm; break;
  }
  const int np = n_passes(sl.rows);

  // Epilogue operands (residual element, int8 row scales) of a pass: requested before the pass -- those of the
  // first pass before the dependency wait -- and first looked at after it, so their latency is hidden.
  uint2 rraw = make_uint2(0u, 0u);                       // residual {value, seq}
  const ActPair* raddr = nullptr;
  int rtask = -1;
  __half sh0 = __float2half(1.f), sh1 = __float2half(1.f);
  auto request_operands = [&](int ps) {
    const int R = pass_rows(sl.rows, ps);
    const int vrow0 = sl.row0 + ps * kPassRows;
    raddr = nullptr;
    if (c.tid < ((kind == OP_GATEUP) ? (R >> 1) : R)) {
      const int vrow = vrow0 + c.tid;
      if (kind == OP_O) {
        raddr = p.x_a + vrow;
        rtask = 5 * (l - 1) + 4;
      } else if (kind == OP_DOWN) {
        raddr = p.x_b + vrow;
        rtask = 5 * l + 2;
      }
      if (raddr) rraw = ld_pair(raddr);
      if (d.wdtype == W_INT8) {
        const __half* scales = reinterpret_cast<const __half*>(
            p.packed + (LMH ? p.lm_scale_off : p.scale_base + (size_t)l * p.scale_layer_stride + p.scale_kind_off[kind]));
        if (kind == OP_GATEUP) {
          sh0 = __ldg(scales + vrow0 + 2 * c.tid);
          sh1 = __ldg(scales + vrow0 + 2 * c.tid + 1);
        } else {
          sh0 = __ldg(scales + vrow);
        }
      }
    }
  };
  if (np > 0) request_operands(0);

  float rnorm = 1.0f;                                    // bf16 weights, normed input: 1/rms, applied to the outputs
  if (src_task >= 0 && !wait_phase(c, src_task)) return false;
  if (np > 0) {
    const unsigned in_seq = seq_of(p, src_task);
    const LoadResult lr = load_input_1pass<WD>(p, c.sh, c.xs, c.cta, K, src, in_seq, src_task, normw, task);
    rnorm = lr.rnorm;
    c.bad = lr.bad;
    if (c.bad) return false;
  }
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_LOADED);

  // ---- passes -------------------------------------------------------------------------------------------
  float best_val = -CUDART_INF_F;
  int best_idx = 0x7fffffff;
  const bool drop = dropped(p, task, c.cta);
  for (int ps = 0; ps < np; ps++) {
    const int R = pass_rows(sl.rows, ps);
    const int gw = (ps == np - 1) ? 1 : 0;             // which precomputed geometry: a full pass or the last one
    const PassGeom g = c.sh->geom[kind][gw];
    const int vrow0 = sl.row0 + ps * kPassRows;
    float* red = c.sh->red[ps & 1];

    const int n_out = (kind == OP_GATEUP) ? (R >> 1) : R;
    const bool outp = c.tid < n_out;
    if (ps > 0) request_operands(ps);

    consume_pass<WD>(c, g, kind, gw, K, red, task);
    if (c.tid == 0 && ps == np - 1) stamp(p, c.cta, task, AMK_TR_REDUCED);
    if (raddr) {
      const unsigned rseq = seq_of(p, rtask);
      if (rraw.y != rseq) {
        rraw = poll_pair_slow(p, raddr, rseq, rtask);
        if (rraw.y != rseq) c.bad = true;
      }
    }
    const float resid = __uint_as_float(rraw.x);
    float sc0 = __half2float(sh0) * rnorm, sc1 = __half2float(sh1) * rnorm;
    c.bad = cons_sync_or(c.bad);
    if (c.bad) return false;

    if (outp && !drop) {
      const int vrow = vrow0 + c.tid;
      if (kind == OP_GATEUP) {
        float gt = 0.f, up = 0.f;
        for (int k = 0; k < g.Wk; k++) {
          gt += red[k * R + 2 * c.tid];
          up += red[k * R + 2 * c.tid + 1];
        }
        gt *= sc0;
        up *= sc1;
        const float mv = silu_f(gt) * up;
        st_pair(p.m + (vrow0 >> 1) + c.tid, mv, my_seq);
      } else {
        float y = 0.f;
        for (int k = 0; k < g.Wk; k++) y += red[k * R + c.tid];
        y *= sc0;
        switch (kind) {
          case OP_QKV:
            st_pair(p.qkv + vrow, y, my_seq);
            if (single_pos(p)) {
              // Position 0: one cache position, softmax weight exactly 1, rotation by angle 0.  The attention
              // output of every q head of a kv group is the rounded v row, and the rows to append are the
              // rounded k and v themselves: the thread that owns the element does it all, and the layer has no
              // attention task (one all-to-all join less on the chain).
              const int qd = p.nq * p.hd, kvd = p.nkv * p.hd;
              const int hs = (p.hd == 128) ? 7 : 6;
              if (vrow >= qd) {
                const bool is_v = vrow >= qd + kvd;
                const int e = vrow - qd - (is_v ? kvd : 0);
                const int g = e >> hs, dd = e & (p.hd - 1);
                unsigned char* cache = is_v ? p.vcache : p.kcache;
                const size_t idx = ((size_t)l * p.nkv + g) * p.S * p.hd + dd;
                float stored;                              // the value the cache now holds
                if (p.kv_esz == 2) {
                  const unsigned short bits = f32_to_bf16_rne(y);
                  reinterpret_cast<unsigned short*>(cache)[idx] = bits;
                  stored = bf16_lo((unsigned)bits);
                } else {
                  const unsigned char code = f32_to_e4m3(y);
                  cache[idx] = code;
                  stored = e4m3_to_f32(code);
                }
                if (is_v) {
                  const unsigned oseq = seq_of(p, 5 * l + 1);
                  for (int h = g * p.n_rep; h < (g + 1) * p.n_rep; h++) st_pair(p.o + (size_t)h * p.hd + dd, stored, oseq);
                }
              }
            }
            break;
          case OP_O: st_pair(p.x_b + vrow, resid + y, my_seq); break;
          case OP_DOWN: {
            const float xn = resid + y;
            st_pair(p.x_a + vrow, xn, my_seq);
            if (p.flags & AMK_FLAG_DEBUG_HIDDEN) p.hidden[(size_t)(l + 1) * p.H + vrow] = xn;
            break;
          }
          default:
            if (p.logits) p.logits[vrow] = y;
            if (y > best_val) { best_val = y; best_idx = vrow; }     // rows ascend, so ties keep the lowest index
            break;
        }
      }
    }
  }
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_COMPUTED);

  if (LMH) {
    // block argmax, then the block that arrives last reduces all blocks' candidates
    if (c.warp < kOutWarps) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best_val, o);
        const int oi = __shfl_xor_sync(0xffffffffu, best_idx, o);
        if (ov > best_val || (ov == best_val && oi < best_idx)) { best_val = ov; best_idx = oi; }
      }
      if (c.lane == 0) { c.sh->cand_val[c.warp] = best_val; c.sh->cand_idx[c.warp] = best_idx; }
    }
    c.bad = cons_sync_or(c.bad);
    if (c.bad) return false;
    if (c.warp == 0) {
      float v = (c.lane < kOutWarps) ? c.sh->cand_val[c.lane] : -CUDART_INF_F;
      int ix = (c.lane < kOutWarps) ? c.sh->cand_idx[c.lane] : 0x7fffffff;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, v, o);
        const int oi = __shfl_xor_sync(0xffffffffu, ix, o);
        if (ov > v || (ov == v && oi < ix)) { v = ov; ix = oi; }
      }
      int last = 0;
      if (c.lane == 0) {
        p.cand_val[c.cta] = v;
        p.cand_idx[c.cta] = ix;
        __threadfence();
        last = (atomicAdd(p.lm_ctr, 1u) == (unsigned)(c.nblk - 1));
        __threadfence();
      }
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) {
        v = -CUDART_INF_F;
        ix = 0x7fffffff;
        for (int b = c.lane; b < c.nblk; b += 32) {
          const float ov = __ldcg(p.cand_val + b);
          const int oi = __ldcg(p.cand_idx + b);
          if (ov > v || (ov == v && oi < ix)) { v = ov; ix = oi; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, v, o);
          const int oi = __shfl_xor_sync(0xffffffffu, ix, o);
          if (ov > v || (ov == v && oi < ix)) { v = ov; ix = oi; }
        }
        if (c.lane == 0) {
          *p.next_ws = ix;
          if (p.next_token) *p.next_token = ix;
          *p.lm_ctr = 0u;                    // next used by the next launch
        }
      }
    }
    return true;
  }

  if (counter_joins(p)) {
    c.bad = cons_sync_or(c.bad);
    if (c.bad) return false;
    signal_phase(c, task);
  }
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_SIGNALLED);
  return true;
}

// ------------------------------------------------------------------------------------------------
// Attention task: RoPE on the group's q heads (and on k, with the KV append, in the chunk that holds the
// new position), online-softmax partial over this chunk of cache positions, then either the final
// output (one chunk) or a partial that the last-arriving chunk of the group combines.
// Scores are kept in the log2 domain: q is pre-scaled by log2(e) / sqrt(hd).
// ------------------------------------------------------------------------------------------------
// Attention scratch in the activation area.  Heads come in sets of four: one tensor-core B operand (8 columns)
// carries the bf16 high and low parts of four heads' vectors.
template <int HD>
struct AttnScratch {
  static constexpr int NKS = HD / 16;                  // k steps of a score product = m tiles of an output product
  int n_sets, nh;                                      // sets of four heads, heads padded to whole sets
  float* qs;                                           // [n_rep][HD] q after the rotation, scaled (fp32)
  uint2* qfrag;                                        // [n_sets][NKS][32 lanes] the same as B fragments {b0, b1}
  float* wp;                                           // [warps][nh][HD (+2)] every warp's partial outputs
  unsigned short* knew;                                // [HD] the new position's K row (bf16) ...
  unsigned short* vnew;                                // ... and V row
  float* S;                                            // [n_rep][Lc] scores, then softmax numerators
  __device__ __forceinline__ AttnScratch(unsigned char* xs, int n_rep) {
    n_sets = (n_rep + 3) >> 2;
    nh = 4 * n_sets;
    qs = reinterpret_cast<float*>(xs);
    qfrag = reinterpret_cast<uint2*>(qs + n_rep * HD);
    wp = reinterpret_cast<float*>(qfrag + n_sets * NKS * 32);
    knew = reinterpret_cast<unsigned short*>(wp + (size_t)kConsumerWarps * nh * (HD + 2));
    vnew = knew + HD;
    S = reinterpret_cast<float*>(vnew + HD);
  }
  // element d of head h goes to column n = 2 (h % 4) + part of set h / 4 (part 0: bf16(v), part 1: bf16(v - part 0)):
  // k step d / 16, inside it kk = d % 16 is held by the lane quad position (kk % 8) / 2 in register kk / 8,
  // half-word kk % 2; the lane is 4 n + quad position
  __device__ __forceinline__ void put_q(int h, int d, float v) const {
    const unsigned short hi = f32_to_bf16_rne(v);
    const unsigned short lo = f32_to_bf16_rne(v - __uint_as_float((unsigned)hi << 16));
    const int ks = d >> 4, kk = d & 15;
    unsigned short* base = reinterpret_cast<unsigned short*>(qfrag + ((h >> 2) * NKS + ks) * 32 + 8 * (h & 3) + ((kk & 7) >> 1)) +
                           (kk >> 3) * 2 + (kk & 1);
    base[0] = hi;                                      // column 2 (h % 4): lane 8 (h % 4) + quad position
    base[16] = lo;                                     // column 2 (h % 4) + 1: four lanes (= 16 half-words) further
  }
};

template <int HD>
__device__ __noinline__ unsigned attn_general(const KParams& p, SmemHeader* sh, unsigned char* xs,
                                              const unsigned char* ring, int cta, int l, int g, int ch, int Lc, int C,
                                              bool bad_in, int stage, unsigned parity);
template <int HD, bool FP8>
__device__ __noinline__ unsigned attn_general_scalar(const KParams& p, SmemHeader* sh, unsigned char* xs,
                                                     const unsigned char* ring, int cta, int l, int g, int ch, int Lc,
                                                     int C, bool bad_in, int stage, unsigned parity);

// (Not inlined and called with scalars only: its many accumulators would otherwise push the per-thread
// state of the task loop out of registers for the whole kernel.)
template <int HD>
__device__ __forceinline__ bool attn_task(const KParams& p, SmemHeader* sh, unsigned char* xs,
                                       const unsigned char* ring, int& stage, unsigned& parity, int cta, int l, int g,
                                       int ch, int Lc, int C, bool bad_in) {
  struct {
    const KParams& p;
    SmemHeader* sh;
    unsigned char* xs;
    int tid, warp, lane, cta;
    bool bad;
  } c{p, sh, xs, (int)threadIdx.x, (int)(threadIdx.x >> 5), (int)(threadIdx.x & 31), cta, bad_in};
  const int n_rep = p.n_rep, half = HD / 2;
  const int n_pos = p.pos + 1;
  const int j0 = ch * Lc, j1 = min(n_pos, j0 + Lc);
  const bool owns_new = (j1 == n_pos);
  const AttnScratch<HD> A(c.xs, n_rep);
  float* qs = A.qs;
  const float2* rope = p.rope + (size_t)p.pos * half;
  const float qscale = 1.4426950408889634f * rsqrtf((float)HD);
  const size_t kvrow = ((size_t)l * p.nkv + g) * p.S;
  const unsigned in_seq = seq_of(p, 5 * l), out_seq = seq_of(p, 5 * l + 1);
  const bool drop = dropped(p, 5 * l + 1, c.cta);

  // ---- gather q (all heads of the group) and, in the chunk that owns the new position, k and v ----------
  // items: [0, n_rep*half) = q pairs (head h, dims e and e + half); then k pairs; then v pairs.
  // Both elements and the rotation are requested before anything is checked, so one round trip serves all.
  unsigned short* knew = A.knew;
  unsigned short* vnew = A.vnew;
  const int n_items = (n_rep + (owns_new ? 2 : 0)) * half;
  // the B-fragment columns of the heads that pad the last set of four are zero
  for (int i = c.tid; i < (A.nh - n_rep) * 2 * A.NKS * 4; i += kConsumerThreads) {
    const int ql = i & 3, ks = (i >> 2) % A.NKS, col = 2 * (n_rep & 3) + (i >> 2) / A.NKS;      // col in [2 (n_rep % 4), 8)
    A.qfrag[((A.n_sets - 1) * A.NKS + ks) * 32 + col * 4 + ql] = make_uint2(0u, 0u);
  }
  // the new row's elements e and e + half: into the cache at its element type, and into shared memory as the bf16
  // pattern of the value the cache now holds (an e4m3 value is exactly a bf16 value)
  auto append2 = [&](unsigned char* cache, unsigned short* fresh, int e, float x0, float x1) {
    unsigned short b0, b1;
    const size_t at = (kvrow + p.pos) * HD;
    if (p.kv_esz == 2) {
      b0 = f32_to_bf16_rne(x0); b1 = f32_to_bf16_rne(x1);
      unsigned short* dst = reinterpret_cast<unsigned short*>(cache) + at;
      dst[e] = b0; dst[e + half] = b1;
    } else {
      const unsigned char c0 = f32_to_e4m3(x0), c1 = f32_to_e4m3(x1);
      cache[at + e] = c0; cache[at + e + half] = c1;
      b0 = f32_to_bf16_rne(e4m3_to_f32(c0)); b1 = f32_to_bf16_rne(e4m3_to_f32(c1));
    }
    fresh[e] = b0; fresh[e + half] = b1;
  };
  for (int i = c.tid; i < n_items; i += kConsumerThreads) {
    const int h = i / half, e = i - h * half;
    const ActPair* base = (h < n_rep) ? p.qkv + (size_t)(g * n_rep + h) * HD
                        : (h == n_rep) ? p.qkv + (size_t)p.nq * HD + (size_t)g * HD
                                       : p.qkv + (size_t)(p.nq + p.nkv) * HD + (size_t)g * HD;
    uint2 ra = ld_pair(base + e), rb = ld_pair(base + e + half);
    const float2 cs = __ldg(rope + e);
    if (ra.y != in_seq) { ra = poll_pair_slow(p, base + e, in_seq, 5 * l); if (ra.y != in_seq) c.bad = true; }
    if (rb.y != in_seq) { rb = poll_pair_slow(p, base + e + half, in_seq, 5 * l); if (rb.y != in_seq) c.bad = true; }
    const float a = __uint_as_float(ra.x), b = __uint_as_float(rb.x);
    if (h < n_rep) {
      const float q0 = (a * cs.x - b * cs.y) * qscale, q1 = (b * cs.x + a * cs.y) * qscale;
      qs[h * HD + e] = q0;
      qs[h * HD + e + half] = q1;
      A.put_q(h, e, q0);                               // and as bf16 high / low parts in tensor-core B-fragment order
      A.put_q(h, e + half, q1);
    } else if (h == n_rep) {
      append2(p.kcache, knew, e, a * cs.x - b * cs.y, b * cs.x + a * cs.y);
    } else {
      append2(p.vcache, vnew, e, a, b);
    }
  }
  c.bad = cons_sync_or(c.bad);           // q and the new cache row are in shared memory
  if (c.tid == 0) stamp(p, c.cta, 5 * l + 1, AMK_TR_LOADED);
  if (c.bad) return true;

  if (C == 1 && n_pos == 1) {
    // one position: its softmax weight is exactly 1, the output is the cached (rounded) v row
    if (!drop)
      for (int i = c.tid; i < n_rep * HD; i += kConsumerThreads) {
        const int h = i / HD, dd = i - h * HD;
        st_pair(p.o + (size_t)(g * n_rep + h) * HD + dd, bf16_lo((unsigned)vnew[dd]), out_seq);
      }
    return c.bad;
  }
  // tensor-core kernel when the accumulators of all sets of four heads fit the registers (every shape measured
  // here: up to 8 q heads per kv head at head_dim 64, 4 at 128); otherwise the scalar one
  // (an fp8 cache: the scalar kernel, which converts the 8-bit entries as it reads them)
  const unsigned r = (p.kv_esz == 1)
                         ? attn_general_scalar<HD, true>(p, sh, xs, ring, cta, l, g, ch, Lc, C, c.bad, stage, parity)
                     : (A.n_sets * A.NKS <= 8)
                         ? attn_general<HD>(p, sh, xs, ring, cta, l, g, ch, Lc, C, c.bad, stage, parity)
                         : attn_general_scalar<HD, false>(p, sh, xs, ring, cta, l, g, ch, Lc, C, c.bad, stage, parity);
  stage = (int)((r >> 1) & 0x7fu);
  parity = (r >> 8) & 1u;
  return (r & 1u) != 0u;
}

// End of a chunk's work, shared by both versions: `partial(h, d)` gives the chunk's unnormalised output (its warps'
// partial sums added in a fixed order).  One chunk: that is the final output.  Several chunks: the partial (max,
// sum, output) is published, and every chunk's block combines an equal share of the group's n_rep * HD outputs.
// The partials carry sequence numbers like every other activation, so the exchange needs no counter and no fence:
// gather what my share needs from all chunks (waiting for it), then combine from shared memory.
template <int HD, class F>
__device__ __forceinline__ unsigned finish_chunk(const KParams& p, SmemHeader* sh, float* scratch, const float* hmax,
                                                 const float* hsum, int cta, int l, int g, int ch, int C, bool bad,
                                                 unsigned ring_pos, F partial) {
  const int tid = threadIdx.x, n_rep = p.n_rep;
  const unsigned out_seq = seq_of(p, 5 * l + 1);
  const bool drop = dropped(p, 5 * l + 1, cta);
  for (int i = tid; i < n_rep * HD; i += kConsumerThreads) {
    const int h = i / HD, dd = i - h * HD;
    const float A = partial(h, dd);
    const int hq = g * n_rep + h;
    if (C == 1) {
      if (!drop) st_pair(p.o + (size_t)hq * HD + dd, A / hsum[h], out_seq);
    } else if (!drop) {
      ActPair* pt = p.part + ((size_t)hq * kMaxChunks + ch) * (HD + 2);
      st_pair(pt + 2 + dd, A, out_seq);
      if (dd == 0) { st_pair(pt, hmax[h], out_seq); st_pair(pt + 1, hsum[h], out_seq); }
    }
  }
  if (C == 1) return ring_pos;

  bad = cons_sync_or(bad);                           // the warps' partial sums are no longer needed
  const int E = n_rep * HD;
  const int e0 = (int)((long long)E * ch / C), e1 = (int)((long long)E * (ch + 1) / C);
  const int n_out = e1 - e0;
  float* G = scratch;                                // [n_out][C] outputs' partials, then [heads touched][C][2] = M, Z
  if (n_out > 0) {
    const int h_lo = e0 / HD, h_hi = (e1 - 1) / HD;
    const int n_a = n_out * C, n_mz = (h_hi - h_lo + 1) * C * 2;
    for (int i = tid; i < n_a + n_mz; i += kConsumerThreads) {
      const ActPair* src;
      if (i < n_a) {
        const int o = i / C, k = i - o * C, e = e0 + o;
        const int h = e / HD, dd = e - h * HD;
        src = p.part + ((size_t)(g * n_rep + h) * kMaxChunks + k) * (HD + 2) + 2 + dd;
      } else {
        const int r = i - n_a, hk = r >> 1, h = h_lo + hk / C, k = hk - (hk / C) * C;
        src = p.part + ((size_t)(g * n_rep + h) * kMaxChunks + k) * (HD + 2) + (r & 1);
      }
      G[i] = read_act(p, bad, src, out_seq, 5 * l + 1);
    }
  }
  bad = cons_sync_or(bad);
  if (bad) return 1u | ring_pos;
  if (tid == 0) stamp(p, cta, 5 * l + 1, AMK_TR_REDUCED);
  for (int o = tid; o < n_out; o += kConsumerThreads) {
    const int e = e0 + o, h = e / HD, dd = e - h * HD;
    const float* mz = G + n_out * C + (size_t)(h - e0 / HD) * C * 2;
    float M = -CUDART_INF_F;
    for (int k = 0; k < C; k++) M = fmaxf(M, mz[2 * k]);
    float Z = 0.f, A = 0.f;
    for (int k = 0; k < C; k++) {                      // fixed order: deterministic
      const float a = exp2f(mz[2 * k] - M);
      Z = fmaf(a, mz[2 * k + 1], Z);
      A = fmaf(a, G[o * C + k], A);
    }
    if (!drop) st_pair(p.o + (size_t)(g * n_rep + h) * HD + dd, A / Z, out_seq);
  }
  return (bad ? 1u : 0u) | ring_pos;
}

// The general case (more than one cache position), on the tensor cores.  Kept out of line so that the code every
// task runs at short contexts stays small; everything it needs is passed as scalars or recomputed.
// The chunk's cache rows [j0, min(j1, pos)) arrive through the weight ring: the producer streams the K rows,
// then the V rows, as ring tiles between the QKV and the O projection's weights (see `producer`), so the
// consumers never wait for a load from HBM.  Three phases, with the chunk's scores in shared memory:
//   1. scores = K q: a warp takes 16 cache rows at a time as the A operand (ldmatrix straight from the ring tile);
//      the B operand's eight columns are the bf16 high and low parts of four q vectors (AttnScratch::qfrag), so
//      the products are exact and the sums fp32;
//   2. softmax within the chunk: one warp per head takes the maximum, exponentiates in place and sums;
//   3. output = P V: a warp takes 16 positions at a time; A is the V tile transposed by ldmatrix (16 output
//      dimensions x 16 positions, for every 16 output dimensions in turn), B the softmax numerators of four heads as
//      bf16 high and low parts; every warp's accumulators go to shared memory and are added in warp order.
// The new position's row is not in the cache tiles: its score and its share of the output are added from the
// copies in shared memory.  The chunk's (max, sum, unnormalised output) is the final output for a single chunk,
// else a partial.  Returns bad | stage << 1 | parity << 8 (the ring position moves on by the tiles walked).
template <int HD>
__device__ __noinline__ unsigned attn_general(const KParams& p, SmemHeader* sh, unsigned char* xs,
                                              const unsigned char* ring, int cta, int l, int g, int ch, int Lc, int C,
                                              bool bad_in, int stage, unsigned parity) {
  struct {
    SmemHeader* sh;
    int tid, warp, lane, cta;
    bool bad;
  } c{sh, (int)threadIdx.x, (int)(threadIdx.x >> 5), (int)(threadIdx.x & 31), cta, bad_in};
  constexpr int NKS = HD / 16;
  constexpr int MAXT = 8;                // accumulator tiles a warp holds: sets of four heads x NKS
  const int n_rep = p.n_rep;
  const AttnScratch<HD> A(xs, n_rep);
  const int n_sets = A.n_sets, nh = A.nh;
  const int n_pos = p.pos + 1;
  const int j0 = ch * Lc, j1 = min(n_pos, j0 + Lc);
  const bool owns_new = (j1 == n_pos);
  const int rows = min(j1, p.pos) - j0;                // rows that come from the cache
  const int n = j1 - j0;                               // + the new row, held in shared memory
  const int rpt = p.stage_bytes / (HD * 2);            // cache rows per ring tile (a multiple of 16)
  const int n_t = (rows + rpt - 1) / rpt;              // ring tiles of K (and again of V)
  float* S = A.S;
  float* hmax = c.sh->red[0];                          // [n_rep] chunk maximum and sum per head
  float* hsum = c.sh->red[1];
  const int gq = c.lane >> 2, q = c.lane & 3;
  const int S_ = p.n_stages;

  // ---- 1. scores -----------------------------------------------------------------------------------------
  {
    uint2 bq[MAXT];                                    // q as B fragments: [set][k step]
#pragma unroll
    for (int i = 0; i < MAXT; i++) bq[i] = (i < n_sets * NKS) ? A.qfrag[i * 32 + c.lane] : make_uint2(0u, 0u);
    // ldmatrix: my row of the 16-row tile and my half of the 16 k of a step
    const unsigned a_off = (unsigned)(((c.lane & 7) + ((c.lane >> 3) & 1) * 8) * (HD * 2) + (c.lane >> 4) * 16);
    for (int k = 0; k < n_t; k++) {
      if (!c.bad && !wait_mbar(p, &c.sh->full[stage], parity, -1)) c.bad = true;
      c.bad = __any_sync(0xffffffffu, c.bad) != 0;
      if (!c.bad) {
        const unsigned char* tile = ring + (size_t)stage * p.stage_bytes;
        const int r_t = min(rpt, rows - k * rpt);
        for (int r0 = c.warp * 16; r0 < r_t; r0 += kConsumerWarps * 16) {
          const unsigned char* rowp = tile + (size_t)r0 * (HD * 2) + a_off;
#pragma unroll
          for (int set = 0; set < MAXT / NKS; set++) {
            if (set < n_sets) {
              float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int ks = 0; ks < NKS; ks++) {
                unsigned a[4];
                ldmatrix_x4(a, rowp + ks * 32);
                mma_bf16(acc, a, bq[set * NKS + ks].x, bq[set * NKS + ks].y);
              }
              // columns 2 q, 2 q + 1 = high and low part of head 4 set + q; rows gq and gq + 8 of the tile
              const int h = 4 * set + q;
              if (h < n_rep) {
                float* sr = S + h * Lc + k * rpt + r0;
                if (r0 + gq < r_t) sr[gq] = acc[0] + acc[1];
                if (r0 + gq + 8 < r_t) sr[gq + 8] = acc[2] + acc[3];
              }
            }
          }
        }
      }
      __syncwarp();
      if (c.lane == 0 && !c.bad) mbar_arrive(&c.sh->empty[stage]);
      if (++stage == S_) { stage = 0; parity ^= 1u; }
    }
    if (owns_new && !c.bad) {                           // the new row, from shared memory: a warp per head
      for (int h = c.warp; h < n_rep; h += kConsumerWarps) {
        float sdot = 0.f;
        for (int d = c.lane; d < HD; d += 32) sdot = fmaf(A.qs[h * HD + d], bf16_lo((unsigned)A.knew[d]), sdot);
        sdot = warp_sum(sdot);
        if (c.lane == 0) S[h * Lc + n - 1] = sdot;
      }
    }
  }
  c.bad = cons_sync_or(c.bad);
  if (c.tid == 0) stamp(p, cta, 5 * l + 1, AMK_TR_PASS_BEGIN);

  // ---- 2. softmax numerators within the chunk (log2 domain) -----------------------------------------------
  for (int h = c.warp; h < n_rep && !c.bad; h += kConsumerWarps) {
    float* sr = S + h * Lc;
    float mx = -CUDART_INF_F;
    for (int t = c.lane; t < n; t += 32) mx = fmaxf(mx, sr[t]);
    mx = warp_max(mx);
    float z = 0.f;
    for (int t = c.lane; t < n; t += 32) {
      const float pw = exp2f(sr[t] - mx);
      sr[t] = pw;
      z += pw;
    }
    z = warp_sum(z);
    if (c.lane == 0) { hmax[h] = mx; hsum[h] = z; }
  }
  c.bad = cons_sync_or(c.bad);
  if (c.tid == 0) stamp(p, cta, 5 * l + 1, AMK_TR_FIRST_TILE);

  // ---- 3. P V ---------------------------------------------------------------------------------------------
  {
    float acc[MAXT][4];                                // [set][16 output dimensions]: rows gq, gq + 8; columns 2 q, 2 q + 1
#pragma unroll
    for (int i = 0; i < MAXT; i++)
#pragma unroll
      for (int e = 0; e < 4; e++) acc[i][e] = 0.f;
    // ldmatrix (transposing): matrix lane / 8 of the four is (positions +0 / +8) x (dimensions +0 / +8)
    const unsigned v_off = (unsigned)(((c.lane & 7) + ((c.lane >> 4) & 1) * 8) * (HD * 2) + ((c.lane >> 3) & 1) * 16);
    for (int k = 0; k < n_t; k++) {
      if (!c.bad && !wait_mbar(p, &c.sh->full[stage], parity, -1)) c.bad = true;
      c.bad = __any_sync(0xffffffffu, c.bad) != 0;
      if (!c.bad) {
        const unsigned char* tile = ring + (size_t)stage * p.stage_bytes;
        const int r_t = min(rpt, rows - k * rpt);
        for (int r0 = c.warp * 16; r0 < r_t; r0 += kConsumerWarps * 16) {
          const int nv = r_t - r0;                     // positions of this step that exist (>= 16: all)
          // B: the numerators of my column's head at positions 2 q, 2 q + 1 (b0) and 8 + 2 q, 9 + 2 q (b1)
          unsigned b0[MAXT / NKS], b1[MAXT / NKS];
#pragma unroll
          for (int set = 0; set < MAXT / NKS; set++) {
            b0[set] = b1[set] = 0u;
            const int h = 4 * set + (gq >> 1);
            if (set < n_sets && h < n_rep) {
              const float* sr = S + h * Lc + k * rpt + r0 + 2 * q;
              const float p0 = (2 * q < nv) ? sr[0] : 0.f, p1 = (2 * q + 1 < nv) ? sr[1] : 0.f;
              const float p8 = (2 * q + 8 < nv) ? sr[8] : 0.f, p9 = (2 * q + 9 < nv) ? sr[9] : 0.f;
              const unsigned h0 = pack_bf16x2(p0, p1), h1 = pack_bf16x2(p8, p9);
              if (gq & 1) {                            // the low parts' column
                b0[set] = pack_bf16x2(p0 - bf16_lo(h0), p1 - bf16_hi(h0));
                b1[set] = pack_bf16x2(p8 - bf16_lo(h1), p9 - bf16_hi(h1));
              } else {
                b0[set] = h0;
                b1[set] = h1;
              }
            }
          }
          const unsigned char* vp = tile + (size_t)r0 * (HD * 2) + v_off;
#pragma unroll
          for (int mt = 0; mt < NKS; mt++) {
            unsigned a[4];
            ldmatrix_x4_trans(a, vp + mt * 32);
            if (nv < 16) {
              // rows past the tile's end hold whatever the stage held before: keep it out of the sums
              // (a0, a1: positions 2 q, 2 q + 1; a2, a3: 8 + 2 q, 9 + 2 q; low half-word = the even position)
              const unsigned m01 = (2 * q >= nv) ? 0u : ((2 * q + 1 >= nv) ? 0x0000ffffu : 0xffffffffu);
              const unsigned m23 = (2 * q + 8 >= nv) ? 0u : ((2 * q + 9 >= nv) ? 0x0000ffffu : 0xffffffffu);
              a[0] &= m01; a[1] &= m01; a[2] &= m23; a[3] &= m23;
            }
#pragma unroll
            for (int set = 0; set < MAXT / NKS; set++)
              if (set < n_sets) mma_bf16(acc[set * NKS + mt], a, b0[set], b1[set]);
          }
        }
      }
      __syncwarp();
      if (c.lane == 0 && !c.bad) mbar_arrive(&c.sh->empty[stage]);
      if (++stage == S_) { stage = 0; parity ^= 1u; }
    }
    // every warp's partial outputs: dimension 16 mt + gq (and + 8), head 4 set + q = high + low column
#pragma unroll
    for (int set = 0; set < MAXT / NKS; set++) {
      const int h = 4 * set + q;
      if (set < n_sets && h < n_rep) {
        float* w = A.wp + ((size_t)c.warp * nh + h) * HD;
#pragma unroll
        for (int mt = 0; mt < NKS; mt++) {
          w[mt * 16 + gq] = acc[set * NKS + mt][0] + acc[set * NKS + mt][1];
          w[mt * 16 + gq + 8] = acc[set * NKS + mt][2] + acc[set * NKS + mt][3];
        }
      }
    }
  }
  c.bad = cons_sync_or(c.bad);
  const unsigned ring_pos = ((unsigned)stage << 1) | (parity << 8);
  if (c.bad) return 1u | ring_pos;
  if (c.tid == 0) stamp(p, cta, 5 * l + 1, AMK_TR_TILES_DONE);

  // the warps' partial outputs in warp order, plus the new position's share
  const float* wp = A.wp;
  const unsigned short* vnew = A.vnew;
  return finish_chunk<HD>(p, sh, A.wp, hmax, hsum, cta, l, g, ch, C, c.bad, ring_pos, [&](int h, int dd) {
    float o = 0.f;
    for (int w = 0; w < kConsumerWarps; w++) o += wp[((size_t)w * nh + h) * HD + dd];
    if (owns_new) o = fmaf(S[h * Lc + n - 1], bf16_lo((unsigned)vnew[dd]), o);
    return o;
  });
}

// Scalar version of the general case, for head configurations the tensor-core version does not cover.
// The chunk's cache rows [j0, min(j1, pos)) arrive through the weight ring: the producer streams the K rows,
// then the V rows, as ring tiles between the QKV and the O projection's weights (see `producer`), so the
// consumers never wait for a load from HBM.  Three phases, with the chunk's scores in shared memory:
//   1. scores: the lanes of a group hold 8 dims each of a K row and of four q vectors; dot products are
//      completed by shuffles;
//   2. softmax within the chunk: one warp per head takes the maximum, exponentiates in place and sums;
//   3. P V: lanes cover the 16-byte pieces of a V row, lane groups and warps cover row slices; the slices
//      are summed by shuffles, then across warps through shared memory.
// The chunk's (max, sum, unnormalised output) is the final output for a single chunk, else a partial.
// Returns bad | stage << 1 | parity << 8 (the ring position moves on by the tiles walked).
template <int HD, bool FP8>
__device__ __noinline__ unsigned attn_general_scalar(const KParams& p, SmemHeader* sh, unsigned char* xs,
                                                     const unsigned char* ring, int cta, int l, int g, int ch, int Lc,
                                                     int C, bool bad_in, int stage, unsigned parity) {
  struct {
    SmemHeader* sh;
    int tid, warp, lane, cta;
    bool bad;
  } c{sh, (int)threadIdx.x, (int)(threadIdx.x >> 5), (int)(threadIdx.x & 31), cta, bad_in};
  constexpr int NC = HD / 8;            // 16-byte pieces per cache row = lanes per row
  constexpr int RPW = 32 / NC;          // rows a warp handles at a time
  const int n_rep = p.n_rep;
  const int n_pos = p.pos + 1;
  const int j0 = ch * Lc, j1 = min(n_pos, j0 + Lc);
  const bool owns_new = (j1 == n_pos);
  const int rows = min(j1, p.pos) - j0;                // rows that come from the cache
  const int n = j1 - j0;                               // + the new row, held in shared memory
  constexpr int RB = HD * (FP8 ? 1 : 2);               // bytes of a cache row
  const int rpt = p.stage_bytes / RB;                  // cache rows per ring tile
  const int n_t = (rows + rpt - 1) / rpt;              // ring tiles of K (and again of V)
  const AttnScratch<HD> AS(xs, n_rep);
  float* qs = AS.qs;                                   // [n_rep][HD]
  float* wp = AS.wp;                                   // used here as [warps][4][HD + 2]
  unsigned short* knew = AS.knew;
  unsigned short* vnew = AS.vnew;
  float* S = AS.S;                                     // [n_rep][Lc] scores, then softmax numerators
  float* hmax = c.sh->red[0];                          // [n_rep] chunk maximum and sum per head
  float* hsum = c.sh->red[1];
  const int n_hb = (n_rep + 3) >> 2;     // blocks of four q heads
  const int wph = kConsumerWarps / n_hb; // warps per head block
  const int hb = c.warp / wph, wi = c.warp - hb * wph;
  const bool busy = hb < n_hb;
  const int dl = c.lane % NC, sub = c.lane / NC;
  const int S_ = p.n_stages;

  // ---- 1. scores -----------------------------------------------------------------------------------------
  {
    float q[4][8];                       // my 8 dims of my block's four q vectors
#pragma unroll
    for (int hh = 0; hh < 4; hh++) {
      const int h = min(hb * 4 + hh, n_rep - 1);
#pragma unroll
      for (int e = 0; e < 8; e++) q[hh][e] = busy ? qs[h * HD + dl * 8 + e] : 0.f;
    }
    auto score_row = [&](const float (&kf)[8], int t) {
#pragma unroll
      for (int hh = 0; hh < 4; hh++) {
        float s = kf[0] * q[hh][0];
#pragma unroll
        for (int e = 1; e < 8; e++) s = fmaf(kf[e], q[hh][e], s);
#pragma unroll
        for (int o = NC / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (dl == 0 && hb * 4 + hh < n_rep && t >= 0) S[(hb * 4 + hh) * Lc + t] = s;
      }
    };
    for (int k = 0; k < n_t; k++) {
      if (!c.bad && !wait_mbar(p, &c.sh->full[stage], parity, -1)) c.bad = true;
      c.bad = __any_sync(0xffffffffu, c.bad) != 0;                         // (shuffles below: the warp stays together)
      if (busy && !c.bad) {
        const unsigned char* tile = ring + (size_t)stage * p.stage_bytes;
        const int r_t = min(rpt, rows - k * rpt);
        for (int r0 = wi * RPW; r0 < r_t; r0 += wph * RPW) {            // (warp-uniform bounds: shuffles inside)
          const int r = r0 + sub;
          float kf[8];
          cache8<FP8>(tile + (size_t)min(r, r_t - 1) * RB + dl * (RB / NC), kf);
          score_row(kf, r < r_t ? k * rpt + r : -1);
        }
      }
      __syncwarp();
      if (c.lane == 0 && !c.bad) mbar_arrive(&c.sh->empty[stage]);
      if (++stage == S_) { stage = 0; parity ^= 1u; }
    }
    if (owns_new && busy && wi == 0 && !c.bad) {                          // the new row, from shared memory
      float kf[8];
      cache8<false>(reinterpret_cast<const unsigned char*>(knew) + dl * 16, kf);
      score_row(kf, sub == 0 ? n - 1 : -1);
    }
  }
  c.bad = cons_sync_or(c.bad);
  if (c.tid == 0) stamp(p, cta, 5 * l + 1, AMK_TR_PASS_BEGIN);

  // ---- 2. softmax numerators within the chunk (log2 domain) -----------------------------------------------
  for (int h = c.warp; h < n_rep && !c.bad; h += kConsumerWarps) {
    float* sr = S + h * Lc;
    float mx = -CUDART_INF_F;
    for (int t = c.lane; t < n; t += 32) mx = fmaxf(mx, sr[t]);
    mx = warp_max(mx);
    float z = 0.f;
    for (int t = c.lane; t < n; t += 32) {
      const float pw = exp2f(sr[t] - mx);
      sr[t] = pw;
      z += pw;
    }
    z = warp_sum(z);
    if (c.lane == 0) { hmax[h] = mx; hsum[h] = z; }
  }
  c.bad = cons_sync_or(c.bad);
  if (c.tid == 0) stamp(p, cta, 5 * l + 1, AMK_TR_FIRST_TILE);

  // ---- 3. P V ---------------------------------------------------------------------------------------------
  {
    float acc[4][8];
#pragma unroll
    for (int hh = 0; hh < 4; hh++)
#pragma unroll
      for (int e = 0; e < 8; e++) acc[hh][e] = 0.f;
    auto add_row = [&](const float (&vf)[8], int t) {
#pragma unroll
      for (int hh = 0; hh < 4; hh++) {
        const float pw = S[min(hb * 4 + hh, n_rep - 1) * Lc + t];
#pragma unroll
        for (int e = 0; e < 8; e++) acc[hh][e] = fmaf(pw, vf[e], acc[hh][e]);
      }
    };
    for (int k = 0; k < n_t; k++) {
      if (!c.bad && !wait_mbar(p, &c.sh->full[stage], parity, -1)) c.bad = true;
      c.bad = __any_sync(0xffffffffu, c.bad) != 0;                         // (shuffles below: the warp stays together)
      if (busy && !c.bad) {
        const unsigned char* tile = ring + (size_t)stage * p.stage_bytes;
        const int r_t = min(rpt, rows - k * rpt);
        for (int r = wi * RPW + sub; r < r_t; r += wph * RPW) {
          float vf[8];
          cache8<FP8>(tile + (size_t)r * RB + dl * (RB / NC), vf);
          add_row(vf, k * rpt + r);
        }
      }
      __syncwarp();
      if (c.lane == 0 && !c.bad) mbar_arrive(&c.sh->empty[stage]);
      if (++stage == S_) { stage = 0; parity ^= 1u; }
    }
    if (owns_new && busy && wi == 0 && sub == 0 && !c.bad) {
      float vf[8];
      cache8<false>(reinterpret_cast<const unsigned char*>(vnew) + dl * 16, vf);
      add_row(vf, n - 1);
    }
    // sum the lane groups of the warp, then leave the warp's partial in shared memory
#pragma unroll
    for (int o = NC; o < 32; o <<= 1)
#pragma unroll
      for (int hh = 0; hh < 4; hh++)
#pragma unroll
        for (int e = 0; e < 8; e++) acc[hh][e] += __shfl_xor_sync(0xffffffffu, acc[hh][e], o);
    if (sub == 0 && busy) {
#pragma unroll
      for (int hh = 0; hh < 4; hh++)
#pragma unroll
        for (int e = 0; e < 8; e++) wp[(size_t)(c.warp * 4 + hh) * (HD + 2) + 2 + dl * 8 + e] = acc[hh][e];
    }
  }
  c.bad = cons_sync_or(c.bad);
  const unsigned ring_pos = ((unsigned)stage << 1) | (parity << 8);
  if (c.bad) return 1u | ring_pos;
  if (c.tid == 0) stamp(p, cta, 5 * l + 1, AMK_TR_TILES_DONE);

  // sum the warps of each head block, in warp order
  return finish_chunk<HD>(p, sh, wp, hmax, hsum, cta, l, g, ch, C, c.bad, ring_pos, [&](int h, int dd) {
    const int hbb = h >> 2, hh = h & 3;
    float A = 0.f;
    for (int w = 0; w < wph; w++) A += wp[(size_t)((hbb * wph + w) * 4 + hh) * (HD + 2) + 2 + dd];
    return A;
  });
}

template <int HD>
__device__ __forceinline__ bool attention_phase(Ctx& c, int l) {
  const KParams& p = c.p;
  if (single_pos(p)) return true;                         // (the QKV projection has done it all)
  // (the chunk plan is the same for every layer: worked out once, at kernel start; no divisions here)
  const int Lc = c.sh->attn_lc, C = c.sh->attn_c;
  const int n_tasks = p.nkv * C;
  const int rot = (l * 29) % c.nblk;
  int t = c.cta + c.nblk - rot;
  if (t >= c.nblk) t -= c.nblk;
  const int task = 5 * l + 1;
  if (!counter_joins(p) && t >= n_tasks) return true;     // nothing to do here and nobody to tell
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_ENTER);
  if (!wait_phase(c, 5 * l + 0)) return false;
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_JOINED);
  if (t < n_tasks) {
    const int g = t / C, ch = t - g * C;
    c.bad = attn_task<HD>(p, c.sh, c.xs, c.ring, c.stage, c.parity, c.cta, l, g, ch, Lc, C, c.bad);
  }
  c.bad = cons_sync_or(c.bad);
  if (c.bad) return false;
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_COMPUTED);
  signal_phase(c, task);
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_SIGNALLED);
  return true;
}

// The last task of the step: final norm, LM head, greedy token.  Out of line and with its own context: the
// per-layer loop above it keeps its registers for the code that runs 4 L times.
template <int WD>
__device__ __noinline__ void lm_head_task(const KParams& p, SmemHeader* sh, unsigned char* xs, unsigned char* ring,
                                          int cta, int nblk, int stage, unsigned parity, int token) {
  const int tid = threadIdx.x;
  Ctx c{p, sh, xs, ring, tid, tid >> 5, tid & 31, cta, nblk, stage, parity, token, false};
  gemv_op<WD, true>(c, (int)OP_LMHEAD, p.L);
}

// ------------------------------------------------------------------------------------------------
// Producer: streams this block's weight tiles, in order, into the ring.  The tile list {offset, bytes,
// task} was laid out by the host, so the producer only waits for a free stage and issues the copy.
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ void producer(const KParams& p, SmemHeader* sh, unsigned char* ring, int cta, int lane) {
  const uint64_t pol = policy_evict_first();
  const unsigned S = (unsigned)p.n_stages;
  const unsigned inflight = (unsigned)p.max_inflight;
  const unsigned ahead = (unsigned)p.l2_ahead;      // tiles kept requested into L2 beyond the ring (<= 32)
  const unsigned begin = __ldg(p.tile_begin + cta), end = __ldg(p.tile_begin + cta + 1);
  unsigned t = 0;                                   // tiles issued so far
  unsigned stage = 0, lap = 0;
#if AMK_TRACE_BUILD
  int cur_task = -1;
#endif
  int ok = 1;
  // the warp holds 64 consecutive table entries: [base, base + 32) in e_cur, [base + 32, base + 64) in e_next
  unsigned long long e_cur = (begin + lane < end) ? __ldg(p.tiles + begin + lane) : 0ull;
  unsigned long long e_next = (begin + 32 + lane < end) ? __ldg(p.tiles + begin + 32 + lane) : 0ull;
  // the first `ahead` tiles are requested right away
  for (unsigned j = 0; j < ahead && begin + j < end; j++) {
    const unsigned long long e = __shfl_sync(0xffffffffu, e_cur, (int)j);
    if (lane == 0 && ((e >> 40) & 0x1fffu))
      bulk_prefetch_l2(p.packed + ((e & ((1ull << 40) - 1)) << 4), (unsigned)((e >> 40) & 0x1fffu) << 4);
  }
  for (unsigned base = begin; base < end && ok; base += 32) {
    const int n = (int)min(32u, end - base);
    for (int j = 0; j < n; j++) {
      const unsigned long long e = __shfl_sync(0xffffffffu, e_cur, j);
      // the tile `ahead` places further on: request it into L2 now
      const int ja = j + (int)ahead;
      const unsigned long long ea = __shfl_sync(0xffffffffu, ja < 32 ? e_cur : e_next, ja & 31);
      if (lane == 0) {
        if (ahead && base + (unsigned)ja < end && ((ea >> 40) & 0x1fffu))
          bulk_prefetch_l2(p.packed + ((ea & ((1ull << 40) - 1)) << 4), (unsigned)((ea >> 40) & 0x1fffu) << 4);
        const unsigned long long off = (e & ((1ull << 40) - 1)) << 4;
        const unsigned bytes = (unsigned)((e >> 40) & 0x1fffu) << 4;
        const int task = (int)(e >> 53);
        // one ring tile: wait for a free stage (and for an older copy to have landed), then issue the copy
        auto issue = [&](const unsigned char* src, unsigned nbytes) {
          if (lap > 0 && !wait_mbar(p, &sh->empty[stage], (lap - 1) & 1u, -2)) ok = 0;
          if (ok && inflight < S && t >= inflight) {
            const unsigned tl = t - inflight;          // this older tile must have landed
            if (!wait_mbar(p, &sh->full[tl % S], (tl / S) & 1u, -2)) ok = 0;
          }
          if (ok) {
            mbar_expect_tx(&sh->full[stage], nbytes);
            bulk_g2s(ring + (size_t)stage * p.stage_bytes, src, nbytes, &sh->full[stage], pol);
#if AMK_TRACE_BUILD
            if (p.trace) {
              if (task != cur_task) { stamp(p, cta, task, AMK_TR_PROD_FIRST); cur_task = task; }
              stamp(p, cta, task, AMK_TR_PROD_LAST);
            }
#endif
            t++;
            if (++stage == S) { stage = 0; lap++; }
          }
        };
        if (bytes) {
          issue(p.packed + off, bytes);
        } else if (p.pos > 0) {
          // Marker of an attention task: stream the cache rows of this block's chunk, K then V, cut into ring
          // tiles -- the same rows, in the same tiles, that attn_general walks.  (Rows of earlier positions
          // only: they were written by earlier launches.  The new row stays in the consumers' shared memory.)
          const int l = task / 5, nblk = (int)gridDim.x;
          int Lc, C;
          attn_chunks(p.pos + 1, nblk, p.nkv, &Lc, &C);
          const int tt = (cta + nblk - (l * 29) % nblk) % nblk;
          if (tt < p.nkv * C) {
            const int g = tt / C, ch = tt - g * C;
            const int j0 = ch * Lc, rows = min(p.pos, j0 + Lc) - j0;
            const int rb = p.hd * p.kv_esz;                                         // bytes of a cache row
            const int rpt = p.stage_bytes / rb;
            const size_t first = (((size_t)l * p.nkv + g) * p.S + j0) * rb;        // in bytes
            for (int which = 0; which < 2 && ok; which++) {
              const unsigned char* cache = which ? p.vcache : p.kcache;
              for (int r0 = 0; r0 < rows && ok; r0 += rpt)
                issue(cache + first + (size_t)r0 * rb, (unsigned)(min(rpt, rows - r0) * rb));
            }
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
    }
    e_cur = e_next;
    e_next = (base + 64 + lane < end) ? __ldg(p.tiles + base + 64 + lane) : 0ull;
  }
  if (!ok && lane == 0) {
    // leaving early: every copy already issued must land before the block's shared memory is released
    const unsigned first = (t > S) ? t - S : 0u;
    for (unsigned i = first; i < t; i++) {
      uint64_t* bar = &sh->full[i % S];
      const unsigned par = (i / S) & 1u;
      for (unsigned spins = 0; spins < (1u << 24) && !mbar_try_wait(bar, par); spins++) {}
    }
  }
}

}  // namespace

// One instantiation per (layer weight dtype, head dimension): only the code a model needs is resident,
// which matters because every task runs its code once and instruction-cache misses cost like L2 misses.
template <int WDL, int HD>
__global__ void __launch_bounds__(kThreads, 1) AMK_KERNEL(const __grid_constant__ KParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  SmemHeader* sh = reinterpret_cast<SmemHeader*>(smem);
  const size_t hdr = (sizeof(SmemHeader) + 127) & ~(size_t)127;
  unsigned char* xs = smem + hdr;
  unsigned char* ring = smem + hdr + p.act_bytes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nblk = gridDim.x;

  if (tid == 0) {
    p.ktime[2 * blockIdx.x] = globaltimer_ns();
    for (int s = 0; s < p.n_stages; s++) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], kConsumerWarps);
    }
    sh->flag = 0;
    // Which share of the work is this block's?  With one block per SM the SM id names the block, and the
    // host's table gives the slot whose share matches what that SM was measured to stream.
    int slot = blockIdx.x;
    if (p.slot_of_smid) {
      unsigned sm;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
      slot = (sm < (unsigned)kMaxSmid) ? __ldg(p.slot_of_smid + sm) : -1;
      if (slot < 0 || slot >= nblk) {
        report_failure(p, (unsigned)AMK_ERR_ABORTED, -3, sm, 0u);     // an SM the plan has not seen
        slot = -1;
      }
    }
    sh->slot = slot;
    if (slot >= 0) {
      for (int k = 0; k < 5; k++) {
        const int* b = p.bounds + k * (nblk + 1);
        sh->slice_row0[k] = __ldg(b + slot) * p.shape[k].unit_rows;
        sh->slice_rows[k] = (__ldg(b + slot + 1) - __ldg(b + slot)) * p.shape[k].unit_rows;
      }
    }
    mbar_fence_init();
  }
  __syncthreads();
  const int cta = sh->slot;
  if (cta < 0) return;
  if (tid == 32) {
    int lc, cc;
    attn_chunks(p.pos + 1, nblk, p.nkv, &lc, &cc);
    sh->attn_lc = lc;
    sh->attn_c = cc;
  }
  if (tid < 10) {
    const int k = tid >> 1, which = tid & 1;
    const int rows = sh->slice_rows[k];
    const int np = n_passes(rows);
    const int R = which ? (np ? pass_rows(rows, np - 1) : 1) : kPassRows;
    const PassGeom g = pass_geom(R, p.shape[k].K, p.shape[k].wdtype, p.stage_bytes);
    sh->geom[k][which] = g;
    sh->step_b[k][which] = g.upt / g.Wr;
    sh->step_r[k][which] = g.upt % g.Wr;
    for (int w = 0; w < kConsumerWarps; w++) {
      sh->wr_of[k][which][w] = (unsigned char)(w % g.Wr);
      sh->wk_of[k][which][w] = (unsigned char)(w / g.Wr);
    }
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    producer(p, sh, ring, cta, lane);
    return;
  }

  int token = p.token_ptr ? __ldcg(p.token_ptr) : p.token;
  token = min(max(token, 0), p.V - 1);
  // Task -1: the embedding row enters the residual stream like every other activation -- every block publishes its
  // share of the row as {value, sequence number} elements, and layer 0 reads it the way layer l reads layer l - 1.
  {
    for (int e = cta * kConsumerThreads + tid; e < p.H; e += nblk * kConsumerThreads) {
      const float v = __uint_as_float((unsigned)__ldg(p.embed + (size_t)token * p.H + e) << 16);
      st_pair(p.x_a + e, v, seq_of(p, -1));
      if (p.flags & AMK_FLAG_DEBUG_HIDDEN) p.hidden[e] = v;
    }
  }
  Ctx c{p, sh, xs, ring, tid, warp, lane, cta, nblk, 0, 0u, token, false};
  // the block's queue: tasks 5 l + {0..4} = QKV, attention, O, gate/up, down of layer l, then the LM head
  // (one call site each, so that the per-thread state stays in registers)
  const int n_layer_tasks = 5 * p.L;
  bool ok = true;
  for (int task = 0; task < n_layer_tasks && ok; task++) {
    const int l = task / 5, k = task - 5 * l;
    if (k == 1) ok = attention_phase<HD>(c, l);
    else ok = gemv_op<WDL, false>(c, k == 0 ? (int)OP_QKV : k - 1, l);
  }
  if (ok) {
    // the LM head is bf16 unless the configuration quantises it like the layers
    if (WDL == W_BF16 || p.shape[OP_LMHEAD].wdtype == W_BF16) lm_head_task<W_BF16>(p, sh, xs, ring, cta, nblk, c.stage, c.parity, token);
    else lm_head_task<WDL>(p, sh, xs, ring, cta, nblk, c.stage, c.parity, token);
  }
  // (every consumer warp stamps; the latest store of the latest block is the kernel's end)
  if (lane == 0) atomicMax(p.ktime + 2 * blockIdx.x + 1, globaltimer_ns());
}

#if !AMK_TRACE_BUILD
// Calibration: every block (one per SM, same shared-memory footprint as the decode kernel) streams
// `bytes_per_block` through a small ring of bulk copies while all the others do the same, and reports its
// SM id and the time it took.  SMs do not all get the same share of the HBM stream; the host can split the
// rows of every op in proportion to these rates.
__global__ void __launch_bounds__(kThreads, 1)
amk_calibrate_kernel(const unsigned char* __restrict__ src, size_t bytes_per_block, unsigned* smid_out,
                     unsigned long long* ns_out) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int S = 4, TILE = 32768;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = full + S;
  unsigned char* ring = smem + 128;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; s++) { mbar_init(full + s, 1); mbar_init(empty + s, kConsumerWarps); }
    mbar_fence_init();
  }
  __syncthreads();
  const unsigned char* base = src + (size_t)blockIdx.x * bytes_per_block;
  const int n_tiles = (int)(bytes_per_block / TILE);
  const unsigned long long t0 = globaltimer_ns();
  const unsigned kSpinLimit = 1u << 26;
  if (warp == kConsumerWarps) {
    if (lane == 0) {
      const uint64_t pol = policy_evict_first();
      for (int t = 0; t < n_tiles; t++) {
        const int s = t % S;
        if (t >= S) {
          unsigned spins = 0;
          while (!mbar_try_wait(empty + s, ((t / S) - 1) & 1u)) if (++spins > kSpinLimit) return;
        }
        mbar_expect_tx(full + s, TILE);
        bulk_g2s(ring + (size_t)s * TILE, base + (size_t)t * TILE, TILE, full + s, pol);
      }
    }
  } else {
    for (int t = 0; t < n_tiles; t++) {
      const int s = t % S;
      unsigned spins = 0;
      bool ok = true;
      while (!mbar_try_wait(full + s, (t / S) & 1u)) if (++spins > kSpinLimit) { ok = false; break; }
      if (!ok) break;
      __syncwarp();
      if (lane == 0) mbar_arrive(empty + s);
    }
    if (threadIdx.x == 0) {
      unsigned sm;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
      smid_out[blockIdx.x] = sm;
      ns_out[blockIdx.x] = globaltimer_ns() - t0;
    }
  }
}

cudaError_t launch_calibrate(const unsigned char* src, size_t bytes_per_block, int n_blocks, size_t smem_bytes,
                             unsigned* smid_out, unsigned long long* ns_out, cudaStream_t stream) {
  const size_t need = 128 + 4 * 32768;
  if (smem_bytes < need) smem_bytes = need;
  cudaError_t e = cudaFuncSetAttribute(amk_calibrate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  amk_calibrate_kernel<<<n_blocks, kThreads, smem_bytes, stream>>>(src, bytes_per_block, smid_out, ns_out);
  return cudaGetLastError();
}

#endif  // !AMK_TRACE_BUILD

typedef void (*DecodeKernel)(const KParams);
static DecodeKernel pick_kernel(int wdtype, int hd) {
  if (hd == 64) {
    if (wdtype == W_BF16) return AMK_KERNEL<W_BF16, 64>;
    if (wdtype == W_INT8) return AMK_KERNEL<W_INT8, 64>;
    if (wdtype == W_INT8G) return AMK_KERNEL<W_INT8G, 64>;
    return AMK_KERNEL<W_INT4, 64>;
  }
  if (wdtype == W_BF16) return AMK_KERNEL<W_BF16, 128>;
  if (wdtype == W_INT8) return AMK_KERNEL<W_INT8, 128>;
  if (wdtype == W_INT8G) return AMK_KERNEL<W_INT8G, 128>;
  return AMK_KERNEL<W_INT4, 128>;
}

cudaError_t AMK_ATTRS(int wdtype, int hd, size_t smem_bytes, int* max_blocks_per_sm) {
  DecodeKernel k = pick_kernel(wdtype, hd);
  // the device's limit, not this handle's need: a handle created later with a smaller plan must not lower the
  // attribute under a handle that is still in use
  int dev = 0, optin = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  if ((size_t)optin < smem_bytes) return cudaErrorInvalidValue;
  e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(max_blocks_per_sm, k, kThreads, smem_bytes);
}

cudaError_t AMK_LAUNCH(const KParams& p, int n_blocks, size_t smem_bytes, cudaStream_t stream) {
  void* args[] = {const_cast<KParams*>(&p)};
  return cudaLaunchCooperativeKernel((const void*)pick_kernel(p.shape[OP_QKV].wdtype, p.hd), dim3(n_blocks),
                                     dim3(kThreads), args, smem_bytes, stream);
}

}  // namespace amk
