// The decode step as one persistent cooperative kernel for sm_100a: one block per SM, each block walks
// its statically known queue of tasks -- wait on a dependency counter, compute, signal -- as in the
// paper's per-SM scheduler loop (Algorithm 1) and counter model (Section 4, "Synchronization model").
//
// What is different from the paper's kernel (written for sm_75..sm_120, where it found the per-tile
// cross-SM synchronisation to be the limiter, Section 7):
//   * Weights do not depend on activations, so a dedicated producer warp streams this block's packed
//     weight bytes -- one contiguous run per block for the whole token -- through a shared-memory ring
//     with bulk asynchronous copies (TMA) and mbarriers, running ahead across dependency joins.  The
//     HBM pipe keeps flowing while the consumer warps wait for an activation.
//   * One counter per join instead of one per tile: five joins per layer, every block signals each once.
//     Counters are never reset: step e waits for e * n_blocks.
//   * RMSNorm is folded into the consuming GEMV's prologue, RoPE and the KV append into the attention
//     task, SiLU*up and the residual adds into GEMV epilogues, the split-K combine and the global argmax
//     into "last arriver finishes" steps, so no extra joins are needed.
//   * Every wait is bounded; on expiry the block records the failure and every block drains and exits.
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <math_constants.h>

#include "amk.h"
#include "amk_internal.h"
#include "amk_ptx.cuh"

namespace amk {

namespace {

constexpr int kBarCons = 1;       // named barrier of the consumer warps
constexpr int kOutWarps = (kPassRows + 31) / 32;   // warps that hold a pass's output rows
constexpr int kNormVec = 4;       // float4 slots per thread held in registers by a norm prologue (H <= 8192)

struct Ctx {
  const KParams& p;
  SmemHeader* sh;
  float* xs;             // activation vector of the current op / attention scratch
  unsigned char* ring;
  int tid, warp, lane, cta, nblk;
  unsigned tile_ctr;     // ring tiles this warp has walked
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

// All consumer threads: wait until every block has signalled `phase` in this step.
__device__ __forceinline__ bool wait_phase(Ctx& c, int phase) {
  if (c.tid == 0) {
    if (!poll_counter(c.p, c.p.phase_ctr + phase, c.p.epoch * (unsigned)c.nblk, phase)) c.bad = true;
  }
  c.bad = cons_sync_or(c.bad);
  return !c.bad;
}
// Called after a consumer barrier that follows the task's last store: release-increment the counter.
__device__ __forceinline__ void signal_phase(Ctx& c, int phase) {
  if (c.tid == 0 && !(phase == c.p.drop_phase && c.cta == c.p.drop_block))
    red_release_gpu_add(c.p.phase_ctr + phase, 1u);
}

// One thread stamps the global timer for (task, event) of this block when tracing is on.
__device__ __forceinline__ void stamp(const KParams& p, int cta, int task, int ev) {
  if (p.trace) p.trace[((size_t)cta * (5 * p.L + 1) + task) * AMK_TRACE_EVENTS + ev] = globaltimer_ns();
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------------------------------------------
// dot product of one lane's 8 weights of one row chunk with its 8 activations
// ------------------------------------------------------------------------------------------------
template <int WD>
__device__ __forceinline__ float dot8(const unsigned char* row, int lane, const float4& x0, const float4& x1);

template <>
__device__ __forceinline__ float dot8<W_BF16>(const unsigned char* row, int lane, const float4& x0, const float4& x1) {
  const uint4 w = *reinterpret_cast<const uint4*>(row + lane * 16);
  float s0 = bf16_lo(w.x) * x0.x;
  float s1 = bf16_lo(w.z) * x1.x;
  s0 = fmaf(bf16_hi(w.x), x0.y, s0);
  s1 = fmaf(bf16_hi(w.z), x1.y, s1);
  s0 = fmaf(bf16_lo(w.y), x0.z, s0);
  s1 = fmaf(bf16_lo(w.w), x1.z, s1);
  s0 = fmaf(bf16_hi(w.y), x0.w, s0);
  s1 = fmaf(bf16_hi(w.w), x1.w, s1);
  return s0 + s1;
}

// int8 codes are stored biased (q + 128) so that one byte-permute builds the float 2^23 + (q + 128).
__device__ __forceinline__ float u8_to_f32_biased(unsigned w, unsigned sel) {
  return __uint_as_float(__byte_perm(w, 0x4B000000u, sel)) - 8388736.0f;   // 2^23 + 128
}
template <>
__device__ __forceinline__ float dot8<W_INT8>(const unsigned char* row, int lane, const float4& x0, const float4& x1) {
  const uint2 w = *reinterpret_cast<const uint2*>(row + lane * 8);
  float s0 = u8_to_f32_biased(w.x, 0x7540u) * x0.x;
  float s1 = u8_to_f32_biased(w.y, 0x7540u) * x1.x;
  s0 = fmaf(u8_to_f32_biased(w.x, 0x7541u), x0.y, s0);
  s1 = fmaf(u8_to_f32_biased(w.y, 0x7541u), x1.y, s1);
  s0 = fmaf(u8_to_f32_biased(w.x, 0x7542u), x0.z, s0);
  s1 = fmaf(u8_to_f32_biased(w.y, 0x7542u), x1.z, s1);
  s0 = fmaf(u8_to_f32_biased(w.x, 0x7543u), x0.w, s0);
  s1 = fmaf(u8_to_f32_biased(w.y, 0x7543u), x1.w, s1);
  return s0 + s1;
}

// int4: 8 codes in one word (element e in nibble e); the row chunk ends with fp16 {s, z} of group 2b and 2b+1.
__device__ __forceinline__ float u4_to_f32(unsigned w, int e, float zbias) {
  return __uint_as_float(((w >> (4 * e)) & 0xFu) | 0x4B000000u) - zbias;           // (2^23 + q) - (2^23 + z)
}
template <>
__device__ __forceinline__ float dot8<W_INT4>(const unsigned char* row, int lane, const float4& x0, const float4& x1) {
  const unsigned w = *reinterpret_cast<const unsigned*>(row + lane * 4);
  const uint2 sz = *reinterpret_cast<const uint2*>(row + 128);
  const float sA = __half2float(__ushort_as_half((unsigned short)(sz.x & 0xffffu)));
  const float zA = __half2float(__ushort_as_half((unsigned short)(sz.x >> 16))) + 8388608.0f;
  const float sB = __half2float(__ushort_as_half((unsigned short)(sz.y & 0xffffu)));
  const float zB = __half2float(__ushort_as_half((unsigned short)(sz.y >> 16))) + 8388608.0f;
  float s0 = u4_to_f32(w, 0, zA) * x0.x;
  float s1 = u4_to_f32(w, 4, zB) * x1.x;
  s0 = fmaf(u4_to_f32(w, 1, zA), x0.y, s0);
  s1 = fmaf(u4_to_f32(w, 5, zB), x1.y, s1);
  s0 = fmaf(u4_to_f32(w, 2, zA), x0.z, s0);
  s1 = fmaf(u4_to_f32(w, 6, zB), x1.z, s1);
  s0 = fmaf(u4_to_f32(w, 3, zA), x0.w, s0);
  s1 = fmaf(u4_to_f32(w, 7, zB), x1.w, s1);
  return fmaf(sA, s0, sB * s1);
}

// ------------------------------------------------------------------------------------------------
// One pass: this warp walks every ring tile of the pass, accumulates its G rows over its column
// blocks, then publishes the warp sums for the cross-k-warp reduction.
// ------------------------------------------------------------------------------------------------
template <int G, int WD>
__device__ __forceinline__ void consume_pass(Ctx& c, const PassGeom& g, float* red) {
  const KParams& p = c.p;
  const int wr = c.warp % g.Wr, wk = c.warp / g.Wr;
  const bool active = wk < g.Wk;
  const int my_rows = active ? min(G, g.R - wr * G) : 0;
  float acc[G];
#pragma unroll
  for (int i = 0; i < G; i++) acc[i] = 0.f;
  const int S = p.n_stages;
  for (int t = 0; t < g.n_tiles; ++t) {
    const int stage = (int)(c.tile_ctr % (unsigned)S);
    const unsigned parity = (c.tile_ctr / (unsigned)S) & 1u;
    if (!c.bad && !wait_mbar(p, &c.sh->full[stage], parity, -1)) c.bad = true;
    if (active && !c.bad) {
      const int u0 = t * g.upt;
      const int u1 = min(u0 + g.upt, g.n_units);
      const unsigned char* sbase = c.ring + (size_t)stage * p.stage_bytes - unit_off(g, u0);
      int b = (u0 > wr) ? (u0 - wr + g.Wr - 1) / g.Wr : 0;            // first column block of row-warp wr in this tile
      b += ((wk - b) % g.Wk + g.Wk) % g.Wk;                           // first one owned by k-warp wk
      for (; b * g.Wr + wr < u1; b += g.Wk) {
        const bool is_tail = g.tail && (b == g.nblk - 1);
        const int wd = is_tail ? g.tail : kBlockCols;
        const int rc = is_tail ? g.rc_tail : g.rc_full;
        const unsigned char* up = sbase + unit_off_br(g, b, wr);
        if (c.lane < (wd >> 3)) {
          const float4 x0 = *reinterpret_cast<const float4*>(c.xs + b * kBlockCols + 4 * c.lane);
          const float4 x1 = *reinterpret_cast<const float4*>(c.xs + b * kBlockCols + (wd >> 1) + 4 * c.lane);
#pragma unroll
          for (int i = 0; i < G; i++)
            if (i < my_rows) acc[i] += dot8<WD>(up + i * rc, c.lane, x0, x1);
        }
      }
    }
    __syncwarp();
    if (c.lane == 0 && !c.bad) mbar_arrive(&c.sh->empty[stage]);
    c.tile_ctr++;
  }
#pragma unroll
  for (int i = 0; i < G; i++) acc[i] = warp_sum(acc[i]);
  if (active && c.lane == 0) {
#pragma unroll
    for (int i = 0; i < G; i++)
      if (i < my_rows) red[wk * g.R + wr * G + i] = acc[i];     // [Wk][R]: Wk * R <= warps * kGMax
  }
}

template <int WD>
__device__ __forceinline__ void consume_pass_g(Ctx& c, const PassGeom& g, float* red) {
  switch (g.G) {
    case 1: consume_pass<1, WD>(c, g, red); break;
    case 2: consume_pass<2, WD>(c, g, red); break;
    case 3: consume_pass<3, WD>(c, g, red); break;
    case 4: consume_pass<4, WD>(c, g, red); break;
    case 5: consume_pass<5, WD>(c, g, red); break;
    case 6: consume_pass<6, WD>(c, g, red); break;
    case 7: consume_pass<7, WD>(c, g, red); break;
    default: consume_pass<8, WD>(c, g, red); break;
  }
}

__device__ __forceinline__ float4 ldcg4(const float* p, int i4) { return __ldcg(reinterpret_cast<const float4*>(p) + i4); }
__device__ __forceinline__ float4 bf16x4_to_f32(uint2 v) {
  return make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
}
__device__ __forceinline__ float silu_f(float z) { return z / (1.0f + expf(-z)); }

// ------------------------------------------------------------------------------------------------
// One matrix-vector product with its fused prologue (gather / RMSNorm) and epilogue.
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ bool gemv_op(Ctx& c, int op_idx, int wait_ph, int sig_ph) {
  const KParams& p = c.p;
  const OpDesc d = p.ops[op_idx];
  const int slot = (c.cta + d.rot) % c.nblk;
  const Slice sl = slot_slice(d.rows, d.unit_rows, c.nblk, slot);
  const int l = d.layer, K = d.K, n4 = K >> 2;
  const bool first_layer = (l == 0);
  const unsigned short* embed_row = p.embed + (size_t)c.token * p.H;

  // input vector and norm weight of this op
  const float* src = nullptr;
  const unsigned short* normw = nullptr;
  bool from_embed = false;
  switch (d.kind) {
    case OP_QKV: src = p.x_a; normw = p.attn_norm + (size_t)l * p.H; from_embed = first_layer; break;
    case OP_O: src = p.o; break;
    case OP_GATEUP: src = p.x_b; normw = p.mlp_norm + (size_t)l * p.H; break;
    case OP_DOWN: src = p.m; break;
    default: src = p.x_a; normw = p.final_norm; break;
  }

  const int task = (d.kind == OP_LMHEAD) ? 5 * p.L : 5 * l + (d.kind == OP_QKV ? 0 : d.kind + 1);
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_ENTER);
  // ---- prologue, part 1: what does not depend on the join (norm weights) -----------------------------
  uint2 gw[kNormVec];
  if (normw) {
#pragma unroll
    for (int k = 0; k < kNormVec; k++) {
      const int i = c.tid + k * kConsumerThreads;
      gw[k] = (i < n4) ? __ldg(reinterpret_cast<const uint2*>(normw) + i) : make_uint2(0u, 0u);
    }
  }
  // ---- the join ---------------------------------------------------------------------------------------
  if (wait_ph >= 0 && !wait_phase(c, wait_ph)) return false;
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_JOINED);

  // ---- prologue, part 2: bring the input vector into shared memory ------------------------------------
  float4* xs4 = reinterpret_cast<float4*>(c.xs);
  if (normw) {
    float4 v[kNormVec];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < kNormVec; k++) {
      const int i = c.tid + k * kConsumerThreads;
      if (i < n4) {
        v[k] = from_embed ? bf16x4_to_f32(__ldg(reinterpret_cast<const uint2*>(embed_row) + i)) : ldcg4(src, i);
        ss = fmaf(v[k].x, v[k].x, ss);
        ss = fmaf(v[k].y, v[k].y, ss);
        ss = fmaf(v[k].z, v[k].z, ss);
        ss = fmaf(v[k].w, v[k].w, ss);
      } else {
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    ss = warp_sum(ss);
    if (c.lane == 0) c.sh->warp_part[c.warp] = ss;
    c.bad = cons_sync_or(c.bad);
    if (c.bad) return false;
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; w++) tot += c.sh->warp_part[w];
    const float r = 1.0f / sqrtf(tot / (float)K + p.eps);
#pragma unroll
    for (int k = 0; k < kNormVec; k++) {
      const int i = c.tid + k * kConsumerThreads;
      if (i < n4) {
        const float4 g = bf16x4_to_f32(gw[k]);
        xs4[i] = make_float4(v[k].x * r * g.x, v[k].y * r * g.y, v[k].z * r * g.z, v[k].w * r * g.w);
        if (from_embed && c.cta == 0 && (p.flags & AMK_FLAG_DEBUG_HIDDEN))
          reinterpret_cast<float4*>(p.hidden)[i] = v[k];
      }
    }
  } else {
    for (int i = c.tid; i < n4; i += kConsumerThreads) xs4[i] = ldcg4(src, i);
  }
  c.bad = cons_sync_or(c.bad);
  if (c.bad) return false;
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_LOADED);

  // ---- passes -------------------------------------------------------------------------------------------
  float best_val = -CUDART_INF_F;
  int best_idx = 0x7fffffff;
  const int np = n_passes(sl.rows);
  for (int ps = 0; ps < np; ps++) {
    const int R = pass_rows(sl.rows, ps);
    const PassGeom g = pass_geom(R, K, d.wdtype, p.stage_bytes);
    const int vrow0 = sl.row0 + ps * kPassRows;
    float* red = c.sh->red[ps & 1];

    // epilogue operands fetched ahead of the pass
    const int n_out = (d.kind == OP_GATEUP) ? (R >> 1) : R;
    const bool outp = c.tid < n_out;
    float resid = 0.f, sc0 = 1.f, sc1 = 1.f;
    if (outp) {
      const int vrow = vrow0 + c.tid;
      if (d.kind == OP_O)
        resid = first_layer ? bf16_lo((unsigned)__ldg(embed_row + vrow)) : __ldcg(p.x_a + vrow);
      else if (d.kind == OP_DOWN)
        resid = __ldcg(p.x_b + vrow);
      if (d.wdtype == W_INT8) {
        const __half* scales = reinterpret_cast<const __half*>(p.packed + d.scale_off);
        if (d.kind == OP_GATEUP) {
          sc0 = __half2float(__ldg(scales + vrow0 + 2 * c.tid));
          sc1 = __half2float(__ldg(scales + vrow0 + 2 * c.tid + 1));
        } else {
          sc0 = __half2float(__ldg(scales + vrow));
        }
      }
    }

    if (d.wdtype == W_BF16) consume_pass_g<W_BF16>(c, g, red);
    else if (d.wdtype == W_INT8) consume_pass_g<W_INT8>(c, g, red);
    else consume_pass_g<W_INT4>(c, g, red);
    c.bad = cons_sync_or(c.bad);
    if (c.bad) return false;

    if (outp) {
      const int vrow = vrow0 + c.tid;
      if (d.kind == OP_GATEUP) {
        float gt = 0.f, up = 0.f;
        for (int k = 0; k < g.Wk; k++) {
          gt += red[k * R + 2 * c.tid];
          up += red[k * R + 2 * c.tid + 1];
        }
        gt *= sc0;
        up *= sc1;
        p.m[(vrow0 >> 1) + c.tid] = silu_f(gt) * up;
      } else {
        float y = 0.f;
        for (int k = 0; k < g.Wk; k++) y += red[k * R + c.tid];
        y *= sc0;
        switch (d.kind) {
          case OP_QKV: p.qkv[vrow] = y; break;
          case OP_O: p.x_b[vrow] = resid + y; break;
          case OP_DOWN: {
            const float xn = resid + y;
            p.x_a[vrow] = xn;
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
  if (d.kind == OP_LMHEAD) {
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
          *p.lm_ctr = 0u;
        }
      }
    }
    return true;
  }

  c.bad = cons_sync_or(c.bad);
  if (c.bad) return false;
  if (sig_ph >= 0) signal_phase(c, sig_ph);
  if (c.tid == 0) stamp(p, c.cta, task, AMK_TR_SIGNALLED);
  return true;
}

// ------------------------------------------------------------------------------------------------
// Attention task: RoPE on the group's q heads (and on k, with the KV append, in the chunk that holds the
// new position), online-softmax partial over this chunk of cache positions, then either the final
// output (one chunk) or a partial that the last-arriving chunk of the group combines.
// Scores are kept in the log2 domain: q is pre-scaled by log2(e) / sqrt(hd).
// ------------------------------------------------------------------------------------------------
template <int HD>
__device__ __forceinline__ void attn_task(Ctx& c, int l, int g, int ch, int Lc, int C) {
  const KParams& p = c.p;
  constexpr int LG = HD / 8;            // lanes per cache position (8 bf16 each)
  constexpr int PPW = 32 / LG;          // positions per warp per step
  constexpr int U = 4;                  // positions in flight per lane group
  const int n_rep = p.n_rep, half = HD / 2;
  const int n_pos = p.pos + 1;
  const int j0 = ch * Lc, j1 = min(n_pos, j0 + Lc);
  const bool owns_new = (j1 == n_pos);
  float* qs = c.xs;                                   // [n_rep][HD]
  float* wp = c.xs + n_rep * HD;                      // [warps][4][HD + 2]
  const float2* rope = p.rope + (size_t)p.pos * half;
  const float qscale = 1.4426950408889634f * rsqrtf((float)HD);
  const size_t kvrow = ((size_t)l * p.nkv + g) * p.S;

  for (int i = c.tid; i < n_rep * half; i += kConsumerThreads) {
    const int h = i / half, e = i - h * half;
    const float* q = p.qkv + (size_t)(g * n_rep + h) * HD;
    const float a = __ldcg(q + e), b = __ldcg(q + e + half);
    const float2 cs = __ldg(rope + e);
    qs[h * HD + e] = (a * cs.x - b * cs.y) * qscale;
    qs[h * HD + e + half] = (b * cs.x + a * cs.y) * qscale;
  }
  if (owns_new) {
    if (c.tid < half) {
      const float* k = p.qkv + (size_t)p.nq * HD + (size_t)g * HD;
      const float a = __ldcg(k + c.tid), b = __ldcg(k + c.tid + half);
      const float2 cs = __ldg(rope + c.tid);
      unsigned short* dst = p.kcache + (kvrow + p.pos) * HD;
      dst[c.tid] = f32_to_bf16_rne(a * cs.x - b * cs.y);
      dst[c.tid + half] = f32_to_bf16_rne(b * cs.x + a * cs.y);
    } else if (c.tid >= 64 && c.tid < 64 + HD) {
      const int e = c.tid - 64;
      const float* v = p.qkv + (size_t)(p.nq + p.nkv) * HD + (size_t)g * HD;
      p.vcache[(kvrow + p.pos) * HD + e] = f32_to_bf16_rne(__ldcg(v + e));
    }
  }
  c.bad = cons_sync_or(c.bad);           // q in shared memory; the new cache row is visible to this block

  const int n_hb = (n_rep + 3) >> 2;     // blocks of four q heads
  const int wph = kConsumerWarps / n_hb; // warps per head block
  const int hb = c.warp / wph, wi = c.warp - hb * wph;
  const int dl = c.lane % LG, sub = c.lane / LG;
  float m[4], lsum[4], acc[4][8];
#pragma unroll
  for (int hh = 0; hh < 4; hh++) {
    m[hh] = -CUDART_INF_F;
    lsum[hh] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; e++) acc[hh][e] = 0.f;
  }
  if (hb < n_hb) {
    const uint4* Kb = reinterpret_cast<const uint4*>(p.kcache + kvrow * HD);
    const uint4* Vb = reinterpret_cast<const uint4*>(p.vcache + kvrow * HD);
    const int stride = wph * PPW;
    for (int jb = j0 + wi * PPW + sub; jb - sub - wi * PPW < j1; jb += U * stride) {
      uint4 kq[U], vq[U];
#pragma unroll
      for (int u = 0; u < U; u++) {
        const int j = min(jb + u * stride, j1 - 1);
        kq[u] = __ldcg(Kb + (size_t)j * LG + dl);
        vq[u] = __ldcg(Vb + (size_t)j * LG + dl);
      }
#pragma unroll
      for (int u = 0; u < U; u++) {
        const bool valid = (jb + u * stride) < j1;
        const float kf[8] = {bf16_lo(kq[u].x), bf16_hi(kq[u].x), bf16_lo(kq[u].y), bf16_hi(kq[u].y),
                             bf16_lo(kq[u].z), bf16_hi(kq[u].z), bf16_lo(kq[u].w), bf16_hi(kq[u].w)};
        const float vf[8] = {bf16_lo(vq[u].x), bf16_hi(vq[u].x), bf16_lo(vq[u].y), bf16_hi(vq[u].y),
                             bf16_lo(vq[u].z), bf16_hi(vq[u].z), bf16_lo(vq[u].w), bf16_hi(vq[u].w)};
#pragma unroll
        for (int hh = 0; hh < 4; hh++) {
          const int h = hb * 4 + hh;
          if (h < n_rep) {
            const float4 q0 = *reinterpret_cast<const float4*>(qs + h * HD + dl * 8);
            const float4 q1 = *reinterpret_cast<const float4*>(qs + h * HD + dl * 8 + 4);
            float s = kf[0] * q0.x;
            s = fmaf(kf[1], q0.y, s);
            s = fmaf(kf[2], q0.z, s);
            s = fmaf(kf[3], q0.w, s);
            s = fmaf(kf[4], q1.x, s);
            s = fmaf(kf[5], q1.y, s);
            s = fmaf(kf[6], q1.z, s);
            s = fmaf(kf[7], q1.w, s);
#pragma unroll
            for (int o = LG / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (valid) {
              const float mn = fmaxf(m[hh], s);
              const float corr = exp2f(m[hh] - mn);          // m = -inf gives 0
              const float pw = exp2f(s - mn);
              lsum[hh] = fmaf(lsum[hh], corr, pw);
#pragma unroll
              for (int e = 0; e < 8; e++) acc[hh][e] = fmaf(acc[hh][e], corr, pw * vf[e]);
              m[hh] = mn;
            }
          }
        }
      }
    }
    // merge the lane groups of the warp
#pragma unroll
    for (int o = LG; o < 32; o <<= 1) {
#pragma unroll
      for (int hh = 0; hh < 4; hh++) {
        const float mo = __shfl_xor_sync(0xffffffffu, m[hh], o);
        const float lo = __shfl_xor_sync(0xffffffffu, lsum[hh], o);
        const float mn = fmaxf(m[hh], mo);
        const float a = (m[hh] == -CUDART_INF_F) ? 0.f : exp2f(m[hh] - mn);
        const float b = (mo == -CUDART_INF_F) ? 0.f : exp2f(mo - mn);
        lsum[hh] = lsum[hh] * a + lo * b;
#pragma unroll
        for (int e = 0; e < 8; e++) {
          const float ao = __shfl_xor_sync(0xffffffffu, acc[hh][e], o);
          acc[hh][e] = acc[hh][e] * a + ao * b;
        }
        m[hh] = mn;
      }
    }
    if (sub == 0) {
#pragma unroll
      for (int hh = 0; hh < 4; hh++) {
        float* w = wp + (size_t)(c.warp * 4 + hh) * (HD + 2);
        if (dl == 0) { w[0] = m[hh]; w[1] = lsum[hh]; }
#pragma unroll
        for (int e = 0; e < 8; e++) w[2 + dl * 8 + e] = acc[hh][e];
      }
    }
  }
  c.bad = cons_sync_or(c.bad);

  // merge the warps of each head block, in warp order
  for (int i = c.tid; i < n_rep * HD; i += kConsumerThreads) {
    const int h = i / HD, dd = i - h * HD;
    const int hbb = h >> 2, hh = h & 3;
    float M = -CUDART_INF_F;
    for (int w = 0; w < wph; w++) M = fmaxf(M, wp[(size_t)((hbb * wph + w) * 4 + hh) * (HD + 2)]);
    float Z = 0.f, A = 0.f;
    for (int w = 0; w < wph; w++) {
      const float* ww = wp + (size_t)((hbb * wph + w) * 4 + hh) * (HD + 2);
      const float a = (ww[0] == -CUDART_INF_F) ? 0.f : exp2f(ww[0] - M);
      Z = fmaf(a, ww[1], Z);
      A = fmaf(a, ww[2 + dd], A);
    }
    const int hq = g * n_rep + h;
    if (C == 1) {
      p.o[(size_t)hq * HD + dd] = A / Z;
    } else {
      float* pt = p.part + ((size_t)hq * kMaxChunks + ch) * (HD + 2);
      pt[2 + dd] = A;
      if (dd == 0) { pt[0] = M; pt[1] = Z; }
    }
  }
  if (C == 1) return;

  // several chunks: the chunk that arrives last for this kv group combines all of them
  c.bad = cons_sync_or(c.bad);
  if (c.tid == 0) {
    __threadfence();
    const unsigned old = atomicAdd(p.group_ctr + g, 1u);
    __threadfence();
    c.sh->flag = (old == (unsigned)(C - 1));
  }
  c.bad = cons_sync_or(c.bad);
  if (c.sh->flag) {
    for (int i = c.tid; i < n_rep * HD; i += kConsumerThreads) {
      const int h = i / HD, dd = i - h * HD;
      const int hq = g * n_rep + h;
      const float* pt = p.part + (size_t)hq * kMaxChunks * (HD + 2);
      float M = -CUDART_INF_F;
      for (int k = 0; k < C; k++) M = fmaxf(M, __ldcg(pt + (size_t)k * (HD + 2)));
      float Z = 0.f, A = 0.f;
      for (int k = 0; k < C; k++) {
        const float a = exp2f(__ldcg(pt + (size_t)k * (HD + 2)) - M);
        Z = fmaf(a, __ldcg(pt + (size_t)k * (HD + 2) + 1), Z);
        A = fmaf(a, __ldcg(pt + (size_t)k * (HD + 2) + 2 + dd), A);
      }
      p.o[(size_t)hq * HD + dd] = A / Z;
    }
    if (c.tid == 0) p.group_ctr[g] = 0u;
  }
}

__device__ __noinline__ bool attention_phase(Ctx& c, int l) {
  const KParams& p = c.p;
  int Lc, C;
  attn_chunks(p.pos + 1, c.nblk, p.nkv, &Lc, &C);
  const int n_tasks = p.nkv * C;
  const int rot = (l * 29) % c.nblk;
  const int t = (c.cta + c.nblk - rot) % c.nblk;
  if (c.tid == 0) stamp(p, c.cta, 5 * l + 1, AMK_TR_ENTER);
  if (!wait_phase(c, 5 * l + 0)) return false;
  if (c.tid == 0) stamp(p, c.cta, 5 * l + 1, AMK_TR_JOINED);
  if (t < n_tasks) {
    const int g = t / C, ch = t - g * C;
    if (p.hd == 64) attn_task<64>(c, l, g, ch, Lc, C);
    else attn_task<128>(c, l, g, ch, Lc, C);
  }
  c.bad = cons_sync_or(c.bad);
  if (c.bad) return false;
  if (c.tid == 0) stamp(p, c.cta, 5 * l + 1, AMK_TR_COMPUTED);
  signal_phase(c, 5 * l + 1);
  if (c.tid == 0) stamp(p, c.cta, 5 * l + 1, AMK_TR_SIGNALLED);
  return true;
}

// ------------------------------------------------------------------------------------------------
// Producer: one thread streams this block's weight tiles, op after op, into the ring.
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ void producer(const KParams& p, SmemHeader* sh, unsigned char* ring, int cta, int nblk) {
  const uint64_t pol = policy_evict_first();
  const int S = p.n_stages;
  const int inflight = p.max_inflight;
  unsigned t = 0;
  bool ok = true;
  for (int op = 0; op < p.n_ops && ok; op++) {
    const OpDesc d = p.ops[op];
    const int slot = (cta + d.rot) % nblk;
    const Slice sl = slot_slice(d.rows, d.unit_rows, nblk, slot);
    const int64_t rb = row_bytes(d.wdtype, d.K);
    const unsigned char* base = p.packed + d.packed_off + (int64_t)sl.row0 * rb;
    const int np = n_passes(sl.rows);
    const int task = (d.kind == OP_LMHEAD) ? 5 * p.L : 5 * d.layer + (d.kind == OP_QKV ? 0 : d.kind + 1);
    bool first = true;
    for (int ps = 0; ps < np && ok; ps++) {
      const PassGeom g = pass_geom(pass_rows(sl.rows, ps), d.K, d.wdtype, p.stage_bytes);
      const unsigned char* pbase = base + (int64_t)ps * kPassRows * rb;
      for (int tt = 0; tt < g.n_tiles; tt++, t++) {
        const int u0 = tt * g.upt;
        const int64_t o0 = unit_off(g, u0), o1 = unit_off(g, u0 + g.upt);
        const int stage = (int)(t % (unsigned)S);
        if (t >= (unsigned)S) {
          if (!wait_mbar(p, &sh->empty[stage], ((t / (unsigned)S) & 1u) ^ 1u, -2)) { ok = false; break; }
        }
        if (inflight < S && t >= (unsigned)inflight) {
          const unsigned tl = t - (unsigned)inflight;      // this older tile must have landed
          if (!wait_mbar(p, &sh->full[tl % (unsigned)S], (tl / (unsigned)S) & 1u, -2)) { ok = false; break; }
        }
        const unsigned bytes = (unsigned)(o1 - o0);
        mbar_expect_tx(&sh->full[stage], bytes);
        bulk_g2s(ring + (size_t)stage * p.stage_bytes, pbase + o0, bytes, &sh->full[stage], pol);
        if (first) { stamp(p, cta, task, AMK_TR_PROD_FIRST); first = false; }
      }
    }
    if (ok) stamp(p, cta, task, AMK_TR_PROD_LAST);
  }
  if (!ok) {
    // leaving early: every copy already issued must land before the block's shared memory is released
    const unsigned first = (t > (unsigned)S) ? t - (unsigned)S : 0u;
    for (unsigned i = first; i < t; i++) {
      uint64_t* bar = &sh->full[i % (unsigned)S];
      const unsigned parity = (i / (unsigned)S) & 1u;
      for (unsigned spins = 0; spins < (1u << 24) && !mbar_try_wait(bar, parity); spins++) {}
    }
  }
}

}  // namespace

__global__ void __launch_bounds__(kThreads, 1) amk_decode_kernel(const __grid_constant__ KParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  SmemHeader* sh = reinterpret_cast<SmemHeader*>(smem);
  const size_t hdr = (sizeof(SmemHeader) + 127) & ~(size_t)127;
  float* xs = reinterpret_cast<float*>(smem + hdr);
  unsigned char* ring = smem + hdr + p.act_bytes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, nblk = gridDim.x;

  if (tid == 0) {
    for (int s = 0; s < p.n_stages; s++) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], kConsumerWarps);
    }
    sh->abort = 0;
    sh->flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    if (lane == 0) producer(p, sh, ring, cta, nblk);
    return;
  }

  int token = p.token_ptr ? __ldcg(p.token_ptr) : p.token;
  token = min(max(token, 0), p.V - 1);
  Ctx c{p, sh, xs, ring, tid, warp, lane, cta, nblk, 0u, token, false};
  bool ok = true;
  for (int l = 0; l < p.L && ok; l++) {
    ok = gemv_op(c, 4 * l + 0, l > 0 ? 5 * (l - 1) + 4 : -1, 5 * l + 0);
    ok = ok && attention_phase(c, l);
    ok = ok && gemv_op(c, 4 * l + 1, 5 * l + 1, 5 * l + 2);
    ok = ok && gemv_op(c, 4 * l + 2, 5 * l + 2, 5 * l + 3);
    ok = ok && gemv_op(c, 4 * l + 3, 5 * l + 3, 5 * l + 4);
  }
  if (ok) gemv_op(c, 4 * p.L, 5 * (p.L - 1) + 4, -1);
}

cudaError_t decode_kernel_attrs(size_t smem_bytes, int* max_blocks_per_sm) {
  cudaError_t e = cudaFuncSetAttribute(amk_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(max_blocks_per_sm, amk_decode_kernel, kThreads, smem_bytes);
}

cudaError_t launch_decode(const KParams& p, int n_blocks, size_t smem_bytes, cudaStream_t stream) {
  void* args[] = {const_cast<KParams*>(&p)};
  return cudaLaunchCooperativeKernel((const void*)amk_decode_kernel, dim3(n_blocks), dim3(kThreads), args, smem_bytes,
                                     stream);
}

}  // namespace amk
