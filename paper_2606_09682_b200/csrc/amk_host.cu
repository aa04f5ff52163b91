// Host side of the C ABI (include/amk.h): configuration checks, the plan (tables, buffer layouts), the
// weight packer's driver, and the launch of the decode kernel.  Nothing here computes any part of the
// decode step: every step of the path runs in the kernels.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "amk.h"
#include "amk_internal.h"

using namespace amk;

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxBlocks = 512;   // upper bound on persistent blocks
inline size_t align_up(size_t v, size_t a = kAlign) { return (v + a - 1) / a * a; }

// One matrix-vector product of the step, as the host plans it.
struct PlanOp {
  int kind, layer;
  OpShape s;
  size_t region_off;                 // byte offset of the op's region in the packed buffer
  size_t scale_off;                  // int8: fp16 row scales (virtual row order)
  std::vector<unsigned long long> slice_off;   // [n_blocks] byte offset of each slot's slice inside the region
};

// Everything that follows from (config, block count): op table, packed-buffer layout, per-block tile lists.
struct Plan {
  int n_blocks = 0;
  uint32_t stage_bytes = 0;
  OpShape shape[5];
  std::vector<PlanOp> ops;
  std::vector<int> bounds[5];        // per op kind: unit boundaries of the slots (n_blocks + 1)
  size_t scale_base = 0, scale_layer_stride = 0, scale_kind_off[4] = {0, 0, 0, 0}, lm_scale_off = 0;
  size_t embed_off = 0, attn_norm_off = 0, mlp_norm_off = 0, final_norm_off = 0, packed_total = 0;
  size_t weight_stream_bytes = 0;    // op regions + scale regions (what a token streams)
  size_t n_tiles = 0;                // total ring tiles over all blocks
};

struct WorkspaceLayout {
  size_t status, phase_ctr, group_ctr, lm_ctr, next_ws, cand_val, cand_idx, x_a, x_b, qkv, o, m, part, hidden, rope,
      trace, ktime, slice_tab, bounds, smid_tab, calib, tile_begin, tiles, total;
};

void plan_to_words(const amk_config* cfg, const Plan& pl, const std::vector<unsigned long long>& tiles,
                   const std::vector<unsigned>& tile_begin, std::vector<uint64_t>& out);

int resolve_blocks(const amk_config* c) {
  if (c->n_blocks) return (int)c->n_blocks;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
    return sms;
  (void)cudaGetLastError();
  return 148;
}

amk_status check_config(const amk_config* c) {
  if (!c) return AMK_ERR_INVALID_ARG;
  if (c->struct_size != sizeof(amk_config) || c->abi_version != AMK_ABI_VERSION) return AMK_ERR_INVALID_ARG;
  if (c->l2_ahead > 33u) return AMK_ERR_INVALID_ARG;
  if (!c->hidden || !c->n_layers || !c->n_q_heads || !c->n_kv_heads || !c->mlp || !c->vocab || !c->max_seq)
    return AMK_ERR_INVALID_ARG;
  if (c->wdtype > AMK_W_INT8_GROUPED || c->sync_mode > 2 || c->kv_dtype > AMK_KV_FP8_E4M3) return AMK_ERR_INVALID_ARG;
  if (5ull * c->n_layers + 1 > 2047ull) return AMK_ERR_UNSUPPORTED;      // a tile entry keeps its task in 11 bits
  if (c->n_blocks > (uint32_t)kMaxBlocks) return AMK_ERR_INVALID_ARG;
  if (c->head_dim != 64 && c->head_dim != 128) return AMK_ERR_UNSUPPORTED;
  if (c->n_q_heads % c->n_kv_heads) return AMK_ERR_UNSUPPORTED;
  if (c->n_q_heads / c->n_kv_heads > (uint32_t)kMaxRep) return AMK_ERR_UNSUPPORTED;
  if (c->quantize_lm_head > 1) return AMK_ERR_INVALID_ARG;
  if (c->quantize_lm_head && c->wdtype == AMK_W_BF16) return AMK_ERR_UNSUPPORTED;   // nothing to quantise it like
  const uint32_t kdiv = grouped((int)c->wdtype) ? 128 : 64;
  const uint32_t qdim = c->n_q_heads * c->head_dim;
  if (c->hidden % kdiv || c->mlp % kdiv || qdim % kdiv) return AMK_ERR_UNSUPPORTED;
  if (c->hidden > 16u * kConsumerThreads) return AMK_ERR_UNSUPPORTED;   // a normed input is gathered in one batch
  if (grouped((int)c->wdtype) && c->group_size != 128) return AMK_ERR_UNSUPPORTED;
  if ((uint64_t)c->vocab * c->hidden > (1ull << 40)) return AMK_ERR_UNSUPPORTED;
  if (c->stage_bytes && (c->stage_bytes % 1024 || c->stage_bytes < 8192 || c->stage_bytes > 65536))
    return AMK_ERR_INVALID_ARG;
  if (c->n_stages > (uint32_t)kMaxStages || c->n_stages == 1) return AMK_ERR_INVALID_ARG;
  return AMK_OK;
}

// Ring stage size.  Default 32 KB; 48 KB for int4, whose consumers do the most work per byte: fewer, larger tiles
// mean fewer waits and arrivals per unit (knob search: Llama-3-8B int4 1254 -> 1222 us; no gain for the others).
uint32_t stage_bytes_of(const amk_config* c) {
  return c->stage_bytes ? c->stage_bytes : (c->wdtype == AMK_W_INT4 ? 49152u : 32768u);
}

// `weights`: relative streaming rate of each slot (nullptr: equal shares).
Plan make_plan(const amk_config* c, int n_blocks, const double* weights, bool with_tiles,
               std::vector<unsigned long long>* tiles, std::vector<unsigned>* tile_begin) {
  Plan pl;
  pl.n_blocks = n_blocks;
  pl.stage_bytes = stage_bytes_of(c);
  const int H = c->hidden, L = c->n_layers, I = c->mlp, V = c->vocab;
  const int qd = c->n_q_heads * c->head_dim, kvd = c->n_kv_heads * c->head_dim;
  const int wd = (int)c->wdtype;
  pl.shape[OP_QKV] = OpShape{H, qd + 2 * kvd, 1, wd};
  pl.shape[OP_O] = OpShape{qd, H, 1, wd};
  pl.shape[OP_GATEUP] = OpShape{H, 2 * I, 2, wd};
  pl.shape[OP_DOWN] = OpShape{I, H, 1, wd};
  pl.shape[OP_LMHEAD] = OpShape{H, V, 1, c->quantize_lm_head ? wd : (int)W_BF16};
  for (int k = 0; k < 5; k++) {
    pl.bounds[k].resize(n_blocks + 1);
    make_bounds(pl.shape[k].rows / pl.shape[k].unit_rows, n_blocks, weights, pl.bounds[k].data());
  }
  size_t off = 0;
  auto add = [&](int kind, int layer) {
    PlanOp op;
    op.kind = kind; op.layer = layer; op.s = pl.shape[kind];
    op.region_off = off;
    op.scale_off = 0;
    op.slice_off.resize(n_blocks);
    size_t o = 0;
    for (int s = 0; s < n_blocks; s++) {
      op.slice_off[s] = o;
      o += (size_t)slice_bytes(slot_slice(pl.bounds[kind].data(), op.s.unit_rows, s).rows, op.s.K, op.s.wdtype,
                               (int)pl.stage_bytes);
    }
    off = align_up(off + o);
    pl.ops.push_back(std::move(op));
  };
  for (int l = 0; l < L; l++) {
    add(OP_QKV, l);
    add(OP_O, l);
    add(OP_GATEUP, l);
    add(OP_DOWN, l);
  }
  add(OP_LMHEAD, L);
  if (wd == W_INT8) {
    pl.scale_base = off;
    size_t k = 0;
    for (int kind = 0; kind < 4; kind++) { pl.scale_kind_off[kind] = k; k = align_up(k + (size_t)pl.shape[kind].rows * 2, 16); }
    pl.scale_layer_stride = k;
    for (auto& op : pl.ops)
      if (op.kind != OP_LMHEAD) op.scale_off = pl.scale_base + (size_t)op.layer * k + pl.scale_kind_off[op.kind];
    off = align_up(off + (size_t)L * k);
    if (c->quantize_lm_head) {
      pl.lm_scale_off = off;
      pl.ops.back().scale_off = off;
      off = align_up(off + (size_t)V * 2);
    }
  }
  pl.weight_stream_bytes = off;
  pl.embed_off = off;      off = align_up(off + (size_t)V * H * 2);
  pl.attn_norm_off = off;  off = align_up(off + (size_t)L * H * 2);
  pl.mlp_norm_off = off;   off = align_up(off + (size_t)L * H * 2);
  pl.final_norm_off = off; off = align_up(off + (size_t)H * 2);
  pl.packed_total = off;

  // per-block tile lists, in the order the block consumes them
  size_t count = 0;
  if (with_tiles) { tiles->clear(); tile_begin->assign(n_blocks + 1, 0); }
  for (int cta = 0; cta < n_blocks; cta++) {
    if (with_tiles) (*tile_begin)[cta] = (unsigned)count;
    for (size_t i = 0; i < pl.ops.size(); i++) {
      const PlanOp& op = pl.ops[i];
      const int slot = cta;
      const Slice sl = slot_slice(pl.bounds[op.kind].data(), op.s.unit_rows, slot);
      const int task = (op.kind == OP_LMHEAD) ? 5 * L : 5 * op.layer + (op.kind == OP_QKV ? 0 : op.kind + 1);
      size_t base = op.region_off + op.slice_off[slot];
      for (int ps = 0; ps < n_passes(sl.rows); ps++) {
        const PassGeom g = pass_geom(pass_rows(sl.rows, ps), op.s.K, op.s.wdtype, (int)pl.stage_bytes);
        for (int t = 0; t < g.n_tiles; t++) {
          const int64_t o0 = unit_off(g, t * g.upt), o1 = unit_off(g, (t + 1) * g.upt);
          if (with_tiles) {
            const unsigned long long e = (unsigned long long)((base + (size_t)o0) >> 4) |
                                         ((unsigned long long)((o1 - o0) >> 4) << 40) |
                                         ((unsigned long long)task << 53);
            tiles->push_back(e);
          }
          count++;
        }
        base += (size_t)pass_bytes(g);
      }
      if (op.kind == OP_QKV) {
        // marker (no bytes) of the layer's attention task: the producer streams the chunk's cache rows here
        if (with_tiles) tiles->push_back((unsigned long long)(5 * op.layer + 1) << 53);
        count++;
      }
    }
  }
  if (with_tiles) (*tile_begin)[n_blocks] = (unsigned)count;
  pl.n_tiles = count;
  return pl;
}

WorkspaceLayout workspace_layout(const amk_config* c, const Plan& pl) {
  WorkspaceLayout w;
  const size_t H = c->hidden, L = c->n_layers, I = c->mlp, S = c->max_seq, hd = c->head_dim;
  const size_t qd = (size_t)c->n_q_heads * hd, kvd = (size_t)c->n_kv_heads * hd;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  w.status = take(sizeof(DevStatus));
  w.phase_ctr = take(5 * L * 4);
  w.group_ctr = take(L * (size_t)c->n_kv_heads * 4);
  w.lm_ctr = take(4);
  w.next_ws = take(4);
  w.cand_val = take(kMaxBlocks * 4);
  w.cand_idx = take(kMaxBlocks * 4);
  w.x_a = take(H * sizeof(ActPair));
  w.x_b = take(H * sizeof(ActPair));
  w.qkv = take((qd + 2 * kvd) * sizeof(ActPair));
  w.o = take(qd * sizeof(ActPair));
  w.m = take(I * sizeof(ActPair));
  w.part = take((size_t)c->n_q_heads * kMaxChunks * (hd + 2) * sizeof(ActPair));
  w.hidden = take((L + 1) * H * 4);
  w.rope = take(S * (hd / 2) * sizeof(float2));
  w.trace = take((size_t)pl.n_blocks * (5 * L + 1) * AMK_TRACE_EVENTS * 8);
  w.ktime = take((size_t)kMaxBlocks * 16);
  w.slice_tab = take(pl.ops.size() * (size_t)pl.n_blocks * 8);
  w.bounds = take(5 * ((size_t)pl.n_blocks + 1) * 4);
  w.smid_tab = take((size_t)kMaxSmid * 4);
  w.calib = take((size_t)pl.n_blocks * 16);
  w.tile_begin = take(((size_t)pl.n_blocks + 1) * 4);
  // the tile count depends a little on how the rows are split over the slots: leave room for any split
  w.tiles = take((pl.n_tiles + pl.ops.size() * (size_t)pl.n_blocks * 2) * 8);
  w.total = off;
  return w;
}

size_t kv_bytes_of(const amk_config* c) {
  return 2ull * c->n_layers * c->n_kv_heads * c->max_seq * c->head_dim * (c->kv_dtype == AMK_KV_FP8_E4M3 ? 1ull : 2ull);
}

}  // namespace

struct amk_handle {
  amk_config cfg;
  amk_plan plan;
  Plan pl;
  WorkspaceLayout wl;
  unsigned char* packed;
  unsigned char* ws;
  KParams base;            // everything but the per-step fields
  unsigned epoch;          // steps launched since the activation area was last cleared (see epoch_would_wrap)
  unsigned ctr_epoch;      // steps since the counters were last zeroed
  cudaStream_t last_stream;
  int drop_phase, drop_block;
  float split_min, split_max;   // smallest / largest share given to a block, relative to the median
  char errmsg[256];
};

extern "C" {

const char* amk_status_str(amk_status s) {
  switch (s) {
    case AMK_OK: return "ok";
    case AMK_ERR_INVALID_ARG: return "invalid argument";
    case AMK_ERR_UNSUPPORTED: return "unsupported configuration";
    case AMK_ERR_CUDA: return "CUDA error";
    case AMK_ERR_OOM: return "out of host memory";
    case AMK_ERR_TIMEOUT: return "device-side wait timed out";
    case AMK_ERR_ABORTED: return "aborted";
    case AMK_ERR_BAD_POS: return "position out of range";
    case AMK_ERR_BAD_TOKEN: return "token out of range";
  }
  return "unknown status";
}

amk_status amk_packed_bytes(const amk_config* cfg, size_t* bytes) {
  if (!bytes) return AMK_ERR_INVALID_ARG;
  amk_status st = check_config(cfg);
  if (st != AMK_OK) return st;
  const Plan pl = make_plan(cfg, resolve_blocks(cfg), nullptr, false, nullptr, nullptr);
  // work units with scales inside are padded to 16 bytes, so the total depends a little on the split: leave room
  *bytes = pl.packed_total + (grouped((int)cfg->wdtype) ? pl.packed_total / 64 : 0);
  return AMK_OK;
}

amk_status amk_workspace_bytes(const amk_config* cfg, size_t* bytes) {
  if (!bytes) return AMK_ERR_INVALID_ARG;
  amk_status st = check_config(cfg);
  if (st != AMK_OK) return st;
  const Plan pl = make_plan(cfg, resolve_blocks(cfg), nullptr, false, nullptr, nullptr);
  *bytes = workspace_layout(cfg, pl).total;
  return AMK_OK;
}

amk_status amk_kv_bytes(const amk_config* cfg, size_t* bytes) {
  if (!bytes) return AMK_ERR_INVALID_ARG;
  amk_status st = check_config(cfg);
  if (st != AMK_OK) return st;
  *bytes = kv_bytes_of(cfg);
  return AMK_OK;
}

#define AMK_CUDA(call)                                                                       \
  do {                                                                                       \
    cudaError_t e_ = (call);                                                                 \
    if (e_ != cudaSuccess) {                                                                 \
      if (h) snprintf(h->errmsg, sizeof(h->errmsg), "%s: %s", #call, cudaGetErrorString(e_)); \
      status = AMK_ERR_CUDA;                                                                 \
      goto fail;                                                                             \
    }                                                                                        \
  } while (0)

amk_status amk_create(const amk_config* cfg, const amk_weights* wts, void* packed_dev, size_t packed_bytes,
                      void* workspace_dev, size_t workspace_bytes, void* cuda_stream, amk_handle** out) {
  if (!out) return AMK_ERR_INVALID_ARG;
  *out = nullptr;
  amk_status status = check_config(cfg);
  if (status != AMK_OK) return status;
  if (!wts || !packed_dev || !workspace_dev) return AMK_ERR_INVALID_ARG;
  if (((uintptr_t)packed_dev | (uintptr_t)workspace_dev) & (kAlign - 1)) return AMK_ERR_INVALID_ARG;
  if (!wts->embed || !wts->final_norm || !wts->attn_norm || !wts->mlp_norm) return AMK_ERR_INVALID_ARG;
  if (!cfg->tied_embeddings && !wts->lm_head && !cfg->quantize_lm_head) return AMK_ERR_INVALID_ARG;
  if (cfg->quantize_lm_head && (!wts->lm_head_q || !wts->lm_head_scale || (cfg->wdtype == AMK_W_INT4 && !wts->lm_head_zero)))
    return AMK_ERR_INVALID_ARG;
  for (int k = 0; k < AMK_LIN_COUNT; k++) {
    if (!wts->linear[k]) return AMK_ERR_INVALID_ARG;
    if (cfg->wdtype != AMK_W_BF16 && !wts->scale[k]) return AMK_ERR_INVALID_ARG;
    if (cfg->wdtype == AMK_W_INT4 && !wts->zero[k]) return AMK_ERR_INVALID_ARG;
  }
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  amk_handle* h = new (std::nothrow) amk_handle();
  if (!h) return AMK_ERR_OOM;
  h->cfg = *cfg;
  h->packed = (unsigned char*)packed_dev;
  h->ws = (unsigned char*)workspace_dev;
  h->drop_phase = -1;
  h->drop_block = -1;
  h->last_stream = stream;
  {
    int dev = 0, sms = 0, coop = 0, smem_optin = 0, cc_major = 0;
    AMK_CUDA(cudaGetDevice(&dev));
    AMK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    AMK_CUDA(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    AMK_CUDA(cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    AMK_CUDA(cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    const int n_blocks = cfg->n_blocks ? (int)cfg->n_blocks : sms;
    if (cc_major != 10 || !coop || sms < 1 || n_blocks > sms || n_blocks > kMaxBlocks ||
        (int)cfg->n_kv_heads > n_blocks) {
      snprintf(h->errmsg, sizeof(h->errmsg),
               "needs a compute-capability-10.x GPU with cooperative launch and at least n_blocks SMs");
      status = AMK_ERR_UNSUPPORTED;
      goto fail;
    }
    // ---- calibration: what share of the HBM stream does each SM get? ------------------------------------
    // (only when every SM runs a block: then the SM id identifies the block, whatever block index it has)
    std::vector<double> weights;
    std::vector<int> slot_of_smid;
    const Plan pl0 = make_plan(cfg, n_blocks, nullptr, false, nullptr, nullptr);
    const WorkspaceLayout wl0 = workspace_layout(cfg, pl0);
    if (packed_bytes < pl0.packed_total || workspace_bytes < wl0.total) {
      snprintf(h->errmsg, sizeof(h->errmsg), "buffers too small: packed %zu < %zu or workspace %zu < %zu", packed_bytes,
               pl0.packed_total, workspace_bytes, wl0.total);
      status = AMK_ERR_INVALID_ARG;
      goto fail;
    }
    const bool by_smid = (n_blocks == sms) && (cfg->flags & AMK_FLAG_MEASURED_SPLIT);
    if (by_smid) {
      size_t per = packed_bytes / (size_t)n_blocks;
      if (per > (8u << 20)) per = 8u << 20;
      per = per / 32768 * 32768;
      if (per >= (1u << 20)) {
        unsigned* smid_dev = (unsigned*)(h->ws + wl0.calib);
        unsigned long long* ns_dev = (unsigned long long*)(h->ws + wl0.calib + (size_t)n_blocks * 4 + 4) ;
        ns_dev = (unsigned long long*)(((uintptr_t)ns_dev + 7) & ~(uintptr_t)7);
        std::vector<unsigned> smid(n_blocks);
        std::vector<unsigned long long> ns(n_blocks);
        for (int rep = 0; rep < 2; rep++)
          AMK_CUDA(launch_calibrate(h->packed, per, n_blocks, (size_t)smem_optin, smid_dev, ns_dev, stream));
        AMK_CUDA(cudaMemcpyAsync(smid.data(), smid_dev, (size_t)n_blocks * 4, cudaMemcpyDeviceToHost, stream));
        AMK_CUDA(cudaMemcpyAsync(ns.data(), ns_dev, (size_t)n_blocks * 8, cudaMemcpyDeviceToHost, stream));
        AMK_CUDA(cudaStreamSynchronize(stream));
        // slot i = the i-th block of the calibration launch; every SM must appear exactly once
        slot_of_smid.assign(kMaxSmid, -1);
        weights.assign(n_blocks, 1.0);
        bool ok_map = true;
        std::vector<double> rates(n_blocks);
        for (int i = 0; i < n_blocks; i++) {
          if (smid[i] >= (unsigned)kMaxSmid || slot_of_smid[smid[i]] >= 0 || ns[i] == 0) { ok_map = false; break; }
          slot_of_smid[smid[i]] = i;
          rates[i] = (double)per / (double)ns[i];
        }
        if (ok_map) {
          std::vector<double> sorted = rates;
          std::sort(sorted.begin(), sorted.end());
          const double med = sorted[n_blocks / 2];
          for (int i = 0; i < n_blocks; i++) {
            double w = rates[i] / med;
            weights[i] = w < 0.8 ? 0.8 : (w > 1.5 ? 1.5 : w);      // a share, not a promise: keep it sane
          }
          if (getenv("AMK_VERBOSE")) {
            fprintf(stderr, "amk_create: per-SM rate GB/s min %.1f p10 %.1f median %.1f p90 %.1f max %.1f (%zu bytes each)\n",
                    sorted[0], sorted[n_blocks / 10], med, sorted[n_blocks * 9 / 10], sorted[n_blocks - 1], per);
          }
        } else {
          weights.clear();
          slot_of_smid.clear();
        }
      }
    }
    std::vector<unsigned long long> tiles;
    std::vector<unsigned> tile_begin;
    h->pl = make_plan(cfg, n_blocks, weights.empty() ? nullptr : weights.data(), true, &tiles, &tile_begin);
    {
      // the static check of the tables: a rejected plan is never launched
      std::vector<uint64_t> words;
      plan_to_words(cfg, h->pl, tiles, tile_begin, words);
      amk_config ccfg = *cfg;
      ccfg.n_blocks = (uint32_t)n_blocks;
      char why[160];
      if (amk_plan_check(&ccfg, words.data(), words.size(), why, sizeof(why)) != AMK_OK) {
        snprintf(h->errmsg, sizeof(h->errmsg), "plan rejected by the static check: %s", why);
        status = AMK_ERR_UNSUPPORTED;
        goto fail;
      }
    }
    h->wl = wl0;
    if (packed_bytes < h->pl.packed_total || tiles.size() * 8 > h->wl.total - h->wl.tiles) {
      snprintf(h->errmsg, sizeof(h->errmsg), "buffers too small for the measured split");
      status = AMK_ERR_INVALID_ARG;
      goto fail;
    }
    const int H = cfg->hidden, L = cfg->n_layers, I = cfg->mlp, hd = cfg->head_dim;
    const int qd = cfg->n_q_heads * hd, n_rep = cfg->n_q_heads / cfg->n_kv_heads;

    // ---- shared-memory plan -----------------------------------------------------------------------
    const size_t hdr = (sizeof(SmemHeader) + 127) & ~(size_t)127;
    size_t kmax = (size_t)(H > I ? H : I);
    if ((size_t)qd > kmax) kmax = qd;
    size_t act = kmax * 4;                                     // bf16 high + low halves
    if (cfg->wdtype != AMK_W_BF16)                             // or three int8 digit columns of whole groups of 128
      act = (kmax + 127) / 128 * (3 * 128 + 32);               //   + 32 bytes per group: digit sums and scale
    if (!cfg->quantize_lm_head && (size_t)H * 4 > act) act = (size_t)H * 4;   // a bf16 LM head in an integer model
    // attention scratch: q vectors, per-warp partial outputs, the new K / V rows, the scores of the longest chunk
    int lc_max = 0, c_max = 0;
    attn_chunks((int)cfg->max_seq, (int)n_blocks, (int)cfg->n_kv_heads, &lc_max, &c_max);
    // (AttnScratch in the kernel: q fp32, q as tensor-core fragments, per-warp partial outputs for the heads padded to
    //  sets of four, the new rows, the scores)
    const size_t n_sets = ((size_t)n_rep + 3) / 4;
    const size_t attn_need = (size_t)n_rep * hd * 4 + n_sets * (hd / 16) * 256 +
                             (size_t)kConsumerWarps * 4 * n_sets * (hd + 2) * 4 + (size_t)hd * 4 + (size_t)n_rep * lc_max * 4;
    if (attn_need > act) act = attn_need;
    act = (act + 127) & ~(size_t)127;
    const uint32_t stage_bytes = h->pl.stage_bytes;
    uint32_t n_stages = cfg->n_stages;
    const size_t avail = (size_t)smem_optin > hdr + act ? (size_t)smem_optin - hdr - act : 0;
    const uint32_t fit = (uint32_t)(avail / stage_bytes);
    if (n_stages == 0) n_stages = fit < (uint32_t)kMaxStages ? fit : (uint32_t)kMaxStages;
    if (n_stages < 2 || n_stages > fit) {
      snprintf(h->errmsg, sizeof(h->errmsg), "shared-memory plan does not fit: need %zu + %u stages of %u, have %d",
               hdr + act, n_stages, stage_bytes, smem_optin);
      status = AMK_ERR_UNSUPPORTED;
      goto fail;
    }
    // default: two copies of 32 KB in flight per block -- enough to saturate HBM from 148 blocks; more only deepens
    // the memory system's queues, which every dependency-carrying load then waits behind (measured: 3 beats 5 by
    // 2-4 %, 2 beats 3 by 0.5-1.3 % on most shapes and ties on the rest); int4 (three 48 KB stages): all three
    uint32_t max_inflight = cfg->max_inflight ? cfg->max_inflight : (cfg->wdtype == AMK_W_INT4 ? 3 : 2);
    if (max_inflight > n_stages) max_inflight = n_stages;
    const size_t smem_bytes = hdr + act + (size_t)n_stages * stage_bytes;
    int per_sm = 0;
    // (both builds of the kernel: the diagnostic one serves tracing, counter joins and the dropped-signal hook)
    AMK_CUDA(decode_kernel_attrs_traced((int)cfg->wdtype, hd, smem_bytes, &per_sm));
    AMK_CUDA(decode_kernel_attrs((int)cfg->wdtype, hd, smem_bytes, &per_sm));
    if (per_sm < 1) {
      snprintf(h->errmsg, sizeof(h->errmsg), "decode kernel does not fit one block per SM");
      status = AMK_ERR_UNSUPPORTED;
      goto fail;
    }

    // ---- workspace: zero it, upload the slice and tile tables and the rotary table ---------------------
    AMK_CUDA(cudaMemsetAsync(h->ws, 0, h->wl.total, stream));
    {
      std::vector<unsigned long long> slices(h->pl.ops.size() * (size_t)n_blocks);
      for (size_t i = 0; i < h->pl.ops.size(); i++)
        memcpy(&slices[i * n_blocks], h->pl.ops[i].slice_off.data(), (size_t)n_blocks * 8);
      AMK_CUDA(cudaMemcpyAsync(h->ws + h->wl.slice_tab, slices.data(), slices.size() * 8, cudaMemcpyHostToDevice, stream));
      std::vector<int> btab(5 * ((size_t)n_blocks + 1));
      for (int k = 0; k < 5; k++) memcpy(&btab[k * ((size_t)n_blocks + 1)], h->pl.bounds[k].data(), ((size_t)n_blocks + 1) * 4);
      AMK_CUDA(cudaMemcpyAsync(h->ws + h->wl.bounds, btab.data(), btab.size() * 4, cudaMemcpyHostToDevice, stream));
      if (!slot_of_smid.empty())
        AMK_CUDA(cudaMemcpyAsync(h->ws + h->wl.smid_tab, slot_of_smid.data(), (size_t)kMaxSmid * 4,
                                 cudaMemcpyHostToDevice, stream));
      AMK_CUDA(cudaMemcpyAsync(h->ws + h->wl.tile_begin, tile_begin.data(), tile_begin.size() * 4,
                               cudaMemcpyHostToDevice, stream));
      AMK_CUDA(cudaMemcpyAsync(h->ws + h->wl.tiles, tiles.data(), tiles.size() * 8, cudaMemcpyHostToDevice, stream));
      // rotary table (cos, sin)[pos][i], angles formed in double
      const int half = hd / 2;
      std::vector<float2> tab((size_t)cfg->max_seq * half);
      for (int i = 0; i < half; i++) {
        const double f = std::pow((double)cfg->rope_theta, -2.0 * (double)i / (double)hd);
        for (uint32_t sp = 0; sp < cfg->max_seq; sp++) {
          const double phi = (double)sp * f;
          tab[(size_t)sp * half + i] = make_float2((float)std::cos(phi), (float)std::sin(phi));
        }
      }
      AMK_CUDA(cudaMemcpyAsync(h->ws + h->wl.rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice,
                               stream));
      AMK_CUDA(cudaStreamSynchronize(stream));     // the host vectors above are pageable memory
    }

    // ---- pack the weights ---------------------------------------------------------------------------------
    for (size_t i = 0; i < h->pl.ops.size(); i++) {
      const PlanOp& op = h->pl.ops[i];
      PackOp d;
      d.s = op.s; d.region_off = op.region_off; d.scale_off = op.scale_off;
      d.bounds = (const int*)(h->ws + h->wl.bounds) + (size_t)op.kind * (n_blocks + 1);
      d.slice_off = (const unsigned long long*)(h->ws + h->wl.slice_tab) + i * (size_t)n_blocks;
      PackSrc s;
      memset(&s, 0, sizeof(s));
      const int l = op.layer;
      auto lin = [&](int slot, int which) {
        s.w[slot] = wts->linear[which][l];
        s.scale[slot] = (cfg->wdtype != AMK_W_BF16) ? wts->scale[which][l] : nullptr;
        s.zero[slot] = (cfg->wdtype == AMK_W_INT4) ? wts->zero[which][l] : nullptr;
        return s.w[slot] && (cfg->wdtype == AMK_W_BF16 || s.scale[slot]) && (cfg->wdtype != AMK_W_INT4 || s.zero[slot]);
      };
      bool okp = true;
      switch (op.kind) {
        case OP_QKV:
          s.mode = 1; s.rows0 = qd; s.rows1 = qd + cfg->n_kv_heads * hd;
          okp = lin(0, AMK_LIN_Q) & lin(1, AMK_LIN_K) & lin(2, AMK_LIN_V);
          break;
        case OP_O: okp = lin(0, AMK_LIN_O); break;
        case OP_GATEUP: s.mode = 2; okp = lin(0, AMK_LIN_GATE) & lin(1, AMK_LIN_UP); break;
        case OP_DOWN: okp = lin(0, AMK_LIN_DOWN); break;
        default:
          if (cfg->quantize_lm_head) {
            s.w[0] = wts->lm_head_q;
            s.scale[0] = wts->lm_head_scale;
            s.zero[0] = wts->lm_head_zero;
          } else {
            s.w[0] = cfg->tied_embeddings ? wts->embed : wts->lm_head;
          }
          break;
      }
      if (!okp) { status = AMK_ERR_INVALID_ARG; goto fail; }
      AMK_CUDA(launch_pack(d, s, h->packed, n_blocks, (int)stage_bytes, false, stream));
    }
    AMK_CUDA(cudaMemcpyAsync(h->packed + h->pl.embed_off, wts->embed, (size_t)cfg->vocab * H * 2,
                             cudaMemcpyDeviceToDevice, stream));
    AMK_CUDA(cudaMemcpyAsync(h->packed + h->pl.final_norm_off, wts->final_norm, (size_t)H * 2,
                             cudaMemcpyDeviceToDevice, stream));
    for (int l = 0; l < L; l++) {
      if (!wts->attn_norm[l] || !wts->mlp_norm[l]) { status = AMK_ERR_INVALID_ARG; goto fail; }
      AMK_CUDA(cudaMemcpyAsync(h->packed + h->pl.attn_norm_off + (size_t)l * H * 2, wts->attn_norm[l], (size_t)H * 2,
                               cudaMemcpyDeviceToDevice, stream));
      AMK_CUDA(cudaMemcpyAsync(h->packed + h->pl.mlp_norm_off + (size_t)l * H * 2, wts->mlp_norm[l], (size_t)H * 2,
                               cudaMemcpyDeviceToDevice, stream));
    }

    // ---- kernel parameters that do not change from step to step ---------------------------------------
    KParams& p = h->base;
    p.H = H; p.L = L; p.nq = cfg->n_q_heads; p.nkv = cfg->n_kv_heads; p.hd = hd; p.I = I; p.V = cfg->vocab;
    p.kv_esz = (cfg->kv_dtype == AMK_KV_FP8_E4M3) ? 1 : 2;
    p.S = cfg->max_seq; p.n_rep = n_rep; p.eps = cfg->rms_eps; p.flags = (int)cfg->flags;
    p.sync_mode = (cfg->sync_mode == 2) ? 0 : 1;      // kernel: 0 = counter joins as well, 1 = sequence numbers only
    for (int k = 0; k < 5; k++) p.shape[k] = h->pl.shape[k];
    p.packed = h->packed;
    p.tiles = (const unsigned long long*)(h->ws + h->wl.tiles);
    p.tile_begin = (const unsigned*)(h->ws + h->wl.tile_begin);
    p.bounds = (const int*)(h->ws + h->wl.bounds);
    p.slot_of_smid = slot_of_smid.empty() ? nullptr : (const int*)(h->ws + h->wl.smid_tab);
    h->split_min = 1.0f; h->split_max = 1.0f;
    for (double w : weights) { if (w < h->split_min) h->split_min = (float)w; if (w > h->split_max) h->split_max = (float)w; }
    p.scale_base = h->pl.scale_base;
    p.scale_layer_stride = (unsigned)h->pl.scale_layer_stride;
    for (int k = 0; k < 4; k++) p.scale_kind_off[k] = (unsigned)h->pl.scale_kind_off[k];
    p.lm_scale_off = h->pl.lm_scale_off;
    p.embed = (const unsigned short*)(h->packed + h->pl.embed_off);
    p.attn_norm = (const unsigned short*)(h->packed + h->pl.attn_norm_off);
    p.mlp_norm = (const unsigned short*)(h->packed + h->pl.mlp_norm_off);
    p.final_norm = (const unsigned short*)(h->packed + h->pl.final_norm_off);
    p.rope = (const float2*)(h->ws + h->wl.rope);
    p.x_a = (ActPair*)(h->ws + h->wl.x_a); p.x_b = (ActPair*)(h->ws + h->wl.x_b);
    p.qkv = (ActPair*)(h->ws + h->wl.qkv); p.o = (ActPair*)(h->ws + h->wl.o); p.m = (ActPair*)(h->ws + h->wl.m);
    p.part = (ActPair*)(h->ws + h->wl.part); p.hidden = (float*)(h->ws + h->wl.hidden);
    p.phase_ctr = (unsigned*)(h->ws + h->wl.phase_ctr); p.group_ctr = (unsigned*)(h->ws + h->wl.group_ctr);
    p.lm_ctr = (unsigned*)(h->ws + h->wl.lm_ctr); p.cand_val = (float*)(h->ws + h->wl.cand_val);
    p.cand_idx = (int*)(h->ws + h->wl.cand_idx); p.next_ws = (int*)(h->ws + h->wl.next_ws);
    p.status = (DevStatus*)(h->ws + h->wl.status);
    p.trace = (cfg->flags & AMK_FLAG_TRACE) ? (unsigned long long*)(h->ws + h->wl.trace) : nullptr;
    p.ktime = (unsigned long long*)(h->ws + h->wl.ktime);
    p.stage_bytes = (int)stage_bytes; p.n_stages = (int)n_stages; p.max_inflight = (int)max_inflight;
    // L2 look-ahead, automatic: two tiles beyond the ring; six where a layer streams so much per block (more than
    // 2 MB: Llama-3-8B bf16) that the step runs at the HBM rate and the deeper look-ahead keeps HBM busier
    // (measured: 2 beats 6 by 0.5-1.6 % on the dependency-bound shapes, 6 beats 2 by 0.7 % on that one)
    {
      const double per_block = (double)(h->pl.weight_stream_bytes) / (L > 0 ? L : 1) / (double)n_blocks;
      const int automatic = (cfg->wdtype == AMK_W_BF16 && per_block > 2.0e6) ? 6 : 2;
      p.l2_ahead = cfg->l2_ahead == 0 ? automatic : (cfg->l2_ahead > 32 ? 0 : (int)cfg->l2_ahead);
    }
    p.act_bytes = (int)act;
    p.timeout_ns = 1000ull * (cfg->wait_timeout_us ? cfg->wait_timeout_us : 200000u);
    p.drop_phase = -1; p.drop_block = -1;

    amk_plan& pn = h->plan;
    pn.n_blocks = n_blocks; pn.threads = kThreads; pn.smem_bytes = (uint32_t)smem_bytes;
    pn.stage_bytes = stage_bytes; pn.n_stages = n_stages; pn.max_inflight = max_inflight;
    pn.l2_ahead = (uint32_t)p.l2_ahead;
    pn.n_gemv_ops = (uint32_t)h->pl.ops.size(); pn.n_phases = 5 * L;
    pn.packed_bytes = h->pl.packed_total; pn.workspace_bytes = h->wl.total; pn.kv_bytes = kv_bytes_of(cfg);
    pn.weight_stream_bytes = h->pl.weight_stream_bytes;
    h->epoch = 0;
    h->ctr_epoch = 0;
  }
  *out = h;
  return AMK_OK;
fail:
  if (getenv("AMK_VERBOSE")) fprintf(stderr, "amk_create: %s: %s\n", amk_status_str(status), h->errmsg);
  delete h;
  return status;
}

// Sequence numbers are 32-bit: step e's task t publishes e * (5 L + 1) + t + 1.  Before that could wrap (after
// 2^32 / (5 L + 1) steps: tens of millions), the activation area is cleared on the step's stream -- everything in
// it then carries sequence number 0, which no task ever waits for -- and the step count starts again.
static bool epoch_would_wrap(const amk_handle* h) {
  const unsigned long long per = 5ull * h->cfg.n_layers + 2ull;
  return ((unsigned long long)h->epoch + 2ull) * per + 2ull > 0xffffffffull;
}

static amk_status launch_step(amk_handle* h, int32_t token, const int* token_ptr, int32_t pos, void* kv, float* logits,
                              int32_t* next_token, cudaStream_t stream) {
  if (epoch_would_wrap(h)) {
    // (stream order puts the clear after every earlier step of this handle and before this one)
    if (cudaMemsetAsync(h->ws + h->wl.x_a, 0, h->wl.hidden - h->wl.x_a, stream) != cudaSuccess) {
      snprintf(h->errmsg, sizeof(h->errmsg), "clearing the activation area at the sequence-number wrap failed");
      return AMK_ERR_CUDA;
    }
    h->epoch = 0;
  }
  KParams p = h->base;
  p.token = token;
  p.token_ptr = token_ptr;
  p.pos = pos;
  p.epoch = ++h->epoch;
  p.ctr_epoch = ++h->ctr_epoch;
  const size_t half = kv_bytes_of(&h->cfg) / 2;
  p.kcache = (unsigned char*)kv;
  p.vcache = (unsigned char*)kv + half;
  p.logits = logits;
  p.next_token = next_token;
  p.drop_phase = h->drop_phase;
  p.drop_block = h->drop_block;
  h->drop_phase = h->drop_block = -1;
  h->last_stream = stream;
  const bool diagnostic = (h->cfg.flags & AMK_FLAG_TRACE) || p.sync_mode == 0 || p.drop_block >= 0;
  cudaError_t e = diagnostic ? launch_decode_traced(p, (int)h->plan.n_blocks, h->plan.smem_bytes, stream)
                             : launch_decode(p, (int)h->plan.n_blocks, h->plan.smem_bytes, stream);
  if (e != cudaSuccess) {
    --h->epoch;
    --h->ctr_epoch;
    snprintf(h->errmsg, sizeof(h->errmsg), "cooperative launch: %s", cudaGetErrorString(e));
    return AMK_ERR_CUDA;
  }
  return AMK_OK;
}

// The kernel reads cache rows with 16-byte bulk copies and writes logits / tokens as 4-byte words.
static bool misaligned(const void* kv, const void* a, const void* b) {
  return ((uintptr_t)kv & 15u) || ((uintptr_t)a & 3u) || ((uintptr_t)b & 3u);
}

amk_status amk_decode_step(amk_handle* h, int32_t token, int32_t pos, void* kv_cache_dev, float* logits_dev,
                           int32_t* next_token_dev, void* cuda_stream) {
  if (!h || !kv_cache_dev) return AMK_ERR_INVALID_ARG;
  if (misaligned(kv_cache_dev, logits_dev, next_token_dev)) return AMK_ERR_INVALID_ARG;
  if (pos < 0 || (uint32_t)pos >= h->cfg.max_seq) return AMK_ERR_BAD_POS;
  if (token < 0 || (uint32_t)token >= h->cfg.vocab) return AMK_ERR_BAD_TOKEN;
  return launch_step(h, token, nullptr, pos, kv_cache_dev, logits_dev, next_token_dev, (cudaStream_t)cuda_stream);
}

amk_status amk_decode_greedy(amk_handle* h, int32_t first_token, int32_t pos0, int32_t n_steps, void* kv_cache_dev,
                             int32_t* tokens_out_dev, float* logits_dev, void* cuda_stream) {
  if (!h || !kv_cache_dev || !tokens_out_dev || n_steps < 1) return AMK_ERR_INVALID_ARG;
  if (misaligned(kv_cache_dev, logits_dev, tokens_out_dev)) return AMK_ERR_INVALID_ARG;
  if (pos0 < 0 || (uint64_t)pos0 + (uint64_t)n_steps > h->cfg.max_seq) return AMK_ERR_BAD_POS;
  if (first_token < 0 || (uint32_t)first_token >= h->cfg.vocab) return AMK_ERR_BAD_TOKEN;
  for (int i = 0; i < n_steps; i++) {
    amk_status st = launch_step(h, first_token, i ? tokens_out_dev + (i - 1) : nullptr, pos0 + i, kv_cache_dev,
                                (i == n_steps - 1) ? logits_dev : nullptr, tokens_out_dev + i, (cudaStream_t)cuda_stream);
    if (st != AMK_OK) return st;
  }
  return AMK_OK;
}

amk_status amk_last_status(amk_handle* h, amk_status* st, char* msg, size_t n) {
  if (!h || !st) return AMK_ERR_INVALID_ARG;
  if (msg && n) msg[0] = 0;
  cudaError_t e = cudaStreamSynchronize(h->last_stream);
  DevStatus ds;
  memset(&ds, 0, sizeof(ds));
  if (e == cudaSuccess) e = cudaMemcpy(&ds, h->ws + h->wl.status, sizeof(ds), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) {
    *st = AMK_ERR_CUDA;
    if (msg && n) snprintf(msg, n, "%s", cudaGetErrorString(e));
    return AMK_ERR_CUDA;
  }
  *st = (amk_status)ds.code;
  if (ds.code == 0 && ds.abort) *st = AMK_ERR_ABORTED;
  if (*st != AMK_OK) {
    if (msg && n)
      snprintf(msg, n, "%s: block %d, %s %d, counter %u of %u", amk_status_str(*st), ds.block,
               ds.phase >= 0 ? "join" : "ring wait", ds.phase, ds.seen, ds.want);
    // the step did not finish: its counters are inconsistent, start over from zero
    e = cudaMemset(h->ws + h->wl.status, 0, sizeof(DevStatus));
    if (e == cudaSuccess) e = cudaMemset(h->ws + h->wl.phase_ctr, 0, h->wl.cand_val - h->wl.phase_ctr);
    // (the activation buffers need no reset: the next step's sequence numbers differ from anything in them)
    if (e != cudaSuccess) return AMK_ERR_CUDA;
    // the counters restart from zero; the sequence numbers keep growing
    h->ctr_epoch = 0;
  }
  return AMK_OK;
}

amk_status amk_plan_info(const amk_handle* h, amk_plan* out) {
  if (!h || !out) return AMK_ERR_INVALID_ARG;
  *out = h->plan;
  return AMK_OK;
}

amk_status amk_debug_hidden(amk_handle* h, float* host_out) {
  if (!h || !host_out) return AMK_ERR_INVALID_ARG;
  if (!(h->cfg.flags & AMK_FLAG_DEBUG_HIDDEN)) return AMK_ERR_INVALID_ARG;
  cudaError_t e = cudaStreamSynchronize(h->last_stream);
  if (e == cudaSuccess)
    e = cudaMemcpy(host_out, h->ws + h->wl.hidden, (size_t)(h->cfg.n_layers + 1) * h->cfg.hidden * 4,
                   cudaMemcpyDeviceToHost);
  return e == cudaSuccess ? AMK_OK : AMK_ERR_CUDA;
}

amk_status amk_debug_trace(amk_handle* h, uint64_t* host_out, size_t n_u64) {
  if (!h || !host_out) return AMK_ERR_INVALID_ARG;
  if (!(h->cfg.flags & AMK_FLAG_TRACE)) return AMK_ERR_INVALID_ARG;
  const size_t need = (size_t)h->plan.n_blocks * (5 * h->cfg.n_layers + 1) * AMK_TRACE_EVENTS;
  if (n_u64 < need) return AMK_ERR_INVALID_ARG;
  cudaError_t e = cudaStreamSynchronize(h->last_stream);
  if (e == cudaSuccess) e = cudaMemcpy(host_out, h->ws + h->wl.trace, need * 8, cudaMemcpyDeviceToHost);
  return e == cudaSuccess ? AMK_OK : AMK_ERR_CUDA;
}

amk_status amk_debug_unpack(amk_handle* h, int layer, int which, void* out_dev, void* scale_dev, void* zero_dev,
                            void* cuda_stream) {
  if (!h || !out_dev) return AMK_ERR_INVALID_ARG;
  const int L = h->cfg.n_layers;
  if (which < 0 || which > AMK_LIN_LM_HEAD) return AMK_ERR_INVALID_ARG;
  if (which != AMK_LIN_LM_HEAD && (layer < 0 || layer >= L)) return AMK_ERR_INVALID_ARG;
  int op, slot = 0, mode = 0;
  switch (which) {
    case AMK_LIN_Q: op = 4 * layer; mode = 1; slot = 0; break;
    case AMK_LIN_K: op = 4 * layer; mode = 1; slot = 1; break;
    case AMK_LIN_V: op = 4 * layer; mode = 1; slot = 2; break;
    case AMK_LIN_O: op = 4 * layer + 1; break;
    case AMK_LIN_GATE: op = 4 * layer + 2; mode = 2; slot = 0; break;
    case AMK_LIN_UP: op = 4 * layer + 2; mode = 2; slot = 1; break;
    case AMK_LIN_DOWN: op = 4 * layer + 3; break;
    default: op = 4 * L; break;
  }
  PackSrc s;
  memset(&s, 0, sizeof(s));
  s.mode = mode;
  s.rows0 = h->cfg.n_q_heads * h->cfg.head_dim;
  s.rows1 = s.rows0 + h->cfg.n_kv_heads * h->cfg.head_dim;
  s.w[slot] = out_dev;
  s.scale[slot] = scale_dev;
  s.zero[slot] = zero_dev;
  const PlanOp& po = h->pl.ops[op];
  PackOp d;
  d.s = po.s; d.region_off = po.region_off; d.scale_off = po.scale_off;
  d.bounds = (const int*)(h->ws + h->wl.bounds) + (size_t)po.kind * (h->plan.n_blocks + 1);
  d.slice_off = (const unsigned long long*)(h->ws + h->wl.slice_tab) + (size_t)op * h->plan.n_blocks;
  cudaError_t e = launch_pack(d, s, h->packed, (int)h->plan.n_blocks, (int)h->plan.stage_bytes, true,
                              (cudaStream_t)cuda_stream);
  return e == cudaSuccess ? AMK_OK : AMK_ERR_CUDA;
}

amk_status amk_debug_drop_signal(amk_handle* h, int phase, int block) {
  if (!h) return AMK_ERR_INVALID_ARG;
  if (block < 0) { h->drop_phase = h->drop_block = -1; return AMK_OK; }
  if (phase < 0 || phase >= 5 * (int)h->cfg.n_layers || block >= (int)h->plan.n_blocks) return AMK_ERR_INVALID_ARG;
  h->drop_phase = phase;
  h->drop_block = block;
  return AMK_OK;
}

amk_status amk_debug_set_step_count(amk_handle* h, uint32_t steps) {
  if (!h) return AMK_ERR_INVALID_ARG;
  // whatever earlier steps left in the activation area could carry the sequence numbers of the steps to come
  if (cudaMemsetAsync(h->ws + h->wl.x_a, 0, h->wl.hidden - h->wl.x_a, h->last_stream) != cudaSuccess) return AMK_ERR_CUDA;
  h->epoch = steps;
  return AMK_OK;
}

amk_status amk_last_kernel_ns(amk_handle* h, uint64_t* ns) {
  if (!h || !ns) return AMK_ERR_INVALID_ARG;
  const int nb = (int)h->plan.n_blocks;
  std::vector<unsigned long long> t((size_t)nb * 2);
  cudaError_t e = cudaStreamSynchronize(h->last_stream);
  if (e == cudaSuccess) e = cudaMemcpy(t.data(), h->ws + h->wl.ktime, t.size() * 8, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return AMK_ERR_CUDA;
  unsigned long long first = ~0ull, last = 0ull;
  for (int b = 0; b < nb; b++) {
    if (t[2 * b] < first) first = t[2 * b];
    if (t[2 * b + 1] > last) last = t[2 * b + 1];
  }
  *ns = (last >= first && first != 0ull) ? (uint64_t)(last - first) : 0u;
  return AMK_OK;
}

amk_status amk_destroy(amk_handle* h) {
  if (!h) return AMK_ERR_INVALID_ARG;
  delete h;
  return AMK_OK;
}

amk_status amk_quantize_int8(const void* w_bf16, int64_t rows, int64_t cols, void* q_out, void* scale_out,
                             void* cuda_stream) {
  if (!w_bf16 || !q_out || !scale_out || rows < 0 || cols <= 0 || rows > 0x7fffffff) return AMK_ERR_INVALID_ARG;
  return launch_quantize_int8(w_bf16, rows, cols, q_out, scale_out, (cudaStream_t)cuda_stream) == cudaSuccess
             ? AMK_OK
             : AMK_ERR_CUDA;
}

amk_status amk_quantize_int8_grouped(const void* w_bf16, int64_t rows, int64_t cols, void* q_out, void* scale_out,
                                     void* cuda_stream) {
  if (!w_bf16 || !q_out || !scale_out || rows < 0 || cols <= 0 || cols % 128) return AMK_ERR_INVALID_ARG;
  return launch_quantize_int8_grouped(w_bf16, rows, cols, q_out, scale_out, (cudaStream_t)cuda_stream) == cudaSuccess
             ? AMK_OK
             : AMK_ERR_CUDA;
}

amk_status amk_quantize_int4(const void* w_bf16, int64_t rows, int64_t cols, void* packed_out, void* scale_out,
                             void* zero_out, void* cuda_stream) {
  if (!w_bf16 || !packed_out || !scale_out || !zero_out || rows < 0 || cols <= 0 || cols % 128)
    return AMK_ERR_INVALID_ARG;
  return launch_quantize_int4(w_bf16, rows, cols, packed_out, scale_out, zero_out, (cudaStream_t)cuda_stream) ==
                 cudaSuccess
             ? AMK_OK
             : AMK_ERR_CUDA;
}

}  // extern "C"

// ====================================================================================================
// Static check of the tables a step runs from (the counterpart of the paper's validate(), Table 2).
// amk_plan_export writes them as one self-describing array of 64-bit words, amk_plan_check verifies such an
// array -- the exported one, or one a test has tampered with -- and amk_create checks its own before upload.
// ====================================================================================================
namespace {

constexpr unsigned long long kPlanMagic = 0x314E414C504B4D41ull;   // "AMKPLAN1"
enum { PH_MAGIC, PH_BLOCKS, PH_LAYERS, PH_OPS, PH_STAGE, PH_WEIGHT_BYTES, PH_TILES, PH_SCHED, PH_WORDS };
constexpr int kOpWords = 8;       // kind, layer, K, rows, unit_rows, wdtype, region_off, region_bytes
constexpr int kSchedWords = 4;    // task kind, buffers read, buffers written, flags
// buffers of the schedule model
enum { B_XA = 1, B_QKV = 2, B_O = 4, B_XB = 8, B_M = 16, B_KVROW = 32, B_OUT = 64, B_MAX = 128, B_PART = 256 };
// flags: every block takes part / the participants together write the whole of each buffer written /
// each participant reads the whole of the buffers in `full_reads` (low 16 bits of word 3 >> 8)
enum { SF_ALL = 1, SF_WRITES_WHOLE = 2 };

struct SchedRow { unsigned kind, reads, writes, flags_fullreads; };
// The per-layer cycle and the head.  `fullreads` = buffers a participant reads entirely (an all-to-all join);
// the other reads are of elements the same block wrote (residual rows) or of another task's slice.
const SchedRow kSchedule[6] = {
    {0, B_XA, B_QKV, SF_ALL | SF_WRITES_WHOLE | (B_XA << 8)},                                   // QKV
    {1, B_QKV | B_PART, B_O | B_KVROW | B_PART, SF_WRITES_WHOLE | (B_PART << 8)},               // attention
    {2, B_O | B_XA, B_XB, SF_ALL | SF_WRITES_WHOLE | (B_O << 8)},                               // O + residual
    {3, B_XB, B_M | B_MAX, SF_ALL | SF_WRITES_WHOLE | (B_XB << 8)},                             // gate/up
    {4, B_M | B_MAX | B_XB, B_XA, SF_ALL | SF_WRITES_WHOLE | ((B_M | B_MAX) << 8)},             // down + residual
    {5, B_XA, B_OUT, SF_ALL | SF_WRITES_WHOLE | (B_XA << 8)},                                   // LM head
};

struct Reject {
  char* msg;
  size_t n;
  amk_status fail(const char* fmt, long long a = 0, long long b = 0, long long c = 0) {
    if (msg && n) snprintf(msg, n, fmt, a, b, c);
    return AMK_ERR_INVALID_ARG;
  }
};

// Schedule model: one step = L cycles of rows 0..4, then row 5.  Checked over enough cycles to cross a
// layer boundary twice.
amk_status check_schedule(const uint64_t* sw, int n_sched, Reject& rj) {
  if (n_sched != 6) return rj.fail("schedule: %lld rows, expected 6", n_sched);
  struct T { unsigned reads, writes, flags, full; };
  std::vector<T> seq;
  const int cycles = 3;
  for (int cyc = 0; cyc <= cycles; cyc++)
    for (int r = 0; r < 6; r++) {
      if ((cyc < cycles) != (r < 5)) continue;
      const uint64_t* w = sw + (size_t)r * kSchedWords;
      if (w[0] != (unsigned long long)r) return rj.fail("schedule: row %lld holds task kind %lld", r, (long long)w[0]);
      seq.push_back(T{(unsigned)w[1], (unsigned)w[2], (unsigned)(w[3] & 0xffu), (unsigned)(w[3] >> 8)});
    }
  const int n = (int)seq.size();
  for (int i = 0; i < n; i++) {
    const T& t = seq[i];
    if (t.full & ~t.reads) return rj.fail("schedule: task %lld reads whole a buffer it does not read", i);
    // wait satisfiability: what a task reads was written earlier in the step (or enters the step from outside:
    // the residual stream from the embedding, cache rows of earlier positions)
    for (unsigned b = 1; b <= B_PART; b <<= 1) {
      if (!(t.reads & b) || b == B_KVROW) continue;
      bool found = (b == B_XA);     // the embedding row
      for (int j = i; j >= 0 && !found; j--) found = (seq[j].writes & b) != 0 && (j < i || b == B_PART);
      if (!found) return rj.fail("schedule: task %lld waits for buffer 0x%llx that nothing before it writes", i, b);
    }
  }
  // output reachability
  if (!(seq[n - 1].writes & B_OUT)) return rj.fail("schedule: no task produces the step's output");
  // Overwrites: before task W overwrites buffer b, every block that read the previous content must be done.
  // after[a][c]: every block of task c starts after every block of task a has finished.  It holds if c reads
  // whole a buffer that a's participants together write (c waits for all of it), and it carries over through
  // program order on either side when the other task runs on at least the same blocks (on all of them, or it
  // is the same task), through chains, and to a task whose every block reads part of what the other wrote.
  std::vector<std::vector<char>> after(n, std::vector<char>(n, 0));
  for (int a = 0; a < n; a++)
    for (int c2 = a + 1; c2 < n; c2++)
      if ((seq[a].flags & SF_WRITES_WHOLE) && (seq[c2].full & seq[a].writes)) after[a][c2] = 1;
  for (bool changed = true; changed;) {
    changed = false;
    for (int a = 0; a < n; a++)
      for (int c2 = a + 1; c2 < n; c2++) {
        if (after[a][c2]) continue;
        bool hold = false;
        for (int m = a; m <= c2 && !hold; m++) {
          // a ..(program order).. m => c2, with m on every block a runs on
          if (m > a && m < c2 && (seq[m].flags & SF_ALL) && after[m][c2]) hold = true;
          // a => m ..(program order).. c2, with m on every block c2 runs on
          if (m > a && m < c2 && (seq[m].flags & SF_ALL) && after[a][m]) hold = true;
          // chains
          if (m > a && m < c2 && after[a][m] && after[m][c2]) hold = true;
          // a => m, and every block of c2 reads something m's blocks wrote last (so each waits for one of them)
          if (m > a && m < c2 && after[a][m]) {
            for (unsigned b = 1; b <= B_PART && !hold; b <<= 1) {
              if (!(seq[m].writes & b) || !(seq[c2].reads & b) || b == B_KVROW) continue;
              bool latest = true;
              for (int j = m + 1; j < c2; j++) latest = latest && !(seq[j].writes & b);
              if (latest) hold = true;
            }
          }
        }
        if (hold) { after[a][c2] = 1; changed = true; }
      }
  }
  for (int w = 0; w < n; w++) {
    for (unsigned b = 1; b <= B_PART; b <<= 1) {
      if (!(seq[w].writes & b) || b == B_KVROW || b == B_OUT) continue;
      int prev = -1;
      for (int j = w - 1; j >= 0; j--)
        if (seq[j].writes & b) { prev = j; break; }
      if (prev < 0) continue;
      for (int r = prev; r < w; r++) {
        if (!(seq[r].reads & b)) continue;
        if (r == prev && b != B_PART) continue;          // (a task does not read what it writes, except the partials)
        if (!after[r][w])
          return rj.fail("schedule: task %lld overwrites buffer 0x%llx while task %lld may still read it", w, b, r);
      }
    }
  }
  return AMK_OK;
}

}  // namespace

namespace {
void plan_to_words(const amk_config* cfg, const Plan& pl, const std::vector<unsigned long long>& tiles,
                   const std::vector<unsigned>& tile_begin, std::vector<uint64_t>& out) {
  const int nb = pl.n_blocks;
  const size_t n_ops = pl.ops.size();
  out.assign(PH_WORDS, 0);
  out[PH_MAGIC] = kPlanMagic; out[PH_BLOCKS] = (uint64_t)nb; out[PH_LAYERS] = cfg->n_layers; out[PH_OPS] = n_ops;
  out[PH_STAGE] = pl.stage_bytes; out[PH_TILES] = tiles.size(); out[PH_SCHED] = 6;
  size_t weight_end = 0;
  for (size_t i = 0; i < n_ops; i++) {
    const PlanOp& op = pl.ops[i];
    size_t bytes = 0;
    for (int s = 0; s < nb; s++)
      bytes += (size_t)slice_bytes(slot_slice(pl.bounds[op.kind].data(), op.s.unit_rows, s).rows, op.s.K, op.s.wdtype,
                                   (int)pl.stage_bytes);
    const uint64_t row[kOpWords] = {(uint64_t)op.kind, (uint64_t)op.layer, (uint64_t)op.s.K, (uint64_t)op.s.rows,
                                    (uint64_t)op.s.unit_rows, (uint64_t)op.s.wdtype, (uint64_t)op.region_off, (uint64_t)bytes};
    out.insert(out.end(), row, row + kOpWords);
    if (op.region_off + bytes > weight_end) weight_end = op.region_off + bytes;
  }
  out[PH_WEIGHT_BYTES] = weight_end;
  for (int k = 0; k < 5; k++)
    for (int s = 0; s <= nb; s++) out.push_back((uint64_t)pl.bounds[k][s]);
  for (int s = 0; s <= nb; s++) out.push_back(tile_begin[s]);
  for (size_t i = 0; i < tiles.size(); i++) out.push_back(tiles[i]);
  for (int r = 0; r < 6; r++) {
    out.push_back(kSchedule[r].kind); out.push_back(kSchedule[r].reads); out.push_back(kSchedule[r].writes);
    out.push_back(kSchedule[r].flags_fullreads);
  }
}
}  // namespace

extern "C" amk_status amk_plan_export(const amk_config* cfg, uint64_t* out, size_t cap_words, size_t* need_words) {
  if (!need_words) return AMK_ERR_INVALID_ARG;
  amk_status st = check_config(cfg);
  if (st != AMK_OK) return st;
  std::vector<unsigned long long> tiles;
  std::vector<unsigned> tile_begin;
  const Plan pl = make_plan(cfg, resolve_blocks(cfg), nullptr, true, &tiles, &tile_begin);
  std::vector<uint64_t> words;
  plan_to_words(cfg, pl, tiles, tile_begin, words);
  *need_words = words.size();
  if (!out) return AMK_OK;
  if (cap_words < words.size()) return AMK_ERR_INVALID_ARG;
  memcpy(out, words.data(), words.size() * 8);
  return AMK_OK;
}

extern "C" amk_status amk_plan_check(const amk_config* cfg, const uint64_t* t, size_t n_words, char* msg,
                                     size_t msg_bytes) {
  Reject rj{msg, msg_bytes};
  if (msg && msg_bytes) msg[0] = 0;
  if (!t) return rj.fail("no tables");
  amk_status st = check_config(cfg);
  if (st != AMK_OK) { rj.fail("configuration rejected"); return st; }
  // ---- well-formedness of the container ------------------------------------------------------------------
  if (n_words < PH_WORDS || t[PH_MAGIC] != kPlanMagic) return rj.fail("not a plan (magic / size)");
  const long long nb = (long long)t[PH_BLOCKS], L = (long long)t[PH_LAYERS], n_ops = (long long)t[PH_OPS];
  const long long stage = (long long)t[PH_STAGE], wbytes = (long long)t[PH_WEIGHT_BYTES], n_tiles = (long long)t[PH_TILES];
  if (nb < 1 || nb > kMaxBlocks) return rj.fail("block count %lld out of range", nb);
  if (cfg->n_blocks && nb != (long long)cfg->n_blocks) return rj.fail("block count %lld differs from the configuration's", nb);
  if (L != (long long)cfg->n_layers || n_ops != 4 * L + 1) return rj.fail("layers %lld / ops %lld do not match the model", L, n_ops);
  if (stage != (long long)stage_bytes_of(cfg)) return rj.fail("stage size %lld differs from the configuration's", stage);
  if (n_tiles < 0 || n_tiles > (1ll << 32)) return rj.fail("tile count out of range");
  const size_t need = PH_WORDS + (size_t)n_ops * kOpWords + 5 * ((size_t)nb + 1) + ((size_t)nb + 1) + (size_t)n_tiles +
                      (size_t)t[PH_SCHED] * kSchedWords;
  if (t[PH_SCHED] > 64 || need != n_words) return rj.fail("array length %lld, sections add up to %lld", (long long)n_words, (long long)need);
  const uint64_t* ops = t + PH_WORDS;
  const uint64_t* bounds = ops + (size_t)n_ops * kOpWords;
  const uint64_t* tbeg = bounds + 5 * ((size_t)nb + 1);
  const uint64_t* tiles = tbeg + (size_t)nb + 1;
  const uint64_t* sched = tiles + (size_t)n_tiles;

  // ---- op table: the model's GEMVs in step order, regions inside the weight area and disjoint -------------
  const int H = cfg->hidden, I = cfg->mlp, V = cfg->vocab, wd = (int)cfg->wdtype;
  const int qd = cfg->n_q_heads * cfg->head_dim, kvd = cfg->n_kv_heads * cfg->head_dim;
  const OpShape want[5] = {{H, qd + 2 * kvd, 1, wd}, {qd, H, 1, wd}, {H, 2 * I, 2, wd}, {I, H, 1, wd},
                           {H, V, 1, cfg->quantize_lm_head ? wd : (int)W_BF16}};
  long long prev_end = 0;
  for (long long i = 0; i < n_ops; i++) {
    const uint64_t* o = ops + (size_t)i * kOpWords;
    const long long kind = (i == n_ops - 1) ? OP_LMHEAD : (i % 4), layer = i / 4;
    if ((long long)o[0] != kind || (long long)o[1] != layer) return rj.fail("op %lld is not the step's op at that place", i);
    const OpShape& s = want[kind];
    if ((long long)o[2] != s.K || (long long)o[3] != s.rows || (long long)o[4] != s.unit_rows || (long long)o[5] != s.wdtype)
      return rj.fail("op %lld: shape or dtype differs from the model's", i);
    const long long off = (long long)o[6], bytes = (long long)o[7];
    if (off < prev_end || (off & 15) || bytes < 0 || off + bytes > wbytes) return rj.fail("op %lld: region [%lld, +%lld) overlaps or leaves the weight area", i, off, bytes);
    prev_end = off + bytes;
  }
  // ---- row bounds: every output row of every GEMV has exactly one producer block --------------------------
  for (int k = 0; k < 5; k++) {
    const uint64_t* b = bounds + (size_t)k * (nb + 1);
    const long long units = want[k].rows / want[k].unit_rows;
    if (b[0] != 0 || (long long)b[nb] != units) return rj.fail("op kind %lld: row bounds do not span [0, %lld]", k, units);
    for (long long s = 0; s < nb; s++)
      if ((long long)b[s + 1] < (long long)b[s]) return rj.fail("op kind %lld: row bounds decrease at block %lld", k, s);
  }
  // ---- per-block queues: exactly the tiles the consumers will wait for, in their order ---------------------
  if (tbeg[0] != 0 || (long long)tbeg[nb] != n_tiles) return rj.fail("tile index does not span the tile list");
  std::vector<int> bnd(nb + 1);
  std::vector<long long> slice_off((size_t)nb);
  for (long long s = 0; s < nb; s++)
    if ((long long)tbeg[s + 1] < (long long)tbeg[s]) return rj.fail("tile index decreases at block %lld", s);
  // offsets of each block's slice inside each op's region follow from the bounds
  std::vector<long long> cursor((size_t)nb);
  for (long long s = 0; s < nb; s++) cursor[s] = (long long)tbeg[s];
  for (long long i = 0; i < n_ops; i++) {
    const uint64_t* o = ops + (size_t)i * kOpWords;
    const int kind = (int)o[0];
    const long long layer = (long long)o[1];
    for (long long s = 0; s <= nb; s++) bnd[s] = (int)bounds[(size_t)kind * (nb + 1) + s];
    long long acc = 0;
    for (long long s = 0; s < nb; s++) {
      slice_off[s] = acc;
      acc += slice_bytes(slot_slice(bnd.data(), want[kind].unit_rows, (int)s).rows, want[kind].K, want[kind].wdtype, (int)stage);
    }
    if (acc != (long long)o[7]) return rj.fail("op %lld: region holds %lld bytes, its slices need %lld", i, (long long)o[7], acc);
    const long long task = (kind == OP_LMHEAD) ? 5 * L : 5 * layer + (kind == OP_QKV ? 0 : kind + 1);
    for (long long s = 0; s < nb; s++) {
      const Slice sl = slot_slice(bnd.data(), want[kind].unit_rows, (int)s);
      long long base = (long long)o[6] + slice_off[s];
      for (int ps = 0; ps < n_passes(sl.rows); ps++) {
        const PassGeom g = pass_geom(pass_rows(sl.rows, ps), want[kind].K, want[kind].wdtype, (int)stage);
        for (int k = 0; k < g.n_tiles; k++) {
          const long long o0 = unit_off(g, k * g.upt), o1 = unit_off(g, (k + 1) * g.upt);
          if (cursor[s] >= (long long)tbeg[s + 1]) return rj.fail("block %lld: queue ends before task %lld's tiles", s, task);
          const uint64_t e = tiles[cursor[s]++];
          const long long eoff = (long long)((e & ((1ull << 40) - 1)) << 4), ebytes = (long long)(((e >> 40) & 0x1fffu) << 4);
          const long long etask = (long long)(e >> 53);
          if (ebytes <= 0 || ebytes > stage) return rj.fail("block %lld: a tile of %lld bytes (stage %lld)", s, ebytes, stage);
          if (eoff + ebytes > wbytes) return rj.fail("block %lld: tile [%lld, +%lld) leaves the weight area", s, eoff, ebytes);
          if (etask != task) return rj.fail("block %lld: tile of task %lld where task %lld is walked", s, etask, task);
          if (eoff != base + o0 || ebytes != o1 - o0)
            return rj.fail("block %lld task %lld: tile is not the one the consumers wait for", s, task);
        }
        base += pass_bytes(g);
      }
      if (kind == OP_QKV) {       // the attention task's marker
        if (cursor[s] >= (long long)tbeg[s + 1]) return rj.fail("block %lld: queue ends before layer %lld's attention marker", s, layer);
        const uint64_t e = tiles[cursor[s]++];
        if (((e >> 40) & 0x1fffu) != 0 || (long long)(e >> 53) != 5 * layer + 1)
          return rj.fail("block %lld: layer %lld's attention marker is missing or misplaced", s, layer);
      }
    }
  }
  for (long long s = 0; s < nb; s++)
    if (cursor[s] != (long long)tbeg[s + 1]) return rj.fail("block %lld: %lld tiles nobody waits for", s, (long long)tbeg[s + 1] - cursor[s]);
  // ---- the dependency model of a step ------------------------------------------------------------------------
  return check_schedule(sched, (int)t[PH_SCHED], rj);
}
