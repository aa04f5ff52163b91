// Structures shared by the host side of the library and the decode kernel (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "amk_layout.h"

namespace amk {

// Device status block: the first error wins; `abort` makes every other wait give up.
struct DevStatus {
  unsigned abort;     // nonzero: leave as soon as possible
  unsigned code;      // amk_status of the first failure
  int phase;          // task whose input never arrived / join that timed out (-1, -2: ring waits)
  int block;          // block that reported
  unsigned seen;      // value seen
  unsigned want;      // value waited for
  unsigned pad[2];
};

// Fixed shared-memory header in front of the activation area and the ring.
constexpr int kMaxSmid = 4096;

struct SmemHeader {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  float red[2][kPassRows];           // cross-k-warp partial sums of a pass: [Wk][R], Wk * R <= warps * kGMax
  float warp_part[2][kConsumerWarps];  // block reductions (sum of squares, max)
  float cand_val[kConsumerWarps];
  int cand_idx[kConsumerWarps];
  int flag;                          // "this block arrived last" broadcast
  int slot;                          // this block's slot (its share of every op, its tile list)
  int slice_row0[5], slice_rows[5];  // its rows of each op kind
  int attn_lc, attn_c;               // this step's split-K plan of the attention: chunk length, chunks per kv group
  int pad[1];
  // Pass geometry of each op kind for this block's slice, worked out once at kernel start (it takes a dozen
  // integer divisions, which would otherwise sit on every task's critical path): [kind][0] a full pass of
  // kPassRows rows (used when the slice has more than one pass), [kind][1] the last pass.
  PassGeom geom[5][2];
  int step_b[5][2], step_r[5][2];                    // tile-to-tile step of the unit walk: upt / Wr, upt % Wr
  unsigned char wr_of[5][2][kConsumerWarps + 1];     // warp -> row-warp index, k-warp index
  unsigned char wk_of[5][2][kConsumerWarps + 1];
};

// An activation element in global memory: the value and the sequence number of the task that wrote it.
// One aligned 8-byte store publishes both, so a reader that sees the expected sequence number has the
// value: no fence and no separate flag are needed.
struct __align__(8) ActPair {
  float v;
  unsigned seq;
};

// Kernel argument, passed by value.
struct KParams {
  // model
  int H, L, nq, nkv, hd, I, V, S, n_rep;
  float eps;
  int flags;
  int sync_mode;                          // 0: counter joins (acquire/release) as well; 1: data-carried sequence numbers only
  OpShape shape[5];                       // per OpKind
  // weights
  const unsigned char* packed;            // packed buffer base
  const unsigned long long* tiles;        // per block: its ring tiles {offset/16 | bytes/16 << 40}, in stream order
  const unsigned* tile_begin;             // [n_blocks + 1] index of each slot's first tile
  const int* bounds;                      // [5][n_blocks + 1] unit boundaries of the slots, per op kind
  const int* slot_of_smid;                // [kMaxSmid] slot of the block running on each SM, or null: slot = blockIdx
  unsigned long long scale_base;          // int8: fp16 row scales, op-major in virtual row order
  unsigned scale_layer_stride;            // bytes per layer
  unsigned scale_kind_off[4];             // byte offset of each op kind inside a layer's scales
  unsigned long long lm_scale_off;        // int8 LM head (quantize_lm_head): its fp16 row scales
  const unsigned short* embed;            // bf16 [V][H], canonical copy
  const unsigned short* attn_norm;        // bf16 [L][H]
  const unsigned short* mlp_norm;         // bf16 [L][H]
  const unsigned short* final_norm;       // bf16 [H]
  const float2* rope;                     // [S][hd/2] (cos, sin)
  // per step
  int token;
  const int* token_ptr;                   // if non-null the token is read from device memory
  int pos;
  unsigned epoch;                         // steps since the activation area was last cleared (the host clears it
                                          // before the 32-bit sequence numbers could wrap)
  unsigned ctr_epoch;                     // steps since the counters were last zeroed
  // caller buffers
  unsigned char* kcache;                  // K cache [L][n_kv][S][hd] of kv_esz-byte elements (2: bf16, 1: fp8 e4m3)
  unsigned char* vcache;
  int kv_esz;
  float* logits;
  int* next_token;
  // workspace
  ActPair* x_a;                           // residual stream entering a layer
  ActPair* x_b;                           // residual stream after attention
  ActPair* qkv;
  ActPair* o;
  ActPair* m;
  ActPair* part;                          // [nq][kMaxChunks][hd + 2]: a chunk's max, sum, unnormalised output
  float* hidden;                          // [(L+1)][H]
  unsigned* phase_ctr;                    // [5 L]
  unsigned* group_ctr;                    // [L][nkv]
  unsigned* lm_ctr;
  float* cand_val;                        // [n_blocks]
  int* cand_idx;
  int* next_ws;
  DevStatus* status;
  unsigned long long* trace;              // [n_blocks][5 L + 1][8] or null
  unsigned long long* ktime;              // [n_blocks][2]: global-timer stamps of each block's first and last instruction
  // plan
  int stage_bytes, n_stages, max_inflight;
  int l2_ahead;                           // ring tiles requested into L2 ahead of the ring (0..32)
  int act_bytes;                          // activation / attention scratch area in shared memory
  unsigned long long timeout_ns;
  int drop_phase, drop_block;             // test hook: this block does not publish this task's output
};

// Launchers implemented in the .cu files.
// (two builds of the decode kernel: without and with the trace stamps compiled in)
cudaError_t launch_decode(const KParams& p, int n_blocks, size_t smem_bytes, cudaStream_t stream);
cudaError_t decode_kernel_attrs(int wdtype, int hd, size_t smem_bytes, int* max_blocks_per_sm);
cudaError_t launch_decode_traced(const KParams& p, int n_blocks, size_t smem_bytes, cudaStream_t stream);
cudaError_t decode_kernel_attrs_traced(int wdtype, int hd, size_t smem_bytes, int* max_blocks_per_sm);

// One op to pack: its shape, rotation and region, plus where the canonical rows come from.
struct PackOp {
  OpShape s;
  const int* bounds;                      // DEVICE [n_blocks + 1]: unit boundaries of the slots for this op kind
  unsigned long long region_off;          // byte offset of the op's region in the packed buffer
  const unsigned long long* slice_off;    // DEVICE [n_blocks]: byte offset of each slot's slice inside the region
  unsigned long long scale_off;           // int8: byte offset of the fp16 row scales (virtual row order)
};
struct PackSrc {
  const void* w[3];
  const void* scale[3];
  const void* zero[3];
  int mode;        // 0 single matrix, 1 three matrices stacked (rows0, rows1 boundaries), 2 two matrices interleaved
  int rows0, rows1;
};
cudaError_t launch_pack(const PackOp& d, const PackSrc& src, unsigned char* packed, int n_blocks, int stage_bytes,
                        bool inverse, cudaStream_t stream);
// Streams `bytes_per_block` per block (one block per SM) and reports each block's SM id and time in ns.
cudaError_t launch_calibrate(const unsigned char* src, size_t bytes_per_block, int n_blocks, size_t smem_bytes,
                             unsigned* smid_out, unsigned long long* ns_out, cudaStream_t stream);
cudaError_t launch_quantize_int8(const void* w, int64_t rows, int64_t cols, void* q, void* scale, cudaStream_t s);
cudaError_t launch_quantize_int8_grouped(const void* w, int64_t rows, int64_t cols, void* q, void* scale, cudaStream_t s);
cudaError_t launch_quantize_int4(const void* w, int64_t rows, int64_t cols, void* packed, void* scale, void* zero,
                                 cudaStream_t s);

}  // namespace amk
