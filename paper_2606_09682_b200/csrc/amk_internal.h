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
  int phase;          // dependency join that timed out (-1: ring wait)
  int block;          // block that reported
  unsigned seen;      // counter value seen
  unsigned want;      // counter value waited for
  unsigned pad[2];
};

// Fixed shared-memory header in front of the activation area and the ring.
struct SmemHeader {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  float red[2][kPassRows];           // cross-k-warp partial sums of a pass (double-buffered)
  float warp_part[kConsumerWarps];   // block reductions (sum of squares)
  float cand_val[kConsumerWarps];
  int cand_idx[kConsumerWarps];
  volatile int abort;                // block-local copy of the abort decision
  int flag;                          // "this block arrived last" broadcast
  int pad[2];
};

// Kernel argument, passed by value.
struct KParams {
  // model
  int H, L, nq, nkv, hd, I, V, S, n_rep;
  float eps;
  int flags;
  // tables and weights
  const OpDesc* ops;
  int n_ops;
  const unsigned char* packed;            // packed buffer base
  const unsigned short* embed;            // bf16 [V][H], canonical copy
  const unsigned short* attn_norm;        // bf16 [L][H]
  const unsigned short* mlp_norm;         // bf16 [L][H]
  const unsigned short* final_norm;       // bf16 [H]
  const float2* rope;                     // [S][hd/2] (cos, sin)
  // per step
  int token;
  const int* token_ptr;                   // if non-null the token is read from device memory
  int pos;
  unsigned epoch;                         // counters of this step count up to epoch * n_blocks
  // caller buffers
  unsigned short* kcache;
  unsigned short* vcache;
  float* logits;
  int* next_token;
  // workspace
  float* x_a;
  float* x_b;
  float* qkv;
  float* o;
  float* m;
  float* part;                            // [nq][kMaxChunks][hd + 2]
  float* hidden;                          // [(L+1)][H]
  unsigned* phase_ctr;                    // [5 L]
  unsigned* group_ctr;                    // [nkv]
  unsigned* lm_ctr;
  float* cand_val;                        // [n_blocks]
  int* cand_idx;
  int* next_ws;
  DevStatus* status;
  unsigned long long* trace;              // [n_blocks][5 L + 1][8] or null
  // plan
  int stage_bytes, n_stages, max_inflight;
  int act_bytes;                          // activation / attention scratch area in shared memory
  unsigned long long timeout_ns;
  int drop_phase, drop_block;             // test hook: this block skips this signal
};

// Launchers implemented in the .cu files.
cudaError_t launch_decode(const KParams& p, int n_blocks, size_t smem_bytes, cudaStream_t stream);
cudaError_t decode_kernel_attrs(size_t smem_bytes, int* max_blocks_per_sm);

struct PackSrc {
  const void* w[3];
  const void* scale[3];
  const void* zero[3];
  int mode;        // 0 single matrix, 1 three matrices stacked (rows0, rows1 boundaries), 2 two matrices interleaved
  int rows0, rows1;
};
cudaError_t launch_pack(const OpDesc& d, const PackSrc& src, unsigned char* packed, int n_blocks, int stage_bytes,
                        bool inverse, cudaStream_t stream);
cudaError_t launch_quantize_int8(const void* w, int64_t rows, int64_t cols, void* q, void* scale, cudaStream_t s);
cudaError_t launch_quantize_int4(const void* w, int64_t rows, int64_t cols, void* packed, void* scale, void* zero,
                                 cudaStream_t s);

}  // namespace amk
