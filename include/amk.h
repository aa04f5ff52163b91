/*
 * amk.h -- C ABI of the B200 single-kernel Llama decode library.
 *
 * What the library does (the paper's statement of the problem, Sections 1, 3 and 4): the weights of a
 * bias-free, full-rotary, SiLU-SwiGLU, RMSNorm, grouped-query-attention Llama-family decoder are laid
 * out once; afterwards ONE launch of one persistent cooperative kernel is one forward pass is one
 * decoded token (batch 1), with the KV cache persisting in device memory between launches.  Weight-only
 * int8 and int4 variants fold the dequantisation into the matrix-vector products while embeddings,
 * scales and every non-GEMV buffer keep their 16-bit types (Section 5, "Quantized generation").
 *
 * Conventions for every entry point
 *   - Plain C, no exceptions, no aborts: every call returns an amk_status.
 *   - Pointers are tagged HOST or DEVICE in the comments.  The library never allocates or frees device
 *     memory: the caller owns the canonical weights, the packed buffer, the workspace, the KV cache and
 *     the outputs.  (The handle and a few small host tables are the only allocations.)
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - One handle is used from one stream at a time; several handles may coexist.
 *   - Same inputs give bit-identical outputs (no floating-point atomics, fixed reduction orders).
 */
#ifndef AMK_H
#define AMK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AMK_ABI_VERSION 3u

typedef enum {
  AMK_OK = 0,
  AMK_ERR_INVALID_ARG = 1, /* NULL pointer, bad struct_size / abi_version, buffer too small            */
  AMK_ERR_UNSUPPORTED = 2, /* a shape or option the kernel's plan cannot serve                          */
  AMK_ERR_CUDA = 3,        /* a CUDA runtime call failed (amk_last_status gives the text)               */
  AMK_ERR_OOM = 4,         /* host allocation failed                                                    */
  AMK_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (read through amk_last_status)         */
  AMK_ERR_ABORTED = 6,     /* the kernel left early because another block reported an error             */
  AMK_ERR_BAD_POS = 7,     /* pos < 0 or pos >= max_seq                                                 */
  AMK_ERR_BAD_TOKEN = 8    /* token < 0 or token >= vocab                                               */
} amk_status;

typedef enum { AMK_W_BF16 = 0, AMK_W_INT8 = 1, AMK_W_INT4 = 2, AMK_W_INT8_GROUPED = 3 } amk_wdtype;
/* element type of the KV cache: bf16 (what the paper's kernels keep, Section 5), or fp8 e4m3 (a variant: the
 * appended rows are rounded to nearest even, saturating at +-448, and attention reads the 8-bit entries) */
typedef enum { AMK_KV_BF16 = 0, AMK_KV_FP8_E4M3 = 1 } amk_kvdtype;

/* amk_config.flags */
#define AMK_FLAG_DEBUG_HIDDEN 1u /* keep the residual stream after the embedding and after every layer */
#define AMK_FLAG_TRACE 2u        /* every block stamps the global timer at the stages of every task          */
#define AMK_FLAG_TRACE_CYCLES 8u /* with AMK_FLAG_TRACE: stamps are the SM's cycle counter, not the global timer (whose
                                    resolution is a quarter microsecond): only differences within one block mean anything */
#define AMK_FLAG_MEASURED_SPLIT 4u /* amk_create measures the HBM rate each SM gets and gives each block a share
                                      of every op in proportion (blocks are then identified by SM id).  Off by
                                      default: on B200 it measured no faster than equal shares.             */

/* Trace layout (amk_debug_trace): uint64 nanosecond stamps [n_blocks][n_tasks][AMK_TRACE_EVENTS], where
 * task 5*l+{0,1,2,3,4} = QKV, attention, O, gate/up, down of layer l and task 5*L = LM head. */
#define AMK_TRACE_EVENTS 12
enum { AMK_TR_ENTER = 0,      /* consumer warps reach the task                                          */
       AMK_TR_JOINED = 1,     /* the dependency wait is over                                            */
       AMK_TR_LOADED = 2,     /* input vector in shared memory (GEMV tasks)                             */
       AMK_TR_COMPUTED = 3,   /* last output stored                                                     */
       AMK_TR_SIGNALLED = 4,  /* counter incremented                                                    */
       AMK_TR_PROD_FIRST = 5, /* producer issued the task's first ring tile (GEMV tasks)                */
       AMK_TR_PROD_LAST = 6,  /* producer issued the task's last ring tile                              */
       AMK_TR_REDUCED = 7,    /* last pass: per-row partial sums are in shared memory                   */
       AMK_TR_PASS_BEGIN = 8, /* last pass: epilogue operands requested, tile walk starts               */
       AMK_TR_FIRST_TILE = 9, /* last pass: its first ring tile has landed                              */
       AMK_TR_TILES_DONE = 10,/* last pass: all ring tiles multiplied                                   */
       /* attention tasks over several positions use 8 = scores done, 9 = softmax done, 10 = P V done (partial
          published), 7 = all chunks' partials gathered */
       AMK_TR_POLLS = 11      /* NOT a time: requests thread 0 made for its first batch of input lines   */
};

/* The seven per-layer linears, in the order used by amk_weights.linear[] and amk_debug_unpack. */
enum { AMK_LIN_Q = 0, AMK_LIN_K = 1, AMK_LIN_V = 2, AMK_LIN_O = 3, AMK_LIN_GATE = 4, AMK_LIN_UP = 5,
       AMK_LIN_DOWN = 6, AMK_LIN_COUNT = 7, AMK_LIN_LM_HEAD = 7 };

/* Model and plan description.  POD; the Python mirror is checked against sizeof/offsetof. */
typedef struct amk_config {
  uint32_t struct_size;      /* = sizeof(amk_config)                                                   */
  uint32_t abi_version;      /* = AMK_ABI_VERSION                                                      */
  uint32_t hidden;           /* H; multiple of 64 (128 for int4); at most 5632: a normed input vector is
                                gathered in one batch of 16 elements per consumer thread               */
  uint32_t n_layers;         /* L; at most 409 (a task id is kept in 11 bits)                          */
  uint32_t n_q_heads;        /* multiple of n_kv_heads; n_q_heads / n_kv_heads <= 16                   */
  uint32_t n_kv_heads;
  uint32_t head_dim;         /* 64 or 128                                                              */
  uint32_t mlp;              /* I; multiple of 64 (128 for int4)                                       */
  uint32_t vocab;            /* V                                                                      */
  uint32_t max_seq;          /* S: positions the KV cache holds                                        */
  uint32_t tied_embeddings;  /* 1: the LM head is the embedding matrix                                 */
  float rms_eps;             /* RMSNorm epsilon (inside the square root)                               */
  float rope_theta;          /* rotary base; pairs (i, i + head_dim/2), no scaling                     */
  uint32_t wdtype;           /* amk_wdtype of the seven per-layer linears                              */
  uint32_t group_size;       /* int4, grouped int8: 128 (the only supported value); ignored otherwise  */
  uint32_t quantize_lm_head; /* 0: the LM head stays bf16 (tied or not), as the paper says of the tied
                                embedding matrix.  1 (int8 / int4 models only): the LM head GEMV streams a
                                copy quantised like the layers (amk_weights.lm_head_q ...); the embedding
                                gather still reads the bf16 matrix                                     */
  uint32_t wait_timeout_us;  /* bound on every device-side wait; 0 = 200000                            */
  uint32_t flags;            /* AMK_FLAG_*                                                             */
  /* tuning knobs, 0 = automatic */
  uint32_t stage_bytes;      /* bytes per shared-memory ring stage (multiple of 1024)                  */
  uint32_t n_stages;         /* ring depth                                                             */
  uint32_t max_inflight;     /* bulk copies a block keeps in flight (<= n_stages; 0 = default 2)        */
  uint32_t sync_mode;        /* 0 = automatic = 1.  1: activations carry sequence numbers, nothing else orders
                                the tasks (no counters, no fences): the mode every published figure uses.
                                2: as 1, AND every task ends with a release-increment that the next task's
                                readers acquire-spin on (the paper's counter model, Section 4), kept so
                                that its cost can be measured.  Same results in both.                    */
  uint32_t n_blocks;         /* persistent blocks; 0 = one per SM of the current device (148 if there is
                                no device).  The packed layout depends on it.                          */
  uint32_t l2_ahead;         /* ring tiles the producer requests into L2 beyond the ring (weight prefetch
                                hint, as in the paper's Algorithm 1); 0 = automatic, 33 = off, max 32    */
  uint32_t kv_dtype;         /* amk_kvdtype of the KV cache; the cache is K then V, each
                                [L][n_kv][max_seq][head_dim] of that type                                */
} amk_config;

/*
 * Canonical (unpacked) weights: every data pointer is a DEVICE pointer to a row-major [out][in] array;
 * the per-layer arrays are HOST arrays of n_layers device pointers.  They are read only inside
 * amk_create and may be freed once the stream passed to amk_create has been synchronised.
 *   bf16 : bf16 [out][in]
 *   int8 : int8 [out][in]; scale fp16 [out]                       w = scale * q, q in [-127, 127]
 *   int4 : uint8 [out][in/2], element j in byte j/2 (even j: bits 0-3); scale fp16 [out][in/128];
 *          zero fp16 [out][in/128] holding an integer 0..15        w = scale * (q - zero)
 *   grouped int8 : int8 [out][in]; scale fp16 [out][in/128]       w = scale * q, q in [-127, 127]
 *          (the paper's ring variant dequantises "per group", Section 7; the group length is the int4 one)
 */
typedef struct amk_weights {
  const void* embed;                        /* bf16 [V][H]                                            */
  const void* lm_head;                      /* bf16 [V][H]; NULL when tied_embeddings                 */
  const void* final_norm;                   /* bf16 [H]                                               */
  const void* const* attn_norm;             /* [L] -> bf16 [H]                                        */
  const void* const* mlp_norm;              /* [L] -> bf16 [H]                                        */
  const void* const* linear[AMK_LIN_COUNT]; /* [L] each: q, k, v, o, gate, up, down                   */
  const void* const* scale[AMK_LIN_COUNT];  /* [L] each; NULL arrays for bf16                         */
  const void* const* zero[AMK_LIN_COUNT];   /* [L] each; int4 only                                    */
  /* quantize_lm_head = 1 only: the LM head matrix (the embedding matrix when tied) quantised like a layer
   * linear of [V][H]: codes, fp16 scales (int8 [V]; int4 and grouped int8 [V][H/128]) and, for int4, fp16 zero
   * points */
  const void* lm_head_q;
  const void* lm_head_scale;
  const void* lm_head_zero;
} amk_weights;

typedef struct amk_handle amk_handle;

/* What the plan looks like; filled by amk_plan_info. */
typedef struct amk_plan {
  uint32_t n_blocks;          /* thread blocks = SMs used (one persistent block per SM)                */
  uint32_t threads;           /* threads per block (one producer warp + consumer warps)                */
  uint32_t smem_bytes;        /* dynamic shared memory per block                                       */
  uint32_t stage_bytes, n_stages, max_inflight;
  uint32_t l2_ahead;          /* ring tiles requested into L2 ahead of the ring                        */
  uint32_t n_gemv_ops;        /* 4 per layer + LM head                                                 */
  uint32_t n_phases;          /* dependency joins per token                                            */
  uint64_t packed_bytes, workspace_bytes, kv_bytes;
  uint64_t weight_stream_bytes; /* packed weight + scale bytes each token streams                      */
} amk_plan;

const char* amk_status_str(amk_status s);

/* Sizes of the three caller-owned device buffers for a configuration.  HOST pointers.
 * Errors: INVALID_ARG (NULL, bad struct_size/abi_version), UNSUPPORTED (shape). */
amk_status amk_packed_bytes(const amk_config* cfg, size_t* bytes);
amk_status amk_workspace_bytes(const amk_config* cfg, size_t* bytes);
amk_status amk_kv_bytes(const amk_config* cfg, size_t* bytes); /* K and V together */

/*
 * Build a decoder: validates the configuration, lays the weights out for streaming (the "weight
 * packer": each block's tiles of each matrix-vector product become one contiguous byte run, column
 * order permuted for conflict-free shared-memory reads, int4 scales and zero points interleaved with
 * their codes), builds the per-op tables and the rotary table in the workspace, all on `cuda_stream`.
 *   cfg, weights            HOST structs (weights' data pointers are DEVICE pointers)
 *   packed_dev / workspace_dev   DEVICE, caller-owned, at least amk_packed_bytes / amk_workspace_bytes,
 *                           256-byte aligned; must outlive the handle; the library fills them
 *   out                     HOST: receives the handle
 * The device must be a compute-capability-10.0 GPU that supports cooperative launch with one block per
 * SM at the plan's shared-memory size; otherwise UNSUPPORTED.  Asynchronous on the stream apart from
 * small synchronous table uploads.
 */
amk_status amk_create(const amk_config* cfg, const amk_weights* weights, void* packed_dev, size_t packed_bytes,
                      void* workspace_dev, size_t workspace_bytes, void* cuda_stream, amk_handle** out);

/*
 * One decode step (Algorithm 1 of the paper: every block walks its queue -- wait, dispatch, signal --
 * inside one cooperative launch): embedding of `token`, L decoder layers at position `pos`, final norm,
 * LM head, greedy token.
 *   kv_cache_dev   DEVICE, caller-owned, amk_kv_bytes: K then V, each [L][n_kv_heads][max_seq][head_dim]
 *                  of cfg.kv_dtype (bf16, or fp8 e4m3 bytes), 16-byte aligned (rows are fetched with 16-byte
 *                  bulk copies).  Entries [0, pos) must be valid; the step writes slot `pos` of every layer
 *                  (K after the rotation, round-to-nearest-even; fp8 saturates at +-448) and reads [0, pos].
 *   logits_dev     DEVICE float[vocab], 4-byte aligned, may be NULL
 *   next_token_dev DEVICE int32[1], 4-byte aligned, may be NULL; lowest index wins an exact tie
 * Asynchronous: returns after the launch.  Synchronous errors: INVALID_ARG (NULL handle or cache, misaligned
 * pointer), BAD_POS, BAD_TOKEN, CUDA.
 * A device-side failure (expired wait) is reported by amk_last_status after the stream has been
 * synchronised; outputs of that step are then undefined, and the next step is legal.
 */
amk_status amk_decode_step(amk_handle* h, int32_t token, int32_t pos, void* kv_cache_dev, float* logits_dev,
                           int32_t* next_token_dev, void* cuda_stream);

/*
 * `n_steps` greedy decode steps with the token fed back on the device (no host round trip between
 * steps): step i decodes position pos0 + i; its input is `first_token` for i = 0 and the previous
 * step's greedy token afterwards.  Goes beyond the paper, which stops at one launch per token and
 * measures the host dispatch between launches separately (Section 5, "Methodology").
 *   tokens_out_dev DEVICE int32[n_steps]: the greedy token of every step
 *   logits_dev     DEVICE float[vocab] or NULL: logits of the LAST step
 * Errors as amk_decode_step; BAD_POS if pos0 + n_steps > max_seq.
 */
amk_status amk_decode_greedy(amk_handle* h, int32_t first_token, int32_t pos0, int32_t n_steps, void* kv_cache_dev,
                             int32_t* tokens_out_dev, float* logits_dev, void* cuda_stream);

/* Synchronises the handle's last stream and reports the device status word of the last step.
 *   st   HOST out: AMK_OK, AMK_ERR_TIMEOUT, ...      msg  HOST out, n bytes, may be NULL. */
amk_status amk_last_status(amk_handle* h, amk_status* st, char* msg, size_t n);

amk_status amk_plan_info(const amk_handle* h, amk_plan* out); /* HOST out */

/* With AMK_FLAG_DEBUG_HIDDEN: copies the residual stream of the last step to HOST memory,
 * float[(L+1)][H]: row 0 after the embedding, row l+1 after layer l.  Synchronises. */
amk_status amk_debug_hidden(amk_handle* h, float* host_out);

/* With AMK_FLAG_TRACE: copies the last step's stamps to HOST memory, n_u64 >= n_blocks * (5 L + 1) *
 * AMK_TRACE_EVENTS.  Synchronises.  This is how the time spent in cross-SM synchronisation is measured. */
amk_status amk_debug_trace(amk_handle* h, uint64_t* host_out, size_t n_u64);

/* Inverse of the packer, for bit-exact layout checks: rebuilds one canonical matrix from the packed
 * buffer into DEVICE memory of the canonical size.  which = AMK_LIN_* (AMK_LIN_LM_HEAD ignores layer).
 *   out_dev    codes / bf16 in the canonical layout
 *   scale_dev  fp16 scales in the canonical layout (int8 / int4), may be NULL
 *   zero_dev   fp16 zero points (int4), may be NULL */
amk_status amk_debug_unpack(amk_handle* h, int layer, int which, void* out_dev, void* scale_dev, void* zero_dev,
                            void* cuda_stream);

/* Test hook for the bounded-wait path: the next step's block `block` skips its signal of dependency
 * join `phase`, so every waiter runs into the time limit and the step ends with AMK_ERR_TIMEOUT
 * (nothing traps or hangs).  block < 0 clears the hook. */
amk_status amk_debug_drop_signal(amk_handle* h, int phase, int block);

/* Kernel-only time of the handle's last step, apart from the launch (the paper's methodology keeps kernel-only
 * and whole-decode figures apart, Section 5): every block stamps the global nanosecond timer when its first
 * thread starts and when its last consumer warp has finished; *ns = latest end - earliest start over all blocks
 * (resolution of that timer: about a quarter of a microsecond).  HOST out.  Synchronises the step's stream. */
amk_status amk_last_kernel_ns(amk_handle* h, uint64_t* ns);

/* Test hook for the 32-bit sequence numbers: sets the handle's count of steps launched since its activation
 * area was last cleared.  Every published activation carries step_count * (5 L + 1) + task + 1; shortly before
 * that would wrap, a step first clears the activation area on its stream and restarts the count (a handle can
 * decode for ever).  Setting the count close to 2^32 / (5 L + 1) lets a test cross that point.  The hook also
 * clears the activation area (on the handle's last stream), since a count set by hand could otherwise meet its
 * own sequence numbers from earlier steps. */
amk_status amk_debug_set_step_count(amk_handle* h, uint32_t steps);

/* Frees host state only.  The caller's buffers are untouched. */
amk_status amk_destroy(amk_handle* h);

/*
 * Round-to-nearest weight quantisers on the device (the paper's "naive round-to-nearest", Section 5),
 * bit-identical to their definition in IEEE fp32 arithmetic:
 *   int8: s = fp16(max|w| / 127) per output row (1 if the row is zero); q = clamp(rint(w / s), -127, 127)
 *   int4: per row and group of 128 columns, mn = min(w, 0), mx = max(w, 0); s = fp16((mx - mn) / 15)
 *         (1 if mx == mn); z = clamp(rint(-mn / s), 0, 15); q = clamp(rint(w / s) + z, 0, 15);
 *         two codes per byte, even column in the low nibble; z stored as an fp16 integer.
 *   grouped int8: the int8 rule per row and group of 128 columns; scale_out is fp16 [rows][cols/128].
 * All pointers DEVICE; w_bf16 is [rows][cols] bf16.  cols % 128 == 0 for int4 and grouped int8.  Asynchronous.
 */
amk_status amk_quantize_int8(const void* w_bf16, int64_t rows, int64_t cols, void* q_out, void* scale_out,
                             void* cuda_stream);
amk_status amk_quantize_int8_grouped(const void* w_bf16, int64_t rows, int64_t cols, void* q_out, void* scale_out,
                                     void* cuda_stream);
amk_status amk_quantize_int4(const void* w_bf16, int64_t rows, int64_t cols, void* packed_out, void* scale_out,
                             void* zero_out, void* cuda_stream);

/*
 * Static check of the tables a decode step runs from -- the counterpart of the paper's validate() (Section 4,
 * "The invariants validate() proves", Table 2), for this kernel's tables: the per-block queues of ring tiles,
 * the row bounds that say which block produces which output rows, and the dependency model of a step.
 * amk_plan_export writes them as one array of 64-bit words (HOST memory; call with out = NULL to learn the
 * size); amk_plan_check accepts such an array or rejects it with the reason in msg.  amk_create runs the
 * check on its own tables and refuses to go on (AMK_ERR_UNSUPPORTED) if it fails, so a rejected plan is never
 * launched.  Neither call touches the GPU; set cfg->n_blocks when no device is present.
 *   words: header {magic, blocks, layers, ops, stage bytes, weight bytes, tiles, schedule rows};
 *          per op {kind, layer, K, rows, unit rows, dtype, region offset, region bytes};
 *          row bounds [5][blocks + 1]; first tile of each block [blocks + 1];
 *          tiles {offset / 16 | bytes / 16 << 40 | task << 53} (bytes = 0: attention marker);
 *          schedule rows {task kind, buffers read, buffers written, flags | buffers read whole << 8}.
 * What is checked (paper's check -> here):
 *   referential integrity, capacity caps -> every tile inside the weight area, 16-byte aligned, non-empty, at most
 *       one ring stage, task ids in range, section sizes consistent with the model;
 *   wait satisfiability, output reachability -> the row bounds of every GEMV partition its rows (every element a
 *       task waits for has exactly one producer); every buffer a task reads is written earlier in the step;
 *   per-SM queue order -> each block's queue is exactly the sequence of tiles its consumers will wait for
 *       (derived again from the pass geometry), one attention marker per layer after the QKV tiles;
 *   DAG acyclicity, transitive happens-before, KV ordering -> in the step's fixed task order no task reads ahead
 *       of its writer, and every overwrite of an activation buffer is ordered, through an all-to-all join, after
 *       every block's read of the previous content.  (Shared-counter all-join does not arise: joins are
 *       carried by the data or wait for all blocks.)
 */
amk_status amk_plan_export(const amk_config* cfg, uint64_t* out, size_t cap_words, size_t* need_words);
amk_status amk_plan_check(const amk_config* cfg, const uint64_t* tables, size_t n_words, char* msg, size_t msg_bytes);

/*
 * Greedy token of a logits vector, with scratch memory that is a fixed array inside the library image.
 * The paper has no counterpart of this call: its kernel picks the token inside the decode step, as
 * amk_decode_step does (the LM-head tail).  This is that tail alone -- every block of 2048 elements
 * publishes its best {value, index}, the block that arrives last reduces them -- for callers that change
 * the logits between the decode step and the choice of the token and want neither a workspace nor an
 * allocation: the call allocates no host or device memory at all.
 *   x      DEVICE in, n floats             token  DEVICE out, one int32 (lowest index among equal maxima;
 *          NaN elements are never chosen, and a vector of nothing but NaNs gives index 0)
 *          Both must be 4-byte-aligned memory of the CURRENT device (the scratch used is that device's).
 *   n      1 .. AMK_ARGMAX_STATIC_MAX_N; larger n returns AMK_ERR_UNSUPPORTED; n < 1, a NULL, misaligned or
 *          host / other-device pointer AMK_ERR_INVALID_ARG; a failed runtime call AMK_ERR_CUDA
 *   msg    HOST out, msg_bytes bytes, may be NULL: the reason in words when the status is not AMK_OK
 * The scratch (4352 bytes per device: an arrival counter and 512 candidates) belongs to the library.  The
 * counter must be zero when the kernel starts: every call clears it on cuda_stream before its launch (so a
 * launch that never finished leaves nothing behind) and the kernel puts it back to zero before it ends; the
 * candidates need no initial value.  Because all calls on a device share
 * the one scratch array, two calls that overlap in time (different streams, or different threads without
 * an order between their streams) race and give wrong tokens: keep the calls of a device in one stream or
 * order them with events.  The first call on each device looks up the scratch address (set-up, a
 * synchronous runtime query under a lock), so make it before any stream capture that is to contain later
 * calls.  Asynchronous on cuda_stream otherwise.
 */
#define AMK_ARGMAX_STATIC_MAX_N (1 << 20)
amk_status amk_argmax_static(const float* x, int64_t n, int32_t* token, char* msg, size_t msg_bytes,
                             void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* AMK_H */
