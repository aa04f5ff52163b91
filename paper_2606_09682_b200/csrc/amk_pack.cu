// The weight packer's device side: canonical row-major matrices -> the streaming layout of amk_layout.h
// (and back, for bit-exact layout checks), plus the round-to-nearest quantisers.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "amk_internal.h"
#include "amk_ptx.cuh"

namespace amk {

namespace {

struct RowSrc {
  unsigned char* w;             // row start in the canonical matrix (nullptr: this row is not wanted)
  unsigned short* scale;        // int8: &scale[row]; int4, grouped int8: &scale[row][0]
  unsigned short* zero;         // int4: &zero[row][0]
};

// Canonical location of virtual row `vrow` of an op.
__device__ __forceinline__ RowSrc row_source(const OpShape& d, const PackSrc& s, int vrow) {
  int which = 0, row = vrow;
  if (s.mode == 1) {
    if (vrow >= s.rows1) { which = 2; row = vrow - s.rows1; }
    else if (vrow >= s.rows0) { which = 1; row = vrow - s.rows0; }
  } else if (s.mode == 2) {
    which = vrow & 1;
    row = vrow >> 1;
  }
  const size_t K = (size_t)d.K;
  const size_t rowb = d.wdtype == W_BF16 ? K * 2 : (d.wdtype == W_INT4 ? K / 2 : K);
  RowSrc r;
  r.w = s.w[which] ? (unsigned char*)s.w[which] + (size_t)row * rowb : nullptr;
  r.scale = nullptr;
  r.zero = nullptr;
  if (d.wdtype == W_INT8 && s.scale[which]) r.scale = (unsigned short*)s.scale[which] + row;
  if (grouped(d.wdtype)) {
    if (s.scale[which]) r.scale = (unsigned short*)s.scale[which] + (size_t)row * (K / 128);
    if (d.wdtype == W_INT4 && s.zero[which]) r.zero = (unsigned short*)s.zero[which] + (size_t)row * (K / 128);
  }
  return r;
}

// grid.x = virtual rows; threads loop over the 16-byte chunks of the row.
// inverse = 0: canonical -> packed;  1: packed -> canonical (s.* then point at writable outputs).
__global__ void pack_kernel(const PackOp d, const PackSrc s, unsigned char* packed, int n_blocks, int stage_bytes,
                            int inverse) {
  const int vrow = blockIdx.x;
  const int wd = d.s.wdtype, K = d.s.K;
  const int slot = slot_of_row(d.bounds, d.s.unit_rows, n_blocks, vrow);
  const Slice sl = slot_slice(d.bounds, d.s.unit_rows, slot);
  const int local = vrow - sl.row0;
  const int ps = local / kPassRows, rp = local - ps * kPassRows;
  int64_t pass_off = 0;
  for (int p = 0; p < ps; p++) pass_off += pass_bytes(pass_geom(pass_rows(sl.rows, p), K, wd, stage_bytes));
  const PassGeom g = pass_geom(pass_rows(sl.rows, ps), K, wd, stage_bytes);
  const int wr = rp / g.G, gi = rp - wr * g.G;
  const int urows = (wr == g.Wr - 1) ? g.g_last : g.G;
  unsigned char* pass_base = packed + d.region_off + d.slice_off[slot] + pass_off;
  const RowSrc src = row_source(d.s, s, vrow);
  if (src.w == nullptr) return;                 // (unpacking one matrix of a stacked op: not this row)

  if (wd == W_INT8 && threadIdx.x == 0 && src.scale) {
    unsigned short* dst = reinterpret_cast<unsigned short*>(packed + d.scale_off) + vrow;
    if (!inverse) *dst = *src.scale;
    else *src.scale = *dst;
  }
  const int cpb = block_chunks(wd), bc = block_cols(wd);
  for (int ci = threadIdx.x; ci < g.nblk * cpb; ci += blockDim.x) {
    const int b = ci / cpb, c = ci - b * cpb;
    unsigned char* unit = pass_base + unit_off_br(g, b, wr);
    uint4* chunk = reinterpret_cast<uint4*>(unit + ((size_t)c * urows + gi) * 16);
    const int col0 = b * bc;
    if (wd == W_BF16) {
      // chunk c = 2 s + hh holds logical k = 16 s + 8 hh + 2 q + j: for q = 0..3 the pair at column 16 q + 4 s + 2 hh
      const int sidx = c >> 1, hh = c & 1;
      unsigned* w32 = reinterpret_cast<unsigned*>(src.w);
      unsigned v[4];
      if (inverse) { const uint4 t = *chunk; v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
      for (int q = 0; q < 4; q++) {
        const int col = col0 + 16 * q + 4 * sidx + 2 * hh;
        if (!inverse) v[q] = w32[col >> 1];
        else w32[col >> 1] = v[q];
      }
      if (!inverse) *chunk = make_uint4(v[0], v[1], v[2], v[3]);
    } else if (wd == W_INT8 || wd == W_INT8G) {
      // chunk c = 2 s + hh holds logical k = 32 s + 16 hh + 4 q + j: for q = 0..3 the word at column
      // 32 q + 8 s + 4 hh (zero codes beyond K: an int8 matrix's last block may be half full)
      const int sidx = c >> 1, hh = c & 1;
      unsigned* w32 = reinterpret_cast<unsigned*>(src.w);
      unsigned v[4];
      if (inverse) { const uint4 t = *chunk; v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
      for (int q = 0; q < 4; q++) {
        const int col = col0 + 32 * q + 8 * sidx + 4 * hh;
        if (col >= K) { if (!inverse) v[q] = 0u; continue; }
        if (!inverse) v[q] = w32[col >> 2];
        else w32[col >> 2] = v[q];
      }
      if (!inverse) *chunk = make_uint4(v[0], v[1], v[2], v[3]);
      if (wd == W_INT8G && c == 0) {
        // {fp16 scale, 0} of this row's group (= this block) after the unit's code bytes
        unsigned* sz = reinterpret_cast<unsigned*>(unit + (size_t)urows * 128 + (size_t)gi * 4);
        if (!inverse) { if (src.scale) *sz = (unsigned)src.scale[b]; }
        else if (src.scale) src.scale[b] = (unsigned short)(*sz & 0xffffu);
      }
    } else {
      // chunk c = 2 x + hh; word q, nibble 2 j + sb holds logical k of step s = 2 x + sb: column 32 q + 8 s + 4 hh + j
      const int x = c >> 1, hh = c & 1;
      unsigned v[4];
      if (inverse) { const uint4 t = *chunk; v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
      for (int q = 0; q < 4; q++) {
        unsigned word = inverse ? v[q] : 0u;
        for (int sb = 0; sb < 2; sb++) {
          for (int jp = 0; jp < 2; jp++) {               // columns 2 jp and 2 jp + 1 share a canonical byte
            const int col = col0 + 32 * q + 8 * (2 * x + sb) + 4 * hh + 2 * jp;
            unsigned char* byte = src.w + (col >> 1);
            const int n0 = 2 * (2 * jp) + sb, n1 = 2 * (2 * jp + 1) + sb;
            if (!inverse) {
              const unsigned bv = *byte;
              word |= (bv & 0xFu) << (4 * n0);
              word |= (bv >> 4) << (4 * n1);
            } else {
              *byte = (unsigned char)(((word >> (4 * n0)) & 0xFu) | (((word >> (4 * n1)) & 0xFu) << 4));
            }
          }
        }
        v[q] = word;
      }
      if (!inverse) *chunk = make_uint4(v[0], v[1], v[2], v[3]);
      if (c == 0) {
        // {fp16 scale, zero point as a 16-bit integer} of this row's group (= this block) after the unit's code
        // bytes (the canonical zero point is an fp16 holding an integer 0..15: the kernel wants the integer)
        unsigned* sz = reinterpret_cast<unsigned*>(unit + (size_t)urows * 64 + (size_t)gi * 4);
        if (!inverse) {
          if (src.scale && src.zero) {
            const unsigned zi = (unsigned)(int)__half2float(__ushort_as_half(src.zero[b])) & 0xffffu;
            *sz = (unsigned)src.scale[b] | (zi << 16);
          }
        } else {
          const unsigned t = *sz;
          if (src.scale) src.scale[b] = (unsigned short)(t & 0xffffu);
          if (src.zero) src.zero[b] = __half_as_ushort(__float2half_rn((float)(t >> 16)));
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------ quantisers
__device__ __forceinline__ float bf16_at(const unsigned short* p, int64_t i) {
  return __uint_as_float((unsigned)p[i] << 16);
}

// one block per row; every operation is an IEEE fp32 operation (no fast-math, no contraction involved)
__global__ void quantize_int8_kernel(const unsigned short* __restrict__ w, int64_t cols, signed char* __restrict__ q,
                                     __half* __restrict__ scale) {
  __shared__ float s_part[32];
  __shared__ float s_scale;
  const int64_t row = blockIdx.x;
  const unsigned short* wr = w + row * cols;
  float amax = 0.f;
  for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) amax = fmaxf(amax, fabsf(bf16_at(wr, j)));
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); i++) a = fmaxf(a, s_part[i]);
    __half h = (a == 0.f) ? __float2half_rn(1.0f) : __float2half_rn(__fdiv_rn(a, 127.0f));
    float s = __half2float(h);
    if (s == 0.f) { h = __float2half_rn(1.0f); s = 1.0f; }
    scale[row] = h;
    s_scale = s;
  }
  __syncthreads();
  const float s = s_scale;
  for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) {
    float r = rintf(__fdiv_rn(bf16_at(wr, j), s));
    r = fminf(fmaxf(r, -127.0f), 127.0f);
    q[row * cols + j] = (signed char)(int)r;
  }
}

// grouped int8: one warp per (row, group of 128), the per-row rule on the group; lane handles 4 consecutive columns
__global__ void quantize_int8_grouped_kernel(const unsigned short* __restrict__ w, int64_t rows, int64_t cols,
                                             signed char* __restrict__ q, __half* __restrict__ scale) {
  const int64_t ng = cols / 128;
  const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (wid >= rows * ng) return;
  const int lane = threadIdx.x & 31;
  const int64_t row = wid / ng, g = wid - row * ng;
  const unsigned short* wp = w + row * cols + g * 128 + lane * 4;
  float v[4];
  float amax = 0.f;
#pragma unroll
  for (int e = 0; e < 4; e++) { v[e] = bf16_at(wp, e); amax = fmaxf(amax, fabsf(v[e])); }
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  __half h = (amax == 0.f) ? __float2half_rn(1.0f) : __float2half_rn(__fdiv_rn(amax, 127.0f));
  float s = __half2float(h);
  if (s == 0.f) { h = __float2half_rn(1.0f); s = 1.0f; }
  signed char* out = q + row * cols + g * 128 + lane * 4;
#pragma unroll
  for (int e = 0; e < 4; e++) {
    float r = rintf(__fdiv_rn(v[e], s));
    r = fminf(fmaxf(r, -127.0f), 127.0f);
    out[e] = (signed char)(int)r;
  }
  if (lane == 0) scale[row * ng + g] = h;
}

// one warp per (row, group of 128): lane handles 4 consecutive columns = 2 output bytes
__global__ void quantize_int4_kernel(const unsigned short* __restrict__ w, int64_t rows, int64_t cols,
                                     unsigned char* __restrict__ packed, __half* __restrict__ scale,
                                     __half* __restrict__ zero) {
  const int64_t ng = cols / 128;
  const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (wid >= rows * ng) return;
  const int lane = threadIdx.x & 31;
  const int64_t row = wid / ng, g = wid - row * ng;
  const unsigned short* wp = w + row * cols + g * 128 + lane * 4;
  float v[4];
  float mn = 0.f, mx = 0.f;
#pragma unroll
  for (int e = 0; e < 4; e++) { v[e] = bf16_at(wp, e); mn = fminf(mn, v[e]); mx = fmaxf(mx, v[e]); }
  for (int o = 16; o > 0; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  __half h = (mx == mn) ? __float2half_rn(1.0f) : __float2half_rn(__fdiv_rn(__fsub_rn(mx, mn), 15.0f));
  float s = __half2float(h);
  if (s == 0.f) { h = __float2half_rn(1.0f); s = 1.0f; }
  float z = rintf(__fdiv_rn(-mn, s));
  if (!(z > 0.f)) z = 0.f;                 // also turns -0 (an all-positive group) into +0
  z = fminf(z, 15.f);
  unsigned code[4];
#pragma unroll
  for (int e = 0; e < 4; e++) {
    float r = __fadd_rn(rintf(__fdiv_rn(v[e], s)), z);
    r = fminf(fmaxf(r, 0.f), 15.f);
    code[e] = (unsigned)(int)r;
  }
  unsigned char* out = packed + row * (cols / 2) + g * 64 + lane * 2;
  out[0] = (unsigned char)(code[0] | (code[1] << 4));
  out[1] = (unsigned char)(code[2] | (code[3] << 4));
  if (lane == 0) { scale[row * ng + g] = h; zero[row * ng + g] = __float2half_rn(z); }
}

}  // namespace

cudaError_t launch_pack(const PackOp& d, const PackSrc& src, unsigned char* packed, int n_blocks, int stage_bytes,
                        bool inverse, cudaStream_t stream) {
  if (d.s.rows <= 0) return cudaSuccess;
  pack_kernel<<<d.s.rows, 128, 0, stream>>>(d, src, packed, n_blocks, stage_bytes, inverse ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t launch_quantize_int8(const void* w, int64_t rows, int64_t cols, void* q, void* scale, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  quantize_int8_kernel<<<(unsigned)rows, 256, 0, s>>>((const unsigned short*)w, cols, (signed char*)q, (__half*)scale);
  return cudaGetLastError();
}

cudaError_t launch_quantize_int8_grouped(const void* w, int64_t rows, int64_t cols, void* q, void* scale, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  const int64_t warps = rows * (cols / 128);
  const int wpb = 8;
  quantize_int8_grouped_kernel<<<(unsigned)((warps + wpb - 1) / wpb), wpb * 32, 0, s>>>(
      (const unsigned short*)w, rows, cols, (signed char*)q, (__half*)scale);
  return cudaGetLastError();
}

cudaError_t launch_quantize_int4(const void* w, int64_t rows, int64_t cols, void* packed, void* scale, void* zero,
                                 cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  const int64_t warps = rows * (cols / 128);
  const int wpb = 8;
  quantize_int4_kernel<<<(unsigned)((warps + wpb - 1) / wpb), wpb * 32, 0, s>>>(
      (const unsigned short*)w, rows, cols, (unsigned char*)packed, (__half*)scale, (__half*)zero);
  return cudaGetLastError();
}

}  // namespace amk
