// The weight packer's device side: canonical row-major matrices -> the streaming layout of amk_layout.h
// (and back, for bit-exact layout checks), plus the round-to-nearest quantisers.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "amk_internal.h"
#include "amk_ptx.cuh"

namespace amk {

namespace {

struct RowSrc {
  const unsigned char* w;       // row start in the canonical matrix
  const unsigned short* scale;  // int8: &scale[row]; int4: &scale[row][0]
  const unsigned short* zero;   // int4: &zero[row][0]
};

// Canonical location of virtual row `vrow` of an op.
__device__ __forceinline__ RowSrc row_source(const OpDesc& d, const PackSrc& s, int vrow) {
  int which = 0, row = vrow;
  if (s.mode == 1) {
    if (vrow >= s.rows1) { which = 2; row = vrow - s.rows1; }
    else if (vrow >= s.rows0) { which = 1; row = vrow - s.rows0; }
  } else if (s.mode == 2) {
    which = vrow & 1;
    row = vrow >> 1;
  }
  const size_t K = (size_t)d.K;
  const size_t rowb = d.wdtype == W_BF16 ? K * 2 : (d.wdtype == W_INT8 ? K : K / 2);
  RowSrc r;
  r.w = s.w[which] ? reinterpret_cast<const unsigned char*>(s.w[which]) + (size_t)row * rowb : nullptr;
  r.scale = nullptr;
  r.zero = nullptr;
  if (d.wdtype == W_INT8 && s.scale[which]) r.scale = reinterpret_cast<const unsigned short*>(s.scale[which]) + row;
  if (d.wdtype == W_INT4) {
    if (s.scale[which]) r.scale = reinterpret_cast<const unsigned short*>(s.scale[which]) + (size_t)row * (K / 128);
    if (s.zero[which]) r.zero = reinterpret_cast<const unsigned short*>(s.zero[which]) + (size_t)row * (K / 128);
  }
  return r;
}

// grid.x = virtual rows; threads loop over (column block, lane) chunks of 8 elements.
// inverse = false: canonical -> packed;  true: packed -> canonical (s.* then point at writable outputs).
__global__ void pack_kernel(const OpDesc d, const PackSrc s, unsigned char* packed, int n_blocks, int stage_bytes,
                            int inverse) {
  const int vrow = blockIdx.x;
  const int slot = slot_of_row(d.rows, d.unit_rows, n_blocks, vrow);
  const Slice sl = slot_slice(d.rows, d.unit_rows, n_blocks, slot);
  const int local = vrow - sl.row0;
  const int ps = local / kPassRows, rp = local - ps * kPassRows;
  const PassGeom g = pass_geom(pass_rows(sl.rows, ps), d.K, d.wdtype, stage_bytes);
  const int wr = rp / g.G, gi = rp - wr * g.G;
  const int64_t rb = row_bytes(d.wdtype, d.K);
  unsigned char* pass_base = packed + d.packed_off + (int64_t)sl.row0 * rb + (int64_t)ps * kPassRows * rb;
  const RowSrc src = row_source(d, s, vrow);
  if (src.w == nullptr) return;                 // (unpacking one matrix of a stacked op: not this row)

  if (d.wdtype == W_INT8 && threadIdx.x == 0 && src.scale) {
    // row scales live in a separate region in virtual-row order
    unsigned short* dst = reinterpret_cast<unsigned short*>(packed + d.scale_off) + vrow;
    if (!inverse) *dst = *src.scale;
    else *const_cast<unsigned short*>(src.scale) = *dst;
  }

  for (int ci = threadIdx.x; ci < g.nblk * 32; ci += blockDim.x) {
    const int b = ci >> 5, lane = ci & 31;
    const bool is_tail = g.tail && (b == g.nblk - 1);
    const int wd = is_tail ? g.tail : kBlockCols;
    const int rc = is_tail ? g.rc_tail : g.rc_full;
    unsigned char* chunk = pass_base + unit_off_br(g, b, wr) + (int64_t)gi * rc;
    if (lane >= (wd >> 3)) continue;
    const int c0 = b * kBlockCols + 4 * lane, c1 = b * kBlockCols + (wd >> 1) + 4 * lane;
    if (d.wdtype == W_BF16) {
      uint2* a0 = (uint2*)(src.w + (size_t)c0 * 2);
      uint2* a1 = (uint2*)(src.w + (size_t)c1 * 2);
      uint4* dst = (uint4*)(chunk + lane * 16);
      if (!inverse) { const uint2 v0 = *a0, v1 = *a1; *dst = make_uint4(v0.x, v0.y, v1.x, v1.y); }
      else { const uint4 v = *dst; *a0 = make_uint2(v.x, v.y); *a1 = make_uint2(v.z, v.w); }
    } else if (d.wdtype == W_INT8) {
      unsigned* a0 = (unsigned*)(src.w + c0);
      unsigned* a1 = (unsigned*)(src.w + c1);
      uint2* dst = (uint2*)(chunk + lane * 8);
      if (!inverse) *dst = make_uint2(*a0 ^ 0x80808080u, *a1 ^ 0x80808080u);      // two's complement -> biased
      else { const uint2 v = *dst; *a0 = v.x ^ 0x80808080u; *a1 = v.y ^ 0x80808080u; }
    } else {
      unsigned short* a0 = (unsigned short*)(src.w + (c0 >> 1));
      unsigned short* a1 = (unsigned short*)(src.w + (c1 >> 1));
      unsigned* dst = (unsigned*)(chunk + lane * 4);
      if (!inverse) *dst = (unsigned)*a0 | ((unsigned)*a1 << 16);
      else { const unsigned v = *dst; *a0 = (unsigned short)(v & 0xffffu); *a1 = (unsigned short)(v >> 16); }
      if (lane == 0) {
        // fp16 {scale, zero} of groups 2b and 2b+1 follow the 128 code bytes of this row chunk
        uint2* sz = (uint2*)(chunk + 128);
        unsigned short* sc = const_cast<unsigned short*>(src.scale);
        unsigned short* zr = const_cast<unsigned short*>(src.zero);
        if (!inverse) {
          if (sc && zr)
            *sz = make_uint2((unsigned)sc[2 * b] | ((unsigned)zr[2 * b] << 16),
                           (unsigned)sc[2 * b + 1] | ((unsigned)zr[2 * b + 1] << 16));
        } else {
          const uint2 v = *sz;
          if (sc) { sc[2 * b] = (unsigned short)(v.x & 0xffffu); sc[2 * b + 1] = (unsigned short)(v.y & 0xffffu); }
          if (zr) { zr[2 * b] = (unsigned short)(v.x >> 16); zr[2 * b + 1] = (unsigned short)(v.y >> 16); }
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

cudaError_t launch_pack(const OpDesc& d, const PackSrc& src, unsigned char* packed, int n_blocks, int stage_bytes,
                        bool inverse, cudaStream_t stream) {
  if (d.rows <= 0) return cudaSuccess;
  pack_kernel<<<d.rows, 256, 0, stream>>>(d, src, packed, n_blocks, stage_bytes, inverse ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t launch_quantize_int8(const void* w, int64_t rows, int64_t cols, void* q, void* scale, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  quantize_int8_kernel<<<(unsigned)rows, 256, 0, s>>>((const unsigned short*)w, cols, (signed char*)q, (__half*)scale);
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
