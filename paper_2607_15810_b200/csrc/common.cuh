// Shared device helpers: NVFP4 block quantization primitives and small utilities.
// sm_100a only.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/quads.h"

namespace quads {

constexpr int kBlock = 16;          // elements per scale block
constexpr float kGlobalDiv = 2688.f; // 6 * 448

// Launch bookkeeping (host side, per thread).
extern thread_local int g_launch_count;
inline void note_launch() { ++g_launch_count; }

#define QUADS_CUDA_OK(expr)                              \
  do {                                                   \
    cudaError_t _e = (expr);                             \
    if (_e != cudaSuccess) return QUADS_ERR_CUDA;        \
  } while (0)

// Programmatic dependent launch: every kernel of the MoE chain starts with this.  It blocks
// until the preceding kernel of the stream has completed and its writes are visible, then
// lets the following kernel begin its own launch (that one blocks at the same point), so
// launch latencies overlap instead of adding up.  A no-op for ordinary launches.
__device__ __forceinline__ void pdl_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Host side: launch with the programmatic-stream-serialization attribute (or plainly).
bool pdl_enabled();
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  note_launch();
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Raise a kernel's dynamic shared-memory limit once per device (the attribute is per device; a
// process may drive several).  `Kernel` must be a distinct function per instantiation.
template <auto Kernel>
inline cudaError_t set_max_dynamic_smem(int bytes) {
  static bool done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
  return e;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b16) { return __uint_as_float(b16 << 16); }

// Unpack 8 bf16 (one 16-byte vector) to float.
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
  f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
  f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}

// 32-byte read-only global load (two 16-byte halves of one scale block).
__device__ __forceinline__ void ldg256(const void* p, uint4& a, uint4& b) {
  asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w)
               : "l"(p));
}

// float -> E4M3 byte, round-to-nearest-even, saturating to 448.
__device__ __forceinline__ uint32_t f32_to_e4m3(float v) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.f), "f"(v));
  return r & 0xFFu;
}

// E4M3 byte -> float (exact).
__device__ __forceinline__ float e4m3_to_f32(uint32_t b) {
  uint32_t h2;
  uint16_t in = (uint16_t)b;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(in));
  return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

// Eight floats -> eight E2M1 codes in one 32-bit word (element i in nibble i),
// round-to-nearest-even, saturating to 6.  The hardware convert keeps the sign bit of
// values that round to zero (-0, small negatives), which is the convention of this
// library; the exhaustive quantizer test pins it.
__device__ __forceinline__ uint32_t f32x8_to_e2m1x8(float v0, float v1, float v2, float v3, float v4, float v5,
                                                    float v6, float v7) {
  uint32_t r;
  asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
      "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
      : "=r"(r) : "f"(v0), "f"(v1), "f"(v2), "f"(v3), "f"(v4), "f"(v5), "f"(v6), "f"(v7));
  return r;
}

// One byte of two E2M1 codes -> two floats (exact): low nibble -> .x, high nibble -> .y.
__device__ __forceinline__ float2 e2m1x2_to_f32x2(uint32_t byte) {
  uint32_t h2;
  uint16_t in = (uint16_t)(byte & 0xFFu);
  asm("{ .reg .b8 t; cvt.u8.u16 t, %1; cvt.rn.f16x2.e2m1x2 %0, t; }" : "=r"(h2) : "h"(in));
  return __half22float2(*reinterpret_cast<__half2*>(&h2));
}

struct BlockQ {
  uint32_t lo, hi;   // 16 codes: elements 0..7 in lo, 8..15 in hi
  uint32_t sf8;      // E4M3 scale byte
  float d;           // decoded block scale sf * gs
};

// Per-tensor constants of the quantizer.  `r6` is the correctly rounded reciprocal of d6 and
// `inv_lut[c]` = 1 / (E4M3(c) * gs) (0 for c = 0), both computed with IEEE operations, so that
// the per-block arithmetic below reproduces the documented single-operation recipe bit for bit
// without a division routine per block.
struct QuantCtx {
  float gs, d6, r6;
  const float* inv_lut;   // 128 entries (shared memory)
};

__device__ __forceinline__ void quant_ctx_scalars(QuantCtx& c, float gs) {
  c.gs = gs;
  c.d6 = __fmul_rn(6.0f, gs);
  c.r6 = __frcp_rn(c.d6);
}
// Entry `code` of the reciprocal table for per-tensor scale gs.
__device__ __forceinline__ float quant_inv_entry(uint32_t code, float gs) {
  const float sf = e4m3_to_f32(code & 0x7Fu);
  return (sf == 0.f || code == 0x7Fu) ? 0.f : __fdiv_rn(1.0f, __fmul_rn(sf, gs));
}

// Quantize one block of 16 floats.  u = amax / d6 is formed as q0 = amax * r6 followed by one
// fused correction step (residual amax - q0 * d6 is exact in an FMA), which yields the correctly
// rounded quotient given a correctly rounded reciprocal; the 1 / d of the element scaling comes
// from the table (kLut) or from the table's own formula evaluated in place.
template <bool kLut = true>
__device__ __forceinline__ BlockQ quantize_block(const float* v, const QuantCtx& c) {
  float a = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) a = fmaxf(a, fabsf(v[i]));
  const float q0 = __fmul_rn(a, c.r6);
  const float u = __fmaf_rn(__fmaf_rn(-q0, c.d6, a), c.r6, q0);
  BlockQ r;
  r.sf8 = f32_to_e4m3(u);
  r.d = __fmul_rn(e4m3_to_f32(r.sf8), c.gs);
  // without the table: the same quotient, one division per block
  const float inv = kLut ? c.inv_lut[r.sf8] : quant_inv_entry(r.sf8, c.gs);
  r.lo = f32x8_to_e2m1x8(__fmul_rn(v[0], inv), __fmul_rn(v[1], inv), __fmul_rn(v[2], inv), __fmul_rn(v[3], inv),
                         __fmul_rn(v[4], inv), __fmul_rn(v[5], inv), __fmul_rn(v[6], inv), __fmul_rn(v[7], inv));
  r.hi = f32x8_to_e2m1x8(__fmul_rn(v[8], inv), __fmul_rn(v[9], inv), __fmul_rn(v[10], inv), __fmul_rn(v[11], inv),
                         __fmul_rn(v[12], inv), __fmul_rn(v[13], inv), __fmul_rn(v[14], inv), __fmul_rn(v[15], inv));
  return r;
}

// Dequantize the 16 codes of a block: value(code) * d, one float32 multiply.
__device__ __forceinline__ void dequant_block(const BlockQ& q, float* out) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 a = e2m1x2_to_f32x2(q.lo >> (8 * i));
    const float2 b = e2m1x2_to_f32x2(q.hi >> (8 * i));
    out[2 * i] = __fmul_rn(a.x, q.d);
    out[2 * i + 1] = __fmul_rn(a.y, q.d);
    out[8 + 2 * i] = __fmul_rn(b.x, q.d);
    out[9 + 2 * i] = __fmul_rn(b.y, q.d);
  }
}

__device__ __forceinline__ uint32_t f32x2_to_bf16x2(float lo, float hi) {
  __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&b);
}

// Byte offset of scale (row, blk) in the tiled layout with kt_count = ceil(K/64) atoms per row tile.
__host__ __device__ __forceinline__ size_t sf_tiled_offset(int64_t row, int64_t blk, int64_t kt_count) {
  return ((size_t)(row >> 7) * (size_t)kt_count + (size_t)(blk >> 2)) * 512u +
         (size_t)((row & 31) * 16 + ((row >> 5) & 3) * 4 + (blk & 3));
}

__device__ __forceinline__ void stg256(void* addr, const uint32_t* v) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]),
               "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}

// Store a warp's 32 rows x 64 accumulator columns (thread = row) as bf16, scaled, to rows of
// `n_out` elements starting at `dst`, rows >= rows_valid skipped.  The 32-byte chunks are first
// transposed inside every group of 4 lanes (two butterfly exchanges), so that each store
// instruction of the warp writes eight complete 128-byte lines instead of a 32-byte piece of 32
// different lines.  All 32 lanes must call it.
__device__ __forceinline__ void store_y_rows(const float* acc, float scale, uint16_t* dst, int n_out, int rows_valid,
                                             int lane) {
  uint32_t w[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) w[i] = f32x2_to_bf16x2(acc[2 * i] * scale, acc[2 * i + 1] * scale);
  // chunk c = w[8c .. 8c+7]; after the exchanges chunk slot c of lane (g, j) holds chunk j of lane (g, c)
#pragma unroll
  for (int s = 1; s < 4; s <<= 1) {
    const bool up = (lane & s) != 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      if (c & s) continue;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint32_t lo = w[8 * c + k], hi = w[8 * (c | s) + k];
        const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, up ? lo : hi, s);
        w[8 * c + k] = up ? got : lo;
        w[8 * (c | s) + k] = up ? hi : got;
      }
    }
  }
  const int g = lane >> 2, j = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = 4 * g + i;
    if (r < rows_valid) stg256(dst + (size_t)r * n_out + 16 * j, w + 8 * i);
  }
}

// One partial column score (a float32 sum of squared residuals, >= 0) as a fixed-point integer with
// `bits` fractional bits in units of gs^2, capped at 2^(cap_bits + bits): a residual is at most half a
// quantization step, 448 gs, so a sum over n rows stays below n * 2^18 gs^2 (cap_bits = 18 + log2 n).
// Added to the column's total with an integer reduction, whose result does not depend on the order of
// the additions.
__device__ __forceinline__ void add_score(unsigned long long* total, float partial, float gs, int bits, int cap_bits = 23) {
  const float u = __fdiv_rn(__fdiv_rn(partial, gs), gs);
  const float cap = __uint_as_float((uint32_t)(127 + cap_bits + bits) << 23);
  const float v = fminf(u * __uint_as_float((uint32_t)(127 + bits) << 23), cap);
  const unsigned long long q = __float2ull_rd(v);
  if (q) asm volatile("red.global.add.u64 [%0], %1;" ::"l"(total), "l"(q) : "memory");
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}

}  // namespace quads
