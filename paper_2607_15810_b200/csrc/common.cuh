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

// Two floats -> one byte of E2M1 codes (lo in bits 0..3, hi in bits 4..7),
// round-to-nearest-even, saturating to 6.  The hardware convert keeps the sign
// bit of values that round to zero (-0, small negatives), which is the
// convention of this library; the exhaustive quantizer test pins it.
__device__ __forceinline__ uint32_t f32x2_to_e2m1x2(float lo, float hi) {
  uint16_t r;
  asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; cvt.u16.u8 %0, t; }"
      : "=h"(r) : "f"(hi), "f"(lo));
  return (uint32_t)r & 0xFFu;
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

// Quantize one block of 16 floats with per-tensor scale gs.  Every step is a
// single IEEE float32 operation, in the order the header documents.
__device__ __forceinline__ BlockQ quantize_block(const float* v, float gs) {
  float a = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) a = fmaxf(a, fabsf(v[i]));
  const float d6 = __fmul_rn(6.0f, gs);
  const float u = __fdiv_rn(a, d6);
  BlockQ r;
  r.sf8 = f32_to_e4m3(u);
  const float sf = e4m3_to_f32(r.sf8);
  r.d = __fmul_rn(sf, gs);
  const float inv = (sf == 0.f) ? 0.f : __fdiv_rn(1.0f, r.d);
  uint32_t lo = 0, hi = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    lo |= f32x2_to_e2m1x2(__fmul_rn(v[2 * i], inv), __fmul_rn(v[2 * i + 1], inv)) << (8 * i);
    hi |= f32x2_to_e2m1x2(__fmul_rn(v[8 + 2 * i], inv), __fmul_rn(v[9 + 2 * i], inv)) << (8 * i);
  }
  r.lo = lo; r.hi = hi;
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

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}

}  // namespace quads
