// FP8 W8A8 comparison path (the paper's "FP8 W8A8" rollout arm): E4M3 elements with fine-grained
// power-of-two scales -- one per (row, 128 channels) of an activation, one per 128 x 128 tile of a
// weight -- and grouped expert GEMMs on the block-scaled FP8 tensor-core path
// (tcgen05.mma.kind::mxf8f6f4, one UE8M0 scale byte per 32 elements: a tile's scale is repeated).
// Same layer, routing, dispatch order and combine as the NVFP4 path; no RAC (there is none in FP8).
// It exists so that the W4A4 / FP8 relations the paper reports can be restated on one layer.
#include "kernels.cuh"
#include "tcgen05.cuh"

namespace quads {

// Smallest e with amax <= 448 * 2^e, as the biased byte e + 127 (clipped to 0..254).
// amax = f * 2^E with 1 <= f < 2:  e = E - 8 when f <= 1.75, else E - 7.
__device__ __forceinline__ uint32_t fp8_scale_code(float amax) {
  const uint32_t b = __float_as_uint(amax);
  const int E = (int)((b >> 23) & 0xFF) - 127;
  int e = E - 8 + (((b & 0x7FFFFFu) > 0x600000u) ? 1 : 0);
  if (amax == 0.f) e = -127;
  e = max(-127, min(127, e));
  return (uint32_t)(e + 127);
}

__device__ __forceinline__ uint32_t f32x4_to_e4m3x4(float a, float b, float c, float d) {
  uint16_t lo, hi;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %2, %1;" : "=h"(lo) : "f"(a), "f"(b));
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %2, %1;" : "=h"(hi) : "f"(c), "f"(d));
  return (uint32_t)lo | ((uint32_t)hi << 16);
}

// Activation quantizer: one warp per (row, 128-channel tile), a lane holds 4 consecutive values.
// codes [rows, K] u8, exps [rows, K/128] u8 (e + 127).
__global__ void __launch_bounds__(256)
fp8_quantize_act_kernel(const uint16_t* __restrict__ x, int64_t rows, int K, uint8_t* __restrict__ codes,
                        uint8_t* __restrict__ exps) {
  pdl_sync();
  const int kt = K >> 7;
  const int64_t n_tiles = rows * kt;
  const int lane = threadIdx.x & 31;
  for (int64_t w = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); w < n_tiles; w += (int64_t)gridDim.x * 8) {
    const int64_t r = w / kt;
    const int t = (int)(w - r * kt);
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(x + r * K + t * 128) + lane);
    const float f0 = __uint_as_float(v.x << 16), f1 = __uint_as_float(v.x & 0xFFFF0000u);
    const float f2 = __uint_as_float(v.y << 16), f3 = __uint_as_float(v.y & 0xFFFF0000u);
    const float a = warp_max(fmaxf(fmaxf(fabsf(f0), fabsf(f1)), fmaxf(fabsf(f2), fabsf(f3))));
    const uint32_t code = fp8_scale_code(a);
    const int e = (int)code - 127;
    reinterpret_cast<uint32_t*>(codes + r * K + t * 128)[lane] =
        f32x4_to_e4m3x4(ldexpf(f0, -e), ldexpf(f1, -e), ldexpf(f2, -e), ldexpf(f3, -e));
    if (lane == 0) exps[r * kt + t] = (uint8_t)code;
  }
}

// Weight quantizer: one CTA per 128 x 128 tile (256 threads, 64 values each: half a row).
// codes [n, N, K] u8; exps [n, N/128, K/128] u8; atoms [n, N/128, K/128, 512] u8: the tile's scale byte
// repeated, the form the tensor-core path copies into tensor memory.
__global__ void __launch_bounds__(256)
fp8_quantize_weight_kernel(const uint16_t* __restrict__ w, int N, int K, uint8_t* __restrict__ codes,
                           uint8_t* __restrict__ exps, uint8_t* __restrict__ atoms) {
  const int kt = K >> 7, nt = N >> 7;
  const int tile = blockIdx.x % (nt * kt), tensor = blockIdx.x / (nt * kt);
  const int tn = tile / kt, tk = tile - tn * kt;
  const int row = threadIdx.x >> 1, half = threadIdx.x & 1;
  const size_t off = ((size_t)tensor * N + (size_t)tn * 128 + row) * K + (size_t)tk * 128 + half * 64;
  uint4 v[8];
  float a = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    v[i] = __ldg(reinterpret_cast<const uint4*>(w + off) + i);
    float f[8];
    unpack8(v[i], f);
#pragma unroll
    for (int k = 0; k < 8; ++k) a = fmaxf(a, fabsf(f[k]));
  }
  a = warp_max(a);
  __shared__ float wm[8];
  __shared__ uint32_t code_sh;
  if ((threadIdx.x & 31) == 0) wm[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < 8; ++i) t = fmaxf(t, wm[i]);
    code_sh = fp8_scale_code(t);
  }
  __syncthreads();
  const uint32_t code = code_sh;
  const int e = (int)code - 127;
#pragma unroll
  for (int i = 0; i < 8; i += 2) {
    float f[16];
    unpack8(v[i], f);
    unpack8(v[i + 1], f + 8);
    uint4 o;
    o.x = f32x4_to_e4m3x4(ldexpf(f[0], -e), ldexpf(f[1], -e), ldexpf(f[2], -e), ldexpf(f[3], -e));
    o.y = f32x4_to_e4m3x4(ldexpf(f[4], -e), ldexpf(f[5], -e), ldexpf(f[6], -e), ldexpf(f[7], -e));
    o.z = f32x4_to_e4m3x4(ldexpf(f[8], -e), ldexpf(f[9], -e), ldexpf(f[10], -e), ldexpf(f[11], -e));
    o.w = f32x4_to_e4m3x4(ldexpf(f[12], -e), ldexpf(f[13], -e), ldexpf(f[14], -e), ldexpf(f[15], -e));
    reinterpret_cast<uint4*>(codes + off)[i >> 1] = o;
  }
  const size_t ti = ((size_t)tensor * nt + tn) * kt + tk;
  if (threadIdx.x == 0) exps[ti] = (uint8_t)code;
  if (threadIdx.x < 32) {
    const uint32_t c4 = code * 0x01010101u;
    reinterpret_cast<uint4*>(atoms + ti * 512)[threadIdx.x] = make_uint4(c4, c4, c4, c4);
  }
}

// Dispatch, driven by the destination tile (as rac_dispatch_kernel): the tile's rows of E4M3 codes
// (H bytes each) and, per 128-channel stage, one 512-byte scale atom with every row's scale byte
// repeated over the stage's four K = 32 MMAs.
__global__ void __launch_bounds__(256)
fp8_dispatch_kernel(int H, const int32_t* __restrict__ header, const int32_t* __restrict__ tile_rows,
                    const int32_t* __restrict__ row_token, const uint8_t* __restrict__ xq, const uint8_t* __restrict__ xe,
                    uint8_t* __restrict__ xq_pad, uint8_t* __restrict__ xsf_atoms) {
  pdl_sync();
  const int mt = blockIdx.x;
  if (mt >= header[kHdrMTiles]) return;
  const int n_rows = tile_rows[mt];
  __shared__ int tok[128];
  if (threadIdx.x < 128) tok[threadIdx.x] = threadIdx.x < n_rows ? row_token[mt * 128 + threadIdx.x] : -1;
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int per_row = H >> 4;                          // 16-byte chunks per row
  for (int c = lane; c < per_row; c += 32)
    for (int r0 = warp; r0 < n_rows; r0 += 32) {
      uint4 v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (r0 + 8 * j < n_rows) v[j] = __ldg(reinterpret_cast<const uint4*>(xq + (size_t)tok[r0 + 8 * j] * H) + c);
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (r0 + 8 * j < n_rows) __stcs(reinterpret_cast<uint4*>(xq_pad + (size_t)(mt * 128 + r0 + 8 * j) * H) + c, v[j]);
    }
  // atoms: word (row % 32) * 4 + row / 32 of atom kt = the row's scale byte, four times
  const int kt = H >> 7;
  for (int i = threadIdx.x; i < kt * 128; i += blockDim.x) {
    const int k = i >> 7, r = i & 127;
    const uint32_t code = r < n_rows ? (uint32_t)xe[(size_t)tok[r] * kt + k] : 0u;
    reinterpret_cast<uint32_t*>(xsf_atoms + ((size_t)mt * kt + k) * 512)[(r & 31) * 4 + (r >> 5)] = code * 0x01010101u;
  }
}

// ---------------------------------------------------------------------------
// Grouped FP8 GEMM: D[row, n] = sum_k A[row, k] W[e(row), n, k] with hardware block scales.
// Persistent, one CTA per SM, 18 warps as in gemm.cu: warp 0 loads (TMA tiles of 128 bytes = 128 E4M3
// per row and stage, 128-byte swizzle; bulk copies of the stage's three scale atoms) into a 4-stage
// ring, warp 1 copies the atoms to tensor memory and issues four 128 x 256 x 32 MMAs per stage (the
// scale byte of MMA j is byte j of the atoms' words), warps 2..17 drain the accumulator and run the
// epilogue: SwiGLU -> bf16 -> E4M3 with one scale per (row, 128 features) -- a tile is exactly one
// such group, its four column quarters meet through shared memory -- or bf16 rows for the combine.
// ---------------------------------------------------------------------------
namespace {

constexpr int k8BM = 128, k8BN = 256;
constexpr int k8TileA = k8BM * 128, k8TileB = k8BN * 128;
constexpr int k8OffB = k8TileA;
constexpr int k8OffSfA = k8OffB + k8TileB;
constexpr int k8OffSfB = k8OffSfA + 512;
constexpr int k8StageBytes = k8OffSfB + 1024 + 512;      // 51200 (1 KB multiple)
constexpr int k8Stages = 4;
constexpr int k8Threads = 576;
constexpr int k8EpiWarps = 16;
constexpr int k8BarOffset = k8Stages * k8StageBytes;
constexpr int k8SmemBytes = k8BarOffset + 256 + 2 * 128 * 4 * 4 + 1024;

struct __align__(8) F8Barriers {
  uint64_t full[k8Stages];
  uint64_t empty[k8Stages];
  uint64_t tmem_full;
  uint64_t tmem_empty;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void tc_mma_mxf8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate) : "memory");
}

template <int EPI>
__global__ void __launch_bounds__(k8Threads, 1)
gemm_fp8_kernel(const Fp8GemmParams p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b) {
  extern __shared__ uint8_t smem_dyn[];
  const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
  F8Barriers* bars = reinterpret_cast<F8Barriers*>(smem_gen + k8BarOffset);
  float* row_amax = reinterpret_cast<float*>(smem_gen + k8BarOffset + 256);     // [2][128][4]
  const uint32_t bar_full = smem_u32(&bars->full[0]), bar_empty = smem_u32(&bars->empty[0]);
  const uint32_t bar_tfull = smem_u32(&bars->tmem_full), bar_tempty = smem_u32(&bars->tmem_empty);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < k8Stages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    mbar_init(bar_tfull, 1);
    mbar_init(bar_tempty, k8EpiWarps);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_b);
  }
  if (warp == 1) tmem_alloc<1>(smem_u32(&bars->tmem_base), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  pdl_sync();

  const int m_tiles = p.header[kHdrMTiles];
  const int total_tiles = m_tiles * p.n_tiles_n;
  const int k_stages = p.K >> 7;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    const bool issuer = elect_one();
    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int mt = tile / p.n_tiles_n, nt = tile - mt * p.n_tiles_n;
      const int e = p.tile_expert[mt];
      const int brow0 = e * p.b_rows_per_expert + nt * (EPI == kEpiSwiGLU ? 128 : 256);
      const int brow1 = brow0 + p.half1_row_offset;
      const bool half1 = (EPI == kEpiSwiGLU) || (nt * 256 + 128 < p.n_out);
      const int rt0 = (brow0 - e * p.b_rows_per_expert) >> 7, rt1 = (brow1 - e * p.b_rows_per_expert) >> 7;
      const uint8_t* bsf = p.b_sf + (size_t)e * p.b_sf_expert_stride;
      const uint8_t* asf = p.a_sf + (size_t)mt * k_stages * 512u;
      for (int ks = 0; ks < k_stages; ++ks) {
        ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status);
        if (!ok) break;
        if (issuer) {
          const uint32_t sb = smem_base + stage * k8StageBytes, full = bar_full + 8 * stage;
          mbar_expect_tx(full, (uint32_t)(k8TileA + (half1 ? k8TileB : k8TileB / 2) + 512 + (half1 ? 1024 : 512)));
          tma_load_2d(sb, &tm_a, ks * 128, mt * k8BM, full);
          tma_load_2d(sb + k8OffB, &tm_b, ks * 128, brow0, full);
          if (half1) tma_load_2d(sb + k8OffB + k8TileA, &tm_b, ks * 128, brow1, full);
          bulk_load(sb + k8OffSfA, asf + (size_t)ks * 512u, 512u, full);
          bulk_load(sb + k8OffSfB, bsf + ((size_t)rt0 * k_stages + ks) * 512u, 512u, full);
          if (half1) bulk_load(sb + k8OffSfB + 512, bsf + ((size_t)rt1 * k_stages + ks) * 512u, 512u, full);
        }
        __syncwarp();
        if (++stage == k8Stages) { stage = 0; phase ^= 1u; }
      }
    }
    for (int s = 0; s < k8Stages && ok; ++s) {
      ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status);
      if (++stage == k8Stages) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    const bool issuer = elect_one();
    uint32_t stage = 0, phase = 0, kcount = 0;
    int it = 0;
    bool ok = true;
    // E4M3 x E4M3, UE8M0 block scales (bit 23), K-major operands, M = 128, N = 256; the scale byte
    // within the 32-bit scale word is chosen per MMA (bits 4..5 for B, 29..30 for A)
    constexpr uint32_t idesc0 = (1u << 23) | ((uint32_t)(k8BN >> 3) << 17) | ((uint32_t)(k8BM >> 4) << 24);
    constexpr uint32_t kSwHi = (uint32_t)((8 * 128) >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t kSfHi = (uint32_t)(128 >> 4) | (1u << 14);
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
      ok = mbar_wait(bar_tempty, (uint32_t)(it & 1) ^ 1u, abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      for (int ks = 0; ks < k_stages; ++ks, ++kcount) {
        ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        if (issuer) {
          const uint32_t sb = smem_base + stage * k8StageBytes;
          const uint32_t sfcol = tmem + 256 + (kcount & 1u) * 16;
          const uint32_t a_lo = ((sb & 0x3FFFFu) >> 4) | (1u << 16);
          const uint32_t b_lo = (((sb + k8OffB) & 0x3FFFFu) >> 4) | (1u << 16);
          tc_cp_sf<1>(sfcol, ((uint64_t)kSfHi << 32) | (((sb + k8OffSfA) & 0x3FFFFu) >> 4));
          tc_cp_sf<1>(sfcol + 4, ((uint64_t)kSfHi << 32) | (((sb + k8OffSfB) & 0x3FFFFu) >> 4));
          tc_cp_sf<1>(sfcol + 8, ((uint64_t)kSfHi << 32) | (((sb + k8OffSfB + 512) & 0x3FFFFu) >> 4));
#pragma unroll
          for (int j = 0; j < 4; ++j)
            tc_mma_mxf8(tmem, ((uint64_t)kSwHi << 32) | (a_lo + 2 * j), ((uint64_t)kSwHi << 32) | (b_lo + 2 * j),
                        idesc0 | ((uint32_t)j << 4) | ((uint32_t)j << 29), sfcol, sfcol + 4, (ks > 0 || j > 0) ? 1u : 0u);
          tc_commit<1>(bar_empty + 8 * stage);
        }
        __syncwarp();
        if (++stage == k8Stages) { stage = 0; phase ^= 1u; }
      }
      if (ok && issuer) tc_commit<1>(bar_tfull);
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3, cq = (warp - 2) >> 2;
    const int row_in_tile = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
      const int mt = tile / p.n_tiles_n, nt = tile - mt * p.n_tiles_n;
      const int e = p.tile_expert[mt];
      const int n_valid = p.tile_rows[mt];
      const bool valid = row_in_tile < n_valid;
      const int prow = mt * k8BM + row_in_tile;
      if (ok) ok = mbar_wait(bar_tfull, (uint32_t)(it & 1), abort_flag, p.status);
      float acc[64];
      if (ok) {
        tc_fence_after();
        if (EPI == kEpiSwiGLU) {
          tmem_ld32(lane_addr + cq * 32, acc);
          tmem_ld32(lane_addr + 128 + cq * 32, acc + 32);
        } else {
          tmem_ld32(lane_addr + cq * 64, acc);
          tmem_ld32(lane_addr + cq * 64 + 32, acc + 32);
        }
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty);
      }
      if (EPI == kEpiSwiGLU) {
        // every epilogue thread takes part in the tile's barrier, whether or not its wait succeeded
        const int I = p.n_out;
        float hb[32];
        float a = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float g = ok ? acc[i] : 0.f, u = ok ? acc[32 + i] : 0.f;
          hb[i] = __bfloat162float(__float2bfloat16_rn(__fdividef(g, 1.0f + __expf(-g)) * u));
          a = fmaxf(a, fabsf(hb[i]));
        }
        float* slot = row_amax + (it & 1) * 512;
        slot[row_in_tile * 4 + cq] = a;
        asm volatile("bar.sync 1, %0;" ::"n"(32 * k8EpiWarps) : "memory");
        const float4 m4 = *reinterpret_cast<const float4*>(slot + row_in_tile * 4);
        const uint32_t code = fp8_scale_code(fmaxf(fmaxf(m4.x, m4.y), fmaxf(m4.z, m4.w)));
        const int ex = (int)code - 127;
        if (ok && valid) {
          uint32_t w8[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)
            w8[i] = f32x4_to_e4m3x4(ldexpf(hb[4 * i], -ex), ldexpf(hb[4 * i + 1], -ex), ldexpf(hb[4 * i + 2], -ex),
                                    ldexpf(hb[4 * i + 3], -ex));
          const int f0 = nt * 128 + cq * 32;
          uint4* dq = reinterpret_cast<uint4*>(p.hq_pad + (size_t)prow * I + f0);
          dq[0] = make_uint4(w8[0], w8[1], w8[2], w8[3]);
          dq[1] = make_uint4(w8[4], w8[5], w8[6], w8[7]);
          if (cq == 0)
            reinterpret_cast<uint32_t*>(p.hsf_atoms + ((size_t)mt * (I >> 7) + nt) * 512)[(row_in_tile & 31) * 4 + (row_in_tile >> 5)] =
                code * 0x01010101u;
          if (p.h_export) {
            const int drow = p.offsets[e] + (mt - p.tile_prefix[e]) * k8BM + row_in_tile;
            uint4* d = reinterpret_cast<uint4*>(p.h_export + (size_t)drow * I + f0);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              d[i] = make_uint4(f32x2_to_bf16x2(hb[8 * i], hb[8 * i + 1]), f32x2_to_bf16x2(hb[8 * i + 2], hb[8 * i + 3]),
                                f32x2_to_bf16x2(hb[8 * i + 4], hb[8 * i + 5]), f32x2_to_bf16x2(hb[8 * i + 6], hb[8 * i + 7]));
            uint4* dc = reinterpret_cast<uint4*>(p.hq_export + (size_t)drow * I + f0);
            dc[0] = make_uint4(w8[0], w8[1], w8[2], w8[3]);
            dc[1] = make_uint4(w8[4], w8[5], w8[6], w8[7]);
            if (cq == 0) p.hexp_export[(size_t)drow * (I >> 7) + nt] = (uint8_t)code;
          }
        } else if (ok && cq == 0) {
          // padding rows of the tile: a defined scale byte (their products are never stored)
          reinterpret_cast<uint32_t*>(p.hsf_atoms + ((size_t)mt * (I >> 7) + nt) * 512)[(row_in_tile & 31) * 4 + (row_in_tile >> 5)] = 0u;
        }
      } else if (ok) {
        const int n0 = nt * 256 + cq * 64;
        if (n0 < p.n_out)
          store_y_rows(acc, 1.0f, p.y_pad + (size_t)(mt * k8BM + q * 32) * p.n_out + n0, p.n_out, n_valid - q * 32, lane);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc<1>(tmem, 512);
}

}  // namespace

quads_status launch_gemm_fp8(int epi, const Fp8GemmParams& p, const CUtensorMap& tm_a, const CUtensorMap& tm_b, int n_sms,
                             cudaStream_t stream) {
  if (epi == kEpiSwiGLU) {
    QUADS_CUDA_OK(set_max_dynamic_smem<gemm_fp8_kernel<kEpiSwiGLU>>(k8SmemBytes));
    QUADS_CUDA_OK(launch_kernel(gemm_fp8_kernel<kEpiSwiGLU>, dim3(n_sms), dim3(k8Threads), (size_t)k8SmemBytes, stream, p, tm_a, tm_b));
  } else {
    QUADS_CUDA_OK(set_max_dynamic_smem<gemm_fp8_kernel<kEpiCombine>>(k8SmemBytes));
    QUADS_CUDA_OK(launch_kernel(gemm_fp8_kernel<kEpiCombine>, dim3(n_sms), dim3(k8Threads), (size_t)k8SmemBytes, stream, p, tm_a, tm_b));
  }
  return QUADS_OK;
}

}  // namespace quads
