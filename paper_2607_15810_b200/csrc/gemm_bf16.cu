// Dense bf16 x bf16 GEMM on the 5th-generation tensor cores (tcgen05, kind::f16) for the
// one-sided rollout modes of the paper's ablations: out[T, N] = A[T, K] B[N, K]^T with float32
// accumulation in tensor memory, bf16 output.
//   W4A16: A = the activations as they are (bf16), B = the NVFP4 weights decoded to bf16;
//   W16A4: A = the decoded NVFP4 activations (Q_A then decode, bf16), B = the bf16 weights.
// The decoded operand is produced by the library's own decode / fake-quant kernels into the
// caller's workspace; this kernel is the contraction.
//
// One persistent CTA per SM, 10 warps: warp 0 issues TMA tile loads (128-byte swizzle, 64 bf16 per
// row and stage) into a 4-stage ring; warp 1 issues four 128 x 256 x 16 MMAs per stage and releases
// stages with tcgen05.commit; warps 2..9 drain one of TWO 128 x 256 float32 accumulators (all 512
// columns of tensor memory) while the MMAs of the next tile fill the other.  Every wait is
// bounded; a wait that gives up records QUADS_ERR_TIMEOUT and all roles leave.
#include "kernels.cuh"
#include "tcgen05.cuh"

namespace quads {
namespace {

constexpr int kFBM = 128, kFBN = 256;
constexpr int kFStageK = 64;                         // bf16 elements per row per stage (128 bytes)
constexpr int kFTileA = kFBM * 128;                  // 16 KB
constexpr int kFTileB = kFBN * 128;                  // 32 KB
constexpr int kFStageBytes = kFTileA + kFTileB;
constexpr int kFStages = 4;
constexpr int kFThreads = 320;
constexpr int kFEpiWarps = 8;
constexpr int kFSmemBytes = kFStages * kFStageBytes + 256 + 1024;

struct __align__(8) FBarriers {
  uint64_t full[kFStages];
  uint64_t empty[kFStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__global__ void __launch_bounds__(kFThreads, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, int T, int N, int K,
                 uint16_t* __restrict__ out, int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_dyn[];
  const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
  FBarriers* bars = reinterpret_cast<FBarriers*>(smem_gen + kFStages * kFStageBytes);
  const uint32_t bar_full = smem_u32(&bars->full[0]), bar_empty = smem_u32(&bars->empty[0]);
  const uint32_t bar_tfull = smem_u32(&bars->tmem_full[0]), bar_tempty = smem_u32(&bars->tmem_empty[0]);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kFStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, kFEpiWarps); }
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
  pdl_sync();                                        // the decoded operand comes from the preceding kernel

  const int m_tiles = (T + kFBM - 1) / kFBM, n_tiles = (N + kFBN - 1) / kFBN;
  const int total = m_tiles * n_tiles;
  const int k_stages = K / kFStageK;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    const bool issuer = elect_one();
    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
      const int mt = tile / n_tiles, nt = tile - mt * n_tiles;
      const bool half1 = nt * kFBN + 128 < N;           // the tile's second 128 weight rows exist
      for (int ks = 0; ks < k_stages; ++ks) {
        ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, status);
        if (!ok) break;
        if (issuer) {
          const uint32_t sb = smem_base + stage * kFStageBytes, full = bar_full + 8 * stage;
          mbar_expect_tx(full, (uint32_t)(kFTileA + (half1 ? kFTileB : kFTileB / 2)));
          tma_load_2d(sb, &tm_a, ks * kFStageK, mt * kFBM, full);
          tma_load_2d(sb + kFTileA, &tm_b, ks * kFStageK, nt * kFBN, full);
          if (half1) tma_load_2d(sb + kFTileA + kFTileB / 2, &tm_b, ks * kFStageK, nt * kFBN + 128, full);
        }
        __syncwarp();
        if (++stage == kFStages) { stage = 0; phase ^= 1u; }
      }
    }
    for (int s = 0; s < kFStages && ok; ++s) {           // drain: every armed stage lands and is consumed
      ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, status);
      if (++stage == kFStages) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    const bool issuer = elect_one();
    uint32_t stage = 0, phase = 0;
    int it = 0;
    bool ok = true;
    // bf16 x bf16 -> float32, both operands K-major, M = 128, N = 256
    constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kFBN >> 3) << 17) | ((uint32_t)(kFBM >> 4) << 24);
    constexpr uint32_t kSwHi = (uint32_t)((8 * 128) >> 4) | (1u << 14) | (2u << 29);
    for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++it) {
      const int buf = it & 1;
      const uint32_t acc = tmem + (uint32_t)(buf * kFBN);
      ok = mbar_wait(bar_tempty + 8 * buf, (uint32_t)((it >> 1) & 1) ^ 1u, abort_flag, status);
      if (!ok) break;
      tc_fence_after();
      for (int ks = 0; ks < k_stages; ++ks) {
        ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, status);
        if (!ok) break;
        tc_fence_after();
        if (issuer) {
          const uint32_t sb = smem_base + stage * kFStageBytes;
          const uint32_t a_lo = ((sb & 0x3FFFFu) >> 4) | (1u << 16);
          const uint32_t b_lo = (((sb + kFTileA) & 0x3FFFFu) >> 4) | (1u << 16);
#pragma unroll
          for (int j = 0; j < 4; ++j)                    // 16 bf16 = 32 bytes along K per MMA
            tc_mma_bf16(acc, ((uint64_t)kSwHi << 32) | (a_lo + 2 * j), ((uint64_t)kSwHi << 32) | (b_lo + 2 * j), idesc,
                        (ks > 0 || j > 0) ? 1u : 0u);
          tc_commit<1>(bar_empty + 8 * stage);
        }
        __syncwarp();
        if (++stage == kFStages) { stage = 0; phase ^= 1u; }
      }
      if (ok && issuer) tc_commit<1>(bar_tfull + 8 * buf);
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ epilogue: thread = row, 128 columns per warp
    const int q = warp & 3, ch = (warp - 2) >> 2;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++it) {
      const int mt = tile / n_tiles, nt = tile - mt * n_tiles;
      const int buf = it & 1;
      const int row = mt * kFBM + q * 32 + lane;
      ok = mbar_wait(bar_tfull + 8 * buf, (uint32_t)((it >> 1) & 1), abort_flag, status);
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int c4 = 0; c4 < 4; ++c4) {
        const int n0 = nt * kFBN + ch * 128 + c4 * 32;
        float v[32];
        tmem_ld32(lane_addr + buf * kFBN + ch * 128 + c4 * 32, v);
        tmem_ld_wait();
        if (row < T && n0 < N) {
          uint4* dst = reinterpret_cast<uint4*>(out + (size_t)row * N + n0);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            dst[i] = make_uint4(f32x2_to_bf16x2(v[8 * i], v[8 * i + 1]), f32x2_to_bf16x2(v[8 * i + 2], v[8 * i + 3]),
                                f32x2_to_bf16x2(v[8 * i + 4], v[8 * i + 5]), f32x2_to_bf16x2(v[8 * i + 6], v[8 * i + 7]));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);   // this accumulator is free again
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc<1>(tmem, 512);
}

}  // namespace

quads_status launch_gemm_bf16(const CUtensorMap& tm_a, const CUtensorMap& tm_b, int T, int N, int K, uint16_t* out,
                              int32_t* status, int n_sms, cudaStream_t stream) {
  QUADS_CUDA_OK(set_max_dynamic_smem<gemm_bf16_kernel>(kFSmemBytes));
  const int tiles = ((T + kFBM - 1) / kFBM) * ((N + kFBN - 1) / kFBN);
  const int grid = tiles < n_sms ? (tiles > 0 ? tiles : 1) : n_sms;
  QUADS_CUDA_OK(launch_kernel(gemm_bf16_kernel, dim3(grid), dim3(kFThreads), (size_t)kFSmemBytes, stream, tm_a, tm_b, T, N,
                              K, out, status));
  return QUADS_OK;
}

}  // namespace quads
