// Tensor-pipe probe: how fast one SM's 5th-generation tensor core takes block-scaled FP4 MMAs when
// nothing else is in the way.  One persistent CTA per SM keeps ONE stage of operands (the grouped
// GEMM's own stage layout: 128 activation rows, 128 residual rows, 256 weight rows of 256 FP4
// values each, plus their UE4M3 scale atoms) resident in shared memory and issues, `k_steps` times,
// what the GEMM's main loop issues per K = 64 step; no global traffic inside the loop.  The
// benchmark turns its duration into the measured dense-FP4 peak that roofline fractions are quoted
// against, and the variants show what the scale copies and the single issuing thread cost.
//
//   mode 0   one MMA per step, scales copied once                      (the bare pipe)
//   mode 1   two MMAs + four scale copies per step                      (first projection with RAC)
//   mode 2   one MMA + three scale copies per step                      (plain W4A4)
//   mode 3   two MMAs per step, scales copied once                      (RAC without its copies)
//   mode 4   as mode 1, but the copies are issued by a second warp      (two issuing threads)
//   mode 5   one N = 128 MMA (128 x 128 x 64) per step, scales copied once
// (M is 128 for every block-scaled kind with cta_group::1: there is no half-height form to probe.)
// Results in tensor memory are never read; every wait is bounded.
#include "kernels.cuh"
#include "tcgen05.cuh"

namespace quads {
namespace {

constexpr int kPTileA = 128 * 128;                 // 128 rows x 128 bytes (256 FP4)
constexpr int kPOffR = kPTileA;
constexpr int kPOffB = 2 * kPTileA;
constexpr int kPOffSfA = kPOffB + 2 * kPTileA;
constexpr int kPOffSfR = kPOffSfA + 2048;
constexpr int kPOffSfB = kPOffSfR + 2048;
constexpr int kPStageBytes = kPOffSfB + 4096;      // 73728, as a stage of the grouped GEMM
constexpr int kPSmemBytes = kPStageBytes + 1024 + 64;

__global__ void __launch_bounds__(128, 1)
fp4_pipe_probe_kernel(const uint8_t* __restrict__ operands, int mode, int k_steps, int32_t* status) {
  extern __shared__ uint8_t smem_dyn[];
  const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + kPStageBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5;
  for (int i = threadIdx.x; i < kPStageBytes / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(smem_gen)[i] = reinterpret_cast<const uint4*>(operands)[i];
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> tensor-core reads
  if (warp == 1) tmem_alloc<1>(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  constexpr uint32_t idesc = (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  constexpr uint32_t kSwHi = (uint32_t)((8 * 128) >> 4) | (1u << 14) | (2u << 29);
  constexpr uint32_t kSfHi = (uint32_t)(128 >> 4) | (1u << 14);
  const uint32_t a_lo = ((smem_base & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t r_lo = (((smem_base + kPOffR) & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t b_lo = (((smem_base + kPOffB) & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t sfa_lo = ((smem_base + kPOffSfA) & 0x3FFFFu) >> 4;
  const uint32_t sfr_lo = ((smem_base + kPOffSfR) & 0x3FFFFu) >> 4;
  const uint32_t sfb_lo = ((smem_base + kPOffSfB) & 0x3FFFFu) >> 4;
  const uint32_t sfcol = tmem + 256;
  auto copy_sf = [&](int j, int buf, bool with_r) {
    const uint32_t c = sfcol + buf * 64;
    tc_cp_sf<1>(c + 4 * j, ((uint64_t)kSfHi << 32) | (sfa_lo + 32 * j));
    if (with_r) tc_cp_sf<1>(c + 16 + 4 * j, ((uint64_t)kSfHi << 32) | (sfr_lo + 32 * j));
    tc_cp_sf<1>(c + 32 + 8 * j, ((uint64_t)kSfHi << 32) | (sfb_lo + 32 * j));
    tc_cp_sf<1>(c + 32 + 8 * j + 4, ((uint64_t)kSfHi << 32) | (sfb_lo + 128 + 32 * j));
  };
  const bool two_mma = mode == 1 || mode == 3 || mode == 4;
  const uint32_t idesc_m = mode == 5 ? ((1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24)) : idesc;
  const bool copies = mode == 1 || mode == 2;
  if (warp == 1) {
    const bool issuer = elect_one();
    if (issuer) {
      for (int j = 0; j < 4; ++j) { copy_sf(j, 0, true); copy_sf(j, 1, true); }
      for (int s = 0; s < k_steps; ++s) {
        const int j = s & 3, buf = (s >> 2) & 1;
        if (copies) copy_sf(j, buf, two_mma);
        const uint32_t c = sfcol + buf * 64;
        const uint64_t bdesc = ((uint64_t)kSwHi << 32) | (b_lo + 2 * j);
        tc_mma_nvf4<1>(tmem, ((uint64_t)kSwHi << 32) | (a_lo + 2 * j), bdesc, idesc_m, c + 4 * j, c + 32 + 8 * j,
                       s > 0 ? 1u : 0u);
        if (two_mma)
          tc_mma_nvf4<1>(tmem, ((uint64_t)kSwHi << 32) | (r_lo + 2 * j), bdesc, idesc, c + 16 + 4 * j, c + 32 + 8 * j, 1u);
      }
      tc_commit<1>(smem_u32(&bars[0]));
    }
    __syncwarp();
    mbar_wait(smem_u32(&bars[0]), 0, abort_flag, status);
  } else if (warp == 2 && mode == 4) {
    // a second issuing thread: the same number of scale copies, into the buffer the MMAs are not reading
    // (no hand-shake with the MMA warp: the probe measures rates, not results)
    const bool issuer = elect_one();
    if (issuer) {
      for (int s = 0; s < k_steps; ++s) copy_sf(s & 3, ((s >> 2) & 1) ^ 1, true);
      tc_commit<1>(smem_u32(&bars[1]));
    }
    __syncwarp();
    mbar_wait(smem_u32(&bars[1]), 0, abort_flag, status);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc<1>(tmem, 512);
}

}  // namespace
}  // namespace quads

using namespace quads;

extern "C" quads_status quads_fp4_pipe_probe(int32_t mode, int32_t k_steps, const void* operands, size_t operand_bytes,
                                             int32_t* status_word, double* flop_out, void* cuda_stream) {
  g_launch_count = 0;
  if (mode < 0 || mode > 5 || k_steps < 1) return QUADS_ERR_SHAPE;
  if (!operands || !status_word) return QUADS_ERR_NULL;
  if (operand_bytes < (size_t)kPStageBytes || (reinterpret_cast<uintptr_t>(operands) & 15)) return QUADS_ERR_WORKSPACE;
  int dev = 0, sms = 0, cc = 0;
  QUADS_CUDA_OK(cudaGetDevice(&dev));
  QUADS_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  QUADS_CUDA_OK(cudaDeviceGetAttribute(&cc, cudaDevAttrComputeCapabilityMajor, dev));
  if (cc != 10) return QUADS_ERR_ARCH;
  QUADS_CUDA_OK(set_max_dynamic_smem<fp4_pipe_probe_kernel>(kPSmemBytes));
  fp4_pipe_probe_kernel<<<sms, 128, kPSmemBytes, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint8_t*>(operands), mode, k_steps, status_word);
  note_launch();
  QUADS_CUDA_OK(cudaGetLastError());
  const int mmas = (mode == 1 || mode == 3 || mode == 4) ? 2 : 1;
  const double shape = mode == 5 ? 128.0 * 128.0 : 128.0 * 256.0;
  if (flop_out) *flop_out = (double)sms * (double)k_steps * mmas * 2.0 * shape * 64.0;
  return QUADS_OK;
}

extern "C" size_t quads_fp4_pipe_probe_operand_bytes(void) { return (size_t)kPStageBytes; }
