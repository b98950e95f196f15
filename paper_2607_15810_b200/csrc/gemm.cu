// Grouped NVFP4 x NVFP4 GEMM on the 5th-generation tensor cores (tcgen05),
// with Residual Activation Compensation folded into the main loop and three
// fused epilogues.
//
//   D[row, n] = sum_k  A^[row,k] W^[e(row), n, k]  +  sum_k  (-M R^)[row,k] W^[e(row), n, k]
//
// A^ / R^ are the quantized activation and its masked, sign-flipped quantized
// residual (padded dispatch order: every expert's rows start at a multiple of
// 128), W^ the expert's quantized weight.  Both products are block-scaled
// `tcgen05.mma.kind::mxf4nvf4` (16-element blocks, UE4M3 scales) into ONE fp32
// accumulator in tensor memory, which is possible because the residual shares
// the per-tensor scale of its activation.
//
// One persistent CTA per SM, 18 warps:
//   warp 0     producer: TMA tile loads of packed FP4 (128-byte swizzle) and bulk
//              copies of 512-byte scale atoms into a 3-stage shared-memory ring;
//   warp 1     tensor-memory allocation; one thread copies scale atoms to TMEM
//              (tcgen05.cp) and issues the MMAs, releasing stages with
//              tcgen05.commit;
//   warps 2..17 epilogue: drain the 128 x 256 accumulator into registers (64
//              columns per thread), free it for the next tile at once, then run
//              the fused epilogue.  Four warps per scheduler hide its latencies.
// Tile = 128 dispatch rows x 256 weight rows; K is consumed 256 elements per
// stage (four K=64 MMAs).  Every wait is bounded; a wait that gives up records
// QUADS_ERR_TIMEOUT in the status word and all roles leave.
#include "kernels.cuh"

namespace quads {

namespace {

constexpr int kBM = 128;
constexpr int kBN = 256;
constexpr int kStageKBytes = 128;                 // 256 FP4 elements per row per stage
constexpr int kStages = 3;
constexpr int kTileA = kBM * kStageKBytes;        // 16384
constexpr int kTileB = kBN * kStageKBytes;        // 32768
constexpr int kSfA = 4 * 512;                     // 4 atoms (128 rows x 4 blocks each)
constexpr int kSfB = 2 * kSfA;
constexpr int kOffR = kTileA;
constexpr int kOffB = 2 * kTileA;
constexpr int kOffSfA = kOffB + kTileB;
constexpr int kOffSfR = kOffSfA + kSfA;
constexpr int kOffSfB = kOffSfR + kSfA;
constexpr int kStageBytes = kOffSfB + kSfB;       // 73728
constexpr int kBarOffset = kStages * kStageBytes; // barriers after the ring
constexpr int kSmemBytes = kBarOffset + 256 + 1024;  // + barrier block + alignment slack
constexpr int kThreads = 576;
constexpr int kEpiWarps = 16;
constexpr int kTmemCols = 512;
constexpr int kTmemSfBase = 256;                  // accumulator: columns 0..255
constexpr int kTmemSfPerBuf = 64;                 // SFA 16 | SFR 16 | SFB 32, double buffered
constexpr uint64_t kWaitNs = 2000000000ull;       // bound of every device-side wait (2 s)

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t globaltimer() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the wait was abandoned (timeout, or another
// role already gave up and raised *abort_flag).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status) {
  if (mbar_try(bar, parity)) return true;
  const uint64_t t0 = globaltimer();
  uint32_t spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (globaltimer() - t0 > kWaitNs) {
        *abort_flag = 1;
        atomicExch(status, (int32_t)QUADS_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tc_mma_nvf4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate) : "memory");
}

// 32 consecutive accumulator columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, K-major operand tile stored as rows of 128
// bytes with the 128-byte swizzle (8-row groups 1024 bytes apart).
__device__ __forceinline__ uint64_t desc_sw128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Descriptor of one 512-byte scale atom for tcgen05.cp: 32 rows of 16 bytes, no
// swizzle, 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t desc_sf_atom(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(128 >> 4) << 32) | ((uint64_t)1 << 46);
}
// Instruction descriptor: E2M1 x E2M1, UE4M3 block scales, both operands
// K-major, M = 128, N = 256, dense.
constexpr uint32_t kIdesc = (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

__device__ __forceinline__ void stg256(void* addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t e,
                                       uint32_t f, uint32_t g, uint32_t h) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(addr), "r"(a), "r"(b), "r"(c), "r"(d),
               "r"(e), "r"(f), "r"(g), "r"(h) : "memory");
}

struct __align__(8) BarrierBlock {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full;
  uint64_t tmem_empty;
  uint32_t tmem_base;
  int abort_flag;
};

// Column sums of 16 per-lane values over the 32 lanes of a warp, fixed order.
// On return lane l holds the sum of column ((l>>4)&1)*8 + ((l>>3)&1)*4 + ((l>>2)&1)*2 + ((l>>1)&1).
__device__ __forceinline__ float warp_colsum16(const float* v, int lane) {
  float a[8], b[4], c[2];
  const bool h4 = lane & 16, h3 = lane & 8, h2 = lane & 4, h1 = lane & 2;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float send = h4 ? v[i] : v[i + 8];
    const float keep = h4 ? v[i + 8] : v[i];
    a[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 16);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float send = h3 ? a[i] : a[i + 4];
    const float keep = h3 ? a[i + 4] : a[i];
    b[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 8);
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const float send = h2 ? b[i] : b[i + 2];
    const float keep = h2 ? b[i + 2] : b[i];
    c[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
  }
  const float send = h1 ? c[0] : c[1];
  const float keep = h1 ? c[1] : c[0];
  float d = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 2);
  d += __shfl_xor_sync(0xFFFFFFFFu, d, 1);
  return d;
}

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_r,
            const __grid_constant__ CUtensorMap tm_b) {
  extern __shared__ uint8_t smem_dyn[];
  const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
  BarrierBlock* bars = reinterpret_cast<BarrierBlock*>(smem_gen + kBarOffset);
  const uint32_t bar_full = smem_u32(&bars->full[0]);
  const uint32_t bar_empty = smem_u32(&bars->empty[0]);
  const uint32_t bar_tfull = smem_u32(&bars->tmem_full);
  const uint32_t bar_tempty = smem_u32(&bars->tmem_empty);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    mbar_init(bar_tfull, 1);
    mbar_init(bar_tempty, kEpiWarps);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_b);
    if (p.has_resid) prefetch_tmap(&tm_r);
  }
  if (warp == 1) tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  const int m_tiles = p.header[kHdrMTiles];
  const int total_tiles = m_tiles * p.n_tiles_n;
  const int kt_count = p.K >> 6;                    // scale atoms (K = 64 each) along K
  const int k_stages = (kt_count + 3) >> 2;
  const bool resid = p.has_resid != 0;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
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
        for (int ks = 0; ks < k_stages; ++ks) {
          ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status);
          if (!ok) break;
          const int atoms = min(4, kt_count - ks * 4);
          const uint32_t sf_bytes = (uint32_t)atoms * 512u;
          const uint32_t sbase = smem_base + stage * kStageBytes;
          const uint32_t full = bar_full + 8 * stage;
          const uint32_t bytes = kTileA + (resid ? kTileA : 0) + (half1 ? kTileB : kTileB / 2) +
                                 sf_bytes * (1u + (resid ? 1u : 0u) + (half1 ? 2u : 1u));
          mbar_expect_tx(full, bytes);
          tma_load_2d(sbase, &tm_a, ks * kStageKBytes, mt * kBM, full);
          if (resid) tma_load_2d(sbase + kOffR, &tm_r, ks * kStageKBytes, mt * kBM, full);
          tma_load_2d(sbase + kOffB, &tm_b, ks * kStageKBytes, brow0, full);
          if (half1) tma_load_2d(sbase + kOffB + kTileB / 2, &tm_b, ks * kStageKBytes, brow1, full);
          const size_t a_off = ((size_t)mt * kt_count + (size_t)ks * 4) * 512u;
          bulk_load(sbase + kOffSfA, p.a_sf + a_off, sf_bytes, full);
          if (resid) bulk_load(sbase + kOffSfR, p.r_sf + a_off, sf_bytes, full);
          bulk_load(sbase + kOffSfB, bsf + ((size_t)rt0 * kt_count + (size_t)ks * 4) * 512u, sf_bytes, full);
          if (half1)
            bulk_load(sbase + kOffSfB + kSfA, bsf + ((size_t)rt1 * kt_count + (size_t)ks * 4) * 512u, sf_bytes, full);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      // drain: let every armed stage land before the CTA may exit
      for (int s = 0; s < kStages && ok; ++s) {
        ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status);
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, kcount = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
        ok = mbar_wait(bar_tempty, (uint32_t)(it & 1) ^ 1u, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        for (int ks = 0; ks < k_stages; ++ks, ++kcount) {
          ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          const int atoms = min(4, kt_count - ks * 4);
          const uint32_t sbase = smem_base + stage * kStageBytes;
          const uint32_t sfcol = tmem + kTmemSfBase + (kcount & 1u) * kTmemSfPerBuf;
          for (int j = 0; j < atoms; ++j) {
            tc_cp_sf(sfcol + 4 * j, desc_sf_atom(sbase + kOffSfA + 512 * j));
            if (resid) tc_cp_sf(sfcol + 16 + 4 * j, desc_sf_atom(sbase + kOffSfR + 512 * j));
            tc_cp_sf(sfcol + 32 + 8 * j, desc_sf_atom(sbase + kOffSfB + 512 * j));
            tc_cp_sf(sfcol + 32 + 8 * j + 4, desc_sf_atom(sbase + kOffSfB + kSfA + 512 * j));
          }
          for (int j = 0; j < atoms; ++j) {
            const uint64_t bdesc = desc_sw128(sbase + kOffB + 32 * j);
            tc_mma_nvf4(tmem, desc_sw128(sbase + 32 * j), bdesc, kIdesc, sfcol + 4 * j, sfcol + 32 + 8 * j,
                        (ks > 0 || j > 0) ? 1u : 0u);
            if (resid)
              tc_mma_nvf4(tmem, desc_sw128(sbase + kOffR + 32 * j), bdesc, kIdesc, sfcol + 16 + 4 * j,
                          sfcol + 32 + 8 * j, 1u);
          }
          tc_commit(bar_empty + 8 * stage);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(bar_tfull);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;                 // TMEM lane quadrant this warp may access
    const int cq = (warp - 2) >> 2;         // which quarter of the tile's columns (0..3)
    const int row_in_tile = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const float a_gs = p.a_gs ? p.a_gs[0]
                              : (__uint_as_float(p.a_amax_bits[0]) > 0.f
                                     ? __fdiv_rn(__uint_as_float(p.a_amax_bits[0]), kGlobalDiv) : 1.0f);
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
      const int mt = tile / p.n_tiles_n, nt = tile - mt * p.n_tiles_n;
      const int e = p.tile_expert[mt];
      const bool valid = row_in_tile < p.tile_rows[mt];
      const int prow = mt * kBM + row_in_tile;
      const float scale = __fmul_rn(a_gs, p.b_gs[e]);
      ok = mbar_wait(bar_tfull, (uint32_t)(it & 1), abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      float acc[64];
      if (EPI == kEpiSwiGLU) {
        // gate columns [cq*32, +32) -> acc[0..31]; up columns [128 + cq*32, +32) -> acc[32..63]
        tmem_ld32(lane_addr + cq * 32, acc);
        tmem_ld32(lane_addr + 128 + cq * 32, acc + 32);
      } else {
        tmem_ld32(lane_addr + cq * 64, acc);
        tmem_ld32(lane_addr + cq * 64 + 32, acc + 32);
      }
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty);     // accumulator is free for the next tile

      if (EPI == kEpiSwiGLU) {
        const float h_gs = p.h_gs[0];
        const int I = p.n_out;
        const int f0 = nt * 128 + cq * 32;        // first feature of this thread's 32
        const int kt2 = I >> 6;
        uint32_t hs = 0, rs = 0;
        int drow = 0;
        if (p.h_export) drow = p.offsets[e] + (mt - p.tile_prefix[e]) * kBM + row_in_tile;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          float hb[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float g = __fmul_rn(acc[16 * c + i], scale);
            const float u = __fmul_rn(acc[32 + 16 * c + i], scale);
            const float h = __fdividef(g, 1.0f + __expf(-g)) * u;
            hb[i] = __bfloat162float(__float2bfloat16_rn(h));
          }
          const BlockQ bq = quantize_block(hb, h_gs);
          hs |= bq.sf8 << (8 * c);
          if (valid) {
            *reinterpret_cast<uint2*>(p.hq_pad + (size_t)prow * (I >> 1) + ((f0 + 16 * c) >> 1)) =
                make_uint2(bq.lo, bq.hi);
            if (p.h_export) {
              uint4* d = reinterpret_cast<uint4*>(p.h_export + (size_t)drow * I + f0 + 16 * c);
              d[0] = make_uint4(f32x2_to_bf16x2(hb[0], hb[1]), f32x2_to_bf16x2(hb[2], hb[3]),
                                f32x2_to_bf16x2(hb[4], hb[5]), f32x2_to_bf16x2(hb[6], hb[7]));
              d[1] = make_uint4(f32x2_to_bf16x2(hb[8], hb[9]), f32x2_to_bf16x2(hb[10], hb[11]),
                                f32x2_to_bf16x2(hb[12], hb[13]), f32x2_to_bf16x2(hb[14], hb[15]));
            }
          }
          if (p.resid2) {
            float r[16];
            dequant_block(bq, r);
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = __fsub_rn(r[i], hb[i]);
            const BlockQ br = quantize_block(r, h_gs);
            rs |= br.sf8 << (8 * c);
            if (valid)
              *reinterpret_cast<uint2*>(p.r2q_pad + (size_t)prow * (I >> 1) + ((f0 + 16 * c) >> 1)) =
                  make_uint2(br.lo ^ 0x88888888u, br.hi ^ 0x88888888u);
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = valid ? r[i] * r[i] : 0.f;
            const float cs = warp_colsum16(r, lane);
            if ((lane & 1) == 0) {
              const int col = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
              p.partials2[(size_t)(mt * 4 + q) * I + f0 + 16 * c + col] = cs;
            }
          }
        }
        if (valid) {
          // this thread's two scale bytes: blocks (f0/16) and (f0/16)+1, adjacent in the atom
          const size_t so = sf_tiled_offset(prow, f0 >> 4, kt2);
          *reinterpret_cast<uint16_t*>(p.hsf_tiled + so) = (uint16_t)hs;
          if (p.resid2) *reinterpret_cast<uint16_t*>(p.r2sf_tiled + so) = (uint16_t)rs;
        }
      } else if (EPI == kEpiCombine) {
        // y = W2 h~ for this dispatched row, rounded to bf16; the weighted sum over a
        // token's experts is taken afterwards in a fixed order (no atomics).
        const int n0 = nt * 256 + cq * 64;
        if (valid && n0 < p.n_out) {
          uint16_t* dst = p.y_pad + (size_t)prow * p.n_out + n0;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            stg256(dst + 16 * i,
                   f32x2_to_bf16x2(acc[16 * i] * scale, acc[16 * i + 1] * scale),
                   f32x2_to_bf16x2(acc[16 * i + 2] * scale, acc[16 * i + 3] * scale),
                   f32x2_to_bf16x2(acc[16 * i + 4] * scale, acc[16 * i + 5] * scale),
                   f32x2_to_bf16x2(acc[16 * i + 6] * scale, acc[16 * i + 7] * scale),
                   f32x2_to_bf16x2(acc[16 * i + 8] * scale, acc[16 * i + 9] * scale),
                   f32x2_to_bf16x2(acc[16 * i + 10] * scale, acc[16 * i + 11] * scale),
                   f32x2_to_bf16x2(acc[16 * i + 12] * scale, acc[16 * i + 13] * scale),
                   f32x2_to_bf16x2(acc[16 * i + 14] * scale, acc[16 * i + 15] * scale));
        }
      } else {
        const int n0 = nt * 256 + cq * 64;
        if (valid && n0 < p.n_out) {
          uint4* dst = reinterpret_cast<uint4*>(p.out_bf16 + (size_t)p.row_token[prow] * p.n_out + n0);
#pragma unroll
          for (int i = 0; i < 8; ++i)
            dst[i] = make_uint4(f32x2_to_bf16x2(acc[8 * i] * scale, acc[8 * i + 1] * scale),
                                f32x2_to_bf16x2(acc[8 * i + 2] * scale, acc[8 * i + 3] * scale),
                                f32x2_to_bf16x2(acc[8 * i + 4] * scale, acc[8 * i + 5] * scale),
                                f32x2_to_bf16x2(acc[8 * i + 6] * scale, acc[8 * i + 7] * scale));
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

quads_status launch_gemm(int epi, const GemmParams& p, const CUtensorMap& tm_a, const CUtensorMap& tm_r,
                         const CUtensorMap& tm_b, int n_sms, cudaStream_t stream) {
  static bool attr_set[3] = {false, false, false};
  void (*fn)(const GemmParams, const CUtensorMap, const CUtensorMap, const CUtensorMap) =
      epi == kEpiStore ? gemm_kernel<kEpiStore> : (epi == kEpiSwiGLU ? gemm_kernel<kEpiSwiGLU> : gemm_kernel<kEpiCombine>);
  if (!attr_set[epi]) {
    QUADS_CUDA_OK(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    attr_set[epi] = true;
  }
  fn<<<n_sms, kThreads, kSmemBytes, stream>>>(p, tm_a, tm_r, tm_b);
  note_launch();
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}

}  // namespace quads
