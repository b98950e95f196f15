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
// Two variants share the code: CG = 1 (one CTA per tile of 128 x 256) and CG = 2
// (a cluster of two CTAs computes a 256 x 256 tile with `cta_group::2` MMAs:
// each CTA holds its own 128 rows of A^ / R^ and HALF of the weight tile, and one
// thread issues the MMAs and scale copies of both SMs; per 128-row tile it is about a
// tenth faster, but every expert's rows must then be padded to a multiple of 256).
// Every CTA loads what it needs itself; no load is shared across the cluster.
//
// One persistent CTA per SM, 19 warps:
//   warp 0     producer: TMA tile loads of packed FP4 (128-byte swizzle) into a 3-stage
//              shared-memory ring;
//   warp 18    second producer: the bulk copies of the stage's 512-byte scale atoms (in the
//              CTA-pair variant warp 0 issues those too, as TMA boxes, and this warp idles);
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
#include "tcgen05.cuh"

namespace quads {

namespace {

constexpr int kBM = 128;
constexpr int kBN = 256;
constexpr int kKSteps = kGemmKSteps;              // K = 64 MMAs per pipeline stage
constexpr int kStageKBytes = kGemmStageKBytes;    // bytes of packed FP4 per row per stage
constexpr int kTileA = kBM * kStageKBytes;
constexpr int kSfA = kKSteps * 512;               // one atom (128 rows x 4 blocks) per K step
constexpr int kSfB = 2 * kSfA;                    // scales of all 256 weight rows
constexpr int kOffR = kTileA;
constexpr int kOffB = 2 * kTileA;
constexpr int kThreads = 608;
constexpr int kEpiWarps = 16;
constexpr int kTmemCols = 512;
constexpr int kMaxTableTiles = 2048;               // M-tiles whose expert / row count fit the shared-memory tables
constexpr int kTmemSfBase = 256;                  // accumulator: columns 0..255
constexpr int kTmemSfPerBuf = 16 * kKSteps;       // SFA 4/step | SFR 4/step | SFB 8/step, double buffered

template <int CG>
struct Cfg {
  static constexpr int kTileB = kBN * kStageKBytes / CG;     // weight rows held by one CTA
  static constexpr int kStages = (CG == 1 ? 12 : 16) / kKSteps;   // ~216 KB of ring either way
  static constexpr int kOffSfA = kOffB + kTileB;
  static constexpr int kOffSfR = kOffSfA + kSfA;
  static constexpr int kOffSfB = kOffSfR + kSfA;
  static constexpr int kStageBytes = kOffSfB + kSfB;         // 73728 / 57344
  static constexpr int kBarOffset = kStages * kStageBytes;   // barriers after the ring
  static constexpr int kMetaBytes = 512 + (CG == 1 ? (2 * kMaxTableTiles + 4 * kMaxExperts) : 0);   // reciprocal table + per-tile tables
  static constexpr int kSmemBytes = kBarOffset + 256 + kMetaBytes + 1024; // + barrier block + tables + alignment slack
};

// Shared-memory matrix descriptors are built where they are used (MMA issuer): 64-bit
//   [0,14) start address >> 4 | [16,30) leading byte offset >> 4 | [32,46) stride byte offset >> 4
//   | [46,48) version = 1 | [61,64) layout (0 none, 2 = 128-byte swizzle, 4 = 64-byte swizzle).
// Operand tiles are K-major rows with the TMA swizzle, 8-row groups 8 * row bytes apart; a scale
// atom for tcgen05.cp is 32 rows of 16 bytes, no swizzle, 8-row groups 128 bytes apart.
// Instruction descriptor: E2M1 x E2M1, UE4M3 block scales, both operands
// K-major, M = 128 per CTA of the group, N = 256, dense.
template <int CG>
__host__ __device__ constexpr uint32_t idesc_nvf4() {
  return (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)((kBM * CG) >> 4) << 24);
}


struct __align__(8) BarrierBlock {
  uint64_t full[8];
  uint64_t empty[8];
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

template <int EPI, int CG>
__device__ __forceinline__ void gemm_body(const GemmParams& p, const CUtensorMap* tm_a, const CUtensorMap* tm_r,
                                          const CUtensorMap* tm_b, const CUtensorMap* tm_sfa,
                                          const CUtensorMap* tm_sfr, const CUtensorMap* tm_sfb) {
  using C = Cfg<CG>;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_dyn[];
  const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
  BarrierBlock* bars = reinterpret_cast<BarrierBlock*>(smem_gen + C::kBarOffset);
  const uint32_t bar_full = smem_u32(&bars->full[0]);
  const uint32_t bar_empty = smem_u32(&bars->empty[0]);
  const uint32_t bar_tfull = smem_u32(&bars->tmem_full);
  const uint32_t bar_tempty = smem_u32(&bars->tmem_empty);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = CG == 1 ? 0u : cluster_ctarank();      // position inside the CTA pair
  const bool leader = rank == 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      // leader: its own producer's arrive + (CG == 2) the peer's "my half has landed" arrive
      mbar_init(bar_full + 8 * s, leader ? CG : 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    mbar_init(bar_tfull, 1);
    mbar_init(bar_tempty, kEpiWarps * CG);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(tm_a);
    prefetch_tmap(tm_b);
    if (p.has_resid) prefetch_tmap(tm_r);
  }
  if (warp == 1) tmem_alloc<CG>(smem_u32(&bars->tmem_base), kTmemCols);
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();          // both CTAs' barriers exist before any remote arrive
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  // Per-tile metadata (expert, valid rows) and the per-expert weight scales are read by every
  // role at every tile; dependent global loads there would sit on the critical path of short K
  // loops, so they are staged in shared memory once (single-CTA variant, when they fit).
  const int m_tiles_all = p.header[kHdrMTiles];
  float* inv_lut = reinterpret_cast<float*>(smem_gen + C::kBarOffset + 256);   // 128 entries, SwiGLU epilogue
  if (EPI == kEpiSwiGLU && threadIdx.x < 128) inv_lut[threadIdx.x] = quant_inv_entry(threadIdx.x, p.h_gs[0]);
  uint8_t* tab_expert = smem_gen + C::kBarOffset + 256 + 512;
  uint8_t* tab_rows = tab_expert + kMaxTableTiles;
  float* tab_gs = reinterpret_cast<float*>(tab_rows + kMaxTableTiles);
  const bool tables = (CG == 1) && m_tiles_all <= kMaxTableTiles && p.n_experts <= kMaxExperts;
  if (tables) {
    for (int i = threadIdx.x; i < m_tiles_all; i += blockDim.x) {
      tab_expert[i] = (uint8_t)p.tile_expert[i];
      tab_rows[i] = (uint8_t)p.tile_rows[i];
    }
    for (int i = threadIdx.x; i < p.n_experts; i += blockDim.x) tab_gs[i] = p.b_gs[i];
  }
  // Everything above reads only what kernels before the preceding one produced (routing tables,
  // weight scales, the static scale of h): it overlaps the preceding kernel's tail.  The operands
  // and the activation amax need that kernel.
  pdl_sync();
  __syncthreads();                          // tables and the reciprocal table are visible to every role
  auto expert_of = [&](int mt) -> int { return tables ? (int)tab_expert[mt] : p.tile_expert[mt]; };
  auto rows_of = [&](int mt) -> int { return tables ? (int)tab_rows[mt] : p.tile_rows[mt]; };
  auto gs_of = [&](int e) -> float { return tables ? tab_gs[e] : p.b_gs[e]; };

  const int m_groups = m_tiles_all / CG;            // M-tiles come in groups of CG (same expert)
  const int total_tiles = m_groups * p.n_tiles_n;
  const int kt_count = p.K >> 6;                    // scale atoms (K = 64 each) along K
  const int k_stages = (kt_count + kKSteps - 1) / kKSteps;
  const bool resid = p.has_resid != 0;
  const int first_tile = blockIdx.x / CG, tile_step = gridDim.x / CG;

  // Two loading warps share a stage's copies: warp 0 the operand tiles (and the byte count), warp 18
  // the scale atoms (single-CTA variant; an asynchronous copy costs its issuing thread tens of
  // nanoseconds whatever its size: first projection 195 -> 193 us, second 116 -> 113.5 us).  All
  // copies of a stage credit the same barrier.
  const int load_role = warp == 0 ? 0 : (warp == 18 ? 1 : -1);
  if (load_role >= 0) {
    // ------------------------------------------------------------ producers (whole warp, one lane issues)
    if (CG == 1 || load_role == 0)                  // (the pair variant keeps one loading warp; warp 18 idles there)
    {
      const bool issuer = elect_one();
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      const uint32_t leader_full = CG == 2 ? map_to_cta(bar_full, 0) : bar_full;
      const int b_atoms_per_expert = (int)(p.b_sf_expert_stride >> 9);
      for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step) {
        const int mg = tile / p.n_tiles_n, nt = tile - mg * p.n_tiles_n;
        const int mt = mg * CG + (int)rank;
        const int e = expert_of(mt) - p.expert_lo;          // index into this call's weights
        const int brow0 = e * p.b_rows_per_expert + nt * (EPI == kEpiSwiGLU ? 128 : 256);
        const int brow1 = brow0 + p.half1_row_offset;
        const bool half1 = (EPI == kEpiSwiGLU) || (nt * 256 + 128 < p.n_out);
        const int rt0 = (brow0 - e * p.b_rows_per_expert) >> 7, rt1 = (brow1 - e * p.b_rows_per_expert) >> 7;
        const uint8_t* bsf = p.b_sf + (size_t)e * p.b_sf_expert_stride;
        const uint8_t* bsf0 = bsf + (size_t)rt0 * kt_count * 512u;
        const uint8_t* bsf1 = bsf + (size_t)rt1 * kt_count * 512u;
        const uint8_t* asf = p.a_sf + (size_t)mt * kt_count * 512u;
        const uint8_t* rsf = p.r_sf + (size_t)mt * kt_count * 512u;
        // weight rows this CTA keeps in shared memory
        const bool load_b0 = CG == 1 || rank == 0;
        const bool load_b1 = half1 && (CG == 1 || rank == 1);
        const uint32_t data_bytes = kTileA + (resid ? kTileA : 0) + ((load_b0 ? 1 : 0) + (load_b1 ? 1 : 0)) * (kBM * kStageKBytes);
        const uint32_t sf_count = 1u + (resid ? 1u : 0u) + (half1 ? 2u : 1u);
        for (int ks = 0; ks < k_stages; ++ks) {
          ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status);
          if (!ok) break;
          const int atoms = min(kKSteps, kt_count - ks * kKSteps);
          const uint32_t sf_bytes = (uint32_t)atoms * 512u;
          const uint32_t sbase = smem_base + stage * C::kStageBytes;
          const uint32_t full = bar_full + 8 * stage;
          const int kc = ks * kStageKBytes;
          const size_t sf_off = (size_t)ks * (size_t)kSfA;
          if (issuer) {
            if (CG == 1) {
              const bool do_tiles = load_role == 0, do_sf = load_role == 1;
              if (do_tiles) {
                mbar_expect_tx(full, data_bytes + sf_bytes * sf_count);
                tma_load_2d(sbase, tm_a, kc, mt * kBM, full);
                if (resid) tma_load_2d(sbase + kOffR, tm_r, kc, mt * kBM, full);
                tma_load_2d(sbase + kOffB, tm_b, kc, brow0, full);
                if (half1) tma_load_2d(sbase + kOffB + kTileA, tm_b, kc, brow1, full);
              }
              if (do_sf) {
                bulk_load(sbase + C::kOffSfA, asf + sf_off, sf_bytes, full);
                if (resid) bulk_load(sbase + C::kOffSfR, rsf + sf_off, sf_bytes, full);
                bulk_load(sbase + C::kOffSfB, bsf0 + sf_off, sf_bytes, full);
                if (half1) bulk_load(sbase + C::kOffSfB + kSfA, bsf1 + sf_off, sf_bytes, full);
              }
            } else {
              // every load of either CTA credits the LEADER's barrier; scale atoms travel as TMA
              // boxes (kKSteps atoms of 512 bytes; a K tail reads, and counts, the full box)
              const uint32_t lfull = leader_full + 8 * stage;
              mbar_expect_tx_cluster(lfull, data_bytes + (uint32_t)kSfA * sf_count);
              tma_load_2d_pair(sbase, tm_a, kc, mt * kBM, lfull);
              if (resid) tma_load_2d_pair(sbase + kOffR, tm_r, kc, mt * kBM, lfull);
              if (load_b0) tma_load_2d_pair(sbase + kOffB, tm_b, kc, brow0, lfull);
              if (load_b1) tma_load_2d_pair(sbase + kOffB, tm_b, kc, brow1, lfull);
              const int a_atom = mt * kt_count + ks * kKSteps;
              const int b_atom = e * b_atoms_per_expert + ks * kKSteps;
              tma_load_2d_pair(sbase + C::kOffSfA, tm_sfa, 0, a_atom, lfull);
              if (resid) tma_load_2d_pair(sbase + C::kOffSfR, tm_sfr, 0, a_atom, lfull);
              tma_load_2d_pair(sbase + C::kOffSfB, tm_sfb, 0, b_atom + rt0 * kt_count, lfull);
              if (half1) tma_load_2d_pair(sbase + C::kOffSfB + kSfA, tm_sfb, 0, b_atom + rt1 * kt_count, lfull);
            }
          }
          __syncwarp();
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      // drain: let every armed stage land and be consumed before the CTA may exit
      for (int s = 0; s < kStages && ok; ++s) {
        ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status);
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1 && !leader) {
    // the leader CTA issues the MMAs of the pair; nothing to do here
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA; whole warp, one lane issues)
    {
      const bool issuer = elect_one();
      uint32_t stage = 0, phase = 0, kcount = 0;
      int it = 0;
      bool ok = true;
      constexpr uint32_t idesc = idesc_nvf4<CG>();
      // constant high words of the two descriptor kinds; the low word carries the address
      // swizzled K-major operand tiles: 8-row groups 8 * row bytes apart; 128-byte rows use the
      // 128-byte swizzle (type 2), 64-byte rows the 64-byte swizzle (type 4)
      constexpr uint32_t kSw128Hi = (uint32_t)((8 * kStageKBytes) >> 4) | (1u << 14) | ((kStageKBytes == 128 ? 2u : 4u) << 29);
      constexpr uint32_t kSfHi = (uint32_t)(128 >> 4) | (1u << 14);
      for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step, ++it) {
        for (int ks = 0; ks < k_stages; ++ks, ++kcount) {
          ok = CG == 1 ? mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status)
                       : mbar_wait_cluster(bar_full + 8 * stage, phase, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          const int atoms = min(kKSteps, kt_count - ks * kKSteps);
          const uint32_t sbase = smem_base + stage * C::kStageBytes;
          const uint32_t sfcol = tmem + kTmemSfBase + (kcount & 1u) * kTmemSfPerBuf;
          // descriptor low words: (address >> 4) [| LBO field for the swizzled operands]
          const uint32_t a_lo = ((sbase & 0x3FFFFu) >> 4) | (1u << 16);
          const uint32_t r_lo = (((sbase + kOffR) & 0x3FFFFu) >> 4) | (1u << 16);
          const uint32_t b_lo = (((sbase + kOffB) & 0x3FFFFu) >> 4) | (1u << 16);
          const uint32_t sfa_lo = ((sbase + C::kOffSfA) & 0x3FFFFu) >> 4;
          const uint32_t sfr_lo = ((sbase + C::kOffSfR) & 0x3FFFFu) >> 4;
          const uint32_t sfb_lo = ((sbase + C::kOffSfB) & 0x3FFFFu) >> 4;
          const bool first = ks == 0;
          // Scale-factor copies run one K step ahead of the MMAs that use them, so that the
          // shared-memory -> tensor-memory copy of step j+1 overlaps the MMAs of step j.
          auto copy_sf = [&](int j) {
            tc_cp_sf<CG>(sfcol + 4 * j, ((uint64_t)kSfHi << 32) | (sfa_lo + 32 * j));
            if (resid) tc_cp_sf<CG>(sfcol + 4 * kKSteps + 4 * j, ((uint64_t)kSfHi << 32) | (sfr_lo + 32 * j));
            tc_cp_sf<CG>(sfcol + 8 * kKSteps + 8 * j, ((uint64_t)kSfHi << 32) | (sfb_lo + 32 * j));
            tc_cp_sf<CG>(sfcol + 8 * kKSteps + 8 * j + 4, ((uint64_t)kSfHi << 32) | (sfb_lo + (kSfA >> 4) + 32 * j));
          };
          if (issuer && atoms > 0) copy_sf(0);
          if (first) {
            // The first scale copies of a tile do not touch the accumulator, so they are issued
            // before waiting for the epilogue to have drained the previous tile out of it.
            ok = CG == 1 ? mbar_wait(bar_tempty, (uint32_t)(it & 1) ^ 1u, abort_flag, p.status)
                         : mbar_wait_cluster(bar_tempty, (uint32_t)(it & 1) ^ 1u, abort_flag, p.status);
            if (!ok) break;
            tc_fence_after();
          }
          if (issuer) {
#pragma unroll
            for (int j = 0; j < kKSteps; ++j) {
              if (j + 1 < atoms) copy_sf(j + 1);
              if (j < atoms) {
                const uint64_t bdesc = ((uint64_t)kSw128Hi << 32) | (b_lo + 2 * j);
                tc_mma_nvf4<CG>(tmem, ((uint64_t)kSw128Hi << 32) | (a_lo + 2 * j), bdesc, idesc, sfcol + 4 * j,
                                sfcol + 8 * kKSteps + 8 * j, (!first || j > 0) ? 1u : 0u);
                if (resid)
                  tc_mma_nvf4<CG>(tmem, ((uint64_t)kSw128Hi << 32) | (r_lo + 2 * j), bdesc, idesc,
                                  sfcol + 4 * kKSteps + 4 * j, sfcol + 8 * kKSteps + 8 * j, 1u);
              }
            }
            tc_commit<CG>(bar_empty + 8 * stage);
          }
          __syncwarp();
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok && issuer) tc_commit<CG>(bar_tfull);
        __syncwarp();
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
    const uint32_t tempty_addr = CG == 1 ? bar_tempty : map_to_cta(bar_tempty, 0);
    for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step, ++it) {
      const int mg = tile / p.n_tiles_n, nt = tile - mg * p.n_tiles_n;
      const int mt = mg * CG + (int)rank;
      const int e = expert_of(mt);
      const bool valid = row_in_tile < rows_of(mt);
      const int prow = mt * kBM + row_in_tile;
      const float scale = __fmul_rn(a_gs, gs_of(e - p.expert_lo));
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
      if (lane == 0) {                            // accumulator is free for the next tile
        if (CG == 1) mbar_arrive(bar_tempty);
        else mbar_arrive_remote_relaxed(tempty_addr);
      }

      if (EPI == kEpiSwiGLU) {
        QuantCtx qc;
        quant_ctx_scalars(qc, p.h_gs[0]);
        qc.inv_lut = inv_lut;
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
          const BlockQ bq = quantize_block(hb, qc);
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
            const BlockQ br = quantize_block(r, qc);
            rs |= br.sf8 << (8 * c);
            if (valid)
              *reinterpret_cast<uint2*>(p.r2q_pad + (size_t)prow * (I >> 1) + ((f0 + 16 * c) >> 1)) =
                  make_uint2(br.lo ^ 0x88888888u, br.hi ^ 0x88888888u);
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = valid ? r[i] * r[i] : 0.f;
            const float cs = warp_colsum16(r, lane);
            if ((lane & 1) == 0) {
              const int col = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
              add_score(p.keys2 + f0 + 16 * c + col, cs, qc.gs, p.score_bits);
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
        if (n0 < p.n_out)
          store_y_rows(acc, scale, p.y_pad + (size_t)(mt * kBM + q * 32) * p.n_out + n0, p.n_out, rows_of(mt) - q * 32, lane);
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
  if (CG == 2) cluster_sync_all();          // the peer may still be signalling this CTA's barriers
  tc_fence_after();
  if (warp == 1) tmem_dealloc<CG>(tmem, kTmemCols);
}

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_r,
            const __grid_constant__ CUtensorMap tm_b) {
  gemm_body<EPI, 1>(p, &tm_a, &tm_r, &tm_b, nullptr, nullptr, nullptr);
}

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_kernel_pair(const GemmParams p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_r,
                 const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_sfa,
                 const __grid_constant__ CUtensorMap tm_sfr, const __grid_constant__ CUtensorMap tm_sfb) {
  gemm_body<EPI, 2>(p, &tm_a, &tm_r, &tm_b, &tm_sfa, &tm_sfr, &tm_sfb);
}

}  // namespace

template <int EPI>
quads_status launch_one(const GemmParams& p, const GemmMaps& m, int n_sms, cudaStream_t stream) {
  QUADS_CUDA_OK(set_max_dynamic_smem<gemm_kernel<EPI>>(Cfg<1>::kSmemBytes));
  QUADS_CUDA_OK(launch_kernel(gemm_kernel<EPI>, dim3(n_sms), dim3(kThreads), (size_t)Cfg<1>::kSmemBytes, stream, p, m.a,
                              m.r, m.b));
  return QUADS_OK;
}
template <int EPI>
quads_status launch_pair(const GemmParams& p, const GemmMaps& m, int n_sms, cudaStream_t stream) {
  QUADS_CUDA_OK(set_max_dynamic_smem<gemm_kernel_pair<EPI>>(Cfg<2>::kSmemBytes));
  QUADS_CUDA_OK(launch_kernel(gemm_kernel_pair<EPI>, dim3((n_sms / 2) * 2), dim3(kThreads), (size_t)Cfg<2>::kSmemBytes,
                              stream, p, m.a, m.r, m.b, m.sfa, m.sfr, m.sfb));
  return QUADS_OK;
}

quads_status launch_gemm(int epi, int cta_group, const GemmParams& p, const GemmMaps& m, int n_sms,
                         cudaStream_t stream) {
  if (cta_group == 2) {
    return epi == kEpiStore ? launch_pair<kEpiStore>(p, m, n_sms, stream)
                            : (epi == kEpiSwiGLU ? launch_pair<kEpiSwiGLU>(p, m, n_sms, stream)
                                                 : launch_pair<kEpiCombine>(p, m, n_sms, stream));
  }
  return epi == kEpiStore ? launch_one<kEpiStore>(p, m, n_sms, stream)
                          : (epi == kEpiSwiGLU ? launch_one<kEpiSwiGLU>(p, m, n_sms, stream)
                                               : launch_one<kEpiCombine>(p, m, n_sms, stream));
}

}  // namespace quads
