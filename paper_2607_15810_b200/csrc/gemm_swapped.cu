// Grouped NVFP4 x NVFP4 GEMM for FEW ROWS PER EXPERT (decode-sized batches), operands swapped.
//
// When an expert receives a handful of tokens, a 128-row activation tile is almost all padding:
// the MMAs run on padding, and half of the bytes an SM pulls in are padding too, while the only
// real cost is streaming every expert's weights once.  Here the WEIGHTS take the M side of the
// MMA (128 weight rows = 128 output features per tile, fully used) and the expert's tokens take
// the N side in chunks of at most 32:
//
//   Dt[f, t] = sum_k  W^[e, f, k] X^[t, k]  +  sum_k  W^[e, f, k] (-M R^)[t, k]
//
// with the same operands, scales and dispatch layout as the row-major kernel (gemm.cu): the
// quantized activations / residuals sit in padded dispatch order (128-row slots per expert), a
// chunk is one quarter (32 consecutive rows) of a slot.  Its block scales are column `chunk` of the
// slot's 128-row scale atom, but the MMA accepts N-side scales only at even column offsets: an odd
// chunk is therefore computed as the second half of a 64-row N tile whose first 32 rows are whatever
// precedes the chunk's rows in shared memory (the operand descriptor starts 4 KB early; those
// accumulator columns are never read), with the scales read from the even column before it.
// Small activation tiles leave room for four (six) stages of weights: what bounds this kernel is
// the number of weight bytes in flight per SM, not the MMAs.
//
//   first projection : tile = 128 features; gate rows and up rows of those features go to two
//                      accumulators; epilogue = SwiGLU, bf16, then the tile is transposed through
//                      shared memory so that 16-feature blocks of one token are quantized exactly
//                      as in the row-major kernel (codes, scales, residual, column scores);
//   second projection: tile = 128 output features; epilogue = bf16 rows for the combine kernel.
//
// Roles: warp 0 producer (TMA + bulk copies, ring of stages), warp 1 MMA issuer, warps 2..9
// epilogue (thread = feature, 16 token columns each).  Two accumulator buffers.  Every wait is
// bounded (status word, as in gemm.cu).
#include "kernels.cuh"
#include "tcgen05.cuh"

namespace quads {

namespace {

constexpr int kKSteps = kGemmKSteps;
constexpr int kStageKBytes = kGemmStageKBytes;
static_assert(kKSteps == 4 && kStageKBytes == 128, "laid out for 256-element K stages");
constexpr int kChunk = 32;                          // tokens per work item (one quarter of a 128-row slot)
constexpr int kBoxRows = 16;                        // activation rows per TMA box
constexpr int kTileW = 128 * kStageKBytes;          // 128 weight rows of one stage
constexpr int kTileX = kChunk * kStageKBytes;       // one chunk of activation rows
constexpr int kSfStage = kKSteps * 512;             // one 128-row scale atom per K step
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kMaxChunkList = 2048;                 // (slot, chunk) entries, 2 bytes each
constexpr int kMaxSlots = kMaxChunkList / 4;
constexpr int kTmemCols = 512;
constexpr int kTmemSfBase = 256;                    // accumulators: buffer b at column 128 b (gate 64 | up 64)
constexpr int kTmemSfPerBuf = 64;

template <int EPI>
struct SCfg {
  static constexpr bool kDual = EPI == kEpiSwiGLU;
  static constexpr int kNumW = kDual ? 2 : 1;
  static constexpr int kOffX = kNumW * kTileW;
  static constexpr int kOffR = kOffX + kTileX;
  static constexpr int kOffSfW = kOffR + kTileX;
  static constexpr int kOffSfX = kOffSfW + kNumW * kSfStage;
  static constexpr int kOffSfR = kOffSfX + kSfStage;
  static constexpr int kStageBytes = kOffSfR + kSfStage;        // 49152 / 30720
  static constexpr int kStages = kDual ? 4 : 6;
  static constexpr int kBarOffset = kStages * kStageBytes;
  // barrier block | reciprocal table | chunk list | expert tables | epilogue staging
  static constexpr int kOffLut = kBarOffset + 256;
  static constexpr int kOffList = kOffLut + 512;
  static constexpr int kOffTab = kOffList + 2 * kMaxChunkList;
  static constexpr int kOffStageH = kOffTab + kMaxSlots * 2 + 4 * kMaxExperts;
  static constexpr int kStageHBytes = kDual ? (kChunk * 128 * 2 + kChunk * 128 * 4) : 0;   // bf16 h | fp32 r^2
  static constexpr int kSmemBytes = kOffStageH + kStageHBytes + 1024;
  static_assert(kSmemBytes <= 232448, "shared memory");
};

struct __align__(8) SBarriers {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  int n_items_chunks;
};

// 16 consecutive accumulator columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory"); }
// Barrier over the epilogue warps that also agrees on `ok` (true only if true in every thread), so
// that the warps leave the item loop together when a wait was abandoned.
__device__ __forceinline__ bool epi_all(bool ok) {
  uint32_t r;
  asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(r) : "r"((uint32_t)ok), "n"(32 * kEpiWarps) : "memory");
  return r != 0;
}

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_swapped_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_r,
                    const __grid_constant__ CUtensorMap tm_w) {
  using C = SCfg<EPI>;
  constexpr bool kDual = C::kDual;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_dyn[];
  const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
  SBarriers* bars = reinterpret_cast<SBarriers*>(smem_gen + C::kBarOffset);
  const uint32_t bar_full = smem_u32(&bars->full[0]), bar_empty = smem_u32(&bars->empty[0]);
  const uint32_t bar_tfull = smem_u32(&bars->tmem_full[0]), bar_tempty = smem_u32(&bars->tmem_empty[0]);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, kEpiWarps); }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tm_x);
    prefetch_tmap(&tm_w);
    if (p.has_resid) prefetch_tmap(&tm_r);
  }
  if (warp == 1) tmem_alloc<1>(smem_u32(&bars->tmem_base), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  // ---- per-CTA tables: slot -> expert / valid rows, expert -> weight scale, and the compact
  // list of non-empty (slot, chunk) pairs in slot order (every CTA builds the same list)
  const int m_slots = p.header[kHdrMTiles];
  float* inv_lut = reinterpret_cast<float*>(smem_gen + C::kOffLut);
  uint16_t* chunk_list = reinterpret_cast<uint16_t*>(smem_gen + C::kOffList);
  uint8_t* tab_expert = smem_gen + C::kOffTab;
  uint8_t* tab_rows = tab_expert + kMaxSlots;
  float* tab_gs = reinterpret_cast<float*>(tab_rows + kMaxSlots);
  if (kDual && threadIdx.x < 128) inv_lut[threadIdx.x] = quant_inv_entry(threadIdx.x, p.h_gs[0]);
  for (int i = threadIdx.x; i < m_slots; i += blockDim.x) {
    tab_expert[i] = (uint8_t)p.tile_expert[i];
    tab_rows[i] = (uint8_t)p.tile_rows[i];
  }
  for (int i = threadIdx.x; i < p.n_experts; i += blockDim.x) tab_gs[i] = p.b_gs[i];
  __syncthreads();
  if (warp == 0) {
    int total = 0;
    for (int base = 0; base < m_slots; base += 32) {
      const int mt = base + lane;
      const int n = mt < m_slots ? ((int)tab_rows[mt] + kChunk - 1) / kChunk : 0;      // 0 .. 4 chunks
      int incl = n;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
      }
      const int pos = total + incl - n;
      for (int c = 0; c < n; ++c) chunk_list[pos + c] = (uint16_t)(mt * 4 + c);
      total += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (lane == 0) bars->n_items_chunks = total;
  }
  // Everything above reads only what kernels before the preceding one produced (routing tables,
  // weight scales): it overlaps the preceding kernel's tail.  The operands need that kernel.
  pdl_sync();
  __syncthreads();
  const int n_chunks = bars->n_items_chunks;
  const int n_ft = p.n_tiles_n;                       // feature tiles of 128
  const int total_items = n_chunks * n_ft;
  const int kt_count = p.K >> 6;
  const int k_stages = (kt_count + kKSteps - 1) / kKSteps;
  const bool resid = p.has_resid != 0;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    const bool issuer = elect_one();
    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      const int ch = item / n_ft, ft = item - ch * n_ft;
      const int mt = chunk_list[ch] >> 2, c = chunk_list[ch] & 3;
      const int e = (int)tab_expert[mt] - p.expert_lo;                 // index into this call's weights
      const int wrow0 = e * p.b_rows_per_expert + ft * 128;            // gate rows (or the only rows)
      const int wrow1 = wrow0 + p.half1_row_offset;                   // up rows
      const int xrow = mt * 128 + c * kChunk;
      const uint8_t* wsf = p.b_sf + (size_t)e * p.b_sf_expert_stride;
      const uint8_t* wsf0 = wsf + (size_t)ft * kt_count * 512u;
      const uint8_t* wsf1 = wsf + (size_t)((p.half1_row_offset >> 7) + ft) * kt_count * 512u;
      const uint8_t* xsf = p.a_sf + (size_t)mt * kt_count * 512u;
      const uint8_t* rsf = p.r_sf + (size_t)mt * kt_count * 512u;
      const int n_box = (min(kChunk, (int)tab_rows[mt] - c * kChunk) + kBoxRows - 1) / kBoxRows;   // 1 or 2
      for (int ks = 0; ks < k_stages; ++ks) {
        ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status);
        if (!ok) break;
        if (issuer) {
          const int atoms = min(kKSteps, kt_count - ks * kKSteps);
          const uint32_t sf_bytes = (uint32_t)atoms * 512u;
          const uint32_t sb = smem_base + stage * C::kStageBytes;
          const uint32_t full = bar_full + 8 * stage;
          const int kc = ks * kStageKBytes;
          const size_t sf_off = (size_t)ks * (size_t)kSfStage;
          mbar_expect_tx(full, (uint32_t)(C::kNumW * kTileW + n_box * (kBoxRows * kStageKBytes) * (resid ? 2 : 1)) +
                                   sf_bytes * (uint32_t)(C::kNumW + (resid ? 2 : 1)));
          tma_load_2d(sb, &tm_w, kc, wrow0, full);
          if (kDual) tma_load_2d(sb + kTileW, &tm_w, kc, wrow1, full);
          for (int b = 0; b < n_box; ++b) {
            tma_load_2d(sb + C::kOffX + b * (kBoxRows * kStageKBytes), &tm_x, kc, xrow + b * kBoxRows, full);
            if (resid) tma_load_2d(sb + C::kOffR + b * (kBoxRows * kStageKBytes), &tm_r, kc, xrow + b * kBoxRows, full);
          }
          bulk_load(sb + C::kOffSfW, wsf0 + sf_off, sf_bytes, full);
          if (kDual) bulk_load(sb + C::kOffSfW + kSfStage, wsf1 + sf_off, sf_bytes, full);
          bulk_load(sb + C::kOffSfX, xsf + sf_off, sf_bytes, full);
          if (resid) bulk_load(sb + C::kOffSfR, rsf + sf_off, sf_bytes, full);
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
    }
    for (int s = 0; s < kStages && ok; ++s) {          // drain
      ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status);
      if (++stage == kStages) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    const bool issuer = elect_one();
    uint32_t stage = 0, phase = 0, kcount = 0;
    int it = 0;
    bool ok = true;
    constexpr uint32_t kSw128Hi = (uint32_t)((8 * kStageKBytes) >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t kSfHi = (uint32_t)(128 >> 4) | (1u << 14);
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++it) {
      const int ch = item / n_ft;
      const int mt = chunk_list[ch] >> 2, c = chunk_list[ch] & 3;
      const int n_rows = min(kChunk, (int)tab_rows[mt] - c * kChunk);
      const int n_pad = (n_rows + 15) & ~15;                          // 16 or 32 token rows
      const int n_lead = (c & 1) * kChunk;                            // odd chunk: 32 rows of filler come first
      const int n_mma = n_lead + n_pad;                               // N of the MMAs: 16 .. 64
      // E2M1 x E2M1, UE4M3 block scales, both operands K-major, M = 128, N = n_mma
      const uint32_t idesc = (1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const int buf = it & 1;
      const uint32_t acc = tmem + (uint32_t)(buf * 128);
      ok = mbar_wait(bar_tempty + 8 * buf, (uint32_t)((it >> 1) & 1) ^ 1u, abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      for (int ks = 0; ks < k_stages; ++ks, ++kcount) {
        ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const int atoms = min(kKSteps, kt_count - ks * kKSteps);
        const uint32_t sb = smem_base + stage * C::kStageBytes;
        const uint32_t sfcol = tmem + kTmemSfBase + (kcount & 1u) * kTmemSfPerBuf;
        const uint32_t w0_lo = ((sb & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t w1_lo = (((sb + kTileW) & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t x_lo = (((sb + C::kOffX - n_lead * kStageKBytes) & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t r_lo = (((sb + C::kOffR - n_lead * kStageKBytes) & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t sfw_lo = ((sb + C::kOffSfW) & 0x3FFFFu) >> 4;
        const uint32_t sfx_lo = ((sb + C::kOffSfX) & 0x3FFFFu) >> 4;
        const uint32_t sfr_lo = ((sb + C::kOffSfR) & 0x3FFFFu) >> 4;
        if (issuer) {
          // scale columns of K step j: weights 0 at 4j, weights 1 at 16+4j, X at 32+4j, R at 48+4j
          auto copy_sf = [&](int j) {
            tc_cp_sf<1>(sfcol + 4 * j, ((uint64_t)kSfHi << 32) | (sfw_lo + 32 * j));
            if (kDual) tc_cp_sf<1>(sfcol + 16 + 4 * j, ((uint64_t)kSfHi << 32) | (sfw_lo + (kSfStage >> 4) + 32 * j));
            tc_cp_sf<1>(sfcol + 32 + 4 * j, ((uint64_t)kSfHi << 32) | (sfx_lo + 32 * j));
            if (resid) tc_cp_sf<1>(sfcol + 48 + 4 * j, ((uint64_t)kSfHi << 32) | (sfr_lo + 32 * j));
          };
          if (atoms > 0) copy_sf(0);
#pragma unroll
          for (int j = 0; j < kKSteps; ++j) {
            if (j + 1 < atoms) copy_sf(j + 1);
            if (j < atoms) {
              const uint32_t accum = (ks > 0 || j > 0) ? 1u : 0u;
              const uint64_t xdesc = ((uint64_t)kSw128Hi << 32) | (x_lo + 2 * j);
              const uint64_t rdesc = ((uint64_t)kSw128Hi << 32) | (r_lo + 2 * j);
              const uint64_t w0desc = ((uint64_t)kSw128Hi << 32) | (w0_lo + 2 * j);
              // token scales: the even column at or before the chunk's own column of the slot's atom
              const uint32_t sfx = sfcol + 32 + 4 * j + (uint32_t)(c & 2), sfr = sfcol + 48 + 4 * j + (uint32_t)(c & 2);
              tc_mma_nvf4<1>(acc, w0desc, xdesc, idesc, sfcol + 4 * j, sfx, accum);
              if (resid) tc_mma_nvf4<1>(acc, w0desc, rdesc, idesc, sfcol + 4 * j, sfr, 1u);
              if (kDual) {
                const uint64_t w1desc = ((uint64_t)kSw128Hi << 32) | (w1_lo + 2 * j);
                tc_mma_nvf4<1>(acc + 64, w1desc, xdesc, idesc, sfcol + 16 + 4 * j, sfx, accum);
                if (resid) tc_mma_nvf4<1>(acc + 64, w1desc, rdesc, idesc, sfcol + 16 + 4 * j, sfr, 1u);
              }
            }
          }
          tc_commit<1>(bar_empty + 8 * stage);
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
      if (ok && issuer) tc_commit<1>(bar_tfull + 8 * buf);
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;                       // TMEM lane quadrant of this warp
    const int th = (warp - 2) >> 2;               // token group: this chunk's columns [16 th, 16 th + 16)
    const int f_in_tile = q * 32 + lane;          // this thread's feature within the tile
    const int etid = (warp - 2) * 32 + lane;      // 0 .. 255
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const float a_gs = p.a_gs ? p.a_gs[0]
                              : (__uint_as_float(p.a_amax_bits[0]) > 0.f
                                     ? __fdiv_rn(__uint_as_float(p.a_amax_bits[0]), kGlobalDiv) : 1.0f);
    uint16_t* hs = reinterpret_cast<uint16_t*>(smem_gen + C::kOffStageH);              // [32 tokens][128 features] bf16
    float* rs = reinterpret_cast<float*>(smem_gen + C::kOffStageH + kChunk * 128 * 2);  // [32][128] squared residuals
    int it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++it) {
      const int ch = item / n_ft, ft = item - ch * n_ft;
      const int mt = chunk_list[ch] >> 2, c = chunk_list[ch] & 3;
      const int e = tab_expert[mt];
      const int n_rows = min(kChunk, (int)tab_rows[mt] - c * kChunk);
      const int n_pad = (n_rows + 15) & ~15;
      const int col0 = (c & 1) * kChunk;          // the chunk's first accumulator column
      const int row0 = mt * 128 + c * kChunk;     // padded dispatch row of the chunk's first token
      const float scale = __fmul_rn(a_gs, tab_gs[e - p.expert_lo]);
      const int buf = it & 1;
      ok = mbar_wait(bar_tfull + 8 * buf, (uint32_t)((it >> 1) & 1), abort_flag, p.status);
      if (kDual) ok = epi_all(ok);               // also: the previous item's readers are done with hs / rs
      if (!ok) break;
      tc_fence_after();
      float g[16], u[16];
      tmem_ld16(lane_addr + buf * 128 + col0 + th * 16, g);
      if (kDual) tmem_ld16(lane_addr + buf * 128 + 64 + col0 + th * 16, u);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);

      if (!kDual) {
        // y rows for the combine kernel: thread = output feature, one 2-byte store per token
        const int n_out = p.n_out;
        const int f = ft * 128 + f_in_tile;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int t = th * 16 + i;
          if (t < n_rows)
            p.y_pad[(size_t)(row0 + t) * n_out + f] = __bfloat16_as_ushort(__float2bfloat16_rn(g[i] * scale));
        }
      } else {
        const int I = p.n_out;
        // (1) SwiGLU in the accumulator layout, rounded to bf16, transposed through shared memory
        if (th * 16 < n_pad) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float gg = __fmul_rn(g[i], scale);
            const float uu = __fmul_rn(u[i], scale);
            const float h = __fdividef(gg, 1.0f + __expf(-gg)) * uu;
            hs[(th * 16 + i) * 128 + f_in_tile] = __bfloat16_as_ushort(__float2bfloat16_rn(h));
          }
        }
        epi_barrier();
        // (2) one 16-feature block of one token per thread: the row-major kernel's arithmetic
        QuantCtx qc;
        quant_ctx_scalars(qc, p.h_gs[0]);
        qc.inv_lut = inv_lut;
        const int kt2 = I >> 6;
        const int t = etid >> 3, b = etid & 7;
        if (t < n_pad) {
          const uint4* src = reinterpret_cast<const uint4*>(hs + t * 128 + 16 * b);
          const uint4 v0 = src[0], v1 = src[1];
          float hb[16];
          unpack8(v0, hb);
          unpack8(v1, hb + 8);
          const bool valid = t < n_rows;
          const int prow = row0 + t;
          const int f0 = ft * 128 + 16 * b;
          const BlockQ bq = quantize_block(hb, qc);
          if (valid) {
            *reinterpret_cast<uint2*>(p.hq_pad + (size_t)prow * (I >> 1) + (f0 >> 1)) = make_uint2(bq.lo, bq.hi);
            p.hsf_tiled[sf_tiled_offset(prow, f0 >> 4, kt2)] = (uint8_t)bq.sf8;
            if (p.h_export) {
              const int drow = p.offsets[e] + (mt - p.tile_prefix[e]) * 128 + c * kChunk + t;
              uint4* d = reinterpret_cast<uint4*>(p.h_export + (size_t)drow * I + f0);
              d[0] = v0;
              d[1] = v1;
            }
          }
          if (p.resid2) {
            float r[16];
            dequant_block(bq, r);
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = __fsub_rn(r[i], hb[i]);
            const BlockQ br = quantize_block(r, qc);
            if (valid) {
              *reinterpret_cast<uint2*>(p.r2q_pad + (size_t)prow * (I >> 1) + (f0 >> 1)) =
                  make_uint2(br.lo ^ 0x88888888u, br.hi ^ 0x88888888u);
              p.r2sf_tiled[sf_tiled_offset(prow, f0 >> 4, kt2)] = (uint8_t)br.sf8;
            }
            float4* rd = reinterpret_cast<float4*>(rs + t * 128 + 16 * b);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              rd[i] = make_float4(r[4 * i] * r[4 * i], r[4 * i + 1] * r[4 * i + 1], r[4 * i + 2] * r[4 * i + 2],
                                  r[4 * i + 3] * r[4 * i + 3]);
          }
        }
        // (3) column scores of the residual: sum over the chunk's tokens in token order, then into the
        // column's integer total
        if (p.resid2) {
          epi_barrier();
          if (etid < 128) {
            float sacc = 0.f;
            for (int tt = 0; tt < n_rows; ++tt) sacc += rs[tt * 128 + etid];
            add_score(p.keys2 + ft * 128 + etid, sacc, p.h_gs[0], p.score_bits);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc<1>(tmem, kTmemCols);
}

}  // namespace

bool gemm_swapped_ok(int64_t assignments, int n_experts, int m_tiles_max) {
  return n_experts > 0 && assignments <= (int64_t)n_experts * 32 && m_tiles_max <= kMaxSlots &&
         n_experts <= kMaxExperts;
}

quads_status launch_gemm_swapped(int epi, const GemmParams& p, const GemmMaps& m, int n_sms, cudaStream_t stream) {
  if (epi == kEpiSwiGLU) {
    QUADS_CUDA_OK(set_max_dynamic_smem<gemm_swapped_kernel<kEpiSwiGLU>>(SCfg<kEpiSwiGLU>::kSmemBytes));
    QUADS_CUDA_OK(launch_kernel(gemm_swapped_kernel<kEpiSwiGLU>, dim3(n_sms), dim3(kThreads),
                                (size_t)SCfg<kEpiSwiGLU>::kSmemBytes, stream, p, m.a, m.r, m.b));
  } else {
    QUADS_CUDA_OK(set_max_dynamic_smem<gemm_swapped_kernel<kEpiCombine>>(SCfg<kEpiCombine>::kSmemBytes));
    QUADS_CUDA_OK(launch_kernel(gemm_swapped_kernel<kEpiCombine>, dim3(n_sms), dim3(kThreads),
                                (size_t)SCfg<kEpiCombine>::kSmemBytes, stream, p, m.a, m.r, m.b));
  }
  return QUADS_OK;
}

}  // namespace quads
