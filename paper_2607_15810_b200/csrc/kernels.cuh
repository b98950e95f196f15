// Kernel declarations shared by the translation units of libquads.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace quads {

constexpr int kRouteTokensPerCta = 32;
constexpr int kMaxTopk = 16;
constexpr int kMaxExperts = 256;

// header words written by the scan (device side sizes of the dispatch)
enum { kHdrMTiles = 0, kHdrPaddedRows = 1, kHdrAssignments = 2, kHdrStatus = 3, kHdrArrivals = 4, kHdrWords = 8 };

constexpr int kAmaxPartsMax = 2048;   // partial maxima left by the first pass of the single-tensor quantizer

// ---- quantize.cu
__global__ void amax_kernel(const uint16_t* x, int64_t rows, int64_t K, int64_t ld, int64_t tensor_stride,
                            uint32_t* amax_bits);
__global__ void fused_quantize_kernel(const uint16_t* x, int64_t rows, int64_t K, int64_t ld, int64_t tensor_stride,
                                      int n_tensors, const float* gs_in, uint32_t* amax_bits, uint32_t* counters,
                                      uint8_t* q, uint8_t* sf, uint16_t* fq, float* gs_out, int sf_tiled,
                                      int64_t sf_tensor_stride, int n_groups, long long wait_cycles,
                                      int extra_arrivals, const uint32_t* amax_parts, int n_amax_parts);
__global__ void amax_partial_kernel(const uint16_t* x, int64_t rows, int64_t K, int64_t ld, uint32_t* partials);
// Fake-quant of a batch of tensors through shared-memory rings of bulk copies (one CTA per SM,
// four groups of 7 consumer warps + 1 producer warp, one ring of 14 KB stages per group).
constexpr int kRingThreads = 1024;
constexpr int kRingDepth = 3;
constexpr int kRingHeaderBytes = 1024;
constexpr int kRingChunkBytes = 7 * 32 * 2 * 32;
constexpr int kRingSmemBytes = kRingHeaderBytes + 4 * kRingDepth * kRingChunkBytes;
__global__ void fake_quant_ring_kernel(const uint16_t* x, int64_t nblk, int64_t tensor_stride, int n_tensors,
                                       uint32_t* pair, int per, int lead, int split, uint8_t* q, uint8_t* sf, uint16_t* fq,
                                       float* gs_out, int sf_tiled, int64_t sf_tensor_stride, uint32_t k16,
                                       int kt_count);
__global__ void dequantize_kernel(const uint8_t* q, const uint8_t* sf, const float* gs, int n_tensors, int64_t nblk,
                                  uint32_t k16, int kt_count, int sf_tiled, int64_t sf_tensor_stride, uint16_t* out);
__global__ void rac_quant_kernel(const uint16_t* x, int T, int H, const float* gs_in, uint32_t* amax_bits,
                                 unsigned int* grid_arrivals, int32_t* status,
                                 float* gs_store, int rows_per_cta, int with_residual, float* partials, uint8_t* xq,
                                 uint8_t* xsf, uint8_t* rq, uint8_t* rsf, uint8_t* xq_exp, uint8_t* xsf_exp,
                                 unsigned long long* score_totals /* or NULL: partial rows */, int score_bits,
                                 int cap_bits);
constexpr int kScoreSlices = 16;
__global__ void score_reduce_kernel(const float* partials, const int* n_part_ptr, int n_part_mul,
                                    int n_part_fixed, int C, double* slice_sums, unsigned int* counters,
                                    unsigned long long* score_keys);
__global__ void rank_select_kernel(const unsigned long long* score_keys, int C, int n_sel, uint8_t* mask);
__global__ void sel_list_kernel(const uint8_t* mask, int C, int32_t* sel_export);
__global__ void rac_scatter_kernel(int T, int H, int parts, const uint8_t* mask, int topk,
                                   const int32_t* pos_pad, const uint8_t* xq, const uint8_t* xsf, const uint8_t* rq,
                                   const uint8_t* rsf, uint8_t* xq_pad, uint8_t* xsf_tiled, uint8_t* rq_pad,
                                   uint8_t* rsf_tiled, uint8_t* rq_exp, uint8_t* rsf_exp);
template <int kParts>   // bit 0: copies of Q(x), bit 1: masked, negated copies of the residual
__global__ void rac_dispatch_kernel(int H, const uint8_t* mask, const int32_t* header,
                                    const int32_t* tile_rows, const int32_t* row_token, const uint8_t* xq,
                                    const uint8_t* xsf, const uint8_t* rq, const uint8_t* rsf, uint8_t* xq_pad,
                                    uint8_t* xsf_tiled, uint8_t* rq_pad, uint8_t* rsf_tiled);
__global__ void mask_codes_kernel(uint8_t* codes, const int* n_rows_ptr, int C, const uint8_t* mask);
__global__ void combine_kernel(const uint16_t* y_pad, const int32_t* pos_pad, const float* wts, int T, int H,
                               int topk, uint16_t* out, float* out_f32);
__global__ void export_site2_kernel(int A, const int32_t* n_rows_ptr, int I, const int32_t* perm, const int32_t* pos_pad,
                                    const uint8_t* hq_pad, const uint8_t* hsf_tiled, const uint8_t* r2q_pad,
                                    const uint8_t* r2sf_tiled, const uint8_t* mask2, uint8_t* hq, uint8_t* hsf,
                                    uint8_t* r2q, uint8_t* r2sf);

__global__ void mismatch_norms_kernel(const uint16_t* a, const uint16_t* b, int64_t n, double* partials,
                                      unsigned int* counter, double* out);

// ---- routing.cu
template <int NJ>
__global__ void route_kernel_t(const float* logits, int T, int E, int topk, int renormalize, int32_t* ids,
                               float* wts, int32_t* chunk_counts, int32_t* expert_total, int32_t* ids_out,
                               float* wts_out, int e_lo, int e_hi);
__global__ void scan_kernel(int E, int n_chunks, int tile_group, const int32_t* chunk_counts,
                            const int32_t* expert_total, int32_t* chunk_base, int32_t* offsets, int32_t* tile_prefix,
                            int32_t* tile_expert, int32_t* tile_rows, int32_t* header, int32_t* offsets_out);
__global__ void permute_kernel(int T, int E, int topk, int n_chunks, const int32_t* ids, const float* wts,
                               const int32_t* chunk_base, const int32_t* offsets, const int32_t* tile_prefix,
                               int32_t* perm, int32_t* pos_pad, int32_t* row_token, float* row_weight,
                               int32_t* perm_out, int e_lo, int e_hi);
__global__ void dense_dispatch_kernel(int T, int tile_group, int32_t* pos_pad, int32_t* row_token, float* row_weight,
                                      int32_t* tile_expert, int32_t* tile_rows, int32_t* header);

// ---- gemm.cu
#ifndef QUADS_GEMM_KSTEPS
#define QUADS_GEMM_KSTEPS 4
#endif
constexpr int kGemmKSteps = QUADS_GEMM_KSTEPS;        // K = 64 MMAs per pipeline stage (2 or 4)
constexpr int kGemmStageKBytes = 32 * kGemmKSteps;    // packed FP4 bytes per operand row per stage
enum { kEpiStore = 0, kEpiSwiGLU = 1, kEpiCombine = 2 };

struct GemmParams {
  int K;                 // contraction length in elements (multiple of 64)
  int n_tiles_n;         // tiles along the output-feature dimension
  int n_out;             // output features (I for SwiGLU, else N)
  int b_rows_per_expert; // weight rows per expert
  int half1_row_offset;  // weight-row distance from the tile's first half to its second half
  int has_resid;         // 1: also accumulate the (negated, masked) residual operand
  int n_experts;         // entries of b_gs (the experts whose weights this call holds)
  int expert_lo;         // global id of the first of them: weights / scales are indexed by (expert - expert_lo)
  const int32_t* header;
  const int32_t* tile_expert;
  const int32_t* tile_rows;
  const uint8_t* a_sf;   // tiled scales of the main activation operand (padded dispatch rows)
  const uint8_t* r_sf;   // tiled scales of the residual operand
  const uint8_t* b_sf;   // tiled weight scales, one block per expert
  size_t b_sf_expert_stride;
  const float* b_gs;     // [E] per-tensor weight scales
  const float* a_gs;     // per-tensor activation scale (pointer), or NULL ...
  const uint32_t* a_amax_bits;  // ... then derived from this amax word
  // epilogue: store / combine
  const int32_t* row_token;
  const float* row_weight;
  uint16_t* out_bf16;    // kEpiStore: [T, n_out]
  uint16_t* y_pad;       // kEpiCombine: bf16 [padded dispatch rows, n_out], one row per assignment
  // epilogue: SwiGLU + requantize (site 2)
  const float* h_gs;     // per-tensor scale of h
  int resid2;            // 1: also emit the residual of h and its column statistics
  uint8_t* hq_pad; uint8_t* hsf_tiled; uint8_t* r2q_pad; uint8_t* r2sf_tiled;
  // column scores of the residual of h (Eq. channel-score), accumulated as integers so that the sum does
  // not depend on the order of arrival: every partial sum of squares (one per tile, lane quadrant and
  // column) is divided by the square of h's per-tensor scale, multiplied by 2^score_bits, rounded down
  // and added with a 64-bit integer reduction; the totals are the selection's order-preserving keys
  unsigned long long* keys2;   // [n_out], zero on entry
  int score_bits;
  uint16_t* h_export;    // optional bf16 [A, n_out] in dispatch order
  const int32_t* tile_prefix;
  const int32_t* offsets;
  int32_t* status;       // device status word (QUADS_ERR_TIMEOUT on a failed wait)
};

// Tensor maps of one GEMM launch: packed codes of the activation / residual / weight operands and
// (CTA-pair variant only) their scale atoms viewed as [atoms, 128 x u32].
struct GemmMaps {
  CUtensorMap a, r, b, sfa, sfr, sfb;
};

// Operand-swapped variant for few rows per expert (weights on the M side, tokens in chunks of 32
// on the N side; epi = kEpiSwiGLU or kEpiCombine).  Maps: a / r = activation / residual codes with
// boxes of 16 rows, b = weight codes with boxes of 128 rows; p.n_tiles_n counts tiles of 128
// output features.  Usable when assignments <= 32 * experts and the slot tables fit.
bool gemm_swapped_ok(int64_t assignments, int n_experts, int m_tiles_max);
quads_status launch_gemm_swapped(int epi, const GemmParams& p, const GemmMaps& m, int n_sms, cudaStream_t stream);

// ---- gemm_bf16.cu: out[T, N] = A[T, K] B[N, K]^T, bf16 operands (tensor maps with boxes of 64 x 128
// elements, 128-byte swizzle), float32 accumulation, bf16 output; K % 64 == 0, N % 128 == 0
quads_status launch_gemm_bf16(const CUtensorMap& tm_a, const CUtensorMap& tm_b, int T, int N, int K, uint16_t* out,
                              int32_t* status, int n_sms, cudaStream_t stream);

// ---- fp8.cu: the FP8 W8A8 comparison path
struct Fp8GemmParams {
  int K;                 // contraction length in elements (multiple of 128)
  int n_tiles_n;         // tiles along the output features
  int n_out;             // output features (I for SwiGLU, else H)
  int b_rows_per_expert;
  int half1_row_offset;
  const int32_t* header;
  const int32_t* tile_expert;
  const int32_t* tile_rows;
  const uint8_t* a_sf;   // activation scale atoms, [m_tiles, K/128, 512]
  const uint8_t* b_sf;   // weight scale atoms, [E, rows/128, K/128, 512]
  size_t b_sf_expert_stride;
  uint16_t* y_pad;       // kEpiCombine: bf16 [padded rows, n_out]
  uint8_t* hq_pad;       // kEpiSwiGLU: E4M3 codes of h, [padded rows, n_out]
  uint8_t* hsf_atoms;    // kEpiSwiGLU: scale atoms of h, [m_tiles, n_out/128, 512]
  uint16_t* h_export;    // optional bf16 [A, n_out], dispatch order (then hq_export / hexp_export too)
  uint8_t* hq_export;
  uint8_t* hexp_export;
  const int32_t* tile_prefix;
  const int32_t* offsets;
  int32_t* status;
};
__global__ void fp8_quantize_act_kernel(const uint16_t* x, int64_t rows, int K, uint8_t* codes, uint8_t* exps);
__global__ void fp8_quantize_weight_kernel(const uint16_t* w, int N, int K, uint8_t* codes, uint8_t* exps, uint8_t* atoms);
__global__ void fp8_dispatch_kernel(int H, const int32_t* header, const int32_t* tile_rows, const int32_t* row_token,
                                    const uint8_t* xq, const uint8_t* xe, uint8_t* xq_pad, uint8_t* xsf_atoms);
quads_status launch_gemm_fp8(int epi, const Fp8GemmParams& p, const CUtensorMap& tm_a, const CUtensorMap& tm_b, int n_sms,
                             cudaStream_t stream);

quads_status launch_gemm(int epi, int cta_group, const GemmParams& p, const GemmMaps& m, int n_sms,
                         cudaStream_t stream);

}  // namespace quads
