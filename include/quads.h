/*
 * quads.h -- C ABI of the B200 (sm_100a) NVFP4 MoE rollout forward and the
 * trainer-side weight fake-quant.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless the comment says "host".  The args
 *     struct and the returned strings are host memory.
 *   - The caller owns every buffer.  The library never allocates or frees
 *     device memory; scratch comes from the `workspace` argument, whose
 *     minimum size the matching *_workspace_bytes() function returns.
 *     Workspaces must be 256-byte aligned.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL =
 *     the legacy default stream) and the call returns without synchronising.
 *   - Argument errors are detected on the host and returned before anything is
 *     launched.  A CUDA launch error is returned as QUADS_ERR_CUDA.  A device
 *     wait that ran out of its iteration budget is recorded in the workspace and
 *     can be read with quads_moe_async_status() after the stream is synchronised.
 *   - Inputs must be finite.  K (and H, I) must be multiples of 16 for the
 *     quantizers and multiples of 128 for GEMM operands.
 *
 * NVFP4 format (paper, Section "Low-Precision Inference", paragraph FP4):
 * E2M1 elements {0,0.5,1,1.5,2,3,4,6} per sign; 16 consecutive elements along
 * the contraction dimension share one E4M3 scale; one FP32 per-tensor scale.
 * Element 2i sits in the low nibble and 2i+1 in the high nibble of byte i.
 * Scale derivation (all float32, in this order):
 *   s_g = amax(tensor) / 2688  (1 for an all-zero tensor)
 *   sf  = E4M3_rne_sat( amax(block) / (6 * s_g) ),  d = sf * s_g
 *   code = E2M1_rne_sat( x * (1 / d) )   (all-zero codes when sf == 0)
 *   dequantized value = value(code) * d
 */
#ifndef QUADS_H_
#define QUADS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t quads_status;

enum {
  QUADS_OK = 0,
  QUADS_ERR_NULL = -1,       /* a required pointer is NULL */
  QUADS_ERR_SHAPE = -2,      /* a size breaks a divisibility or range rule */
  QUADS_ERR_WORKSPACE = -3,  /* workspace missing, misaligned or too small */
  QUADS_ERR_ARCH = -4,       /* the current device is not sm_100 */
  QUADS_ERR_CUDA = -5,       /* a CUDA runtime / driver call failed */
  QUADS_ERR_TIMEOUT = -6,    /* a bounded device-side wait gave up */
  QUADS_ERR_LIMIT = -7       /* size beyond the fixed capacity of an allocation-free entry point */
};

enum {
  QUADS_SF_LINEAR = 0, /* scale bytes as [rows, K/16], row-major (the parity layout) */
  QUADS_SF_TILED = 1   /* 512-byte atoms of 128 rows x 4 blocks for the tensor-core path:
                          atom (row/128, blk/4) at ((row/128) * ceil(K/64) + blk/4) * 512,
                          byte (row%32)*16 + ((row%128)/32)*4 + blk%4 inside it; rows are
                          padded to a multiple of 128 and K to a multiple of 64 */
};

/* Human-readable name of a status code (host string, never NULL). */
const char* quads_status_string(quads_status s);

/* Bytes of a QUADS_SF_TILED scale buffer for one [rows, K] tensor. */
size_t quads_sf_tiled_bytes(int64_t rows, int64_t K);

/*
 * (1) Online NVFP4 activation quantization, the operator Q_A of
 * Eq. "act-error-def" (Section "Methods"), format as in Section "Low-Precision
 * Inference", paragraph FP4.
 *   x      bf16 [rows, K], row stride `ld` elements (ld >= K, ld % 16 == 0),
 *          32-byte aligned
 *   gs_in  float[1] per-tensor scale, or NULL: amax(x)/2688 computed on device
 *   q      out, u8 [rows, K/2]
 *   sf     out, u8, layout per `sf_layout` ([rows, K/16] when linear)
 *   gs_out out, float[1]: the per-tensor scale that was used (may be NULL)
 *   workspace  >= quads_quantize_workspace_bytes() bytes
 * rows == 0 is allowed (nothing is written except gs_out = 1 when gs_in is NULL).
 * With gs_in == NULL the call is two ordinary launches (per-CTA partial maxima,
 * then the quantization, which finds the tensor in L2); with gs_in given it is
 * one.  Neither contains a wait of one CTA for another.  (Setting the environment
 * variable QUADS_QUANT_COOPERATIVE selects the single cooperative kernel that
 * batches of large tensors use, whose CTAs meet at a counter once the amax is
 * complete; that wait is bounded, about two seconds, and if it ever gives up
 * the call still ends, q and sf are unspecified and gs_out[0] = NaN says so.)
 * The same holds for quads_fake_quant_activations.
 * A tensor holds fewer than 2^31 scale blocks (rows * K / 16), else QUADS_ERR_SHAPE;
 * the same limit applies to every tensor of quads_fake_quant_weights.
 */
quads_status quads_quantize_nvfp4(const void* x, int64_t rows, int64_t K, int64_t ld,
                                  const float* gs_in, uint8_t* q, uint8_t* sf, float* gs_out,
                                  int sf_layout, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream);
size_t quads_quantize_workspace_bytes(void);

/*
 * (4) Trainer-side Asymmetric-QAT weight fake-quant QDQ_W (Eq. "w4a16-qat-forward")
 * and the pack for rollout weight sync (Eqs. "weight-sync", "weight-qdq-align"):
 * one quantization decides both outputs, so the bf16 the trainer multiplies by
 * equals, bit for bit, the bf16 dequantization of the bytes the rollout loads.
 *   w       bf16 [n_tensors, N, K], K contiguous; every [N, K] slice is one tensor
 *           with its own per-tensor scale
 *   w_fq    out, bf16 [n_tensors, N, K]  (NULL to skip)
 *   q       out, u8 [n_tensors, N, K/2]  (NULL to skip)
 *   sf      out, u8 per `sf_layout`, one [N, K/16] (or tiled) block per tensor (NULL to skip)
 *   gs      out, float [n_tensors] (required)
 *   workspace >= quads_fake_quant_workspace_bytes(n_tensors) bytes
 * The kernel is one cooperative launch whose CTAs meet at a counter per tensor
 * (a tensor's scale needs every CTA's share of its amax).  Every such wait is
 * bounded (2 s); if one ever gives up, the call still ends, the outputs of the
 * tensors concerned are unspecified and gs[t] = NaN marks them.  The launch
 * needs the whole GPU: it fails with QUADS_ERR_CUDA if the device cannot hold
 * all of its CTAs at once (for instance under a partitioned context).
 */
quads_status quads_fake_quant_weights(const void* w, int64_t n_tensors, int64_t N, int64_t K,
                                      void* w_fq, uint8_t* q, uint8_t* sf, float* gs,
                                      int sf_layout, void* workspace, size_t workspace_bytes,
                                      void* cuda_stream);
size_t quads_fake_quant_workspace_bytes(int64_t n_tensors);

/*
 * NVFP4 -> bf16 decode of packed tensors: out = value(code) * (E4M3 block scale *
 * per-tensor scale), one float32 multiply rounded to bf16 -- the right-hand side
 * of Eq. "weight-qdq-align", i.e. what the rollout side holds after loading the
 * bytes quads_fake_quant_weights produced (out equals that call's w_fq bit for
 * bit), and the weight operand of a W4A16 rollout.
 *   q    u8 [n_tensors, rows, K/2], 8-byte aligned
 *   sf   u8, one [rows, K/16] (or tiled) block per tensor, per `sf_layout`
 *   gs   float [n_tensors] per-tensor scales (device)
 *   out  bf16 [n_tensors, rows, K], 32-byte aligned
 * rows * K / 16 < 2^31 per tensor.  n_tensors == 0 or rows == 0 does nothing.
 */
quads_status quads_dequantize_nvfp4(const uint8_t* q, const uint8_t* sf, const float* gs,
                                    int64_t n_tensors, int64_t rows, int64_t K, int sf_layout,
                                    void* out, void* cuda_stream);

/*
 * Activation fake-quant QDQ_A for the learner-side ablations of the paper
 * (Table "qdq-alignment": a W16A4- or W4A4-QAT learner quantizes and
 * dequantizes its own activations; Section "Asymmetric Quantization-Aware
 * Training" argues against it, and keeps activations in BF16).  The same NVFP4
 * quantizer as quads_quantize_nvfp4, followed by the same dequantization as
 * quads_fake_quant_weights, so x_fq is bit for bit what the rollout's
 * activation operand decodes to.  The straight-through backward of the node is
 * the identity and needs no kernel.
 *   x      bf16 [rows, K], row stride `ld` elements (ld >= K, ld % 16 == 0), 32-byte aligned
 *   gs_in  float[1] per-tensor scale, or NULL: amax(x)/2688 computed on device
 *   x_fq   out, bf16 [rows, K] contiguous, 32-byte aligned
 *   gs_out out, float[1]: the scale that was used (may be NULL)
 *   workspace  >= quads_quantize_workspace_bytes() bytes
 */
quads_status quads_fake_quant_activations(const void* x, int64_t rows, int64_t K, int64_t ld,
                                          const float* gs_in, void* x_fq, float* gs_out,
                                          void* workspace, size_t workspace_bytes,
                                          void* cuda_stream);

/*
 * Allocation-free variant of quads_fake_quant_weights (the paper has no
 * counterpart; it exists for callers that cannot provide scratch memory).
 * Some hosts of this library may not call cudaMalloc where they use it: a
 * trainer whose device memory belongs entirely to its own caching pool, a
 * plugin that is forbidden to allocate after start-up, or code on a path where
 * the implicit device synchronisation of an allocation is not acceptable.  For
 * them this entry point takes no workspace: its scratch, two 4-byte words per
 * tensor (the running amax and an arrival counter), is a fixed array sized for
 * QUADS_NOALLOC_MAX_TENSORS tensors inside the library image (32 KiB, resident
 * on every GPU that loads the library until the process exits).  Arguments, outputs and results are those of
 * quads_fake_quant_weights, bit for bit.
 *   - n_tensors > QUADS_NOALLOC_MAX_TENSORS returns QUADS_ERR_LIMIT and
 *     launches nothing; split the batch.
 *   - The first call on each device looks up the array's device address (a
 *     host-side query, no allocation).  Make that first call outside any
 *     stream capture.
 *   - The call allocates and frees nothing: no cudaMalloc, no cudaFree, no
 *     allocating library routine.
 *   - Every call on a device shares the one array.  Each call zeroes the words
 *     it uses, on its stream, before use, so earlier contents do not matter;
 *     but two calls that may run at the same time on one GPU (different
 *     streams, or different host threads) race on it and must be serialised
 *     by the caller.
 */
#define QUADS_NOALLOC_MAX_TENSORS 4096
quads_status quads_fake_quant_weights_noalloc(const void* w, int64_t n_tensors, int64_t N, int64_t K,
                                              void* w_fq, uint8_t* q, uint8_t* sf, float* gs,
                                              int sf_layout, void* cuda_stream);

/*
 * (2)+(3) MoE expert layer forward with native W4A4 grouped GEMMs and Residual
 * Activation Compensation (Section "Activation Error Compensation for
 * Rollout-side", Eqs. "residual-def", "residual-recon", "channel-score",
 * "channel-select"):
 *   X~ = Q_A(X) - M_S (.) Q_A(Q_A(X) - X),  S = the n_sel channels with the
 *   largest residual L2 norm over the current token batch,
 * evaluated as  W X~ = W Q_A(X) - W (M_S (.) Q_A(dX)), two W4A4 tensor-core
 * products into one accumulator (the residual shares the per-tensor scale of
 * its activation).  Per token: top-k experts by router logit (ties to the lower
 * id), weights = softmax over all experts restricted to the chosen ones
 * (renormalised when `renormalize`), h = silu(W1 x) * (W3 x) rounded to bf16,
 * requantized with `a2_gs`, out = sum_k weight_k * W2 h~.
 * The output is reproducible bit for bit: every floating-point sum runs in a
 * fixed order, and the channel scores that cross CTAs are added as 64-bit
 * integers (partial sum of squares / scale^2, at most 26 fractional bits), so
 * the selection does not depend on the order in which CTAs finish.
 *
 * Dense mode (I == 0): one projection out[T, N] = W X~ with E = topk = 1, the
 * weight in w13_*, no routing, no SwiGLU ("single dense W4A4+RAC GEMM").  With
 * operand_mode = QUADS_W4A16 / QUADS_W16A4 the same projection is computed with
 * only the weights / only the activations in NVFP4 (see the enum below).
 *
 * Weight buffers are exactly what quads_fake_quant_weights() writes with
 * QUADS_SF_TILED: w13 is [E, 2I, H] (gate rows first, then up rows), w2 is
 * [E, H, I]; H % 128 == 0, I % 128 == 0 (dense: N % 128 == 0).
 * Limits: E <= 256, topk <= 16 and <= E, H <= 16384, I <= 16384; a size outside
 * them returns QUADS_ERR_SHAPE before anything is launched.
 *
 * The call allocates nothing and never synchronises the host.  Part of the
 * work (routing, the dispatched copies of Q_A(X)) is enqueued on a second
 * stream of the library's own, forked from and joined back into the caller's
 * stream with events, so the call as a whole is ordered like any other work on
 * `cuda_stream` and can be captured into a CUDA graph (make one ordinary call
 * first: kernel attributes are set on first use).  Device-side waits are bounded;
 * one that gives up writes QUADS_ERR_TIMEOUT to a status word in the workspace,
 * read with quads_moe_async_status().  Every call resets that word on its stream
 * before its first kernel: poll after each call whose status matters.
 * One side stream per device serves all callers: calls on one device are
 * serialised on the host by a lock while they enqueue, and a CUDA-graph capture
 * of a call must not overlap, in time, other MoE calls on the same device (they
 * would enqueue into the capturing side stream).  The timing and trace aids
 * below keep process-wide state and are not thread-safe.
 */
enum {
  QUADS_W4A4 = 0,   /* both operands NVFP4, block-scaled FP4 tensor-core product (+ RAC) */
  QUADS_W4A16 = 1,  /* NVFP4 weights (w13_q / w13_sf / w13_gs) decoded to bf16, x stays bf16: out = bf16(W^) x,
                       a bf16 tensor-core product with float32 accumulation -- also the learner's forward of
                       Eq. "w4a16-qat-forward" */
  QUADS_W16A4 = 2,  /* x quantized online (a13_gs or amax-derived) and decoded to bf16, weights bf16 (w13_bf16):
                       out = W bf16(Q_A(x)) */
  QUADS_W16A16 = 3  /* neither side quantized (x and w13_bf16 in bf16): Y_train of Eq. "linear-mismatch", the
                       reference the mismatch of the other modes is measured against */
};

typedef struct {
  int32_t T, H, I, E, topk;
  int32_t N;                    /* dense mode only */
  const void* x;                /* bf16 [T, H] */
  const float* router_logits;   /* float [T, E]; ignored in dense mode */
  const uint8_t* w13_q;         /* u8 [E, 2I, H/2]  (dense: [N, H/2]) */
  const uint8_t* w13_sf;        /* tiled, E blocks of quads_sf_tiled_bytes(2I, H) */
  const float* w13_gs;          /* float [E] */
  const uint8_t* w2_q;          /* u8 [E, H, I/2] */
  const uint8_t* w2_sf;         /* tiled, E blocks of quads_sf_tiled_bytes(H, I) */
  const float* w2_gs;           /* float [E] */
  int32_t rac_nsel_13;          /* channels compensated at the W13 input, 0..H */
  int32_t rac_nsel_2;           /* channels compensated at the W2 input, 0..I */
  const float* a13_gs;          /* float[1] per-tensor scale of x, NULL: amax-derived on device */
  const float* a2_gs;           /* float[1] per-tensor scale of h; required when I > 0 */
  int32_t renormalize;
  void* out;                    /* bf16 [T, H]  (dense: [T, N]) */
  /* Optional exports for verification; each may be NULL. Dispatch order means
     assignments (token, slot) sorted by (expert, token, slot); A = T * topk. */
  int32_t* topk_ids;            /* [T, topk] */
  float* topk_w;                /* [T, topk] */
  int32_t* expert_offsets;      /* [E + 1] */
  int32_t* perm;                /* [A] flat assignment index t*topk+slot per dispatched row */
  uint8_t* xq;                  /* [T, H/2]  Q_A(x) codes, token order */
  uint8_t* xsf;                 /* [T, H/16] linear */
  uint8_t* rq;                  /* [T, H/2]  masked residual codes */
  uint8_t* rsf;                 /* [T, H/16] */
  int32_t* sel13;               /* [rac_nsel_13] ascending */
  float* a13_gs_out;            /* float[1] */
  void* h_bf16;                 /* bf16 [A, I], dispatch order */
  uint8_t* hq;                  /* [A, I/2] */
  uint8_t* hsf;                 /* [A, I/16] linear */
  uint8_t* r2q;                 /* [A, I/2] masked residual codes of h */
  uint8_t* r2sf;                /* [A, I/16] */
  int32_t* sel2;                /* [rac_nsel_2] ascending */
  void* workspace;
  size_t workspace_bytes;       /* >= quads_moe_workspace_bytes(T, H, I, E, topk, N) */
  /* Dense mode only: which operands are NVFP4 (the one-sided rollout modes of Table
     "qdq-alignment" and Section "Train-inference mismatch ...").  Modes 1 and 2 take no RAC
     (rac_nsel_13 must be 0): they exist to isolate one side's quantization error. */
  int32_t operand_mode;         /* QUADS_W4A4 (0, default), QUADS_W4A16, QUADS_W16A4 or QUADS_W16A16 */
  const void* w13_bf16;         /* QUADS_W16A4 / QUADS_W16A16: the unquantized weight, bf16 [N, H], 16-byte aligned */
  /* Expert-sharded execution (MoE mode; the paper's engines run the experts expert-parallel, Section
     "Experimental setup"): this call holds the weights of experts [expert_lo, expert_lo + expert_count)
     only -- w13_* / w2_* are arrays over those experts -- while x, router_logits and the routing are
     those of the whole layer (E experts).  It computes the contributions of its experts to every token:
     quantization, channel statistics and both selections run over the whole token batch at site 13
     (identical on every shard) and over the shard's own dispatched rows at site 2.  The partial sums are
     written unrounded to out_f32; the shards' partial sums add up to the layer output (an all-reduce when
     the shards live on several GPUs).  expert_count == 0 means all E experts (the default). */
  int32_t expert_lo, expert_count;
  float* out_f32;               /* optional float [T, H]: the call's sum before rounding; `out` may then be NULL */
} quads_moe_args;

quads_status quads_moe_w4a4_rac(const quads_moe_args* args /* host */, void* cuda_stream);
size_t quads_moe_workspace_bytes(int32_t T, int32_t H, int32_t I, int32_t E, int32_t topk,
                                 int32_t N);
/* Reads (with a device-to-host copy and a stream synchronise) the status word
   that device-side bounded waits write into the workspace of an earlier
   quads_moe_w4a4_rac call: QUADS_OK or QUADS_ERR_TIMEOUT. */
quads_status quads_moe_async_status(const void* workspace, void* cuda_stream);

/*
 * Measurement aid (no counterpart in the paper).  When enabled, every later
 * MoE-mode quads_moe_w4a4_rac call records CUDA events on its stream right
 * before and after each of its two grouped GEMM kernels; quads_moe_last_kernel_ms
 * waits for the most recent call's events and returns the two durations in
 * milliseconds (host pointers).  Off by default; the events are created on the
 * device that is current at the first enable.  Returns QUADS_ERR_SHAPE when no
 * timed call has been made.
 */
quads_status quads_moe_set_kernel_timing(int32_t enable);
quads_status quads_moe_last_kernel_ms(float* gemm1_ms /* host */, float* gemm2_ms /* host */);

/*
 * Measurement aid (no counterpart in the paper): when enabled, a MoE-mode call
 * records a CUDA event on its stream after every stage; get_stage_trace waits
 * for the last call and fills, for each stage, its name (static host string)
 * and the time since the previous mark in milliseconds; returns the number of
 * entries written (at most `cap`).  Off by default; not thread-safe.
 */
quads_status quads_moe_set_stage_trace(int32_t enable);
int32_t quads_moe_get_stage_trace(const char** names /* host */, float* ms /* host */, int32_t cap);

/*
 * FP8 W8A8 comparison path: the "FP8 W8A8" rollout arm that the paper measures NVFP4 against
 * (Section "Low-Precision Inference", paragraph FP8; Section "Rollout Throughput Comparison").  E4M3
 * elements (maximum 448) with fine-grained power-of-two scales: one per (row, 128 channels) of an
 * activation, one per 128 x 128 tile of a weight; scale = 2^e with e the smallest integer for which the
 * tile's amax fits (amax <= 448 * 2^e), stored as the byte e + 127; element = E4M3_rne_sat(x * 2^-e).
 * The same MoE layer as quads_moe_w4a4_rac (top-k routing, dispatch order, SwiGLU, h rounded to bf16
 * and requantized per (row, 128 features), weighted combine) on block-scaled FP8 tensor-core GEMMs;
 * there is no residual compensation in this format.
 *
 * quads_fp8_quantize_weights:  w bf16 [n, N, K] (N % 128 == 0, K % 128 == 0, 16-byte aligned) ->
 *   q u8 [n, N, K], exps u8 [n, N/128, K/128], atoms u8 [n, N/128, K/128, 512] (each tile's scale byte
 *   repeated 512 times: what the GEMM copies into tensor memory; 16-byte aligned).
 * quads_moe_fp8_w8a8: H % 128 == 0, I % 128 == 0, limits on E / topk as for quads_moe_w4a4_rac; the
 *   optional exports (dispatch order, A = T * topk rows) serve verification.  Enqueued on one stream;
 *   device-side waits are bounded and report through quads_moe_async_status(workspace).
 */
quads_status quads_fp8_quantize_weights(const void* w, int64_t n_tensors, int64_t N, int64_t K, uint8_t* q,
                                        uint8_t* exps, uint8_t* atoms, void* cuda_stream);
typedef struct {
  int32_t T, H, I, E, topk;
  const void* x;                 /* bf16 [T, H] */
  const float* router_logits;    /* float [T, E] */
  const uint8_t* w13_q;          /* u8 [E, 2I, H], gate rows first */
  const uint8_t* w13_atoms;      /* u8 [E, 2I/128, H/128, 512] */
  const uint8_t* w2_q;           /* u8 [E, H, I] */
  const uint8_t* w2_atoms;       /* u8 [E, H/128, I/128, 512] */
  int32_t renormalize;
  void* out;                     /* bf16 [T, H] */
  int32_t* topk_ids;             /* optional exports: [T, topk] */
  int32_t* perm;                 /* [A] */
  uint8_t* xq;                   /* [T, H] E4M3 codes of x, token order */
  uint8_t* xexp;                 /* [T, H/128] */
  void* h_bf16;                  /* bf16 [A, I]; with it hq [A, I] and hexp [A, I/128] must be given too */
  uint8_t* hq;
  uint8_t* hexp;
  void* workspace;
  size_t workspace_bytes;        /* >= quads_moe_fp8_workspace_bytes(T, H, I, E, topk), 256-byte aligned */
} quads_moe_fp8_args;
quads_status quads_moe_fp8_w8a8(const quads_moe_fp8_args* args /* host */, void* cuda_stream);
size_t quads_moe_fp8_workspace_bytes(int32_t T, int32_t H, int32_t I, int32_t E, int32_t topk);

/*
 * Diagnostics of the paper's mismatch analysis, computed on the device.
 *
 * quads_rac_channel_scores: s_j^2 = sum over the token batch of (Q_A(X) - X)[:, j]^2, the squared
 * channel score of Eq. "channel-score" -- the per-channel residual map whose heavy channels are the
 * "vertical bands" of Fig. "residual-distribution" and whose largest entries RAC selects.
 *   x       bf16 [T, H], 32-byte aligned, H % 128 == 0
 *   gs_in   float[1] per-tensor scale of x, or NULL: amax-derived on the device
 *   scores  out, double [H] (per-CTA float32 partial sums over <= 14 rows, then float64, fixed order)
 *   workspace >= quads_rac_channel_scores_workspace_bytes(T, H) bytes, 256-byte aligned
 *
 * quads_mismatch_norms: out = { ||A - B||_F^2, ||A||_F^2, ||B||_F^2 } for two bf16 tensors of n
 * elements, float64 accumulation in a fixed order -- the layer-wise forward mismatch of Eq.
 * "linear-mismatch" for A = Y_infer, B = Y_train (take the square root of out[0]), and, with the
 * one-sided modes of quads_moe_w4a4_rac as A, its activation-error and weight-error terms.
 *   a, b    bf16 [n], 16-byte aligned;  out  double [3] (device)
 *   workspace >= quads_mismatch_norms_workspace_bytes() bytes, 256-byte aligned
 */
quads_status quads_rac_channel_scores(const void* x, int64_t T, int64_t H, const float* gs_in, double* scores,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t quads_rac_channel_scores_workspace_bytes(int64_t T, int64_t H);
quads_status quads_mismatch_norms(const void* a, const void* b, int64_t n, double* out, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream);
size_t quads_mismatch_norms_workspace_bytes(void);

/*
 * Measurement aid (no counterpart in the paper): the tensor-pipe probe.  One
 * persistent CTA per SM keeps one pipeline stage of FP4 operands and UE4M3 scale
 * atoms (the grouped GEMM's stage layout, quads_fp4_pipe_probe_operand_bytes()
 * bytes copied once from `operands`, device memory, 16-byte aligned) resident in
 * shared memory and issues `k_steps` times what the GEMM's main loop issues per
 * K = 64 step, with no global traffic in the loop:
 *   mode 0  one 128 x 256 x 64 block-scaled MMA per step (the bare pipe);
 *   mode 1  two MMAs + four scale copies per step (first projection with RAC);
 *   mode 2  one MMA + three scale copies (plain W4A4);
 *   mode 3  two MMAs, no copies;  mode 4  as mode 1 with the copies issued by a
 *   second thread;  mode 5  one 128 x 128 x 64 MMA.
 * Time it with events on `cuda_stream`; *flop_out (host, may be NULL) receives
 * the floating-point operations of the launch (2 * M * N * 64 per MMA and SM).  Scale bytes in `operands` should avoid the NaN code 0x7F.  The wait for
 * the pipe to drain is bounded; a give-up writes QUADS_ERR_TIMEOUT to
 * *status_word (device int32, zero it first).
 */
quads_status quads_fp4_pipe_probe(int32_t mode, int32_t k_steps, const void* operands, size_t operand_bytes,
                                  int32_t* status_word, double* flop_out /* host */, void* cuda_stream);
size_t quads_fp4_pipe_probe_operand_bytes(void);

/*
 * Test hook (no counterpart in the paper): exercises the give-up path of a
 * bounded device-side wait without faulting or hanging anything.  It sets the
 * bound, in SM clock cycles, of the wait in which the CTAs of the cooperative
 * quantization kernel (quads_fake_quant_weights on tensors above 32 MB, or any
 * quantizing call under QUADS_QUANT_COOPERATIVE / QUADS_NO_RING_QUANT) meet at a
 * tensor's arrival counter in global memory, and
 * a surplus of arrivals to expect that nothing will ever deliver.  With a
 * surplus > 0 every such wait runs out after `clock_cycles`: the call still
 * completes, its outputs are unspecified and gs_out = NaN marks them.
 * clock_cycles <= 0 and extra_arrivals <= 0 restore the defaults (about two
 * seconds, no surplus).  Process-wide; meant for tests only.
 */
void quads_debug_set_quantize_wait(int64_t clock_cycles, int32_t extra_arrivals);

/* Number of kernels the last quads_* call on this host thread enqueued. */
int32_t quads_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* QUADS_H_ */
