// Streaming kernels: tensor amax, NVFP4 quantize / fake-quant, RAC statistics,
// channel selection, masked residual quantize + dispatch scatter, small fix-ups.
// All HBM- or latency-bound; no tensor cores here.
#include "kernels.cuh"

namespace quads {

// ---------------------------------------------------------------------------
// amax over bf16 tensors.  gridDim.y = tensor; magnitudes compared as 15-bit
// integers (two per 32-bit word); result = bf16 bit pattern << 16 = float bits.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) amax_kernel(const uint16_t* __restrict__ x, int64_t rows, int64_t K,
                                                   int64_t ld, int64_t tensor_stride,
                                                   uint32_t* __restrict__ amax_bits) {
  pdl_sync();
  const uint16_t* base = x + (size_t)blockIdx.y * tensor_stride;
  const int64_t k8 = K >> 3;
  const int64_t chunks = rows * k8;
  uint32_t m = 0;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  if (ld == K) {
    const uint4* p = reinterpret_cast<const uint4*>(base);
    int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; c + 3 * stride < chunks; c += 4 * stride) {
      uint4 v0 = __ldg(p + c), v1 = __ldg(p + c + stride), v2 = __ldg(p + c + 2 * stride),
            v3 = __ldg(p + c + 3 * stride);
      uint32_t a = __vmaxu2(__vmaxu2(v0.x & 0x7FFF7FFFu, v0.y & 0x7FFF7FFFu),
                            __vmaxu2(v0.z & 0x7FFF7FFFu, v0.w & 0x7FFF7FFFu));
      uint32_t b = __vmaxu2(__vmaxu2(v1.x & 0x7FFF7FFFu, v1.y & 0x7FFF7FFFu),
                            __vmaxu2(v1.z & 0x7FFF7FFFu, v1.w & 0x7FFF7FFFu));
      uint32_t c2 = __vmaxu2(__vmaxu2(v2.x & 0x7FFF7FFFu, v2.y & 0x7FFF7FFFu),
                             __vmaxu2(v2.z & 0x7FFF7FFFu, v2.w & 0x7FFF7FFFu));
      uint32_t d = __vmaxu2(__vmaxu2(v3.x & 0x7FFF7FFFu, v3.y & 0x7FFF7FFFu),
                            __vmaxu2(v3.z & 0x7FFF7FFFu, v3.w & 0x7FFF7FFFu));
      m = __vmaxu2(m, __vmaxu2(__vmaxu2(a, b), __vmaxu2(c2, d)));
    }
    for (; c < chunks; c += stride) {
      uint4 v = __ldg(p + c);
      m = __vmaxu2(m, __vmaxu2(__vmaxu2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu),
                               __vmaxu2(v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu)));
    }
  } else {
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < chunks; c += stride) {
      const int64_t r = c / k8, cc = c - r * k8;
      uint4 v = __ldg(reinterpret_cast<const uint4*>(base + r * ld + cc * 8));
      m = __vmaxu2(m, __vmaxu2(__vmaxu2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu),
                               __vmaxu2(v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu)));
    }
  }
  uint32_t s = max(m & 0xFFFFu, m >> 16);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s = max(s, __shfl_xor_sync(0xFFFFFFFFu, s, o));
  __shared__ uint32_t wmax[8];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t t = 0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t = max(t, wmax[i]);
    if (t) atomicMax(amax_bits + blockIdx.y, t << 16);
  }
}

__device__ __forceinline__ float gs_from_amax_bits(uint32_t bits) {
  const float amax = __uint_as_float(bits);
  return amax > 0.f ? __fdiv_rn(amax, kGlobalDiv) : 1.0f;
}

// ---------------------------------------------------------------------------
// Fused amax + NVFP4 quantize / fake-quant in ONE cooperative launch.
// The CTAs form `n_groups` groups (CTA c belongs to group c % n_groups, so every
// group spans all SMs).  A group takes tensors group, group + n_groups, ...:
//   phase 1  its CTAs stream the tensor once (kept in L2: evict_last), reduce
//            |x| max, publish it with atomicMax and meet at a per-tensor counter;
//   phase 2  they read the tensor again (from L2), quantize, and stream the
//            outputs out (evict_first).
// Other groups overlap their phases with this group's barrier wait.  DRAM sees
// each input byte once: 2 B read + the outputs per element.
// `amax_bits` and `counters` (one word each per tensor) must be zero on entry.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void ldg256_keep(const void* p, uint4& a, uint4& b) {
  asm volatile("ld.global.L2::evict_last.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(p));
}
__device__ __forceinline__ void ldg256_stream(const void* p, uint4& a, uint4& b) {
  asm volatile("ld.global.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(p));
}
__device__ __forceinline__ uint32_t absmax8(const uint4& v) {
  return __vmaxu2(__vmaxu2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu), __vmaxu2(v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu));
}

__global__ void __launch_bounds__(256, 4)
fused_quantize_kernel(const uint16_t* __restrict__ x, int64_t rows, int64_t K, int64_t ld, int64_t tensor_stride,
                      int n_tensors, const float* __restrict__ gs_in, uint32_t* __restrict__ amax_bits,
                      uint32_t* __restrict__ counters, uint8_t* __restrict__ q, uint8_t* __restrict__ sf,
                      uint16_t* __restrict__ fq, float* __restrict__ gs_out, int sf_tiled, int64_t sf_tensor_stride,
                      int n_groups) {
  const int group = blockIdx.x % n_groups;
  const int rank = blockIdx.x / n_groups;
  const int gsize = ((int)gridDim.x - group + n_groups - 1) / n_groups;
  const int64_t k16 = K >> 4;
  const int64_t nblk = rows * k16;
  const int64_t gthreads = (int64_t)gsize * blockDim.x;
  const int64_t gtid = (int64_t)rank * blockDim.x + threadIdx.x;
  __shared__ uint32_t wmax[8];
  __shared__ float gs_sh;
  __shared__ float inv_lut[128];
  for (int t = group; t < n_tensors; t += n_groups) {
    const uint16_t* base = x + (size_t)t * tensor_stride;
    float gs;
    if (gs_in) {
      gs = gs_in[t];
    } else {
      // ---- phase 1: tensor amax, one 32-byte block per load
      uint32_t m = 0;
      if (ld == K) {
        int64_t b = gtid;
        for (; b + 3 * gthreads < nblk; b += 4 * gthreads) {
          uint4 a0, a1, b0, b1, c0, c1, d0, d1;
          ldg256_keep(base + b * 16, a0, a1);
          ldg256_keep(base + (b + gthreads) * 16, b0, b1);
          ldg256_keep(base + (b + 2 * gthreads) * 16, c0, c1);
          ldg256_keep(base + (b + 3 * gthreads) * 16, d0, d1);
          m = __vmaxu2(m, __vmaxu2(__vmaxu2(__vmaxu2(absmax8(a0), absmax8(a1)), __vmaxu2(absmax8(b0), absmax8(b1))),
                                   __vmaxu2(__vmaxu2(absmax8(c0), absmax8(c1)), __vmaxu2(absmax8(d0), absmax8(d1)))));
        }
        for (; b < nblk; b += gthreads) {
          uint4 a0, a1;
          ldg256_keep(base + b * 16, a0, a1);
          m = __vmaxu2(m, __vmaxu2(absmax8(a0), absmax8(a1)));
        }
      } else {
        for (int64_t b = gtid; b < nblk; b += gthreads) {
          const int64_t r = b / k16, kb = b - r * k16;
          uint4 a0, a1;
          ldg256_keep(base + r * ld + kb * 16, a0, a1);
          m = __vmaxu2(m, __vmaxu2(absmax8(a0), absmax8(a1)));
        }
      }
      uint32_t sm = max(m & 0xFFFFu, m >> 16);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sm = max(sm, __shfl_xor_sync(0xFFFFFFFFu, sm, o));
      if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = sm;
      __syncthreads();
      if (threadIdx.x == 0) {
        uint32_t tm = 0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) tm = max(tm, wmax[i]);
        if (tm) atomicMax(amax_bits + t, tm << 16);
        __threadfence();
        atomicAdd(counters + t, 1u);
        // bounded wait for the rest of the group (cooperative launch: all CTAs are resident)
        const long long t0 = clock64();
        while (atomicAdd(counters + t, 0u) < (uint32_t)gsize) {
          __nanosleep(64);
          if (clock64() - t0 > 4000000000ll) break;
        }
        __threadfence();
        gs_sh = gs_from_amax_bits(atomicAdd(amax_bits + t, 0u));
      }
      __syncthreads();
      gs = gs_sh;
      __syncthreads();
    }
    if (gs_out && rank == 0 && threadIdx.x == 0) gs_out[t] = gs;
    __syncthreads();                              // the previous tensor's table is no longer read
    if (threadIdx.x < 128) inv_lut[threadIdx.x] = quant_inv_entry(threadIdx.x, gs);
    __syncthreads();
    QuantCtx qc;
    quant_ctx_scalars(qc, gs);
    qc.inv_lut = inv_lut;
    // ---- phase 2: quantize (16-element blocks), stream the outputs
    uint8_t* qt = q ? q + (size_t)t * rows * (K >> 1) : nullptr;
    uint8_t* sft = sf ? sf + (size_t)t * sf_tensor_stride : nullptr;
    uint16_t* fqt = fq ? fq + (size_t)t * rows * K : nullptr;
    const int kt_count = (int)((K + 63) >> 6);
    const bool contiguous = (ld == K);
    const uint32_t k16u = (uint32_t)k16;
    auto emit = [&](int64_t b, const uint4& v0, const uint4& v1) {
      float f[16];
      unpack8(v0, f);
      unpack8(v1, f + 8);
      const BlockQ bq = quantize_block(f, qc);
      // outputs are contiguous per tensor: block b owns bytes [8b, 8b+8) of q and [32b, 32b+32) of fq
      if (qt) __stcs(reinterpret_cast<uint2*>(qt + b * 8), make_uint2(bq.lo, bq.hi));
      if (sft) {
        if (sf_tiled) {
          const uint32_t r = (uint32_t)(b / k16u), kb = (uint32_t)(b - (int64_t)r * k16u);
          sft[sf_tiled_offset(r, kb, kt_count)] = (uint8_t)bq.sf8;
        } else {
          sft[b] = (uint8_t)bq.sf8;
        }
      }
      if (fqt) {
        float o[16];
        dequant_block(bq, o);
        uint4* dst = reinterpret_cast<uint4*>(fqt + b * 16);
        __stcs(dst, make_uint4(f32x2_to_bf16x2(o[0], o[1]), f32x2_to_bf16x2(o[2], o[3]),
                               f32x2_to_bf16x2(o[4], o[5]), f32x2_to_bf16x2(o[6], o[7])));
        __stcs(dst + 1, make_uint4(f32x2_to_bf16x2(o[8], o[9]), f32x2_to_bf16x2(o[10], o[11]),
                                   f32x2_to_bf16x2(o[12], o[13]), f32x2_to_bf16x2(o[14], o[15])));
      }
    };
    auto src_of = [&](int64_t b) -> const uint16_t* {
      if (contiguous) return base + b * 16;
      const int64_t r = b / k16, kb = b - r * k16;
      return base + r * ld + kb * 16;
    };
    int64_t b = gtid;
    for (; b + 3 * gthreads < nblk; b += 4 * gthreads) {     // four loads in flight per thread
      uint4 a0, a1, c0, c1, d0, d1, e0, e1;
      ldg256_stream(src_of(b), a0, a1);
      ldg256_stream(src_of(b + gthreads), c0, c1);
      ldg256_stream(src_of(b + 2 * gthreads), d0, d1);
      ldg256_stream(src_of(b + 3 * gthreads), e0, e1);
      emit(b, a0, a1);
      emit(b + gthreads, c0, c1);
      emit(b + 2 * gthreads, d0, d1);
      emit(b + 3 * gthreads, e0, e1);
    }
    for (; b < nblk; b += gthreads) {
      uint4 a0, a1;
      ldg256_stream(src_of(b), a0, a1);
      emit(b, a0, a1);
    }
  }
}

// ---------------------------------------------------------------------------
// Site-13 quantization pass, token order.  For every row and 16-channel block:
// Q_A(x) codes + scale; the residual Q_A(x) - x in float32 (Eq. residual-def);
// its squared sum per channel over the rows this CTA owns (Eq. channel-score,
// one partial row per CTA, reduced later in a fixed order); and the residual's
// own quantization with the same per-tensor scale (the mask of Eq.
// residual-recon is applied later, when rows are copied into dispatch order:
// quantizing the residual does not depend on the selection).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
rac_quant_kernel(const uint16_t* __restrict__ x, int T, int H, const float* __restrict__ gs_in,
                 uint32_t* __restrict__ amax_bits, unsigned int* __restrict__ grid_arrivals, int32_t* __restrict__ status,
                 float* __restrict__ gs_store, int rows_per_cta,
                 int with_residual, float* __restrict__ partials, uint8_t* __restrict__ xq,
                 uint8_t* __restrict__ xsf, uint8_t* __restrict__ rq, uint8_t* __restrict__ rsf,
                 uint8_t* __restrict__ xq_exp, uint8_t* __restrict__ xsf_exp) {
  pdl_sync();
  const int k16 = H >> 4;
  const int r0 = blockIdx.x * rows_per_cta;
  const int r1 = min(T, r0 + rows_per_cta);
  __shared__ float gs_sh;
  if (grid_arrivals) {
    // Cooperative launch with no per-tensor scale given: first the tensor's amax over this
    // CTA's rows (the same rows it quantizes below, so the second read hits L1 / L2), then a
    // bounded wait until every CTA has contributed.
    __shared__ uint32_t wmax[8];
    uint32_t m = 0;
    for (int kb = threadIdx.x; kb < k16; kb += blockDim.x)
      for (int r = r0; r < r1; ++r) {
        uint4 v0, v1;
        ldg256(x + (size_t)r * H + kb * 16, v0, v1);
        m = __vmaxu2(m, __vmaxu2(absmax8(v0), absmax8(v1)));
      }
    uint32_t smx = max(m & 0xFFFFu, m >> 16);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) smx = max(smx, __shfl_xor_sync(0xFFFFFFFFu, smx, o));
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = smx;
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t tm = 0;
      for (int i = 0; i < (int)((blockDim.x + 31) >> 5); ++i) tm = max(tm, wmax[i]);
      if (tm) atomicMax(amax_bits, tm << 16);
      __threadfence();
      atomicAdd(grid_arrivals, 1u);
      const long long t0 = clock64();
      unsigned int seen;
      for (;;) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(grid_arrivals) : "memory");
        if (seen >= gridDim.x) break;
        __nanosleep(200);
        if (clock64() - t0 > 4000000000ll) { atomicExch(status, (int32_t)QUADS_ERR_TIMEOUT); break; }
      }
      gs_sh = gs_from_amax_bits(atomicAdd(amax_bits, 0u));
    }
    __syncthreads();
  } else if (threadIdx.x == 0) {
    gs_sh = gs_in ? gs_in[0] : gs_from_amax_bits(amax_bits[0]);
  }
  __syncthreads();
  const float gs = gs_sh;
  if (gs_store && blockIdx.x == 0 && threadIdx.x == 0) gs_store[0] = gs;
  __shared__ float inv_lut[128];
  for (int i = threadIdx.x; i < 128; i += blockDim.x) inv_lut[i] = quant_inv_entry(i, gs);
  __syncthreads();
  QuantCtx qc;
  quant_ctx_scalars(qc, gs);
  qc.inv_lut = inv_lut;
  for (int kb = threadIdx.x; kb < k16; kb += blockDim.x) {
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.f;
    uint4 n0 = make_uint4(0, 0, 0, 0), n1 = n0;
    if (r0 < r1) ldg256(x + (size_t)r0 * H + kb * 16, n0, n1);
    for (int r = r0; r < r1; ++r) {
      const uint4 v0 = n0, v1 = n1;
      if (r + 1 < r1) ldg256(x + (size_t)(r + 1) * H + kb * 16, n0, n1);   // next row's block, ahead of this row's arithmetic
      float f[16], o[16];
      unpack8(v0, f);
      unpack8(v1, f + 8);
      const BlockQ bq = quantize_block(f, qc);
      const size_t qo = (size_t)r * (H >> 1) + kb * 8, so = (size_t)r * k16 + kb;
      *reinterpret_cast<uint2*>(xq + qo) = make_uint2(bq.lo, bq.hi);
      xsf[so] = (uint8_t)bq.sf8;
      if (xq_exp) *reinterpret_cast<uint2*>(xq_exp + qo) = make_uint2(bq.lo, bq.hi);
      if (xsf_exp) xsf_exp[so] = (uint8_t)bq.sf8;
      if (with_residual) {
        dequant_block(bq, o);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          o[i] = __fsub_rn(o[i], f[i]);
          acc[i] = __fmaf_rn(o[i], o[i], acc[i]);
        }
        const BlockQ br = quantize_block(o, qc);
        *reinterpret_cast<uint2*>(rq + qo) = make_uint2(br.lo, br.hi);
        rsf[so] = (uint8_t)br.sf8;
      }
    }
    if (with_residual) {
      float4* dst = reinterpret_cast<float4*>(partials + (size_t)blockIdx.x * H + kb * 16);
      dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
      dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
      dst[2] = make_float4(acc[8], acc[9], acc[10], acc[11]);
      dst[3] = make_float4(acc[12], acc[13], acc[14], acc[15]);
    }
  }
}

// Channel scores (Eq. channel-score).  The partial rows are split into
// kScoreSlices contiguous slices; CTA (column group, slice) adds its slice's
// rows in float64.  The CTA of a column group that finishes last adds the
// slice sums in slice order (a fixed order, whichever CTA does it) and stores
// the group's 32 scores as order-preserving 64-bit keys (scores are >= 0).
// grid = (ceil(C/32), kScoreSlices), 256 threads = 32 columns x 8 row lanes.
// `counters` (one per column group) must be zero on entry.
__global__ void __launch_bounds__(256)
score_reduce_kernel(const float* __restrict__ partials, const int* __restrict__ n_part_ptr, int n_part_mul,
                    int n_part_fixed, int C, double* __restrict__ slice_sums, unsigned int* __restrict__ counters,
                    unsigned long long* __restrict__ score_keys) {
  pdl_sync();
  const int n_part = n_part_ptr ? *n_part_ptr * n_part_mul : n_part_fixed;
  const int per = (n_part + kScoreSlices - 1) / kScoreSlices;
  const int p0 = blockIdx.y * per, p1 = min(n_part, p0 + per);
  const int col = blockIdx.x * 32 + (threadIdx.x & 31);
  const int rl = threadIdx.x >> 5;
  double s = 0.0;
  if (col < C)
    for (int p = p0 + rl; p < p1; p += 8) s += (double)partials[(size_t)p * C + col];
  __shared__ double sm[8][32];
  __shared__ unsigned int last;
  sm[rl][threadIdx.x & 31] = s;
  __syncthreads();
  if (rl == 0 && col < C) {
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) t += sm[i][threadIdx.x & 31];
    slice_sums[(size_t)blockIdx.y * C + col] = t;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = atomicAdd(counters + blockIdx.x, 1u);
  __syncthreads();
  if (last == kScoreSlices - 1 && rl == 0 && col < C) {
    __threadfence();
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < kScoreSlices; ++i) t += __ldcg(slice_sums + (size_t)i * C + col);
    score_keys[col] = (unsigned long long)__double_as_longlong(t);
  }
}

// Channel selection (Eq. channel-select): rank_j = #{i : s_i > s_j, or s_i ==
// s_j and i < j}; channel j is selected iff rank_j < n_sel (the n_sel largest,
// ties to the lower index).  Every CTA loads all C score keys into shared
// memory and ranks 16 channels with 16 threads each.
// grid = ceil(C/16), 256 threads, smem = C * 8 bytes.
__global__ void __launch_bounds__(256)
rank_select_kernel(const unsigned long long* __restrict__ score_keys, int C, int n_sel, uint8_t* __restrict__ mask) {
  pdl_sync();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* sc = reinterpret_cast<unsigned long long*>(smem_raw);
  for (int i = threadIdx.x; i < C; i += blockDim.x) sc[i] = score_keys[i];
  __syncthreads();
  const int j = blockIdx.x * 16 + (threadIdx.x >> 4);
  const int sub = threadIdx.x & 15;
  int rank = 0;
  if (j < C) {
    const unsigned long long sj = sc[j];
#pragma unroll 8
    for (int i = sub; i < C; i += 16) {
      const unsigned long long si = sc[i];
      rank += (si > sj || (si == sj && i < j)) ? 1 : 0;
    }
  }
#pragma unroll
  for (int o = 1; o < 16; o <<= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
  if (j < C && sub == 0) mask[j] = rank < n_sel ? 1 : 0;
}

// Ascending list of the selected channels (verification export only).  One CTA.
__global__ void __launch_bounds__(1024)
sel_list_kernel(const uint8_t* __restrict__ mask, int C, int32_t* __restrict__ sel_export) {
  pdl_sync();
  __shared__ int chunk_tot[1024];
  const int tid = threadIdx.x, nt = blockDim.x;
  const int per = (C + nt - 1) / nt;
  const int c0 = tid * per, c1 = min(C, c0 + per);
  int cnt = 0;
  for (int i = c0; i < c1; ++i) cnt += mask[i];
  chunk_tot[tid] = cnt;
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int i = 0; i < nt; ++i) { const int c = chunk_tot[i]; chunk_tot[i] = run; run += c; }
  }
  __syncthreads();
  int pos = chunk_tot[tid];
  for (int i = c0; i < c1; ++i)
    if (mask[i]) sel_export[pos++] = i;
}

// ---------------------------------------------------------------------------
// Site-13 dispatch: copy every token row's codes and scales into each of its
// dispatched copies (padded dispatch order, tiled scale layout).  The residual
// is masked on the way (Eq. residual-recon: codes of unselected channels are
// cleared) and stored NEGATED (sign bits flipped) so that the GEMM can
// accumulate W Q(x) + W (-M Q(dx)) with two plain MMAs.  Pure data movement:
// one thread per (token, 32 channels = 16 code bytes).
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t nibble_mask8(const uint8_t* m) {
  // m[0..7] in {0,1} -> 0xF per selected nibble
  const uint2 v = *reinterpret_cast<const uint2*>(m);
  uint32_t out = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out |= ((v.x >> (8 * i)) & 1u) * (0xFu << (4 * i));
    out |= ((v.y >> (8 * i)) & 1u) * (0xFu << (16 + 4 * i));
  }
  return out;
}

__global__ void __launch_bounds__(256)
rac_scatter_kernel(int T, int H, int parts, const uint8_t* __restrict__ mask, int topk,
                   const int32_t* __restrict__ pos_pad, const uint8_t* __restrict__ xq,
                   const uint8_t* __restrict__ xsf, const uint8_t* __restrict__ rq, const uint8_t* __restrict__ rsf,
                   uint8_t* __restrict__ xq_pad, uint8_t* __restrict__ xsf_tiled, uint8_t* __restrict__ rq_pad,
                   uint8_t* __restrict__ rsf_tiled, uint8_t* __restrict__ rq_exp, uint8_t* __restrict__ rsf_exp) {
  pdl_sync();
  const int per_row = H >> 5;                         // 16-byte chunks of codes per row
  const int64_t n_chunks = (int64_t)T * per_row;
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < n_chunks; g += (int64_t)gridDim.x * blockDim.x) {
  const int t = (int)(g / per_row), c = (int)(g - (int64_t)t * per_row);
  const size_t co = (size_t)t * (H >> 1) + c * 16;
  const bool do_x = (parts & 1) != 0, with_residual = (parts & 2) != 0;
  uint4 xv = make_uint4(0, 0, 0, 0), rv = make_uint4(0, 0, 0, 0);
  const bool sf_owner = (c & 1) == 0;                 // even chunks also move 4 scale bytes (64 channels)
  uint32_t xs = 0, rs = 0;
  if (do_x) {
    xv = __ldg(reinterpret_cast<const uint4*>(xq + co));
    if (sf_owner) xs = __ldg(reinterpret_cast<const uint32_t*>(xsf + (size_t)t * (H >> 4) + c * 2));
  }
  if (with_residual) {
    rv = __ldg(reinterpret_cast<const uint4*>(rq + co));
    const uint8_t* m = mask + c * 32;
    rv.x &= nibble_mask8(m); rv.y &= nibble_mask8(m + 8);
    rv.z &= nibble_mask8(m + 16); rv.w &= nibble_mask8(m + 24);
    if (sf_owner) rs = __ldg(reinterpret_cast<const uint32_t*>(rsf + (size_t)t * (H >> 4) + c * 2));
    if (rq_exp) *reinterpret_cast<uint4*>(rq_exp + co) = rv;
    if (rsf_exp && sf_owner) *reinterpret_cast<uint32_t*>(rsf_exp + (size_t)t * (H >> 4) + c * 2) = rs;
    rv.x ^= 0x88888888u; rv.y ^= 0x88888888u; rv.z ^= 0x88888888u; rv.w ^= 0x88888888u;
  }
  const int kt_count = H >> 6;
  for (int s0 = 0; s0 < topk; s0 += 8) {
    int p[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) p[j] = (s0 + j < topk) ? __ldg(pos_pad + t * topk + s0 + j) : -1;   // all loads first
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (p[j] < 0) continue;
      const size_t po = (size_t)p[j] * (H >> 1) + c * 16;
      if (do_x) __stcs(reinterpret_cast<uint4*>(xq_pad + po), xv);
      if (with_residual) __stcs(reinterpret_cast<uint4*>(rq_pad + po), rv);
      if (sf_owner) {
        const size_t so = sf_tiled_offset(p[j], c * 2, kt_count);
        if (do_x) *reinterpret_cast<uint32_t*>(xsf_tiled + so) = xs;
        if (with_residual) *reinterpret_cast<uint32_t*>(rsf_tiled + so) = rs;
      }
    }
  }
  }
}

// Clear (in place) the codes of unselected channels of a padded [rows, C/2]
// code matrix; one thread per 16 bytes (32 channels).  A thread keeps its column
// chunk (its four nibble-mask words are formed once) and walks down the rows.
__global__ void __launch_bounds__(256)
mask_codes_kernel(uint8_t* __restrict__ codes, const int* __restrict__ n_rows_ptr, int C,
                  const uint8_t* __restrict__ mask) {
  pdl_sync();
  const int per_row = C >> 5;
  const int n_rows = *n_rows_ptr;
  if (per_row <= 256) {
    const int rows_per_pass = 256 / per_row;
    const int c = threadIdx.x % per_row, rl = threadIdx.x / per_row;
    if (rl >= rows_per_pass) return;
    const uint8_t* m = mask + c * 32;
    const uint32_t m0 = nibble_mask8(m), m1 = nibble_mask8(m + 8), m2 = nibble_mask8(m + 16), m3 = nibble_mask8(m + 24);
    if ((m0 & m1 & m2 & m3) == 0xFFFFFFFFu) return;          // every channel of this chunk is selected
    for (int r = blockIdx.x * rows_per_pass + rl; r < n_rows; r += gridDim.x * rows_per_pass) {
      uint4* p = reinterpret_cast<uint4*>(codes + (size_t)r * (C >> 1)) + c;
      uint4 v = *p;
      v.x &= m0; v.y &= m1; v.z &= m2; v.w &= m3;
      *p = v;
    }
    return;
  }
  const int64_t n = (int64_t)n_rows * per_row;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int c = (int)(i % per_row);
    uint4* p = reinterpret_cast<uint4*>(codes) + i;
    uint4 v = *p;
    const uint8_t* m = mask + c * 32;
    v.x &= nibble_mask8(m); v.y &= nibble_mask8(m + 8);
    v.z &= nibble_mask8(m + 16); v.w &= nibble_mask8(m + 24);
    *p = v;
  }
}

// Weighted top-k combine: out[t, :] = sum over the token's slots, in slot order,
// of weight * y[row of (t, slot), :], accumulated in float32, rounded to bf16.
// One thread per (token, 8 columns).
__global__ void __launch_bounds__(256)
combine_kernel(const uint16_t* __restrict__ y_pad, const int32_t* __restrict__ pos_pad,
               const float* __restrict__ wts, int T, int H, int topk, uint16_t* __restrict__ out) {
  pdl_sync();
  const int per_row = H >> 3;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)T * per_row) return;
  const int t = (int)(i / per_row), c = (int)(i - (int64_t)t * per_row);
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  // eight slots at a time: all row positions first, then all row loads, so that the loads of a
  // token's rows are in flight together; the sum itself runs in slot order
  for (int s0 = 0; s0 < topk; s0 += 8) {
    int p[8];
    float w[8];
    uint4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const bool on = s0 + j < topk;
      p[j] = on ? __ldg(pos_pad + t * topk + s0 + j) : -1;
      w[j] = on ? __ldg(wts + t * topk + s0 + j) : 0.f;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
      v[j] = p[j] >= 0 ? __ldcs(reinterpret_cast<const uint4*>(y_pad + (size_t)p[j] * H) + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (p[j] < 0) continue;
      float f[8];
      unpack8(v[j], f);
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = __fmaf_rn(w[j], f[k], acc[k]);
    }
  }
  reinterpret_cast<uint4*>(out + (size_t)t * H)[c] =
      make_uint4(f32x2_to_bf16x2(acc[0], acc[1]), f32x2_to_bf16x2(acc[2], acc[3]),
                 f32x2_to_bf16x2(acc[4], acc[5]), f32x2_to_bf16x2(acc[6], acc[7]));
}

// Export of padded dispatch-order buffers into linear dispatch order.
// One thread per (dispatched row, 16-channel block).
__global__ void __launch_bounds__(256)
export_site2_kernel(int A, int I, const int32_t* __restrict__ perm, const int32_t* __restrict__ pos_pad,
                    const uint8_t* __restrict__ hq_pad, const uint8_t* __restrict__ hsf_tiled,
                    const uint8_t* __restrict__ r2q_pad, const uint8_t* __restrict__ r2sf_tiled,
                    const uint8_t* __restrict__ mask2, uint8_t* __restrict__ hq, uint8_t* __restrict__ hsf, uint8_t* __restrict__ r2q,
                    uint8_t* __restrict__ r2sf) {
  pdl_sync();
  const int k16 = I >> 4;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)A * k16) return;
  const int row = (int)(i / k16), kb = (int)(i - (int64_t)row * k16);
  const int p = pos_pad[perm[row]];
  const size_t so = sf_tiled_offset(p, kb, I >> 6);
  if (hq) *reinterpret_cast<uint2*>(hq + (size_t)row * (I >> 1) + kb * 8) =
      *reinterpret_cast<const uint2*>(hq_pad + (size_t)p * (I >> 1) + kb * 8);
  if (hsf) hsf[(size_t)row * k16 + kb] = hsf_tiled[so];
  if (r2q) {
    uint2 v = *reinterpret_cast<const uint2*>(r2q_pad + (size_t)p * (I >> 1) + kb * 8);
    // stored negated: flip the signs back, then clear the unselected channels again
    v.x = (v.x ^ 0x88888888u) & nibble_mask8(mask2 + kb * 16);
    v.y = (v.y ^ 0x88888888u) & nibble_mask8(mask2 + kb * 16 + 8);
    *reinterpret_cast<uint2*>(r2q + (size_t)row * (I >> 1) + kb * 8) = v;
  }
  if (r2sf) r2sf[(size_t)row * k16 + kb] = r2sf_tiled[so];
}

}  // namespace quads
