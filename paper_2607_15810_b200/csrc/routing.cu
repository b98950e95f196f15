// Top-k routing, per-expert histogram, exclusive scan and the stable dispatch
// permutation.  Integer outputs are deterministic: assignments (token, slot)
// end up sorted by (expert, token, slot).
#include "kernels.cuh"

namespace quads {

// Order-preserving map float -> uint32 (larger float <=> larger uint).
__device__ __forceinline__ uint32_t float_key(float v) {
  const uint32_t b = __float_as_uint(v);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Each warp routes kRouteTokensPerWarp tokens at once (independent chains hide
// the reduction latency).  E <= 256.  Top-k by logit, ties to the lower expert
// id, slots in descending-logit order; weights = softmax over all experts at
// the chosen ones, optionally renormalised.  Each CTA (kRouteTokensPerCta
// tokens) also writes its per-expert assignment counts: chunk_counts[expert][cta],
// and adds them to expert_total[expert] (zero on entry).
constexpr int kRouteTokensPerWarp = 4;
// NJ = logits per lane = ceil(E / 32) rounded up to 1, 2, 4 or 8.
template <int NJ>
__global__ void __launch_bounds__(256)
route_kernel_t(const float* __restrict__ logits, int T, int E, int topk, int renormalize,
             int32_t* __restrict__ ids, float* __restrict__ wts, int32_t* __restrict__ chunk_counts,
             int32_t* __restrict__ expert_total, int32_t* __restrict__ ids_out, float* __restrict__ wts_out,
             int e_lo, int e_hi) {
  pdl_sync();
  __shared__ int hist[kMaxExperts];
  for (int i = threadIdx.x; i < E; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t0 = blockIdx.x * kRouteTokensPerCta + warp * kRouteTokensPerWarp;
  constexpr int TW = kRouteTokensPerWarp;
  float v[TW][NJ];
  float mx[TW], sum[TW], wsum[TW], my_w[TW];
  int my_id[TW];
#pragma unroll
  for (int a = 0; a < TW; ++a) {
    const int t = t0 + a;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      const int e = j * 32 + lane;
      v[a][j] = (t < T && e < E) ? logits[(size_t)t * E + e] : -INFINITY;
    }
  }
#pragma unroll
  for (int a = 0; a < TW; ++a) {
    float m = v[a][0];
#pragma unroll
    for (int j = 1; j < NJ; ++j) m = fmaxf(m, v[a][j]);
    mx[a] = m;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int a = 0; a < TW; ++a) mx[a] = fmaxf(mx[a], __shfl_xor_sync(0xFFFFFFFFu, mx[a], o));
#pragma unroll
  for (int a = 0; a < TW; ++a) {
    float sacc = 0.f;
#pragma unroll
    for (int j = 0; j < NJ; ++j) sacc += (j * 32 + lane < E && t0 + a < T) ? expf(v[a][j] - mx[a]) : 0.f;
    sum[a] = sacc; wsum[a] = 0.f; my_w[a] = 0.f; my_id[a] = 0;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int a = 0; a < TW; ++a) sum[a] += __shfl_xor_sync(0xFFFFFFFFu, sum[a], o);
  for (int s = 0; s < topk; ++s) {
    uint32_t bk[TW];
    int be[TW];
#pragma unroll
    for (int a = 0; a < TW; ++a) {
      float bv = -INFINITY;
      int e1 = 0x7FFFFFFF;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const int e = j * 32 + lane;
        if (e < E && v[a][j] > bv) { bv = v[a][j]; e1 = e; }   // ascending e: the first maximum wins
      }
      bk[a] = (e1 == 0x7FFFFFFF) ? 0u : float_key(bv);
      be[a] = e1;
    }
    uint32_t gk[TW];
#pragma unroll
    for (int a = 0; a < TW; ++a) gk[a] = __reduce_max_sync(0xFFFFFFFFu, bk[a]);
#pragma unroll
    for (int a = 0; a < TW; ++a)
      be[a] = (int)__reduce_min_sync(0xFFFFFFFFu, (unsigned)((bk[a] == gk[a]) ? be[a] : 0x7FFFFFFF));
#pragma unroll
    for (int a = 0; a < TW; ++a) {
      // the winner's logit: recover from the key
      const uint32_t kb = gk[a];
      const float bv = __uint_as_float((kb & 0x80000000u) ? (kb & 0x7FFFFFFFu) : ~kb);
      const float w = expf(bv - mx[a]) / sum[a];
      wsum[a] += w;
      if (lane == s) { my_w[a] = w; my_id[a] = be[a]; }
#pragma unroll
      for (int j = 0; j < NJ; ++j)
        if (j * 32 + lane == be[a]) v[a][j] = -INFINITY;       // remove the winner
    }
  }
#pragma unroll
  for (int a = 0; a < TW; ++a) {
    const int t = t0 + a;
    if (t < T && lane < topk) {
      const float w = renormalize ? my_w[a] / wsum[a] : my_w[a];
      ids[(size_t)t * topk + lane] = my_id[a];
      wts[(size_t)t * topk + lane] = w;
      if (ids_out) ids_out[(size_t)t * topk + lane] = my_id[a];
      if (wts_out) wts_out[(size_t)t * topk + lane] = w;
      if (my_id[a] >= e_lo && my_id[a] < e_hi) atomicAdd(&hist[my_id[a]], 1);   // only this call's experts get rows
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < E; i += blockDim.x) {
    chunk_counts[(size_t)i * gridDim.x + blockIdx.x] = hist[i];
    if (hist[i]) atomicAdd(expert_total + i, hist[i]);          // integer sums: order does not matter
  }
}

template __global__ void route_kernel_t<1>(const float*, int, int, int, int, int32_t*, float*, int32_t*, int32_t*, int32_t*, float*, int, int);
template __global__ void route_kernel_t<2>(const float*, int, int, int, int, int32_t*, float*, int32_t*, int32_t*, int32_t*, float*, int, int);
template __global__ void route_kernel_t<4>(const float*, int, int, int, int, int32_t*, float*, int32_t*, int32_t*, int32_t*, float*, int, int);
template __global__ void route_kernel_t<8>(const float*, int, int, int, int, int32_t*, float*, int32_t*, int32_t*, int32_t*, float*, int, int);

// One CTA per expert, 256 threads.  From the experts' totals: the exclusive scan over experts of
// counts (offsets) and of 128-row tile counts (tile_prefix; every expert gets a multiple of
// `tile_group` tiles, so that a CTA pair never straddles experts); for its own expert the
// exclusive prefix of the counts over chunks (chunk_base) and the tile -> (expert, valid rows)
// map; the last expert's CTA also writes the header.  E <= 256.
__global__ void __launch_bounds__(256)
scan_kernel(int E, int n_chunks, int tile_group, const int32_t* __restrict__ chunk_counts,
            const int32_t* __restrict__ expert_total, int32_t* __restrict__ chunk_base, int32_t* __restrict__ offsets,
            int32_t* __restrict__ tile_prefix, int32_t* __restrict__ tile_expert, int32_t* __restrict__ tile_rows,
            int32_t* __restrict__ header, int32_t* __restrict__ offsets_out) {
  pdl_sync();
  __shared__ int wsum[2][8];
  __shared__ int carry;
  const int e = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // (1) offsets and tile prefix of this expert: block-wide sums over the experts below it
  const int cnt = threadIdx.x < E ? expert_total[threadIdx.x] : 0;
  const int tiles = ((cnt + 128 * tile_group - 1) / (128 * tile_group)) * tile_group;
  int a_lo = threadIdx.x < e ? cnt : 0, t_lo = threadIdx.x < e ? tiles : 0;
  int a_all = cnt, t_all = tiles;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a_lo += __shfl_xor_sync(0xFFFFFFFFu, a_lo, o);
    t_lo += __shfl_xor_sync(0xFFFFFFFFu, t_lo, o);
    a_all += __shfl_xor_sync(0xFFFFFFFFu, a_all, o);
    t_all += __shfl_xor_sync(0xFFFFFFFFu, t_all, o);
  }
  __shared__ int red[4][8];
  if (lane == 0) { red[0][warp] = a_lo; red[1][warp] = t_lo; red[2][warp] = a_all; red[3][warp] = t_all; }
  __syncthreads();
  int off_e = 0, tpre_e = 0, a_tot = 0, t_tot = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w) { off_e += red[0][w]; tpre_e += red[1][w]; a_tot += red[2][w]; t_tot += red[3][w]; }
  const int my_cnt = expert_total[e];
  const int my_tiles = ((my_cnt + 128 * tile_group - 1) / (128 * tile_group)) * tile_group;
  if (threadIdx.x == 0) {
    offsets[e] = off_e;
    tile_prefix[e] = tpre_e;
    if (offsets_out) offsets_out[e] = off_e;
    if (e == E - 1) {
      offsets[E] = a_tot;
      tile_prefix[E] = t_tot;
      if (offsets_out) offsets_out[E] = a_tot;
      header[kHdrMTiles] = t_tot;
      header[kHdrPaddedRows] = t_tot * 128;
      header[kHdrAssignments] = a_tot;
    }
  }
  for (int m = threadIdx.x; m < my_tiles; m += blockDim.x) {
    tile_expert[tpre_e + m] = e;
    tile_rows[tpre_e + m] = max(0, min(128, my_cnt - m * 128));
  }
  // (2) exclusive prefix of this expert's counts over the chunks, 256 chunks per pass
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int c0 = 0; c0 < n_chunks; c0 += 256) {
    const int c = c0 + threadIdx.x;
    const int v = c < n_chunks ? chunk_counts[(size_t)e * n_chunks + c] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += n;
    }
    const int p = (c0 >> 8) & 1;
    if (lane == 31) wsum[p][warp] = incl;
    __syncthreads();
    int before = carry;
#pragma unroll
    for (int w = 0; w < 8; ++w) before += w < warp ? wsum[p][w] : 0;
    if (c < n_chunks) chunk_base[(size_t)e * n_chunks + c] = before + incl - v;
    __syncthreads();
    if (threadIdx.x == 255) carry = before + incl;
    __syncthreads();
  }
}

// One CTA (4 warps) per routing chunk.  The chunk's assignments in (token, slot) order are split
// into four consecutive segments, one per warp; a warp first counts its segment per expert
// (lanes holding the same expert find each other with match_any), then every assignment's row
// inside its expert is chunk_base + (counts of the earlier warps) + (its rank inside the warp's
// walk), so every expert hands out consecutive rows in (token, slot) order.
__global__ void __launch_bounds__(128)
permute_kernel(int T, int E, int topk, int n_chunks, const int32_t* __restrict__ ids, const float* __restrict__ wts,
               const int32_t* __restrict__ chunk_base, const int32_t* __restrict__ offsets,
               const int32_t* __restrict__ tile_prefix, int32_t* __restrict__ perm, int32_t* __restrict__ pos_pad,
               int32_t* __restrict__ row_token, float* __restrict__ row_weight, int32_t* __restrict__ perm_out,
               int e_lo, int e_hi) {
  pdl_sync();
  __shared__ int run[4][kMaxExperts];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = blockIdx.x;
  const int t0 = chunk * kRouteTokensPerCta;
  const int n = min(kRouteTokensPerCta, T - t0) * topk;
  const int seg = (((n + 3) / 4) + 31) & ~31;               // assignments per warp, a multiple of 32
  const int i_begin = warp * seg, i_end = min(n, i_begin + seg);
  for (int e = lane; e < E; e += 32) run[warp][e] = 0;
  __syncwarp();
  // pass 1: this warp's count per expert
  for (int i0 = i_begin; i0 < i_end; i0 += 32) {
    const int i = i0 + lane;
    int e = i < i_end ? ids[t0 * topk + i] : -1;
    const bool active = e >= e_lo && e < e_hi;              // an assignment to an expert of this call
    if (!active) e = 0x40000000 + lane;
    const unsigned same = __match_any_sync(0xFFFFFFFFu, e);
    if (active && (same & ((1u << lane) - 1u)) == 0) run[warp][e] += __popc(same);
    __syncwarp();
  }
  __syncthreads();
  // starting row of each warp inside every expert: chunk base + the earlier warps' counts
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int b = chunk_base[(size_t)e * n_chunks + chunk];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int c = run[w][e];
      run[w][e] = b;
      b += c;
    }
  }
  __syncthreads();
  // pass 2: hand out the rows
  for (int i0 = i_begin; i0 < i_end; i0 += 32) {
    const int i = i0 + lane;
    const int flat = t0 * topk + i;
    int e = i < i_end ? ids[flat] : -1;
    const bool active = e >= e_lo && e < e_hi;
    if (i < i_end && !active) pos_pad[flat] = -1;           // another call's expert (expert-sharded execution)
    if (!active) e = 0x40000000 + lane;
    const unsigned same = __match_any_sync(0xFFFFFFFFu, e);
    const int rank = __popc(same & ((1u << lane) - 1u));
    int base = 0;
    if (active) base = run[warp][e];
    __syncwarp();
    if (active && rank == 0) run[warp][e] = base + __popc(same);
    __syncwarp();
    if (active) {
      const int r = base + rank;
      const int row = offsets[e] + r;
      perm[row] = flat;
      if (perm_out) perm_out[row] = flat;
      const int p = tile_prefix[e] * 128 + r;
      pos_pad[flat] = p;
      row_token[p] = flat / topk;
      row_weight[p] = wts[flat];
    }
  }
}

// Dense mode: identity dispatch of T rows to a single "expert".
__global__ void __launch_bounds__(256)
dense_dispatch_kernel(int T, int tile_group, int32_t* __restrict__ pos_pad, int32_t* __restrict__ row_token,
                      float* __restrict__ row_weight, int32_t* __restrict__ tile_expert,
                      int32_t* __restrict__ tile_rows, int32_t* __restrict__ header) {
  pdl_sync();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int m_tiles = ((T + 128 * tile_group - 1) / (128 * tile_group)) * tile_group;
  if (i < T) { pos_pad[i] = i; row_token[i] = i; row_weight[i] = 1.f; }
  if (i < m_tiles) { tile_expert[i] = 0; tile_rows[i] = max(0, min(128, T - i * 128)); }
  if (i == 0) { header[kHdrMTiles] = m_tiles; header[kHdrPaddedRows] = m_tiles * 128; header[kHdrAssignments] = T; }
}

}  // namespace quads
