// Top-k routing, per-expert histogram, exclusive scan and the stable dispatch
// permutation.  Integer outputs are deterministic: assignments (token, slot)
// end up sorted by (expert, token, slot).
#include "kernels.cuh"

namespace quads {

// One warp per token.  E <= 256.  Top-k by logit, ties to the lower expert id,
// slots in descending-logit order; weights = softmax over all experts at the
// chosen ones, optionally renormalised.  Each CTA (kRouteTokensPerCta tokens)
// also writes its per-expert assignment counts: chunk_counts[cta][E].
__global__ void __launch_bounds__(256)
route_kernel(const float* __restrict__ logits, int T, int E, int topk, int renormalize,
             int32_t* __restrict__ ids, float* __restrict__ wts, int32_t* __restrict__ chunk_counts,
             int32_t* __restrict__ ids_out, float* __restrict__ wts_out) {
  __shared__ int hist[kMaxExperts];
  for (int i = threadIdx.x; i < E; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t0 = blockIdx.x * kRouteTokensPerCta;
  for (int tt = warp; tt < kRouteTokensPerCta; tt += (int)(blockDim.x >> 5)) {
    const int t = t0 + tt;
    if (t >= T) break;
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int e = j * 32 + lane;
      v[j] = e < E ? logits[(size_t)t * E + e] : -INFINITY;
    }
    // softmax denominator over all experts
    float mx = v[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) mx = fmaxf(mx, v[j]);
    mx = warp_max(mx);
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) sum += (j * 32 + lane < E) ? expf(v[j] - mx) : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    float my_w = 0.f;      // lane s keeps slot s
    int my_id = -1;
    float wsum = 0.f;
    for (int s = 0; s < topk; ++s) {
      float bv = -INFINITY;
      int be = 0x7FFFFFFF;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int e = j * 32 + lane;
        if (e < E && (v[j] > bv)) { bv = v[j]; be = e; }    // ascending e within a lane: first max wins
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
        const int oe = __shfl_xor_sync(0xFFFFFFFFu, be, o);
        if (ov > bv || (ov == bv && oe < be)) { bv = ov; be = oe; }
      }
      const float w = expf(bv - mx) / sum;
      wsum += w;
      if (lane == s) { my_w = w; my_id = be; }
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (j * 32 + lane == be) v[j] = -INFINITY;         // remove the winner
    }
    if (lane < topk) {
      if (renormalize) my_w = my_w / wsum;
      ids[(size_t)t * topk + lane] = my_id;
      wts[(size_t)t * topk + lane] = my_w;
      if (ids_out) ids_out[(size_t)t * topk + lane] = my_id;
      if (wts_out) wts_out[(size_t)t * topk + lane] = my_w;
      atomicAdd(&hist[my_id], 1);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < E; i += blockDim.x) chunk_counts[(size_t)blockIdx.x * E + i] = hist[i];
}

// One CTA of 1024 threads.  A warp per expert (round robin): exclusive prefix of
// the expert's counts over chunks and its total; then the exclusive scan over
// experts of counts (offsets) and of 128-row tile counts (tile_prefix), the
// tile -> (expert, valid rows) map, and the header.
__global__ void __launch_bounds__(1024)
scan_kernel(int E, int n_chunks, const int32_t* __restrict__ chunk_counts, int32_t* __restrict__ chunk_base,
            int32_t* __restrict__ offsets, int32_t* __restrict__ tile_prefix, int32_t* __restrict__ tile_expert,
            int32_t* __restrict__ tile_rows, int32_t* __restrict__ header, int32_t* __restrict__ offsets_out) {
  __shared__ int cnt[kMaxExperts];
  __shared__ int off[kMaxExperts + 1];
  __shared__ int tpre[kMaxExperts + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int e = warp; e < E; e += n_warps) {
    int run = 0;
    for (int c0 = 0; c0 < n_chunks; c0 += 32) {
      const int c = c0 + lane;
      const int v = c < n_chunks ? chunk_counts[(size_t)c * E + e] : 0;
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += n;
      }
      if (c < n_chunks) chunk_base[(size_t)c * E + e] = run + incl - v;
      run += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (lane == 0) cnt[e] = run;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int a = 0, t = 0;
    for (int i = 0; i < E; ++i) {
      off[i] = a; tpre[i] = t;
      a += cnt[i];
      t += (cnt[i] + 127) >> 7;
    }
    off[E] = a; tpre[E] = t;
    header[kHdrMTiles] = t;
    header[kHdrPaddedRows] = t * 128;
    header[kHdrAssignments] = a;
  }
  __syncthreads();
  for (int i = threadIdx.x; i <= E; i += blockDim.x) {
    offsets[i] = off[i];
    tile_prefix[i] = tpre[i];
    if (offsets_out) offsets_out[i] = off[i];
  }
  for (int e = warp; e < E; e += n_warps) {
    const int n_t = tpre[e + 1] - tpre[e];
    for (int m = lane; m < n_t; m += 32) {
      tile_expert[tpre[e] + m] = e;
      tile_rows[tpre[e] + m] = min(128, cnt[e] - m * 128);
    }
  }
}

// One warp per routing chunk: walk the chunk's assignments in (token, slot)
// order, 32 at a time; lanes holding the same expert rank themselves with
// match_any, so every expert hands out consecutive rows in that order.
__global__ void __launch_bounds__(128)
permute_kernel(int T, int E, int topk, int n_chunks, const int32_t* __restrict__ ids, const float* __restrict__ wts,
               const int32_t* __restrict__ chunk_base, const int32_t* __restrict__ offsets,
               const int32_t* __restrict__ tile_prefix, int32_t* __restrict__ perm, int32_t* __restrict__ pos_pad,
               int32_t* __restrict__ row_token, float* __restrict__ row_weight, int32_t* __restrict__ perm_out) {
  __shared__ int run[4][kMaxExperts];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = blockIdx.x * 4 + warp;
  if (chunk >= n_chunks) return;
  for (int e = lane; e < E; e += 32) run[warp][e] = chunk_base[(size_t)chunk * E + e];
  __syncwarp();
  const int t0 = chunk * kRouteTokensPerCta;
  const int n = min(kRouteTokensPerCta, T - t0) * topk;
  for (int i0 = 0; i0 < n; i0 += 32) {
    const int i = i0 + lane;
    const bool active = i < n;
    const int flat = t0 * topk + i;
    const int e = active ? ids[flat] : (0x40000000 + lane);
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
dense_dispatch_kernel(int T, int32_t* __restrict__ pos_pad, int32_t* __restrict__ row_token,
                      float* __restrict__ row_weight, int32_t* __restrict__ tile_expert,
                      int32_t* __restrict__ tile_rows, int32_t* __restrict__ header) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int m_tiles = (T + 127) >> 7;
  if (i < T) { pos_pad[i] = i; row_token[i] = i; row_weight[i] = 1.f; }
  if (i < m_tiles) { tile_expert[i] = 0; tile_rows[i] = min(128, T - i * 128); }
  if (i == 0) { header[kHdrMTiles] = m_tiles; header[kHdrPaddedRows] = m_tiles * 128; header[kHdrAssignments] = T; }
}

}  // namespace quads
