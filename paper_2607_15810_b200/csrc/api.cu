// C ABI entry points: argument checks, workspace carving, TMA descriptors and
// the launch sequence of each public call.
#include <algorithm>
#include <cstdlib>
#include <atomic>
#include <mutex>

#include "kernels.cuh"

namespace quads {

thread_local int g_launch_count = 0;

bool pdl_enabled() {
  static const bool on = [] { const char* e = getenv("QUADS_NO_PDL"); return !(e && e[0] == '1'); }();
  return on;
}

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct DeviceInfo {
  int sm_count = 0;
  int cc_major = 0;
  bool ok = false;
};

quads_status device_info(DeviceInfo* out) {
  static std::mutex mu;
  static DeviceInfo cache[64];
  int dev = 0;
  QUADS_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QUADS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (!cache[dev].ok) {
    QUADS_CUDA_OK(cudaDeviceGetAttribute(&cache[dev].sm_count, cudaDevAttrMultiProcessorCount, dev));
    QUADS_CUDA_OK(cudaDeviceGetAttribute(&cache[dev].cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    cache[dev].ok = true;
  }
  *out = cache[dev];
  return cache[dev].cc_major == 10 ? QUADS_OK : QUADS_ERR_ARCH;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  });
  return fn;
}

// 2D map over packed FP4 codes viewed as bytes: [rows, row_bytes], box 128 bytes x
// box_rows rows, 128-byte swizzle, zero fill outside.
quads_status make_codes_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t row_bytes,
                            uint32_t box_rows = 128) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return QUADS_ERR_CUDA;
  if (rows == 0) rows = 1;
  cuuint64_t dims[2] = {row_bytes, rows};
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {(cuuint32_t)kGemmStageKBytes, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE,
                  kGemmStageKBytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QUADS_OK : QUADS_ERR_CUDA;
}

// 2D map over tiled scale factors viewed as [atoms, 128 x u32] (512-byte atoms), box =
// kGemmKSteps atoms, no swizzle; used by the CTA-pair GEMM only.
quads_status make_sf_map(CUtensorMap* map, const void* base, uint64_t atoms) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return QUADS_ERR_CUDA;
  if (atoms == 0) atoms = 1;
  cuuint64_t dims[2] = {128, atoms};
  cuuint64_t strides[1] = {512};
  cuuint32_t box[2] = {128, (cuuint32_t)kGemmKSteps};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QUADS_OK : QUADS_ERR_CUDA;
}

// 2D map over a bf16 matrix [rows, K] (K contiguous): box 64 elements (128 bytes) x 128 rows,
// 128-byte swizzle, zero fill outside.
quads_status make_bf16_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t K) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return QUADS_ERR_CUDA;
  if (rows == 0) rows = 1;
  cuuint64_t dims[2] = {K, rows};
  cuuint64_t strides[1] = {K * 2};
  cuuint32_t box[2] = {64, 128};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QUADS_OK : QUADS_ERR_CUDA;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// ------------------------------------------------------------------ workspace
struct MoeLayout {
  size_t header, amax, counters13, keys13, keys2, expert_total, ids, wts, chunk_counts, chunk_base, offsets, tile_prefix, tile_expert, tile_rows;
  size_t perm, pos_pad, row_token, row_weight;
  size_t partials13, scores13, sel13, mask13, xq_tok, xsf_tok, rq_tok, rsf_tok, xq_pad, xsf, rq_pad, rsf;
  size_t hq_pad, hsf, r2q_pad, r2sf, sel2, mask2, y_pad, dec;
  size_t total;
  int n_chunks, m_tiles_max, stats_ctas, rows_per_cta;
};

MoeLayout moe_layout(int T, int H, int I, int E, int topk, int N) {
  MoeLayout L{};
  const bool dense = (I == 0);
  const int64_t A = dense ? T : (int64_t)T * topk;
  const int Ee = dense ? 1 : E;
  L.n_chunks = (T + kRouteTokensPerCta - 1) / kRouteTokensPerCta;
  L.m_tiles_max = ((int)(A / 256) + Ee) * 2;      // enough for either tile grouping (1 or 2)
  L.stats_ctas = T < 592 * 4 ? (T + 3) / 4 : 592;
  if (L.stats_ctas < 1) L.stats_ctas = 1;
  L.rows_per_cta = (T + L.stats_ctas - 1) / L.stats_ctas;
  if (L.rows_per_cta < 1) L.rows_per_cta = 1;
  L.stats_ctas = (T + L.rows_per_cta - 1) / L.rows_per_cta;
  if (L.stats_ctas < 1) L.stats_ctas = 1;
  const size_t pad_rows = (size_t)L.m_tiles_max * 128;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
  L.header = take(kHdrWords * 4);
  L.amax = take((size_t)kAmaxPartsMax * 4);    // the amax word; also the quantizer's scratch in the one-sided modes
  L.counters13 = take((size_t)((H + 31) / 32) * 4);
  L.keys13 = take((size_t)H * 8);                  // integer column scores of site 13 (small batches), zeroed with the header
  L.keys2 = take((size_t)I * 8);                   // zeroed with the header: the first projection's epilogue adds to it
  L.expert_total = take((size_t)Ee * 4);           // zeroed with the header: the routing kernel adds to it
  L.ids = take((size_t)A * 4);
  L.wts = take((size_t)A * 4);
  L.chunk_counts = take((size_t)L.n_chunks * Ee * 4);
  L.chunk_base = take((size_t)L.n_chunks * Ee * 4);
  L.offsets = take((size_t)(Ee + 1) * 4);
  L.tile_prefix = take((size_t)(Ee + 1) * 4);
  L.tile_expert = take((size_t)L.m_tiles_max * 4);
  L.tile_rows = take((size_t)L.m_tiles_max * 4);
  L.perm = take((size_t)A * 4);
  L.pos_pad = take((size_t)A * 4);
  L.row_token = take(pad_rows * 4);
  L.row_weight = take(pad_rows * 4);
  L.partials13 = take((size_t)L.stats_ctas * H * 4);
  L.scores13 = take((size_t)H * 8 * kScoreSlices);
  L.sel13 = take((size_t)H * 4);
  L.mask13 = take((size_t)H);
  L.xq_tok = take((size_t)T * (H / 2));
  L.xsf_tok = take((size_t)T * (H / 16));
  L.rq_tok = take((size_t)T * (H / 2));
  L.rsf_tok = take((size_t)T * (H / 16));
  L.xq_pad = take(pad_rows * (H / 2));
  L.xsf = take((size_t)L.m_tiles_max * (H / 64) * 512);
  L.rq_pad = take(pad_rows * (H / 2));
  L.rsf = take((size_t)L.m_tiles_max * (H / 64) * 512);
  if (!dense) {
    L.hq_pad = take(pad_rows * (I / 2));
    L.hsf = take((size_t)L.m_tiles_max * (I / 64) * 512);
    L.r2q_pad = take(pad_rows * (I / 2));
    L.r2sf = take((size_t)L.m_tiles_max * (I / 64) * 512);
    L.sel2 = take((size_t)I * 4);
    L.mask2 = take((size_t)I);
    L.y_pad = take(pad_rows * (size_t)H * 2);
  }
  if (dense) L.dec = take((size_t)std::max(T, N) * (size_t)H * 2);   // decoded bf16 operand of the one-sided modes
  L.total = o;
  return L;
}

// Optional per-kernel timing of the two grouped GEMMs (off by default).
struct GemmTimers {
  bool enabled = false;
  bool created = false;
  bool valid = false;
  cudaEvent_t ev[4];
};
GemmTimers g_timers;

// Optional stage trace of one MoE call: an event after every stage (off by default).
struct StageTrace {
  bool enabled = false;
  int n = 0;
  cudaEvent_t ev[40];
  const char* name[40];
  bool created = false;
};
StageTrace g_trace;
inline void trace_mark(const char* name, cudaStream_t st) {
  if (!g_trace.enabled || g_trace.n >= 40) return;
  g_trace.name[g_trace.n] = name;
  cudaEventRecord(g_trace.ev[g_trace.n], st);
  ++g_trace.n;
}

// Side stream on which the routing chain (route -> scan -> permute) runs next to the
// activation chain (amax -> quantize -> select); both are joined before the dispatch copy.
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, mid = nullptr, tables = nullptr, join = nullptr;
  bool ok = false;
};
std::mutex g_side_mu;
// Call with g_side_mu held (the per-device objects are created on first use).
SideStream* side_stream() {
  static SideStream per_device[64];
  static const bool disabled = [] { const char* e = getenv("QUADS_NO_OVERLAP"); return e && e[0] == '1'; }();
  if (disabled) return nullptr;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  SideStream& s = per_device[dev];
  if (!s.ok) {
    if (cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s.mid, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s.tables, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    s.ok = true;
  }
  return &s;
}

// Joins the side stream back into the caller's stream when the scope is left before the regular
// join (an error return between fork and join): without it the side stream would stay forked
// and, under stream capture, the captured graph would be left with an unjoined branch.
struct SideJoinGuard {
  SideStream* side = nullptr;
  cudaStream_t main = nullptr;
  bool joined = true;
  void arm(SideStream* s, cudaStream_t st) { side = s; main = st; joined = false; }
  void join() {
    if (joined || !side) return;
    joined = true;
    if (cudaEventRecord(side->join, side->stream) == cudaSuccess) cudaStreamWaitEvent(main, side->join, 0);
  }
  ~SideJoinGuard() { join(); }
};

// GEMM variant of a call.  1: single-CTA tiles of 128 x 256; 2: CTA pairs computing 256 x 256
// tiles with cta_group::2 MMAs: about 7 % (first projection) / 5 % (second) faster per tile, but
// every expert's rows are then padded to a multiple of 256, i.e. half a tile more per expert on
// average than padding to 128.  That pays from roughly 1000 rows per expert, which is the rule used
// here; QUADS_GEMM_CTA_GROUP=1|2 forces a variant.  (When the experts' tile counts happen to be
// even -- the skewed prefill benchmark: 410 rows = 4 tiles for most experts -- pairs already win at
// 512 rows per expert: 477 vs 488 us per layer.)
int gemm_cta_group_for(int64_t rows, int experts) {
  static const int forced = [] {
    const char* e = getenv("QUADS_GEMM_CTA_GROUP");
    return (e && (e[0] == '1' || e[0] == '2')) ? e[0] - '0' : 0;
  }();
  if (forced) return forced;
  return rows >= (int64_t)1024 * (experts > 0 ? experts : 1) ? 2 : 1;
}

// Ranking of C order-preserving 64-bit score keys: mask of the n_sel largest (+ their ascending list).
quads_status run_rank(const unsigned long long* keys, int C, int n_sel, uint8_t* mask, int32_t* sel_export,
                      cudaStream_t st) {
  QUADS_CUDA_OK(set_max_dynamic_smem<rank_select_kernel>(128 * 1024));
  QUADS_CUDA_OK(launch_kernel(rank_select_kernel, dim3((C + 15) / 16), dim3(256), (size_t)((size_t)C * 8), st, keys, C, n_sel, mask));
  if (sel_export) {
    QUADS_CUDA_OK(launch_kernel(sel_list_kernel, dim3(1), dim3(1024), (size_t)(0), st, mask, C, sel_export));
  }
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}

quads_status run_select(const float* partials, const int* n_part_ptr, int n_part_mul, int n_part_fixed, int C,
                        int n_sel, double* slice_sums, unsigned int* counters, unsigned long long* keys,
                        uint8_t* mask, int32_t* sel_export, cudaStream_t st) {
  QUADS_CUDA_OK(launch_kernel(score_reduce_kernel, dim3((C + 31) / 32, kScoreSlices), dim3(256), (size_t)(0), st, partials, n_part_ptr, n_part_mul, n_part_fixed, C, slice_sums, counters, keys));
  return run_rank(keys, C, n_sel, mask, sel_export, st);
}

}  // namespace
}  // namespace quads

using namespace quads;

extern "C" {

const char* quads_status_string(quads_status s) {
  switch (s) {
    case QUADS_OK: return "QUADS_OK";
    case QUADS_ERR_NULL: return "QUADS_ERR_NULL: a required pointer is NULL";
    case QUADS_ERR_SHAPE: return "QUADS_ERR_SHAPE: a size breaks a divisibility or range rule";
    case QUADS_ERR_WORKSPACE: return "QUADS_ERR_WORKSPACE: workspace missing, misaligned or too small";
    case QUADS_ERR_ARCH: return "QUADS_ERR_ARCH: the current device is not sm_100";
    case QUADS_ERR_CUDA: return "QUADS_ERR_CUDA: a CUDA runtime or driver call failed";
    case QUADS_ERR_TIMEOUT: return "QUADS_ERR_TIMEOUT: a bounded device-side wait gave up";
    case QUADS_ERR_LIMIT: return "QUADS_ERR_LIMIT: the size exceeds the fixed capacity of an allocation-free entry point";
    default: return "QUADS: unknown status";
  }
}

size_t quads_sf_tiled_bytes(int64_t rows, int64_t K) {
  if (rows < 0 || K < 0) return 0;
  return (size_t)((rows + 127) / 128) * (size_t)((K + 63) / 64) * 512u;
}

size_t quads_quantize_workspace_bytes(void) { return (size_t)kAmaxPartsMax * 4; }
size_t quads_fake_quant_workspace_bytes(int64_t n_tensors) {
  return std::max(align_up((size_t)(n_tensors > 0 ? n_tensors : 1) * 8, 256), (size_t)kAmaxPartsMax * 4);
}
int32_t quads_last_launch_count(void) { return g_launch_count; }

// Bound of the per-tensor arrival wait of fused_quantize_kernel in SM clock cycles (about two
// seconds), and a test-only surplus of expected arrivals (see quads_debug_set_quantize_wait).
static std::atomic<long long> g_quant_wait_cycles{4000000000ll};
static std::atomic<int> g_quant_extra_arrivals{0};

void quads_debug_set_quantize_wait(int64_t clock_cycles, int32_t extra_arrivals) {
  g_quant_wait_cycles.store(clock_cycles > 0 ? (long long)clock_cycles : 4000000000ll);
  g_quant_extra_arrivals.store(extra_arrivals > 0 ? (int)extra_arrivals : 0);
}

static quads_status quantize_common(const void* x, int64_t n_tensors, int64_t rows, int64_t K, int64_t ld,
                                    int64_t tensor_stride, const float* gs_in, void* fq, uint8_t* q, uint8_t* sf,
                                    float* gs_out, int sf_layout, void* workspace, size_t workspace_bytes,
                                    cudaStream_t st) {
  g_launch_count = 0;
  if (rows < 0 || n_tensors < 0 || K <= 0 || (K % 16) != 0 || ld < K || (ld % 16) != 0) return QUADS_ERR_SHAPE;
  if (sf_layout != QUADS_SF_LINEAR && sf_layout != QUADS_SF_TILED) return QUADS_ERR_SHAPE;
  if (rows * (K / 16) > (int64_t)0x7FFFFFFF || n_tensors > 65535) return QUADS_ERR_SHAPE;   // block indices are 31-bit
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < quads_fake_quant_workspace_bytes(n_tensors))
    return QUADS_ERR_WORKSPACE;
  if (n_tensors > 0 && rows > 0 && !x) return QUADS_ERR_NULL;
  if (!aligned(x, 32) || !aligned(q, 8) || !aligned(fq, 32) || !aligned(sf, 4)) return QUADS_ERR_SHAPE;
  DeviceInfo di;
  quads_status s = device_info(&di);
  if (s != QUADS_OK) return s;
  if (n_tensors == 0) return QUADS_OK;
  // scratch: one amax word and one arrival counter per tensor, zero on entry
  uint32_t* amax_bits = static_cast<uint32_t*>(workspace);
  uint32_t* counters = amax_bits + n_tensors;
  const uint16_t* xp = static_cast<const uint16_t*>(x);
  // One tensor, scale to be derived: two ordinary launches instead of a cooperative one.  The first
  // leaves one partial maximum per CTA in the workspace (no initialisation, no atomics) and asks L2 to
  // keep the tensor; the second, launched as a programmatic dependent, reduces the partials and
  // quantizes out of L2.  The kernel boundary is the only synchronisation.
  const bool two_pass = !gs_in && n_tensors == 1 && rows > 0 && !getenv("QUADS_QUANT_COOPERATIVE");
  if (!gs_in && !two_pass) QUADS_CUDA_OK(cudaMemsetAsync(amax_bits, 0, (size_t)n_tensors * 8, st));
  int n_parts = 0;
  if (two_pass) {
    const int64_t chunks = rows * (K / 8);
    n_parts = (int)std::max<int64_t>(1, std::min<int64_t>((chunks + 2047) / 2048, std::min(di.sm_count * 8, kAmaxPartsMax)));
    QUADS_CUDA_OK(launch_kernel(amax_partial_kernel, dim3(n_parts), dim3(256), (size_t)0, st, xp, rows, K, ld, amax_bits));
  }
  uint16_t* fqp = static_cast<uint16_t*>(fq);
  int nt = (int)n_tensors;
  int tiled = sf_layout == QUADS_SF_TILED;
  int64_t sf_stride = tiled ? (int64_t)quads_sf_tiled_bytes(rows, K) : rows * (K / 16);
  const int64_t nblk = rows * (K / 16);
  // A batch of tensors with no scales given: the ring kernel (pipelines of bulk copies, the amax
  // stream running ahead of the quantization by a tensor or two, which must stay in L2).
  if (!gs_in && ld == K && n_tensors >= 2 && nblk > 0 && !getenv("QUADS_NO_RING_QUANT")) {
    // small tensors are dealt to 2 or 4 sets of CTAs (tensor t to set t mod split), so that a CTA's
    // share is a few 14 KB chunks; the grid is a multiple of the split
    int split = 1;
    const int64_t chunk_blocks = kRingChunkBytes / 32;
    while (split < 4 && n_tensors >= 2 * split && di.sm_count % (2 * split) == 0 &&
           (nblk + di.sm_count / split - 1) / (di.sm_count / split) < 3 * chunk_blocks)
      split *= 2;
    if (const char* e = getenv("QUADS_RING_SPLIT")) {
      const int v = atoi(e);
      if ((v == 1 || v == 2 || v == 4) && di.sm_count % v == 0) split = v;
    }
    const int ctas_per_tensor = di.sm_count / split;
    const int64_t per64 = ((nblk + ctas_per_tensor - 1) / ctas_per_tensor + 3) / 4 * 4;   // blocks per CTA, 128-byte granules
    const int64_t tensor_bytes = nblk * 32;
    if (per64 < (int64_t)1 << 24 && tensor_bytes * 2 <= (int64_t)64 << 20) {
      // A's lead over Q: a group's chunks of one tensor (so Q never catches up with A inside a
      // tensor) plus a few for the time it takes a maximum to travel between the CTAs
      const int chunks_per_tensor = (int)((per64 * 32 + 4 * kRingChunkBytes - 1) / (4 * kRingChunkBytes));
      int lead = chunks_per_tensor + (tensor_bytes > ((int64_t)16 << 20) ? 2 : 3);   // large tensors: mind the L2 footprint
      if (const char* e = getenv("QUADS_RING_LEAD")) lead = chunks_per_tensor + std::max(0, atoi(e));
      int per = (int)per64;
      uint32_t k16 = (uint32_t)(K / 16);
      int kt_count = (int)((K + 63) / 64);
      int64_t stride = tensor_stride;
      int64_t nb = nblk;
      QUADS_CUDA_OK(set_max_dynamic_smem<fake_quant_ring_kernel>(kRingSmemBytes));
      void* rargs[] = {&xp, &nb, &stride, &nt, &amax_bits, &per, &lead, &split, &q, &sf, &fqp,
                       &gs_out, &tiled, &sf_stride, &k16, &kt_count};
      QUADS_CUDA_OK(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(fake_quant_ring_kernel), dim3(di.sm_count),
                                                dim3(kRingThreads), rargs, (size_t)kRingSmemBytes, st));
      note_launch();
      QUADS_CUDA_OK(cudaGetLastError());
      return QUADS_OK;
    }
  }
  static std::atomic<int> blocks_per_sm_cache{0};   // same kernel and block size on every sm_100 device
  int blocks_per_sm = blocks_per_sm_cache.load();
  if (blocks_per_sm == 0) {
    int b = 0;
    QUADS_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, fused_quantize_kernel, 256, 0));
    blocks_per_sm = b < 1 ? 1 : (b > 8 ? 8 : b);
    blocks_per_sm_cache.store(blocks_per_sm);
  }
  int max_groups = 4;
  int n_groups = n_tensors < max_groups ? (int)n_tensors : max_groups;
  int64_t want = (nblk * n_groups + 255) / 256;            // no more CTAs than there is work
  int grid = di.sm_count * blocks_per_sm;
  if (want < grid) grid = (int)want;
  if (grid < n_groups) grid = n_groups;
  long long wait_cycles = g_quant_wait_cycles.load();
  int extra_arrivals = g_quant_extra_arrivals.load();
  const uint32_t* amax_parts = two_pass ? amax_bits : nullptr;
  if (two_pass || gs_in) {
    // no CTA waits for another one: an ordinary launch
    QUADS_CUDA_OK(launch_kernel(fused_quantize_kernel, dim3(grid), dim3(256), (size_t)0, st, xp, rows, K, ld, tensor_stride, nt,
                                gs_in, amax_bits, counters, q, sf, fqp, gs_out, tiled, sf_stride, n_groups, wait_cycles,
                                extra_arrivals, amax_parts, n_parts));
  } else {
    void* args[] = {&xp, &rows, &K, &ld, &tensor_stride, &nt, &gs_in, &amax_bits, &counters, &q, &sf, &fqp,
                    &gs_out, &tiled, &sf_stride, &n_groups, &wait_cycles, &extra_arrivals, &amax_parts, &n_parts};
    QUADS_CUDA_OK(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(fused_quantize_kernel), dim3(grid), dim3(256),
                                              args, 0, st));
    note_launch();
  }
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}

quads_status quads_quantize_nvfp4(const void* x, int64_t rows, int64_t K, int64_t ld, const float* gs_in,
                                  uint8_t* q, uint8_t* sf, float* gs_out, int sf_layout, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream) {
  if (rows > 0 && (!q || !sf)) return QUADS_ERR_NULL;
  return quantize_common(x, 1, rows, K, ld, 0, gs_in, nullptr, q, sf, gs_out, sf_layout, workspace,
                         workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

quads_status quads_dequantize_nvfp4(const uint8_t* q, const uint8_t* sf, const float* gs, int64_t n_tensors,
                                    int64_t rows, int64_t K, int sf_layout, void* out, void* cuda_stream) {
  g_launch_count = 0;
  if (rows < 0 || n_tensors < 0 || K <= 0 || (K % 16) != 0) return QUADS_ERR_SHAPE;
  if (sf_layout != QUADS_SF_LINEAR && sf_layout != QUADS_SF_TILED) return QUADS_ERR_SHAPE;
  const int64_t nblk = rows * (K / 16);
  if (nblk > (int64_t)0x7FFFFFFF || n_tensors > 65535) return QUADS_ERR_SHAPE;
  if (n_tensors == 0 || rows == 0) return QUADS_OK;
  if (!q || !sf || !gs || !out) return QUADS_ERR_NULL;
  if (!aligned(q, 8) || !aligned(out, 32)) return QUADS_ERR_SHAPE;
  DeviceInfo di;
  quads_status s = device_info(&di);
  if (s != QUADS_OK) return s;
  const int tiled = sf_layout == QUADS_SF_TILED;
  const int64_t sf_stride = tiled ? (int64_t)quads_sf_tiled_bytes(rows, K) : nblk;
  const int64_t want = (nblk * n_tensors + 255) / 256;
  const int grid = (int)std::min<int64_t>(want, (int64_t)di.sm_count * 16);
  QUADS_CUDA_OK(launch_kernel(dequantize_kernel, dim3(grid), dim3(256), (size_t)0, static_cast<cudaStream_t>(cuda_stream),
                              q, sf, gs, (int)n_tensors, nblk, (uint32_t)(K / 16), (int)((K + 63) / 64), tiled, sf_stride,
                              static_cast<uint16_t*>(out)));
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}

quads_status quads_fake_quant_activations(const void* x, int64_t rows, int64_t K, int64_t ld, const float* gs_in,
                                          void* x_fq, float* gs_out, void* workspace, size_t workspace_bytes,
                                          void* cuda_stream) {
  if (rows > 0 && !x_fq) return QUADS_ERR_NULL;
  return quantize_common(x, 1, rows, K, ld, 0, gs_in, x_fq, nullptr, nullptr, gs_out, QUADS_SF_LINEAR, workspace,
                         workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

quads_status quads_fake_quant_weights(const void* w, int64_t n_tensors, int64_t N, int64_t K, void* w_fq,
                                      uint8_t* q, uint8_t* sf, float* gs, int sf_layout, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream) {
  if (!gs && n_tensors > 0) return QUADS_ERR_NULL;
  return quantize_common(w, n_tensors, N, K, K, N * K, nullptr, w_fq, q, sf, gs, sf_layout, workspace,
                         workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------
// Allocation-free fake-quant.  Its scratch (an amax word and an arrival counter per tensor) lives in
// the library image, so a caller that must not allocate device memory -- for
// instance code running under a memory pool it does not own, or inside a
// region where cudaMalloc's implicit device synchronisation is forbidden --
// needs no workspace.  In host code `g_noalloc_amax` is only a handle for the
// symbol; the device address comes from cudaGetSymbolAddress, looked up once
// per device with that device current.
// ---------------------------------------------------------------------------
static __device__ __align__(256) uint32_t g_noalloc_amax[2 * QUADS_NOALLOC_MAX_TENSORS];

static quads_status noalloc_scratch(uint32_t** out) {
  static std::mutex mu;
  static uint32_t* per_device[64] = {nullptr};
  int dev = 0;
  QUADS_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QUADS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (!per_device[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_amax) != cudaSuccess || !p) return QUADS_ERR_CUDA;
    per_device[dev] = static_cast<uint32_t*>(p);
  }
  *out = per_device[dev];
  return QUADS_OK;
}

quads_status quads_fake_quant_weights_noalloc(const void* w, int64_t n_tensors, int64_t N, int64_t K, void* w_fq,
                                              uint8_t* q, uint8_t* sf, float* gs, int sf_layout,
                                              void* cuda_stream) {
  if (n_tensors > QUADS_NOALLOC_MAX_TENSORS) return QUADS_ERR_LIMIT;
  if (!gs && n_tensors > 0) return QUADS_ERR_NULL;
  uint32_t* scratch = nullptr;
  quads_status s = noalloc_scratch(&scratch);
  if (s != QUADS_OK) return s;
  // quantize_common zeroes the words it is about to use on the stream before
  // the kernel, so the previous call's contents never leak in.
  return quantize_common(w, n_tensors, N, K, K, N * K, nullptr, w_fq, q, sf, gs, sf_layout, scratch,
                         sizeof(uint32_t) * 2 * QUADS_NOALLOC_MAX_TENSORS, static_cast<cudaStream_t>(cuda_stream));
}

// ---- diagnostics
static int score_stats_ctas(int64_t T, int* rows_per_cta) {
  int ctas = T < 592 * 4 ? (int)((T + 3) / 4) : 592;
  if (ctas < 1) ctas = 1;
  int rpc = (int)((T + ctas - 1) / ctas);
  if (rpc < 1) rpc = 1;
  ctas = (int)((T + rpc - 1) / rpc);
  *rows_per_cta = rpc;
  return ctas < 1 ? 1 : ctas;
}

size_t quads_rac_channel_scores_workspace_bytes(int64_t T, int64_t H) {
  if (T < 0 || H <= 0) return 0;
  int rpc;
  const int ctas = score_stats_ctas(T, &rpc);
  return 512 + align_up((size_t)((H + 31) / 32) * 4, 256) + align_up((size_t)ctas * H * 4, 256) +
         align_up((size_t)H * 8 * kScoreSlices, 256);
}

quads_status quads_rac_channel_scores(const void* x, int64_t T, int64_t H, const float* gs_in, double* scores,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
  g_launch_count = 0;
  if (T < 0 || T > 0x3FFFFFFF || H <= 0 || (H % 128) != 0 || H > 16384) return QUADS_ERR_SHAPE;
  if (!scores || (T > 0 && !x)) return QUADS_ERR_NULL;
  if (!aligned(x, 32) || !aligned(scores, 8)) return QUADS_ERR_SHAPE;
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < quads_rac_channel_scores_workspace_bytes(T, H))
    return QUADS_ERR_WORKSPACE;
  DeviceInfo di;
  quads_status s = device_info(&di);
  if (s != QUADS_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (T == 0) { QUADS_CUDA_OK(cudaMemsetAsync(scores, 0, (size_t)H * 8, st)); return QUADS_OK; }
  int rpc;
  const int ctas = score_stats_ctas(T, &rpc);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint32_t* amax_bits = reinterpret_cast<uint32_t*>(ws);                 // [0, 256): amax word; [256, 512): status word
  int32_t* status_word = reinterpret_cast<int32_t*>(ws + 256);
  unsigned int* counters = reinterpret_cast<unsigned int*>(ws + 512);
  const size_t n_counter_bytes = align_up((size_t)((H + 31) / 32) * 4, 256);
  float* partials = reinterpret_cast<float*>(ws + 512 + n_counter_bytes);
  double* slices = reinterpret_cast<double*>(ws + 512 + n_counter_bytes + align_up((size_t)ctas * H * 4, 256));
  QUADS_CUDA_OK(cudaMemsetAsync(ws, 0, 512 + n_counter_bytes, st));
  const uint16_t* xp = static_cast<const uint16_t*>(x);
  if (!gs_in) {
    const int64_t chunks = T * (H / 8);
    int gx = (int)std::min<int64_t>((chunks + 2047) / 2048, (int64_t)di.sm_count * 8);
    QUADS_CUDA_OK(launch_kernel(amax_kernel, dim3(gx, 1), dim3(256), (size_t)0, st, xp, T, H, H, (int64_t)0, amax_bits));
  }
  const int block = H / 16 > 256 ? 256 : (int)((H / 16 + 31) / 32 * 32);
  QUADS_CUDA_OK(launch_kernel(rac_quant_kernel, dim3(ctas), dim3(block), (size_t)0, st, xp, (int)T, (int)H, gs_in, amax_bits,
                              (unsigned int*)nullptr, status_word, (float*)nullptr, rpc, 1, partials, (uint8_t*)nullptr,
                              (uint8_t*)nullptr, (uint8_t*)nullptr, (uint8_t*)nullptr, (uint8_t*)nullptr, (uint8_t*)nullptr,
                              (unsigned long long*)nullptr, 0, 0));
  // the order-preserving 64-bit keys of non-negative scores are the scores' own bit patterns
  QUADS_CUDA_OK(launch_kernel(score_reduce_kernel, dim3((unsigned)((H + 31) / 32), kScoreSlices), dim3(256), (size_t)0, st,
                              (const float*)partials, (const int*)nullptr, 1, ctas, (int)H, slices, counters,
                              reinterpret_cast<unsigned long long*>(scores)));
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}

size_t quads_mismatch_norms_workspace_bytes(void) { return 256 + 1184 * 3 * sizeof(double); }

quads_status quads_mismatch_norms(const void* a, const void* b, int64_t n, double* out, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream) {
  g_launch_count = 0;
  if (n < 0) return QUADS_ERR_SHAPE;
  if (!out || (n > 0 && (!a || !b))) return QUADS_ERR_NULL;
  if (!aligned(a, 16) || !aligned(b, 16) || !aligned(out, 8)) return QUADS_ERR_SHAPE;
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < quads_mismatch_norms_workspace_bytes())
    return QUADS_ERR_WORKSPACE;
  DeviceInfo di;
  quads_status s = device_info(&di);
  if (s != QUADS_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  QUADS_CUDA_OK(cudaMemsetAsync(ws, 0, 256, st));
  const int64_t want = (n / 8 + 256 * 4 - 1) / (256 * 4);
  const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(want, 1184));
  QUADS_CUDA_OK(launch_kernel(mismatch_norms_kernel, dim3(grid), dim3(256), (size_t)0, st, static_cast<const uint16_t*>(a),
                              static_cast<const uint16_t*>(b), n, reinterpret_cast<double*>(ws + 256),
                              reinterpret_cast<unsigned int*>(ws), out));
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}

size_t quads_moe_workspace_bytes(int32_t T, int32_t H, int32_t I, int32_t E, int32_t topk, int32_t N) {
  if (T < 0 || H <= 0 || I < 0 || E < 1 || topk < 1) return 0;
  return moe_layout(T, H, I, E, topk, N).total;
}

quads_status quads_moe_async_status(const void* workspace, void* cuda_stream) {
  if (!workspace) return QUADS_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int32_t v = 0;
  QUADS_CUDA_OK(cudaMemcpyAsync(&v, static_cast<const int32_t*>(workspace) + kHdrStatus, 4, cudaMemcpyDeviceToHost, st));
  QUADS_CUDA_OK(cudaStreamSynchronize(st));
  return v == 0 ? QUADS_OK : (quads_status)v;
}

quads_status quads_moe_set_stage_trace(int32_t enable) {
  if (enable && !g_trace.created) {
    for (int i = 0; i < 40; ++i) QUADS_CUDA_OK(cudaEventCreate(&g_trace.ev[i]));
    g_trace.created = true;
  }
  g_trace.enabled = enable != 0;
  g_trace.n = 0;
  return QUADS_OK;
}

int32_t quads_moe_get_stage_trace(const char** names, float* ms, int32_t cap) {
  if (!names || !ms || g_trace.n < 2) return 0;
  if (cudaEventSynchronize(g_trace.ev[g_trace.n - 1]) != cudaSuccess) return 0;
  int n = 0;
  for (int i = 1; i < g_trace.n && n < cap; ++i, ++n) {
    names[n] = g_trace.name[i];
    if (cudaEventElapsedTime(&ms[n], g_trace.ev[i - 1], g_trace.ev[i]) != cudaSuccess) return n;
  }
  return n;
}

quads_status quads_moe_set_kernel_timing(int32_t enable) {
  if (enable && !g_timers.created) {
    for (int i = 0; i < 4; ++i) QUADS_CUDA_OK(cudaEventCreate(&g_timers.ev[i]));
    g_timers.created = true;
  }
  g_timers.enabled = enable != 0;
  g_timers.valid = false;
  return QUADS_OK;
}

quads_status quads_moe_last_kernel_ms(float* gemm1_ms, float* gemm2_ms) {
  if (!gemm1_ms || !gemm2_ms) return QUADS_ERR_NULL;
  if (!g_timers.valid) return QUADS_ERR_SHAPE;
  QUADS_CUDA_OK(cudaEventSynchronize(g_timers.ev[3]));
  QUADS_CUDA_OK(cudaEventElapsedTime(gemm1_ms, g_timers.ev[0], g_timers.ev[1]));
  QUADS_CUDA_OK(cudaEventElapsedTime(gemm2_ms, g_timers.ev[2], g_timers.ev[3]));
  return QUADS_OK;
}

quads_status quads_moe_w4a4_rac(const quads_moe_args* a, void* cuda_stream) {
  g_launch_count = 0;
  if (!a) return QUADS_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool dense = (a->I == 0);
  const int T = a->T, H = a->H, I = a->I;
  const int E = dense ? 1 : a->E, topk = dense ? 1 : a->topk;
  const int N1 = dense ? a->N : 2 * I;            // weight rows of the first projection
  if (T < 0 || H <= 0 || (H % 128) != 0 || I < 0 || (I % 128) != 0) return QUADS_ERR_SHAPE;
  if (dense && (a->N <= 0 || (a->N % 128) != 0)) return QUADS_ERR_SHAPE;
  if (!dense && (E < 1 || E > kMaxExperts || topk < 1 || topk > kMaxTopk || topk > E)) return QUADS_ERR_SHAPE;
  if (H > 16384 || I > 16384 || a->rac_nsel_13 < 0 || a->rac_nsel_13 > H || (!dense && (a->rac_nsel_2 < 0 || a->rac_nsel_2 > I)))
    return QUADS_ERR_SHAPE;
  if ((int64_t)T * topk > 0x3FFFFFFF) return QUADS_ERR_SHAPE;
  if (a->operand_mode != QUADS_W4A4) {
    if (!dense || a->operand_mode < QUADS_W4A16 || a->operand_mode > QUADS_W16A16 || a->rac_nsel_13 != 0)
      return QUADS_ERR_SHAPE;
  }
  // expert-sharded execution: this call's experts
  const int e_lo = (dense || a->expert_count == 0) ? 0 : a->expert_lo;
  const int e_cnt = (dense || a->expert_count == 0) ? E : a->expert_count;
  if (e_lo < 0 || e_cnt < 1 || e_lo + e_cnt > E) return QUADS_ERR_SHAPE;
  if (dense && (a->expert_count != 0 || a->out_f32)) return QUADS_ERR_SHAPE;
  if (T == 0) return QUADS_OK;                      // nothing to do; x / out may be NULL
  if (a->operand_mode == QUADS_W16A4 || a->operand_mode == QUADS_W16A16) {
    if (!a->x || !a->w13_bf16 || !a->out) return QUADS_ERR_NULL;
    if (!aligned(a->w13_bf16, 16)) return QUADS_ERR_SHAPE;
  } else if (!a->x || !a->w13_q || !a->w13_sf || !a->w13_gs || (!a->out && !a->out_f32)) {
    return QUADS_ERR_NULL;
  }
  if (!aligned(a->out_f32, 16)) return QUADS_ERR_SHAPE;
  if (!dense && (!a->router_logits || !a->w2_q || !a->w2_sf || !a->w2_gs || !a->a2_gs)) return QUADS_ERR_NULL;
  if (!aligned(a->x, 32) || !aligned(a->w13_q, 16) || !aligned(a->w13_sf, 16) || !aligned(a->out, 16) ||
      (!dense && (!aligned(a->w2_q, 16) || !aligned(a->w2_sf, 16))))
    return QUADS_ERR_SHAPE;
  const MoeLayout L = moe_layout(T, H, I, E, topk, a->N);
  if (!a->workspace || !aligned(a->workspace, 256) || a->workspace_bytes < L.total) return QUADS_ERR_WORKSPACE;
  DeviceInfo di;
  quads_status s = device_info(&di);
  if (s != QUADS_OK) return s;
  if (T == 0) return QUADS_OK;

  uint8_t* ws = static_cast<uint8_t*>(a->workspace);
  auto P = [&](size_t off) { return ws + off; };
  int32_t* header = reinterpret_cast<int32_t*>(P(L.header));
  uint32_t* amax_bits = reinterpret_cast<uint32_t*>(P(L.amax));
  int32_t* ids = reinterpret_cast<int32_t*>(P(L.ids));
  float* wts = reinterpret_cast<float*>(P(L.wts));
  int32_t* offsets = reinterpret_cast<int32_t*>(P(L.offsets));
  int32_t* tile_prefix = reinterpret_cast<int32_t*>(P(L.tile_prefix));
  int32_t* tile_expert = reinterpret_cast<int32_t*>(P(L.tile_expert));
  int32_t* tile_rows = reinterpret_cast<int32_t*>(P(L.tile_rows));
  int32_t* perm = reinterpret_cast<int32_t*>(P(L.perm));
  int32_t* pos_pad = reinterpret_cast<int32_t*>(P(L.pos_pad));
  int32_t* row_token = reinterpret_cast<int32_t*>(P(L.row_token));
  float* row_weight = reinterpret_cast<float*>(P(L.row_weight));
  const uint16_t* x = static_cast<const uint16_t*>(a->x);
  const int A = T * topk;
  const size_t pad_rows = (size_t)L.m_tiles_max * 128;
  const int cta_group = gemm_cta_group_for(dense ? (int64_t)T : (int64_t)A, dense ? 1 : E);

  g_trace.n = 0;
  trace_mark("start", st);
  // header (status word included) and the amax word start at zero
  QUADS_CUDA_OK(cudaMemsetAsync(ws, 0, L.ids, st));
  trace_mark("memset", st);

  if (dense && a->operand_mode != QUADS_W4A4) {
    // ---- one-sided modes: decode the NVFP4 side to bf16 with the library's own kernels, then one
    // bf16 tensor-core product
    uint16_t* dec = reinterpret_cast<uint16_t*>(P(L.dec));
    const void *A_op = a->x, *B_op = a->w13_bf16;
    if (a->operand_mode == QUADS_W4A16) {
      const int64_t nblk = (int64_t)a->N * (H / 16);
      const int grid = (int)std::min<int64_t>((nblk + 255) / 256, (int64_t)di.sm_count * 16);
      QUADS_CUDA_OK(launch_kernel(dequantize_kernel, dim3(grid), dim3(256), (size_t)0, st, a->w13_q, a->w13_sf, a->w13_gs, 1,
                                  nblk, (uint32_t)(H / 16), (int)(H / 64), 1, (int64_t)quads_sf_tiled_bytes(a->N, H), dec));
      B_op = dec;
    } else if (a->operand_mode == QUADS_W16A4) {
      // Q_A(x) then decode, in one pass of the quantizer (its scratch: the 256 bytes at the amax slot)
      const int launches = g_launch_count;
      s = quantize_common(a->x, 1, T, H, H, 0, a->a13_gs, dec, a->xq, a->xsf, a->a13_gs_out, QUADS_SF_LINEAR, P(L.amax), (size_t)kAmaxPartsMax * 4, st);
      g_launch_count += launches;
      if (s != QUADS_OK) return s;
      A_op = dec;
    }
    CUtensorMap tm_a, tm_b;
    if ((s = make_bf16_map(&tm_a, A_op, (uint64_t)T, (uint64_t)H)) != QUADS_OK) return s;
    if ((s = make_bf16_map(&tm_b, B_op, (uint64_t)a->N, (uint64_t)H)) != QUADS_OK) return s;
    s = launch_gemm_bf16(tm_a, tm_b, T, a->N, H, static_cast<uint16_t*>(a->out), header + kHdrStatus, di.sm_count, st);
    if (s != QUADS_OK) return s;
    QUADS_CUDA_OK(cudaGetLastError());
    return QUADS_OK;
  }

  // ---- routing and dispatch order: on a side stream, next to the activation chain below
  // (declared in this order: on an early return the guard joins first, then the lock is released)
  std::unique_lock<std::mutex> side_lock(g_side_mu, std::defer_lock);
  SideJoinGuard side_guard;
  SideStream* side = nullptr;
  if (!dense && !g_trace.enabled) {
    side_lock.lock();                       // event record / wait pairs of two host threads must not interleave
    side = side_stream();
    if (!side) side_lock.unlock();
  }
  cudaStream_t rs = st;
  if (side) {
    QUADS_CUDA_OK(cudaEventRecord(side->fork, st));
    QUADS_CUDA_OK(cudaStreamWaitEvent(side->stream, side->fork, 0));
    side_guard.arm(side, st);
    rs = side->stream;
  }
  if (dense) {
    QUADS_CUDA_OK(launch_kernel(dense_dispatch_kernel, dim3((T + 255) / 256), dim3(256), (size_t)(0), st, T, cta_group, pos_pad, row_token, row_weight, tile_expert, tile_rows, header));
  } else {
    int32_t* chunk_counts = reinterpret_cast<int32_t*>(P(L.chunk_counts));
    int32_t* chunk_base = reinterpret_cast<int32_t*>(P(L.chunk_base));
    int32_t* expert_total = reinterpret_cast<int32_t*>(P(L.expert_total));
    {
      auto route = E <= 32 ? route_kernel_t<1> : (E <= 64 ? route_kernel_t<2> : (E <= 128 ? route_kernel_t<4> : route_kernel_t<8>));
      QUADS_CUDA_OK(launch_kernel(route, dim3(L.n_chunks), dim3(256), (size_t)(0), rs, a->router_logits, T, E, topk,
                                  a->renormalize, ids, wts, chunk_counts, expert_total, a->topk_ids, a->topk_w, e_lo, e_lo + e_cnt));
    }
    trace_mark("route", st);
    QUADS_CUDA_OK(launch_kernel(scan_kernel, dim3(E), dim3(256), (size_t)(0), rs, E, L.n_chunks, cta_group, chunk_counts, expert_total, chunk_base, offsets, tile_prefix, tile_expert, tile_rows, header, a->expert_offsets));
    trace_mark("scan", st);
    QUADS_CUDA_OK(launch_kernel(permute_kernel, dim3(L.n_chunks), dim3(128), (size_t)(0), rs, T, E, topk, L.n_chunks, ids, wts, chunk_base, offsets, tile_prefix, perm, pos_pad, row_token, row_weight, a->perm, e_lo, e_lo + e_cnt));
  }
  trace_mark("permute", st);

  // ---- per-tensor scale of x
  // ---- per-tensor scale of x: folded into the quantization kernel (cooperative launch, grid
  // barrier) when all of its CTAs fit on the GPU at once; else a kernel of its own
  const int rq_block = H / 16 > 256 ? 256 : (H / 16 + 31) / 32 * 32;
  static const bool no_fused_amax = getenv("QUADS_NO_FUSED_AMAX") != nullptr;
  bool fused_amax = false;
  if (!a->a13_gs && !no_fused_amax && !g_trace.enabled) {
    // resident CTAs per SM for the two block sizes in use (128 and 256 threads); same on every sm_100 device
    static std::atomic<int> per_sm_cache[2] = {{0}, {0}};
    std::atomic<int>& slot = per_sm_cache[rq_block > 128 ? 1 : 0];
    int per_sm = slot.load();
    if (per_sm == 0) {
      QUADS_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rac_quant_kernel, rq_block > 128 ? 256 : 128, 0));
      slot.store(per_sm);
    }
    fused_amax = (int64_t)per_sm * di.sm_count >= L.stats_ctas;
  }
  if (!a->a13_gs && !fused_amax) {
    const int64_t chunks = (int64_t)T * (H / 8);
    int gx = (int)((chunks + 2047) / 2048);
    if (gx > di.sm_count * 8) gx = di.sm_count * 8;
    QUADS_CUDA_OK(launch_kernel(amax_kernel, dim3(gx, 1), dim3(256), (size_t)(0), st, x, T, H, H, 0, amax_bits));
  }
  trace_mark("amax", st);
  // ---- site 13: quantize (+ residual + statistics), selection, dispatch scatter
  const int nsel13 = a->rac_nsel_13;
  const bool totals13 = (int64_t)L.stats_ctas * H <= ((int64_t)1 << 18);
  uint8_t* mask13 = P(L.mask13);
  {
    const uint16_t* xp = x;
    int Tt = T, Hh = H, rows_per_cta = L.rows_per_cta, with_res = nsel13 > 0 ? 1 : 0;
    const float* gs13 = a->a13_gs;
    unsigned int* arrivals = fused_amax ? reinterpret_cast<unsigned int*>(header + kHdrArrivals) : nullptr;
    int32_t* status_word = header + kHdrStatus;
    float* gs_store = a->a13_gs_out;
    // Column scores of site 13: integer totals added by every CTA when there are few of them (the
    // selection is then one ranking kernel; decode-sized batches), else one partial row per CTA and a
    // reduction kernel (586 x 2048 integer reductions at the end of the kernel cost 20 us, the
    // reduction kernel 9)
    float* partials = totals13 ? nullptr : reinterpret_cast<float*>(P(L.partials13));
    unsigned long long* totals = totals13 ? reinterpret_cast<unsigned long long*>(P(L.keys13)) : nullptr;
    // a CTA's partial sum covers rows_per_cta rows (< rows * 2^18 in units of the squared scale); the
    // stats_ctas partial sums of a column must fit 62 bits together
    int cap_bits = 18, ctas_log2 = 0;
    while ((1 << (cap_bits - 18)) < rows_per_cta) ++cap_bits;
    while ((1 << ctas_log2) < L.stats_ctas) ++ctas_log2;
    int score_bits = std::max(0, std::min(26, 62 - cap_bits - ctas_log2));
    uint8_t *xq_tok = P(L.xq_tok), *xsf_tok = P(L.xsf_tok), *rq_tok = P(L.rq_tok), *rsf_tok = P(L.rsf_tok);
    uint8_t *xq_exp = a->xq, *xsf_exp = a->xsf;
    if (fused_amax) {
      void* args[] = {&xp, &Tt, &Hh, &gs13, &amax_bits, &arrivals, &status_word, &gs_store, &rows_per_cta, &with_res,
                      &partials, &xq_tok, &xsf_tok, &rq_tok, &rsf_tok, &xq_exp, &xsf_exp, &totals, &score_bits, &cap_bits};
      QUADS_CUDA_OK(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(rac_quant_kernel), dim3(L.stats_ctas),
                                                dim3(rq_block), args, 0, st));
      note_launch();
    } else {
      QUADS_CUDA_OK(launch_kernel(rac_quant_kernel, dim3(L.stats_ctas), dim3(rq_block), (size_t)(0), st, xp, Tt, Hh, gs13,
                                  amax_bits, arrivals, status_word, gs_store, rows_per_cta, with_res, partials, xq_tok,
                                  xsf_tok, rq_tok, rsf_tok, xq_exp, xsf_exp, totals, score_bits, cap_bits));
    }
  }
  trace_mark("rac_stats", st);
  // The dispatched copies of Q(x) need only the dispatch order and the codes: with a side stream
  // they are written there, next to the channel selection; the residual copies (which need the
  // selection and the dispatch tables, not the other copies) follow on the main stream and may run
  // beside them: the two streams meet again only in front of the first projection.
  const bool split_scatter = side != nullptr && nsel13 > 0;
  auto dispatch = [&](int parts, cudaStream_t s_) {
    auto k = parts == 1 ? rac_dispatch_kernel<1> : (parts == 2 ? rac_dispatch_kernel<2> : rac_dispatch_kernel<3>);
    return launch_kernel(k, dim3(L.m_tiles_max), dim3(256), (size_t)(0), s_, H, mask13, header,
                         tile_rows, row_token, P(L.xq_tok), P(L.xsf_tok), P(L.rq_tok), P(L.rsf_tok), P(L.xq_pad),
                         P(L.xsf), P(L.rq_pad), P(L.rsf));
  };
  if (side) {
    if (split_scatter) {
      QUADS_CUDA_OK(cudaEventRecord(side->tables, side->stream));      // routing tables complete
      QUADS_CUDA_OK(cudaEventRecord(side->mid, st));
      QUADS_CUDA_OK(cudaStreamWaitEvent(side->stream, side->mid, 0));
      QUADS_CUDA_OK(dispatch(1, side->stream));
    }
  }
  if (nsel13 > 0) {
    if (totals13)
      s = run_rank(reinterpret_cast<unsigned long long*>(P(L.keys13)), H, nsel13, mask13, a->sel13, st);
    else
      s = run_select(reinterpret_cast<float*>(P(L.partials13)), nullptr, 1, L.stats_ctas, H, nsel13,
                     reinterpret_cast<double*>(P(L.scores13)), reinterpret_cast<unsigned int*>(P(L.counters13)),
                     reinterpret_cast<unsigned long long*>(P(L.keys13)), mask13, a->sel13, st);
    if (s != QUADS_OK) return s;
  }
  trace_mark("select13", st);
  if (split_scatter) {
    QUADS_CUDA_OK(cudaStreamWaitEvent(st, side->tables, 0));
  } else if (side) {
    side_guard.join();
    side_lock.unlock();
  }
  {
    const int parts = split_scatter ? 2 : (nsel13 > 0 ? 3 : 1);
    QUADS_CUDA_OK(dispatch(parts, st));
    if (nsel13 > 0 && (a->rq || a->rsf)) {
      // verification export of the masked residual in token order (no dispatched copies: top-k of 0)
      const int64_t chunks = (int64_t)T * (H / 32);
      QUADS_CUDA_OK(launch_kernel(rac_scatter_kernel, dim3((unsigned)((chunks + 255) / 256)), dim3(256), (size_t)(0), st, T, H, 2, mask13, 0, pos_pad, P(L.xq_tok), P(L.xsf_tok), P(L.rq_tok), P(L.rsf_tok), P(L.xq_pad), P(L.xsf), P(L.rq_pad), P(L.rsf), a->rq, a->rsf));
    }
  }
  if (split_scatter) {
    side_guard.join();
    side_lock.unlock();
  }
  trace_mark("rac_dispatch", st);
  // ---- tensor maps
  // few rows per expert (decode-sized batches): operands swapped, weights on the M side
  static const bool no_swap = getenv("QUADS_NO_SWAP") != nullptr;
  const bool swapped = !dense && !no_swap && cta_group == 1 && gemm_swapped_ok(A, E, L.m_tiles_max);
  const uint32_t act_box = swapped ? 16 : 128;
  GemmMaps m1;
  if ((s = make_codes_map(&m1.a, P(L.xq_pad), pad_rows, H / 2, act_box)) != QUADS_OK) return s;
  if ((s = make_codes_map(&m1.r, P(L.rq_pad), pad_rows, H / 2, act_box)) != QUADS_OK) return s;
  if ((s = make_codes_map(&m1.b, a->w13_q, (uint64_t)e_cnt * N1, H / 2)) != QUADS_OK) return s;
  if (cta_group == 2) {
    const uint64_t a_atoms = (uint64_t)(pad_rows / 128) * (H / 64);
    if ((s = make_sf_map(&m1.sfa, P(L.xsf), a_atoms)) != QUADS_OK) return s;
    if ((s = make_sf_map(&m1.sfr, P(L.rsf), a_atoms)) != QUADS_OK) return s;
    if ((s = make_sf_map(&m1.sfb, a->w13_sf, (uint64_t)e_cnt * (quads_sf_tiled_bytes(N1, H) / 512))) != QUADS_OK) return s;
  }

  GemmParams g{};
  g.K = H;
  g.has_resid = nsel13 > 0;
  g.header = header; g.tile_expert = tile_expert; g.tile_rows = tile_rows;
  g.a_sf = P(L.xsf); g.r_sf = P(L.rsf);
  g.b_sf = a->w13_sf; g.b_sf_expert_stride = quads_sf_tiled_bytes(N1, H);
  g.b_gs = a->w13_gs; g.a_gs = a->a13_gs; g.a_amax_bits = amax_bits;
  g.row_token = row_token; g.row_weight = row_weight;
  g.tile_prefix = tile_prefix; g.offsets = offsets;
  g.status = header + kHdrStatus;
  g.b_rows_per_expert = N1;
  g.n_experts = e_cnt;
  g.expert_lo = e_lo;
  if (dense) {
    g.n_out = a->N;
    g.n_tiles_n = (a->N + 255) / 256;
    g.half1_row_offset = 128;
    g.out_bf16 = static_cast<uint16_t*>(a->out);
    return launch_gemm(kEpiStore, cta_group, g, m1, di.sm_count, st);
  }
  g.n_out = I;
  g.n_tiles_n = I / 128;                          // both variants: 128 features per tile (gate + up rows)
  g.half1_row_offset = I;
  g.h_gs = a->a2_gs;
  g.resid2 = a->rac_nsel_2 > 0 || a->r2q || a->r2sf;
  g.hq_pad = P(L.hq_pad); g.hsf_tiled = P(L.hsf); g.r2q_pad = P(L.r2q_pad); g.r2sf_tiled = P(L.r2sf);
  g.keys2 = reinterpret_cast<unsigned long long*>(P(L.keys2));
  {
    // fractional bits of the integer column scores: a partial sum stays below 2^23 (in units of the
    // squared scale), there are at most 4 per row tile, and their total must fit 62 bits
    int rows_log2 = 0;
    while (((int64_t)1 << rows_log2) < (int64_t)L.m_tiles_max * 4) ++rows_log2;
    g.score_bits = std::max(0, std::min(26, 62 - 23 - rows_log2));
  }
  g.h_export = static_cast<uint16_t*>(a->h_bf16);
  const bool timing = g_timers.enabled && g_timers.created;
  if (timing) QUADS_CUDA_OK(cudaEventRecord(g_timers.ev[0], st));
  s = swapped ? launch_gemm_swapped(kEpiSwiGLU, g, m1, di.sm_count, st)
              : launch_gemm(kEpiSwiGLU, cta_group, g, m1, di.sm_count, st);
  if (s != QUADS_OK) return s;
  if (timing) QUADS_CUDA_OK(cudaEventRecord(g_timers.ev[1], st));

  trace_mark("gemm1", st);
  // ---- site 2: selection and masking of the residual of h
  const int nsel2 = a->rac_nsel_2;
  uint8_t* mask2 = P(L.mask2);
  if (nsel2 > 0) {
    // the scores are complete when the first projection ends (integer totals): ranking only
    s = run_rank(g.keys2, I, nsel2, mask2, a->sel2, st);
    if (s != QUADS_OK) return s;
    QUADS_CUDA_OK(launch_kernel(mask_codes_kernel, dim3(di.sm_count * 8), dim3(256), (size_t)(0), st, P(L.r2q_pad), header + kHdrPaddedRows, I, mask2));
  } else if (a->r2q) {
    QUADS_CUDA_OK(cudaMemsetAsync(mask2, 0, I, st));
  }
  if (a->hq || a->hsf || a->r2q || a->r2sf) {
    const int64_t n = (int64_t)A * (I / 16);
    QUADS_CUDA_OK(launch_kernel(export_site2_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), (size_t)(0), st, A, header + kHdrAssignments, I, perm, pos_pad, P(L.hq_pad), P(L.hsf), P(L.r2q_pad), P(L.r2sf), mask2, a->hq, a->hsf, a->r2q, a->r2sf));
  }

  trace_mark("select2+mask", st);
  // ---- second projection + weighted combine
  uint16_t* y_pad = reinterpret_cast<uint16_t*>(P(L.y_pad));
  GemmMaps m2;
  if ((s = make_codes_map(&m2.a, P(L.hq_pad), pad_rows, I / 2, act_box)) != QUADS_OK) return s;
  if ((s = make_codes_map(&m2.r, P(L.r2q_pad), pad_rows, I / 2, act_box)) != QUADS_OK) return s;
  if ((s = make_codes_map(&m2.b, a->w2_q, (uint64_t)e_cnt * H, I / 2)) != QUADS_OK) return s;
  if (cta_group == 2) {
    const uint64_t a_atoms = (uint64_t)(pad_rows / 128) * (I / 64);
    if ((s = make_sf_map(&m2.sfa, P(L.hsf), a_atoms)) != QUADS_OK) return s;
    if ((s = make_sf_map(&m2.sfr, P(L.r2sf), a_atoms)) != QUADS_OK) return s;
    if ((s = make_sf_map(&m2.sfb, a->w2_sf, (uint64_t)e_cnt * (quads_sf_tiled_bytes(H, I) / 512))) != QUADS_OK) return s;
  }
  GemmParams g2 = g;
  g2.K = I;
  g2.has_resid = nsel2 > 0;
  g2.a_sf = P(L.hsf); g2.r_sf = P(L.r2sf);
  g2.b_sf = a->w2_sf; g2.b_sf_expert_stride = quads_sf_tiled_bytes(H, I);
  g2.b_gs = a->w2_gs; g2.a_gs = a->a2_gs; g2.a_amax_bits = nullptr;
  g2.b_rows_per_expert = H;
  g2.n_out = H;
  g2.n_tiles_n = swapped ? H / 128 : (H + 255) / 256;
  g2.half1_row_offset = 128;
  g2.y_pad = y_pad;
  if (timing) QUADS_CUDA_OK(cudaEventRecord(g_timers.ev[2], st));
  s = swapped ? launch_gemm_swapped(kEpiCombine, g2, m2, di.sm_count, st)
              : launch_gemm(kEpiCombine, cta_group, g2, m2, di.sm_count, st);
  if (s != QUADS_OK) return s;
  if (timing) {
    QUADS_CUDA_OK(cudaEventRecord(g_timers.ev[3], st));
    g_timers.valid = true;
  }
  trace_mark("gemm2", st);
  const int64_t n8 = (int64_t)T * (H / 8);
  QUADS_CUDA_OK(launch_kernel(combine_kernel, dim3((unsigned)((n8 + 255) / 256)), dim3(256), (size_t)(0), st, y_pad, pos_pad, wts, T, H, topk, static_cast<uint16_t*>(a->out), a->out_f32));
  trace_mark("combine", st);
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}


// ---------------------------------------------------------------------------
// FP8 W8A8 comparison path
// ---------------------------------------------------------------------------
namespace {
struct Fp8Layout {
  size_t header, expert_total, ids, wts, chunk_counts, chunk_base, offsets, tile_prefix, tile_expert, tile_rows;
  size_t perm, pos_pad, row_token, row_weight, xq_tok, xe_tok, xq_pad, xsf, hq_pad, hsf, y_pad, total;
  int n_chunks, m_tiles_max;
};
Fp8Layout fp8_layout(int T, int H, int I, int E, int topk) {
  Fp8Layout L{};
  const int64_t A = (int64_t)T * topk;
  L.n_chunks = (T + kRouteTokensPerCta - 1) / kRouteTokensPerCta;
  L.m_tiles_max = (int)(A / 128) + E;
  const size_t pad_rows = (size_t)L.m_tiles_max * 128;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
  L.header = take(kHdrWords * 4);
  L.expert_total = take((size_t)E * 4);
  L.ids = take((size_t)A * 4);
  L.wts = take((size_t)A * 4);
  L.chunk_counts = take((size_t)L.n_chunks * E * 4);
  L.chunk_base = take((size_t)L.n_chunks * E * 4);
  L.offsets = take((size_t)(E + 1) * 4);
  L.tile_prefix = take((size_t)(E + 1) * 4);
  L.tile_expert = take((size_t)L.m_tiles_max * 4);
  L.tile_rows = take((size_t)L.m_tiles_max * 4);
  L.perm = take((size_t)A * 4);
  L.pos_pad = take((size_t)A * 4);
  L.row_token = take(pad_rows * 4);
  L.row_weight = take(pad_rows * 4);
  L.xq_tok = take((size_t)T * H);
  L.xe_tok = take((size_t)T * (H / 128));
  L.xq_pad = take(pad_rows * (size_t)H);
  L.xsf = take((size_t)L.m_tiles_max * (H / 128) * 512);
  L.hq_pad = take(pad_rows * (size_t)I);
  L.hsf = take((size_t)L.m_tiles_max * (I / 128) * 512);
  L.y_pad = take(pad_rows * (size_t)H * 2);
  L.total = o;
  return L;
}
}  // namespace

quads_status quads_fp8_quantize_weights(const void* w, int64_t n_tensors, int64_t N, int64_t K, uint8_t* q,
                                        uint8_t* exps, uint8_t* atoms, void* cuda_stream) {
  g_launch_count = 0;
  if (n_tensors < 0 || N <= 0 || K <= 0 || (N % 128) != 0 || (K % 128) != 0) return QUADS_ERR_SHAPE;
  if (n_tensors * (N / 128) * (K / 128) > (int64_t)0x7FFFFFFF) return QUADS_ERR_SHAPE;
  if (n_tensors == 0) return QUADS_OK;
  if (!w || !q || !exps || !atoms) return QUADS_ERR_NULL;
  if (!aligned(w, 16) || !aligned(q, 16) || !aligned(atoms, 16)) return QUADS_ERR_SHAPE;
  DeviceInfo di;
  quads_status s = device_info(&di);
  if (s != QUADS_OK) return s;
  const unsigned grid = (unsigned)(n_tensors * (N / 128) * (K / 128));
  QUADS_CUDA_OK(launch_kernel(fp8_quantize_weight_kernel, dim3(grid), dim3(256), (size_t)0, static_cast<cudaStream_t>(cuda_stream),
                              static_cast<const uint16_t*>(w), (int)N, (int)K, q, exps, atoms));
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}

size_t quads_moe_fp8_workspace_bytes(int32_t T, int32_t H, int32_t I, int32_t E, int32_t topk) {
  if (T < 0 || H <= 0 || I <= 0 || E < 1 || topk < 1) return 0;
  return fp8_layout(T, H, I, E, topk).total;
}


quads_status quads_moe_fp8_w8a8(const quads_moe_fp8_args* a, void* cuda_stream) {
  g_launch_count = 0;
  if (!a) return QUADS_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int T = a->T, H = a->H, I = a->I, E = a->E, topk = a->topk;
  if (T < 0 || H <= 0 || (H % 128) != 0 || I <= 0 || (I % 128) != 0 || H > 16384 || I > 16384) return QUADS_ERR_SHAPE;
  if (E < 1 || E > kMaxExperts || topk < 1 || topk > kMaxTopk || topk > E) return QUADS_ERR_SHAPE;
  if ((int64_t)T * topk > 0x3FFFFFFF) return QUADS_ERR_SHAPE;
  if (T == 0) return QUADS_OK;
  if (!a->x || !a->router_logits || !a->w13_q || !a->w13_atoms || !a->w2_q || !a->w2_atoms || !a->out) return QUADS_ERR_NULL;
  if (a->h_bf16 && (!a->hq || !a->hexp)) return QUADS_ERR_NULL;
  if (!aligned(a->x, 16) || !aligned(a->w13_q, 16) || !aligned(a->w13_atoms, 16) || !aligned(a->w2_q, 16) ||
      !aligned(a->w2_atoms, 16) || !aligned(a->out, 16) || !aligned(a->h_bf16, 16) || !aligned(a->hq, 16))
    return QUADS_ERR_SHAPE;
  const Fp8Layout L = fp8_layout(T, H, I, E, topk);
  if (!a->workspace || !aligned(a->workspace, 256) || a->workspace_bytes < L.total) return QUADS_ERR_WORKSPACE;
  DeviceInfo di;
  quads_status s = device_info(&di);
  if (s != QUADS_OK) return s;
  uint8_t* ws = static_cast<uint8_t*>(a->workspace);
  auto P = [&](size_t off) { return ws + off; };
  int32_t* header = reinterpret_cast<int32_t*>(P(L.header));
  int32_t* ids = reinterpret_cast<int32_t*>(P(L.ids));
  float* wts = reinterpret_cast<float*>(P(L.wts));
  int32_t* chunk_counts = reinterpret_cast<int32_t*>(P(L.chunk_counts));
  int32_t* chunk_base = reinterpret_cast<int32_t*>(P(L.chunk_base));
  int32_t* expert_total = reinterpret_cast<int32_t*>(P(L.expert_total));
  int32_t* offsets = reinterpret_cast<int32_t*>(P(L.offsets));
  int32_t* tile_prefix = reinterpret_cast<int32_t*>(P(L.tile_prefix));
  int32_t* tile_expert = reinterpret_cast<int32_t*>(P(L.tile_expert));
  int32_t* tile_rows = reinterpret_cast<int32_t*>(P(L.tile_rows));
  int32_t* perm = reinterpret_cast<int32_t*>(P(L.perm));
  int32_t* pos_pad = reinterpret_cast<int32_t*>(P(L.pos_pad));
  int32_t* row_token = reinterpret_cast<int32_t*>(P(L.row_token));
  float* row_weight = reinterpret_cast<float*>(P(L.row_weight));
  const size_t pad_rows = (size_t)L.m_tiles_max * 128;
  QUADS_CUDA_OK(cudaMemsetAsync(ws, 0, L.ids, st));            // header, status word, per-expert totals
  // ---- routing and dispatch order (the NVFP4 path's kernels)
  {
    auto route = E <= 32 ? route_kernel_t<1> : (E <= 64 ? route_kernel_t<2> : (E <= 128 ? route_kernel_t<4> : route_kernel_t<8>));
    QUADS_CUDA_OK(launch_kernel(route, dim3(L.n_chunks), dim3(256), (size_t)0, st, a->router_logits, T, E, topk, a->renormalize,
                                ids, wts, chunk_counts, expert_total, a->topk_ids, (float*)nullptr, 0, E));
  }
  QUADS_CUDA_OK(launch_kernel(scan_kernel, dim3(E), dim3(256), (size_t)0, st, E, L.n_chunks, 1, chunk_counts, expert_total,
                              chunk_base, offsets, tile_prefix, tile_expert, tile_rows, header, (int32_t*)nullptr));
  QUADS_CUDA_OK(launch_kernel(permute_kernel, dim3(L.n_chunks), dim3(128), (size_t)0, st, T, E, topk, L.n_chunks, ids, wts,
                              chunk_base, offsets, tile_prefix, perm, pos_pad, row_token, row_weight, a->perm, 0, E));
  // ---- activation quantization (token order) and dispatch
  uint8_t* xq_tok = a->xq ? a->xq : P(L.xq_tok);
  uint8_t* xe_tok = a->xexp ? a->xexp : P(L.xe_tok);
  {
    const int64_t tiles = (int64_t)T * (H / 128);
    const unsigned grid = (unsigned)std::min<int64_t>((tiles + 7) / 8, (int64_t)di.sm_count * 16);
    QUADS_CUDA_OK(launch_kernel(fp8_quantize_act_kernel, dim3(grid), dim3(256), (size_t)0, st, static_cast<const uint16_t*>(a->x),
                                (int64_t)T, H, xq_tok, xe_tok));
  }
  QUADS_CUDA_OK(launch_kernel(fp8_dispatch_kernel, dim3(L.m_tiles_max), dim3(256), (size_t)0, st, H, header, tile_rows, row_token,
                              xq_tok, xe_tok, P(L.xq_pad), P(L.xsf)));
  // ---- first projection: W13, SwiGLU, requantize
  CUtensorMap ma, mb;
  if ((s = make_codes_map(&ma, P(L.xq_pad), pad_rows, (uint64_t)H)) != QUADS_OK) return s;
  if ((s = make_codes_map(&mb, a->w13_q, (uint64_t)E * 2 * I, (uint64_t)H)) != QUADS_OK) return s;
  Fp8GemmParams g{};
  g.K = H; g.n_tiles_n = I / 128; g.n_out = I; g.b_rows_per_expert = 2 * I; g.half1_row_offset = I;
  g.header = header; g.tile_expert = tile_expert; g.tile_rows = tile_rows;
  g.a_sf = P(L.xsf); g.b_sf = a->w13_atoms; g.b_sf_expert_stride = (size_t)(2 * I / 128) * (H / 128) * 512;
  g.hq_pad = P(L.hq_pad); g.hsf_atoms = P(L.hsf);
  g.h_export = static_cast<uint16_t*>(a->h_bf16); g.hq_export = a->hq; g.hexp_export = a->hexp;
  g.tile_prefix = tile_prefix; g.offsets = offsets; g.status = header + kHdrStatus;
  const bool timing = g_timers.enabled && g_timers.created;
  if (timing) QUADS_CUDA_OK(cudaEventRecord(g_timers.ev[0], st));
  if ((s = launch_gemm_fp8(kEpiSwiGLU, g, ma, mb, di.sm_count, st)) != QUADS_OK) return s;
  if (timing) QUADS_CUDA_OK(cudaEventRecord(g_timers.ev[1], st));
  // ---- second projection and weighted combine
  CUtensorMap m2a, m2b;
  if ((s = make_codes_map(&m2a, P(L.hq_pad), pad_rows, (uint64_t)I)) != QUADS_OK) return s;
  if ((s = make_codes_map(&m2b, a->w2_q, (uint64_t)E * H, (uint64_t)I)) != QUADS_OK) return s;
  Fp8GemmParams g2 = g;
  g2.K = I; g2.n_tiles_n = (H + 255) / 256; g2.n_out = H; g2.b_rows_per_expert = H; g2.half1_row_offset = 128;
  g2.a_sf = P(L.hsf); g2.b_sf = a->w2_atoms; g2.b_sf_expert_stride = (size_t)(H / 128) * (I / 128) * 512;
  g2.y_pad = reinterpret_cast<uint16_t*>(P(L.y_pad));
  g2.h_export = nullptr;
  if (timing) QUADS_CUDA_OK(cudaEventRecord(g_timers.ev[2], st));
  if ((s = launch_gemm_fp8(kEpiCombine, g2, m2a, m2b, di.sm_count, st)) != QUADS_OK) return s;
  if (timing) {
    QUADS_CUDA_OK(cudaEventRecord(g_timers.ev[3], st));
    g_timers.valid = true;
  }
  const int64_t n8 = (int64_t)T * (H / 8);
  QUADS_CUDA_OK(launch_kernel(combine_kernel, dim3((unsigned)((n8 + 255) / 256)), dim3(256), (size_t)0, st, g2.y_pad, pos_pad, wts,
                              T, H, topk, static_cast<uint16_t*>(a->out), (float*)nullptr));
  QUADS_CUDA_OK(cudaGetLastError());
  return QUADS_OK;
}

}  // extern "C"
