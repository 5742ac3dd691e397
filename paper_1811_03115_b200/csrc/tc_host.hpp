// Host side of the tensor-core projection: TMA tensor maps, K-split planning and launches.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <map>
#include <mutex>
#include <tuple>

#include "gemm_tc.cuh"
#include "host.hpp"

namespace bpd {
namespace tc {

// Resident CTA slots the planner aims to fill: 2 CTAs on each of the 148 SMs of a B200.
constexpr int kSlots = 296;
constexpr int kMinChunksPerSplit = 2;

struct Plan {
  int tiles, chunks, splits, chunks_per_split;
};
// Depends on (N, K) only -- never on the number of tokens -- so that a position
// scored alone and the same position scored inside a block add up in the same order.
// wide_ttiles: 0 for sessions whose passes carry few rows (one token tile, two CTAs per SM, split K finely);
// otherwise the number of token tiles the split is planned for (the session's widest pass, unless the launch
// says otherwise): those launches already have tiles x token tiles CTAs, so K is split only as far as that
// leaves of the `slots` CTA slots idle.  Both are properties of the session and of the matrix, so greedy and
// blockwise passes of one session still agree.
inline Plan plan_splits(int N, int K, int wide_ttiles = 0, int slots = kSlots / 2) {
  Plan pl;
  pl.tiles = (N + kBM - 1) / kBM;
  pl.chunks = (K + kBK - 1) / kBK;
  int splits;
  if (wide_ttiles > 0) splits = std::max(1, std::min(pl.chunks / 8, slots / (pl.tiles * wide_ttiles)));
  else splits = std::max(1, std::min(pl.chunks / kMinChunksPerSplit, kSlots / pl.tiles));
  pl.chunks_per_split = (pl.chunks + splits - 1) / splits;
  pl.splits = (pl.chunks + pl.chunks_per_split - 1) / pl.chunks_per_split;
  return pl;
}
inline int token_bn(int T, int ttiles);
// Token tiling of a launch: as few tiles of at most 128 tokens as possible, but -- in sessions with many rows --
// the tiling (tiles of 32 to 64 tokens) that leaves the busiest SM the fewest bytes to stage: with
// `ctas_per_ttile` CTAs per token tile, a CTA stages 16 KB of weights and bn / 4 KB of activation planes per
// K chunk, and the busiest SM runs ceil(CTAs / 148) of them.  Ties go to the finer tiling (more loads in
// flight).  The tile width only changes the MMA's N; every output element is still the same sum in the same order.
inline int token_tiles(int T, int ctas_per_ttile = 0) {
  int tt = std::max(1, (T + kMaxBN - 1) / kMaxBN);
  if (ctas_per_ttile > 0) {
    // at most 64 tokens per tile: two CTAs fit on an SM, and one's epilogue overlaps the other's main loop
    // (measured on the batch-32 workload: 1428 -> 1338 us per iteration against tiles of 80-112 tokens)
    tt = std::max(tt, (T + 63) / 64);
    const int hi = std::max(tt, (T + 31) / 32);
    long best_cost = -1;
    int best_tt = tt;
    for (int cand = tt; cand <= hi; ++cand) {
      const int bn = token_bn(T, cand);
      if ((long)(cand - 1) * bn >= T) continue;                   // its last tile would be empty
      const long per_sm = ((long)ctas_per_ttile * cand + 147) / 148;
      const long cost = per_sm * (64 + bn);                       // quarter KB per K chunk
      if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best_tt = cand; }
    }
    tt = best_tt;
  }
  return tt;
}
inline int token_bn(int T, int ttiles) {
  const int per = (T + ttiles - 1) / ttiles;
  return std::max(16, (per + 15) / 16 * 16);
}
inline int token_bn(int T) { return token_bn(T, token_tiles(T)); }
inline int max_token_tiles(int T) { return std::max(token_tiles(T), (T + 31) / 32); }
// fp32 elements of split-K workspace a launch with these sizes needs.
inline size_t ws_floats(int N, int K, int T, int zslices, int wide_ttiles = 0, int slots = kSlots / 2) {
  const Plan pl = plan_splits(N, K, wide_ttiles, slots);
  if (pl.splits == 1) return 0;
  // upper bound over every token tiling the launch may pick: tiles * bn <= T + 16 per tile
  return (size_t)zslices * pl.tiles * pl.splits * ((size_t)T + 16 * max_token_tiles(T)) * kBM;
}
inline size_t counters_needed(int N, int T, int zslices) {
  return (size_t)max_token_tiles(T) * zslices * ((N + kBM - 1) / kBM);
}

struct Scratch {
  float* ws; size_t ws_floats;
  unsigned* tile_counters; size_t n_counters;
  unsigned* done_counter;
  unsigned long long* best; size_t best_elems;
  int* error;
  int wide_ttiles;   // see plan_splits
  int l2_hints;      // 1: weights that a launch reads once are loaded "evict first"
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline int get_encode_fn(EncodeTiledFn* out) {
  static EncodeTiledFn fn = nullptr;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p)
      return fail(BPD_E_CUDA, "cuTensorMapEncodeTiled is not available: %s", cudaGetErrorString(e));
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  *out = fn;
  return BPD_OK;
}

constexpr size_t kMapCacheMax = 4096;   // descriptors kept per process (128 bytes each)

// bf16 matrix [rows, cols] with `ld` elements between rows; boxes of (64 columns, box_rows rows), 128-byte swizzle.
inline int make_map(const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows, CUtensorMap* out) {
  typedef std::tuple<const void*, uint64_t, uint64_t, uint64_t, uint32_t> Key;
  static std::map<Key, CUtensorMap> cache;
  static std::mutex mu;
  const Key key(ptr, rows, cols, ld, box_rows);
  {
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return BPD_OK; }
  }
  if ((uintptr_t)ptr % 16 || (ld * 2) % 16) return fail(BPD_E_INVALID, "tensor-map operand is not 16-byte aligned");
  if (box_rows < 1 || box_rows > 256) return fail(BPD_E_INVALID, "tensor-map box of %u rows", box_rows);
  EncodeTiledFn enc;
  int rc = get_encode_fn(&enc);
  if (rc) return rc;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(BPD_E_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  std::lock_guard<std::mutex> lock(mu);
  // A descriptor is a pure function of its key, so an entry never goes stale (a freed and reused address yields
  // the same descriptor); the cache only saves the encode call.  Keep it bounded: sessions come and go in a
  // long-lived process, each with its own activation buffers.
  if (cache.size() >= kMapCacheMax) cache.clear();
  cache[key] = *out;
  return BPD_OK;
}

// A general 2-D map (not cached): `rows` x `cols` elements of `elem_bytes` (2: bf16, 4: fp32) with `ld` elements
// between rows, boxes of box_cols x box_rows, swizzle chosen by the box's inner extent in bytes (128 -> 128-byte
// mode, 64 -> 64-byte mode, anything else -> none).
inline int make_map_2d(const void* ptr, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_cols,
                       uint32_t box_rows, bool swizzle, CUtensorMap* out) {
  if ((uintptr_t)ptr % 16 || (ld * elem_bytes) % 16) return fail(BPD_E_INVALID, "tensor-map operand is not 16-byte aligned");
  if (box_rows < 1 || box_rows > 256 || box_cols < 1 || box_cols > 256) return fail(BPD_E_INVALID, "tensor-map box %u x %u", box_cols, box_rows);
  EncodeTiledFn enc;
  int rc = get_encode_fn(&enc);
  if (rc) return rc;
  const uint32_t inner = box_cols * (uint32_t)elem_bytes;
  CUtensorMapSwizzle sw = CU_TENSOR_MAP_SWIZZLE_NONE;
  if (swizzle && inner == 128) sw = CU_TENSOR_MAP_SWIZZLE_128B;
  else if (swizzle && inner == 64) sw = CU_TENSOR_MAP_SWIZZLE_64B;
  else if (swizzle) return fail(BPD_E_INVALID, "no swizzle mode for boxes of %u bytes per row", inner);
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * (uint64_t)elem_bytes};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(out, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                   const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(BPD_E_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return BPD_OK;
}

// The same over `layers` tensors that lie `layer_stride_bytes` apart: dimensions (columns, rows, layer), boxes of
// box_cols x box_rows x 1.
inline int make_map_3d(const void* ptr, int elem_bytes, uint64_t layers, uint64_t layer_stride_bytes, uint64_t rows, uint64_t cols,
                       uint64_t ld, uint32_t box_cols, uint32_t box_rows, bool swizzle, CUtensorMap* out) {
  if ((uintptr_t)ptr % 16 || (ld * elem_bytes) % 16 || layer_stride_bytes % 16)
    return fail(BPD_E_INVALID, "tensor-map operand is not 16-byte aligned");
  if (box_rows < 1 || box_rows > 256 || box_cols < 1 || box_cols > 256) return fail(BPD_E_INVALID, "tensor-map box %u x %u", box_cols, box_rows);
  EncodeTiledFn enc;
  int rc = get_encode_fn(&enc);
  if (rc) return rc;
  const uint32_t inner = box_cols * (uint32_t)elem_bytes;
  CUtensorMapSwizzle sw = CU_TENSOR_MAP_SWIZZLE_NONE;
  if (swizzle && inner == 128) sw = CU_TENSOR_MAP_SWIZZLE_128B;
  else if (swizzle && inner == 64) sw = CU_TENSOR_MAP_SWIZZLE_64B;
  else if (swizzle) return fail(BPD_E_INVALID, "no swizzle mode for boxes of %u bytes per row", inner);
  const cuuint64_t dims[3] = {cols, rows, layers};
  const cuuint64_t strides[2] = {ld * (uint64_t)elem_bytes, layers > 1 ? layer_stride_bytes : ld * (uint64_t)elem_bytes * rows};
  const cuuint32_t box[3] = {box_cols, box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(out, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3,
                   const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(BPD_E_CUDA, "cuTensorMapEncodeTiled (3-D) failed with code %d", (int)r);
  return BPD_OK;
}

struct Operands {
  const void* w; int w_rows;            // weights [w_rows, K] (all slices stacked)
  const void* x; long long x_plane;     // activation planes: hi at x, lo at x + x_plane (elements)
  long long ldx; int x_rows; int x_cols;  // allocated rows, total columns per row
  const void* x_lo = nullptr;           // the lo plane when it lives in another allocation (x_plane unused then)
};

template <int EPI>
int launch(const Operands& op, int N, int K, int T, TcParams p, const Scratch& sc, cudaStream_t st, int zslices = 1,
           int a_rows_per_slice = 0, int b_cols_per_slice = 0, bool pdl = false, int plan_n = 0, int plan_tt = 0) {
  {
    int rc0 = ensure_smem_limit(reinterpret_cast<const void*>(gemm_tc_kernel<EPI, false>), smem_bytes(16));
    if (!rc0) rc0 = ensure_smem_limit(reinterpret_cast<const void*>(gemm_tc_kernel<EPI, true>), std::max(smem_bytes(kMaxBN), smem_bytes(64)));
    if (rc0) return rc0;
  }
  // plan_n: the feature count the K split is planned for.  A launch that computes only the first features of a
  // matrix (fewer heads) passes the full count so that every feature is summed in the same order either way.
  // plan_tt: in a session with many rows, a launch whose results need not agree bit for bit with any other
  // launch (the second stage of the lazy heads) plans its K split for its own token tiles and for two CTAs per SM.
  Plan pl = (sc.wide_ttiles && plan_tt > 0) ? plan_splits(plan_n > 0 ? plan_n : N, K, plan_tt, kSlots)
                                            : plan_splits(plan_n > 0 ? plan_n : N, K, sc.wide_ttiles);
  pl.tiles = (N + kBM - 1) / kBM;
  const int ttiles = token_tiles(T, sc.wide_ttiles ? pl.tiles * pl.splits * zslices : 0), bn = token_bn(T, ttiles);
  const size_t need_ws = pl.splits == 1 ? 0 : (size_t)ttiles * zslices * pl.tiles * pl.splits * bn * kBM;
  const size_t need_cnt = (size_t)ttiles * zslices * pl.tiles;
  if (need_ws > sc.ws_floats || need_cnt > sc.n_counters)
    return fail(BPD_E_NOMEM, "split-K workspace too small (%zu floats, %zu counters needed)", need_ws, need_cnt);
  if (EPI == kTcArgmax && (size_t)T > sc.best_elems) return fail(BPD_E_NOMEM, "top-1 workspace too small");
  CUtensorMap ma, mh, ml;
  int rc = make_map(op.w, (uint64_t)op.w_rows, (uint64_t)K, (uint64_t)K, kBM, &ma);
  if (rc) return rc;
  rc = make_map(op.x, (uint64_t)op.x_rows, (uint64_t)op.x_cols, (uint64_t)op.ldx, (uint32_t)bn, &mh);
  if (rc) return rc;
  rc = make_map(op.x_lo ? static_cast<const bf16*>(op.x_lo) : static_cast<const bf16*>(op.x) + op.x_plane, (uint64_t)op.x_rows, (uint64_t)op.x_cols, (uint64_t)op.ldx,
                (uint32_t)bn, &ml);
  if (rc) return rc;
  p.T = T; p.N = N; p.K = K; p.bn = bn; p.splits = pl.splits; p.chunks_per_split = pl.chunks_per_split;
#ifdef BPD_TC_TRACE
  { static int next_trace_id = 0; p.trace_id = next_trace_id++ & 127; }
#endif
  p.ws = sc.ws; p.tile_counters = sc.tile_counters; p.done_counter = sc.done_counter;
  p.best = sc.best; p.error = sc.error;
  p.stream_weights = (ttiles == 1 && sc.l2_hints) ? 1 : 0;
  {
    // vector stores in the epilogue of wide tiles: every row offset and pointer involved must allow them
    auto al = [](const void* q, size_t a) { return q == nullptr || (uintptr_t)q % a == 0; };
    p.vec = (N % 4 == 0 && p.ldo % 4 == 0 && p.plane % 4 == 0 && p.xg_plane % 4 == 0 && p.zofs_n % 4 == 0 &&
             (p.d % 4 == 0) && al(p.out_f32, 16) && al(p.out_hi, 8) && al(p.xg_hi, 8) && al(p.h, 16) && al(p.bias, 8) &&
             al(p.g_next, 8) && al(p.kcache, 8) && al(p.vcache, 8)) ? 1 : 0;
  }
  if ((p.stat_in || p.stat_out) && !(p.vec && bn >= 32 && N % kBM == 0 && EPI != kTcArgmax && !p.ln_x))
    return fail(BPD_E_UNSUPPORTED, "per-tile layer-norm statistics need wide, vectorisable tiles (N = %d, %d tokens per tile)", N, bn);
  dim3 grid(pl.tiles, pl.splits, ttiles * zslices);
  if (bn >= 32)
    BPD_CUDA(launch_k(gemm_tc_kernel<EPI, true>, grid, dim3(kThreads), smem_bytes(bn), st, pdl, ma, mh, ml, p, zslices,
                      a_rows_per_slice, b_cols_per_slice));
  else
    BPD_CUDA(launch_k(gemm_tc_kernel<EPI, false>, grid, dim3(kThreads), smem_bytes(bn), st, pdl, ma, mh, ml, p, zslices,
                      a_rows_per_slice, b_cols_per_slice));
  return BPD_OK;
}

}  // namespace tc
}  // namespace bpd
