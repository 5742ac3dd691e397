// Shared device helpers and parameter structs for the decoding kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bpd {

constexpr int kPage = 64;        // positions per KV-cache page
constexpr int kMaxK = 16;        // largest block size / head count

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// Load 8 consecutive elements (16-byte aligned for bf16, 32-byte for float) as floats.
__device__ __forceinline__ void load8(const bf16* p, float (&out)[8]) {
  uint4 raw = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void load8(const float* p, float (&out)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
  out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
}
// Same, read from L2 (data another SM may have written earlier in the same launch must not come from L1).
__device__ __forceinline__ void load8_cg(const bf16* p, float (&out)[8]) {
  uint4 raw = __ldcg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void load8_cg(const float* p, float (&out)[8]) {
  float4 a = __ldcg(reinterpret_cast<const float4*>(p));
  float4 b = __ldcg(reinterpret_cast<const float4*>(p + 4));
  out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
  out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
}
// Same, bypassing L1 (weights are streamed once).
__device__ __forceinline__ void load8_stream(const bf16* p, float (&out)[8]) {
  uint4 raw = __ldcs(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void load8_stream(const float* p, float (&out)[8]) {
  float4 a = __ldcs(reinterpret_cast<const float4*>(p));
  float4 b = __ldcs(reinterpret_cast<const float4*>(p + 4));
  out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
  out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// (value, index) ordering used by every top-1: larger value wins, equal values go to the lower index.
__device__ __forceinline__ bool better(float v, int i, float bv, int bi) {
  return (v > bv) || (v == bv && i < bi);
}
__device__ __forceinline__ void warp_argmax(float& v, int& i) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, v, o);
    int oi = __shfl_xor_sync(0xffffffffu, i, o);
    if (better(ov, oi, v, i)) { v = ov; i = oi; }
  }
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start while
// its predecessor still runs.  launch_dependents lets the successor start early; wait blocks until the
// predecessor grids have completed and their writes are visible.  Both are no-ops without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Per-row decode state living in the session buffer (device memory).
struct RowState {
  int* len;        // [B] committed decoder inputs (cache length)
  int* j;          // [B] tokens emitted
  int* finished;   // [B]
  int* src_len;    // [B]
  int* block;      // [B][kMaxK] proposals to score next
  int* cur_block;  // [B][kMaxK] proposals scored by the running pass (after forcing)
  int* khat;       // [B]
  int* table;      // [B][kcur][kh]
  int* out_ids;    // [B][max_tgt]
  int* all_done;   // [1]
  int* error;      // [1] first device-side error code
  int* signal;     // [2] epoch of the running decode, passes verified in it
  int* host_flags; // [8] pinned host memory (device address): slot (pass number mod 8) = epoch * 4 + 1, + 1 if all
                   //     rows are finished; the host reads it instead of waiting for a copy between passes
  long long* stats;  // [0] row_iterations, [1] tokens, [2] iterations, [3] priming passes, [4..4+kMaxK] khat histogram
  const int* page_table;  // [B][pages_per_row]
  int pages_per_row;
  int max_tgt;
};

// kModePredict: the Predict call of the two-call form -- like the priming pass, one row per sequence with all heads,
// but at the position of the last accepted token instead of the start token.
enum PassMode { kModePrime = 0, kModeBlock = 1, kModeGreedy = 2, kModePredict = 3 };

// Acceptance criteria of the Verify substep (values match the public header).
enum AcceptKind { kAcceptExact = 0, kAcceptTopN = 1, kAcceptDistance = 2 };

// Top-n acceptance asks how many vocabulary entries beat each proposal under p_1 at the position before it.
// Position pr = row * kcur + r (r-th block position) holds proposal r+1's token, its own logit and the count.
struct RankState {
  float* thr;   // [B*kcur] logit of the proposal under p_1 at position pr
  int* tok;     // [B*kcur] the proposal's token id, -1 where there is none (last position of a block)
  int* cnt;     // [B*kcur] entries that beat it (filled by the vocabulary projection)
};

}  // namespace bpd
