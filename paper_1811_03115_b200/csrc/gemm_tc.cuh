// Weight-streaming projection on the 5th-generation tensor cores (sm_100a):
//   y[t][n] = sum_c x[t][c] * w[n][c]        t < T tokens (few), n < N features (many)
// The weight matrix is the MMA's M operand (128 features per tile), the tokens are
// its N operand.  Weights (bf16, [N, K] row-major) and activations (two bf16
// planes hi + lo that together carry an fp32 value, [rows, K] row-major) are
// brought into 128-byte-swizzled shared memory by TMA; one elected thread issues
// tcgen05.mma with the fp32 accumulator in tensor memory; four warps read it
// back with tcgen05.ld and run the fused epilogue.  K can be split over CTAs
// (grid.y): partial tiles go to a workspace and the CTA that arrives last for a
// tile adds them in split order, so the summation order is fixed by (N, K) alone.
//
// Every wait on an mbarrier is bounded; on expiry the CTA records an error code,
// skips its remaining work, waits (bounded) for copies in flight, frees its
// tensor memory and returns.
#pragma once
#include <type_traits>
#include <cuda.h>

#include "common.cuh"

namespace bpd {
namespace tc {

#ifdef BPD_TC_TRACE
// Development builds only: per-CTA step timestamps of the projection kernel (16 words per CTA, up to 4096 CTAs of
// the launches that run while the pointer is set; 128 regions chosen by the host's launch counter).
__device__ unsigned long long* g_tc_trace = nullptr;
__device__ __forceinline__ void tc_stamp(int region, int slot) {
  if (!g_tc_trace) return;
  const unsigned cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
  if (cta >= 2047) return;
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  g_tc_trace[((size_t)region * 2048 + cta) * 16 + slot] = t;
}
#define BPD_TC_STAMP(slot) tc_stamp(p.trace_id, slot)
#else
#define BPD_TC_STAMP(slot) do { } while (0)
#endif

constexpr int kBM = 128;          // features per tile (MMA M)
constexpr int kBK = 64;           // K elements per pipeline stage (128 bytes of bf16: one swizzle row)
constexpr int kMaxStages = 4;     // pipeline depth is chosen per launch (2..4) so that two CTAs fit on an SM when possible
constexpr int kThreads = 192;     // warp 0: TMA, warp 1: MMA + tensor-memory allocation, warps 2-5: epilogue
constexpr int kMaxBN = 128;       // tokens per CTA (MMA N), a multiple of 16
// Words between the top-1 keys of successive tokens: every key has a 128-byte line of its own.  Hundreds of
// tiles send one atomic max per token; keys that share a line queue behind one another in L2.
constexpr int kBestStride = 16;
constexpr unsigned long long kSpinCycles = 2000000000ull;   // about a second

enum TcEpilogue {
  kTcPlanes = 0,    // out planes (hi, lo) = split(act(v + bias))
  kTcF32 = 1,       // out fp32 = act(v + bias)
  kTcResidual = 2,  // x fp32 += v + bias
  kTcQkv = 3,       // n < d: q fp32; else key / value (bf16) into the paged cache
  kTcHeadOut = 4,   // out planes = split(v + bias + h[t][n mod d])
  kTcArgmax = 5     // per-token top-1 over all features (two-level merge), optional logits dump
};

struct TcParams {
  int T, N, K;                 // tokens in this launch, features, reduction length
  int bn;                      // MMA N: T rounded up to 16 (per token tile)
  int splits;                  // grid.y
  int chunks_per_split;        // K chunks (of kBK) each split owns
  const bf16* bias;            // [N] or null
  int relu;
  // outputs
  bf16* out_hi; long long plane; long long ldo;   // planes: lo plane = hi + plane
  float* out_f32;              // kTcF32 / kTcResidual / kTcQkv(q): [T, ldo]
  const float* h; int d;       // kTcHeadOut residual; kTcQkv model width
  int head_identity;
  int zofs_n;                  // column offset of this z-slice inside the output row (block-diagonal heads)
  bf16* kcache; bf16* vcache;  // kTcQkv
  RowState st; int rows_per_b;
  // split-K workspace
  float* ws;                   // [z][tile][split][bn][128]
  unsigned* tile_counters;     // [z][tiles]
  // top-1
  unsigned long long* best;         // [T][kBestStride] packed (orderable value, ~index) in the first word of each
                                    // token's 128 bytes, zero between launches
  unsigned* done_counter;           // [1]
  int* out_idx; float* out_val; float* logits;
  RankState rank; int rank_kh;      // top-n acceptance: count entries beating each proposal (rank.cnt null = off)
  // layer norm folded into the projection: the activation planes hold x * gain (not normalised); the
  // epilogue finishes y = rstd * (acc - mean * ln_s[n]) + ln_c[n] with per-token statistics of ln_x
  const float* ln_x; int ln_d; float ln_eps;   // residual stream [rows, ln_d] fp32, or null
  const float* ln_s; const float* ln_c;        // [N]: sum_c gain_c w[n][c]  and  sum_c shift_c w[n][c] + bias[n]
  // kTcResidual: also write planes of the updated stream times the next layer norm's gain
  const bf16* g_next; bf16* xg_hi; long long xg_plane;
  // Wide token tiles (more than 16 tokens) cannot afford to read whole rows of the residual stream for the folded
  // layer norm.  There the kernel that updates the stream also writes, per (128-feature tile, token), the mean and
  // the sum of squared deviations of its 128 new values (stat_out, [tiles][stat_T][2]); the projection that
  // consumes the normalised stream merges the stat_parts tiles of a token in tile order (stat_in).
  float* stat_out; const float* stat_in; int stat_parts; int stat_T;
#ifdef BPD_TC_TRACE
  int trace_id;
#endif
  int* error;                  // device error word
  const int* all_done;
  int stream_weights;          // 1: the weights are read once per launch (one token tile): load them "evict first"
  int vec;                     // 1: wide token tiles finish through shared memory with 8- and 16-byte stores (the
                               // host has checked sizes and alignment)
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// Bounded wait: false if the phase did not complete within about a second.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_cycles = kSpinCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if ((unsigned long long)(clock64() - t0) > limit_cycles) return false;
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// Same with an L2 policy: weights that are read once per pass are marked "evict first", so that streaming
// hundreds of MB through the 126 MB L2 does not push out what every pass reads again (caches, small vectors).
__device__ __forceinline__ unsigned long long l2_evict_first() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                                 unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(policy) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffff) >> 4);          // start address, 16-byte units
  d |= (uint64_t)1 << 16;                           // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                 // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                           // descriptor version
  d |= (uint64_t)2 << 61;                           // layout: 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

// (value, index) packed so that an unsigned 64-bit max picks the larger value and, among equal values, the
// lower index.  Zero is below every real entry.
__device__ __forceinline__ unsigned long long pack_best(float v, int idx) {
  const unsigned b = __float_as_uint(v);
  const unsigned ord = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return ((unsigned long long)ord << 32) | (unsigned long long)(0xffffffffu - (unsigned)idx);
}
__device__ __forceinline__ float unpack_value(unsigned long long key) {
  const unsigned ord = (unsigned)(key >> 32);
  return __uint_as_float((ord & 0x80000000u) ? (ord & 0x7fffffffu) : ~ord);
}

// Warp-wide (value, index) maximum with ties to the lower index, for lanes whose indices grow with the lane
// number: one integer max-reduction on the orderable pattern of the value, one ballot for the first lane that
// holds it -- instead of a five-level shuffle butterfly on two registers.
__device__ __forceinline__ void warp_argmax_lanes(float& v, int& idx) {
  const unsigned b = __float_as_uint(v);
  const unsigned ord = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  const unsigned m = __reduce_max_sync(0xffffffffu, ord);
  const int src = __ffs(__ballot_sync(0xffffffffu, ord == m)) - 1;
  idx = __shfl_sync(0xffffffffu, idx, src);
  v = __uint_as_float((m & 0x80000000u) ? (m & 0x7fffffffu) : ~m);
}

// Arrival on a device-wide counter with release (our earlier writes, and those of the CTA's other threads
// ordered before us by the barrier, become visible) and acquire (we see what earlier arrivals released).
__device__ __forceinline__ unsigned atom_add_acq_rel(unsigned* addr, unsigned v) {
  unsigned old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(addr), "r"(v) : "memory");
  return old;
}

// Top-n acceptance: among this warp's 32 features, how many beat the proposal that follows token t's position.
__device__ __forceinline__ void count_beats(const TcParams& p, int t, int n, float x, int lane) {
  if (!p.rank.cnt || t >= p.T || (t % p.rank_kh) != 0) return;   // uniform over the warp
  const int pr = t / p.rank_kh, tok = p.rank.tok[pr];
  const bool beat = tok >= 0 && n < p.N && n != tok && better(x, n, p.rank.thr[pr], tok);
  const unsigned m = __ballot_sync(0xffffffffu, beat);
  if (lane == 0 && m) atomicAdd(&p.rank.cnt[pr], __popc(m));
}

__device__ __forceinline__ void split_bf16(float v, bf16& hi, bf16& lo) {
  hi = __float2bfloat16_rn(v);
  lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Shared-memory footprint of one CTA.
__host__ __device__ inline size_t stage_bytes(int bn) { return (size_t)kBM * 128 + 2 * (size_t)bn * 128; }
__host__ __device__ inline int stages_for(int bn) { return bn <= 16 ? 5 : (bn <= 32 ? 4 : (bn <= 64 ? 3 : 4)); }
__host__ __device__ inline size_t smem_bytes(int bn) { return stages_for(bn) * stage_bytes(bn) + 1024 /*alignment*/ + 256; }

// ---------------------------------------------------------------- final epilogue for one (feature, token)
// Finishes up to 8 tokens of one feature.  Everything that has to be read (old residual values, the head
// residual, cache slots) is fetched for all tokens first, so the loads overlap instead of queueing behind
// the stores of the previous token.
template <int EPI>
__device__ __forceinline__ void tc_store8(const TcParams& p, int z, int t_first, int ntok, int n, const float (&vin)[8],
                                          const float* s_mean, const float* s_rstd, int stat0,
                                          const unsigned long long* s_slot) {
  float lns = 0.f, lnc = 0.f, bias = 0.f, gnext = 0.f;
  if (p.ln_x) { lns = p.ln_s[n]; lnc = p.ln_c[n]; }
  else if (p.bias) bias = __bfloat162float(p.bias[n + p.zofs_n * z]);
  if (EPI == kTcResidual && p.g_next) gnext = __bfloat162float(p.g_next[n]);
  float pre[8];
  const bool need_old = (EPI == kTcResidual) && p.g_next != nullptr;   // otherwise the add is a fire-and-forget reduction
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    pre[c] = 0.f;
    if (c < ntok) {
      const int t = t_first + c;
      if (need_old) pre[c] = p.out_f32[(long long)t * p.ldo + n];
      if (EPI == kTcHeadOut) pre[c] = __ldg(&p.h[(size_t)t * p.d + (n % p.d)]);
    }
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    if (c < ntok) {
      const int t = t_first + c;
      float v = vin[c];
      if (p.ln_x) v = s_rstd[(stat0 + c) & 15] * (v - s_mean[(stat0 + c) & 15] * lns) + lnc;
      else v += bias;
      if (p.relu) v = fmaxf(v, 0.f);
      if (EPI == kTcPlanes) {
        bf16 hi, lo;
        split_bf16(v, hi, lo);
        const long long o = (long long)t * p.ldo + n + (long long)p.zofs_n * z;
        p.out_hi[o] = hi;
        p.out_hi[o + p.plane] = lo;
      } else if (EPI == kTcF32) {
        p.out_f32[(long long)t * p.ldo + n] = v;
      } else if (EPI == kTcResidual) {
        if (!need_old) {
          atomicAdd(&p.out_f32[(long long)t * p.ldo + n], v);   // single writer per element: just x += v without a read
          continue;
        }
        const float xnew = pre[c] + v;
        p.out_f32[(long long)t * p.ldo + n] = xnew;
        if (p.g_next) {
          bf16 hi, lo;
          split_bf16(xnew * gnext, hi, lo);
          p.xg_hi[(long long)t * p.ldo + n] = hi;
          p.xg_hi[(long long)t * p.ldo + n + p.xg_plane] = lo;
        }
      } else if (EPI == kTcHeadOut) {
        const int nz = n + p.zofs_n * z;
        v = (p.head_identity && nz < p.d) ? pre[c] : v + pre[c];
        bf16 hi, lo;
        split_bf16(v, hi, lo);
        const long long o = (long long)t * p.ldo + nz;
        p.out_hi[o] = hi;
        p.out_hi[o + p.plane] = lo;
      } else if (EPI == kTcQkv) {
        const int d = p.d;
        if (n < d) p.out_f32[(long long)t * p.ldo + n] = v;
        else if (n < 2 * d) p.kcache[s_slot[stat0 + c] + (n - d)] = __float2bfloat16_rn(v);
        else p.vcache[s_slot[stat0 + c] + (n - 2 * d)] = __float2bfloat16_rn(v);
      }
    }
  }
}

// ---------------------------------------------------------------- final epilogue of a wide tile
// The tile lies in shared memory with one row per token (row stride tstride floats, a multiple of 4).  An item is
// (token, four consecutive features); the 128 epilogue threads take the items in order, so a warp finishes 128
// consecutive features of a token with one 16-byte (fp32) or 8-byte (bf16) access per lane instead of 32-lane
// scalar stores per token.  Same arithmetic per element as tc_store8 (no folded layer norm here).
__device__ __forceinline__ uint2 pack4_bf16(const bf16 (&b)[4]) {
  return make_uint2((uint32_t)__bfloat16_as_ushort(b[0]) | ((uint32_t)__bfloat16_as_ushort(b[1]) << 16),
                    (uint32_t)__bfloat16_as_ushort(b[2]) | ((uint32_t)__bfloat16_as_ushort(b[3]) << 16));
}
// A 16-byte load from L2 that stays where it is written: the compiler otherwise sinks such loads to their first use,
// which turns a batch of independent loads into a chain of round trips.
__device__ __forceinline__ float4 ld_cg_v4_here(const float* ptr) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr) : "memory");
  return v;
}

// Per-thread constants of an item's four features.
struct FinishCtx {
  float bias[4], gn[4], lns[4];
  bool folded;     // y = rstd * (acc - mean * ln_s) + ln_c; ln_c holds the bias
  int n, g;
};
template <int EPI>
__device__ __forceinline__ bool tc_finish_setup(const TcParams& p, int z, int tile, int et, FinishCtx& c) {
  c.g = et & 31;
  c.n = tile * kBM + c.g * 4;                       // first of this item's four features (within the slice)
  if (c.n >= p.N) return false;
#pragma unroll
  for (int e = 0; e < 4; ++e) { c.bias[e] = 0.f; c.gn[e] = 0.f; c.lns[e] = 0.f; }
  c.folded = (p.stat_in != nullptr);
  if (c.folded) {
    const float4 s4 = *reinterpret_cast<const float4*>(p.ln_s + c.n), c4 = *reinterpret_cast<const float4*>(p.ln_c + c.n);
    c.lns[0] = s4.x; c.lns[1] = s4.y; c.lns[2] = s4.z; c.lns[3] = s4.w;
    c.bias[0] = c4.x; c.bias[1] = c4.y; c.bias[2] = c4.z; c.bias[3] = c4.w;
  } else if (p.bias) {
    const uint2 bw = *reinterpret_cast<const uint2*>(p.bias + c.n + p.zofs_n * z);
    c.bias[0] = __uint_as_float(bw.x << 16); c.bias[1] = __uint_as_float(bw.x & 0xffff0000u);
    c.bias[2] = __uint_as_float(bw.y << 16); c.bias[3] = __uint_as_float(bw.y & 0xffff0000u);
  }
  if (EPI == kTcResidual && p.g_next) {
    const uint2 gw = *reinterpret_cast<const uint2*>(p.g_next + c.n);
    c.gn[0] = __uint_as_float(gw.x << 16); c.gn[1] = __uint_as_float(gw.x & 0xffff0000u);
    c.gn[2] = __uint_as_float(gw.y << 16); c.gn[3] = __uint_as_float(gw.y & 0xffff0000u);
  }
  return true;
}
// Finishes one item: token t (row tr of the tile), features c.n .. c.n + 3, accumulated values a; `old` is the
// residual stream's current content (only read by the caller when the new value is needed: residual with g_next).
template <int EPI>
__device__ __forceinline__ void tc_finish_item(const TcParams& p, const FinishCtx& c, int z, int t, int tr, const float4& a,
                                               float4& old, const unsigned long long* s_slot, const float* s_mean,
                                               const float* s_rstd) {
  const int n = c.n;
  float v[4] = {a.x + c.bias[0], a.y + c.bias[1], a.z + c.bias[2], a.w + c.bias[3]};
  if (c.folded) {
    const float mu = s_mean[tr], rs = s_rstd[tr];
    v[0] = rs * (a.x - mu * c.lns[0]) + c.bias[0]; v[1] = rs * (a.y - mu * c.lns[1]) + c.bias[1];
    v[2] = rs * (a.z - mu * c.lns[2]) + c.bias[2]; v[3] = rs * (a.w - mu * c.lns[3]) + c.bias[3];
  }
  if (p.relu) {
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = fmaxf(v[e], 0.f);
  }
  if (EPI == kTcPlanes || EPI == kTcHeadOut) {
    const int nz = n + p.zofs_n * z;
    if (EPI == kTcHeadOut) {
      const float4 h = __ldg(reinterpret_cast<const float4*>(p.h + (size_t)t * p.d + (n % p.d)));
      const float pre[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) v[e] = (p.head_identity && nz < p.d) ? pre[e] : v[e] + pre[e];
    }
    bf16 hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) split_bf16(v[e], hi[e], lo[e]);
    const long long o = (long long)t * p.ldo + nz;
    *reinterpret_cast<uint2*>(p.out_hi + o) = pack4_bf16(hi);
    *reinterpret_cast<uint2*>(p.out_hi + o + p.plane) = pack4_bf16(lo);
  } else if (EPI == kTcF32) {
    *reinterpret_cast<float4*>(p.out_f32 + (long long)t * p.ldo + n) = make_float4(v[0], v[1], v[2], v[3]);
  } else if (EPI == kTcResidual) {
    float4* xp = reinterpret_cast<float4*>(p.out_f32 + (long long)t * p.ldo + n);
    if (!p.g_next) {
      // one writer per element: x += v as a 16-byte reduction, nothing to read back
      asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(xp), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
      return;
    }
    const float xn[4] = {old.x + v[0], old.y + v[1], old.z + v[2], old.w + v[3]};
    *xp = make_float4(xn[0], xn[1], xn[2], xn[3]);
    {
      bf16 hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) split_bf16(xn[e] * c.gn[e], hi[e], lo[e]);
      *reinterpret_cast<uint2*>(p.xg_hi + (long long)t * p.ldo + n) = pack4_bf16(hi);
      *reinterpret_cast<uint2*>(p.xg_hi + (long long)t * p.ldo + n + p.xg_plane) = pack4_bf16(lo);
    }
    old = make_float4(xn[0], xn[1], xn[2], xn[3]);   // handed back for the per-tile statistics
  } else if (EPI == kTcQkv) {
    const int d = p.d;
    if (n < d) {
      *reinterpret_cast<float4*>(p.out_f32 + (long long)t * p.ldo + n) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
      const bf16 b4[4] = {__float2bfloat16_rn(v[0]), __float2bfloat16_rn(v[1]), __float2bfloat16_rn(v[2]), __float2bfloat16_rn(v[3])};
      bf16* dst = (n < 2 * d) ? p.kcache + s_slot[tr] + (n - d) : p.vcache + s_slot[tr] + (n - 2 * d);
      *reinterpret_cast<uint2*>(dst) = pack4_bf16(b4);
    }
  }
}
// Per-tile statistics of TB tokens at once (kTcResidual with stat_out): the warp holds the tile's 128 new values of
// each token, four per lane (N is a multiple of 128 here: every lane is live).  Sums of deviations from the token's
// first value in the tile, and of their squares, are reduced for all TB tokens together so that the shuffles of one
// token hide behind those of the others; mean and squared deviations about the mean follow exactly from the two.
template <int TB>
__device__ __forceinline__ void tc_tile_stats(const TcParams& p, const FinishCtx& c, int t0, int tb, int nt, const float4 (&xn)[TB]) {
  float s1[TB], s2[TB], pivot[TB];
#pragma unroll
  for (int i = 0; i < TB; ++i) {
    pivot[i] = __shfl_sync(0xffffffffu, xn[i].x, 0);
    const float d0 = xn[i].x - pivot[i], d1 = xn[i].y - pivot[i], d2 = xn[i].z - pivot[i], d3 = xn[i].w - pivot[i];
    s1[i] = (d0 + d1) + (d2 + d3);
    s2[i] = (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
    for (int i = 0; i < TB; ++i) {
      s1[i] += __shfl_xor_sync(0xffffffffu, s1[i], o);
      s2[i] += __shfl_xor_sync(0xffffffffu, s2[i], o);
    }
  }
  if (c.g == 0) {
#pragma unroll
    for (int i = 0; i < TB; ++i) {
      const int tr = tb + 4 * i;
      if (tr < nt) {
        const float dm = s1[i] * (1.0f / kBM);              // mean - pivot
        reinterpret_cast<float2*>(p.stat_out)[(size_t)(c.n / kBM) * p.stat_T + t0 + tr] =
            make_float2(pivot[i] + dm, fmaxf(s2[i] - s1[i] * dm, 0.f));
      }
    }
  }
}

// The complete tile lies in shared memory (one row per token).  Warp w of the four takes tokens w, w + 4, ...; four
// tokens are in flight per lane so that the loads of the old residual values overlap.
template <int EPI>
__device__ __forceinline__ void tc_finish_tile(const TcParams& p, int z, int t0, int nt, int tile, const float* s_t, int tstride,
                                               const unsigned long long* s_slot, int et, const float* s_mean,
                                               const float* s_rstd) {
  FinishCtx c;
  if (!tc_finish_setup<EPI>(p, z, tile, et, c)) return;
  const bool need_old = (EPI == kTcResidual) && p.g_next != nullptr;
  constexpr int TB = 4;
  for (int tb = et >> 5; tb < nt; tb += 4 * TB) {
    float4 old[TB];
#pragma unroll
    for (int i = 0; i < TB; ++i) {
      const int tr = tb + 4 * i;
      old[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (need_old && tr < nt) old[i] = ld_cg_v4_here(p.out_f32 + (long long)(t0 + tr) * p.ldo + c.n);
    }
#pragma unroll
    for (int i = 0; i < TB; ++i) {
      const int tr = tb + 4 * i;
      if (tr < nt) {
        const float4 a = *reinterpret_cast<const float4*>(s_t + tr * tstride + c.g * 4);
        tc_finish_item<EPI>(p, c, z, t0 + tr, tr, a, old[i], s_slot, s_mean, s_rstd);
      }
    }
    if (EPI == kTcResidual && p.stat_out) tc_tile_stats<TB>(p, c, t0, tb, nt, old);
  }
}
// The tile is the sum of `splits` partial tiles in the workspace ([split][token][128 features]): the CTA that
// arrived last adds them in split order and finishes the items straight from registers -- TB tokens x up to four
// splits of 16-byte loads (and the old residual values) are in flight per lane.
template <int EPI, int TB>
__device__ __forceinline__ void tc_merge_finish_tile(const TcParams& p, int z, int t0, int nt, int tile, const float* wsz, int bn,
                                                     const unsigned long long* s_slot, int et, const float* s_mean,
                                                     const float* s_rstd) {
  FinishCtx c;
  if (!tc_finish_setup<EPI>(p, z, tile, et, c)) return;
  const bool need_old = (EPI == kTcResidual) && p.g_next != nullptr;
  constexpr int SB = 16 / TB;                       // 16 partial loads in flight
  if (et == 0) BPD_TC_STAMP(8);
  for (int tb = et >> 5; tb < nt; tb += 4 * TB) {
    float4 old[TB], acc[TB];
#pragma unroll
    for (int i = 0; i < TB; ++i) {
      const int tr = tb + 4 * i;
      old[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (need_old && tr < nt) old[i] = ld_cg_v4_here(p.out_f32 + (long long)(t0 + tr) * p.ldo + c.n);
    }
    for (int s0 = 0; s0 < p.splits; s0 += SB) {
      float4 v[SB][TB];
#pragma unroll
      for (int ss = 0; ss < SB; ++ss)
#pragma unroll
        for (int i = 0; i < TB; ++i) {
          const int tr = tb + 4 * i;
          v[ss][i] = (s0 + ss < p.splits && tr < nt) ? ld_cg_v4_here(wsz + ((size_t)(s0 + ss) * bn + tr) * kBM + c.g * 4)
                                                      : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
      for (int ss = 0; ss < SB; ++ss)
#pragma unroll
        for (int i = 0; i < TB; ++i) {
          acc[i].x += v[ss][i].x; acc[i].y += v[ss][i].y; acc[i].z += v[ss][i].z; acc[i].w += v[ss][i].w;
        }
    }
#pragma unroll
    for (int i = 0; i < TB; ++i) {
      const int tr = tb + 4 * i;
      if (tr < nt) tc_finish_item<EPI>(p, c, z, t0 + tr, tr, acc[i], old[i], s_slot, s_mean, s_rstd);
    }
    if (EPI == kTcResidual && p.stat_out) tc_tile_stats<TB>(p, c, t0, tb, nt, old);
  }
  if (et == 0) BPD_TC_STAMP(12);
}

// ---------------------------------------------------------------- bounded-wait self test
// One CTA waits on an mbarrier that nothing ever arrives on, gives up after `limit_cycles`, records the same
// error code the projection kernel would and returns normally: the context stays usable.
static __global__ void wait_probe_kernel(int* error, unsigned long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait(b, 0, limit_cycles)) atomicCAS(error, 0, 103);
  }
}

// Top-1 epilogue: threads that share a token (a power of two, at most 8, with tpt * bn <= 128).
__host__ __device__ inline int topk_threads_per_token(int bn) { return bn <= 16 ? 8 : (bn <= 32 ? 4 : (bn <= 64 ? 2 : 1)); }

// ---------------------------------------------------------------- epilogue of one (tile, split) unit
// Shared by the one-shot projection kernel and the persistent layer kernel.  Called by the four epilogue warps
// (128 threads, named barrier 1).
struct EpiShared {
  float* s_t;                   // top-1: the tile transposed, [token][128 features], rows of topk_stride() floats
  float* s_mean; float* s_rstd;
  unsigned long long* s_slot;
  volatile uint32_t* ctl;       // [1] reduces the tile, [2] merges the top-1, [3] accumulator arrived
};
struct EpiUnit {
  uint32_t tmem, acc_bar, acc_parity;
  int tile, split, slice, zidx, ntiles, zcount, t0, nt, bn, nchunks;
  bool skip;
};
// WIDE: the launch has token tiles of 32 or more tokens.  Everything that only such tiles use (the way out through
// shared memory, per-tile statistics, the merge that finishes items from registers) is compiled into that variant
// alone, so that the few-row launches of the weight-streaming kernels carry none of it.
template <int EPI, bool WIDE>
__device__ __forceinline__ void tc_epilogue(const TcParams& p, const EpiShared& sh, const EpiUnit& u, int warp, int lane) {
  float* s_t = sh.s_t;
  float* s_mean = sh.s_mean;
  float* s_rstd = sh.s_rstd;
  unsigned long long* s_slot = sh.s_slot;
  volatile uint32_t* ctl = sh.ctl;
  const uint32_t tmem = u.tmem;
  const int tile = u.tile, split = u.split, slice = u.slice, t0 = u.t0, nt = u.nt, bn = u.bn, nchunks = u.nchunks;
  const bool skip = u.skip;
  const int q = warp & 3;                          // tensor-memory lane quarter this warp may read
  const int row = q * 32 + lane;
  const int n = tile * kBM + row;                  // feature index within the slice
  const int et = threadIdx.x - 64;                 // 0..127
  const int tpt = topk_threads_per_token(bn), tstride = kBM + tpt;   // row stride = tpt mod 32: conflict-free scans
  // the debug dump of the logits and the rank counting of top-n acceptance are rare: kept out of the common loops
  const bool extras = (EPI == kTcArgmax) && (p.logits != nullptr || p.rank.cnt != nullptr);
  // wide tiles of the other epilogues leave through shared memory too (see tc_finish_tile)
  const bool vec = WIDE && (EPI != kTcArgmax) && p.vec && bn >= 32 && !p.ln_x;   // a folded layer norm on wide tiles comes with stat_in
  constexpr int vstride = kBM + 4;
  if (EPI == kTcQkv && !skip && et < nt) {
    const int t = t0 + et;
    const int b = t / p.rows_per_b, i = t % p.rows_per_b;
    const int pos = p.st.len[b] + i;
    const int page = p.st.page_table[b * p.st.pages_per_row + pos / kPage];
    s_slot[et] = ((unsigned long long)page * kPage + (pos % kPage)) * p.d;
  }
  if (WIDE && p.stat_in && !skip && et < nt) {
    // per-token statistics from the per-tile partial results of the kernel that wrote the stream: merged in
    // tile order (pairwise update of mean and sum of squared deviations), the same for every consumer
    const float2* sp = reinterpret_cast<const float2*>(p.stat_in) + (t0 + et);
    float2 part[8];
    float mean = 0.f, m2 = 0.f, cnt = 0.f;
    for (int i0 = 0; i0 < p.stat_parts; i0 += 8) {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (i0 + i < p.stat_parts) part[i] = __ldcg(sp + (size_t)(i0 + i) * p.stat_T);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (i0 + i < p.stat_parts) {
          const float nb = (float)kBM, tot = cnt + nb;
          const float delta = part[i].x - mean;
          mean += delta * (nb / tot);
          m2 += part[i].y + delta * delta * (cnt * nb / tot);
          cnt = tot;
        }
      }
    }
    s_mean[et] = mean;
    s_rstd[et] = rsqrtf(m2 / cnt + p.ln_eps);
  }
  if (p.ln_x && !skip) {
    // per-token mean and 1/std of the residual stream, computed while the main loop runs: 8 threads per
    // token (at most 16 tokens per tile in this mode), two passes, fixed order
    const int tr = et >> 3, part = et & 7;
    const int trc = min(tr, nt - 1);               // threads beyond the live tokens shadow the last one
    const float4* xr = reinterpret_cast<const float4*>(p.ln_x + (size_t)(t0 + trc) * p.ln_d);
    const int nv = p.ln_d >> 2;
    float sum = 0.f;
#pragma unroll 8
    for (int i = part; i < nv; i += 8) { const float4 a = xr[i]; sum += (a.x + a.y) + (a.z + a.w); }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    sum += __shfl_xor_sync(0xffffffffu, sum, 4);
    const float mean = sum / (float)p.ln_d;
    float sq = 0.f;
#pragma unroll 8
    for (int i = part; i < nv; i += 8) {
      const float4 a = xr[i];
      const float d0 = a.x - mean, d1 = a.y - mean, d2 = a.z - mean, d3 = a.w - mean;
      sq += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
    }
    sq += __shfl_xor_sync(0xffffffffu, sq, 1);
    sq += __shfl_xor_sync(0xffffffffu, sq, 2);
    sq += __shfl_xor_sync(0xffffffffu, sq, 4);
    const float rstd = rsqrtf(sq / (float)p.ln_d + p.ln_eps);
    if (part == 0 && tr < nt) { s_mean[tr] = mean; s_rstd[tr] = rstd; }
  }
  // one thread waits for the accumulator; the other 127 learn the outcome through the named barrier
  if (et == 0) {
    bool done = !skip;
    if (nchunks > 0 && !skip) done = mbar_wait(u.acc_bar, u.acc_parity);
    if (!done && !skip) atomicCAS(p.error, 0, 103);
    ctl[3] = done ? 1u : 0u;
    BPD_TC_STAMP(5);
  }
  asm volatile("bar.sync 1, 128;" ::: "memory");
  const bool ok = (ctl[3] != 0);
  tc_fence_after();
  const int ntiles = u.ntiles;
  const bool direct = (p.splits == 1);
  float* wsz = p.ws + ((size_t)u.zidx * ntiles + tile) * p.splits * (size_t)bn * kBM;
  if (ok) {
    if (direct) {
      for (int cb = 0; cb < bn; cb += 16) {
        float v[16];
        tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + cb, v);
        if (EPI != kTcArgmax && vec) {
#pragma unroll
          for (int c = 0; c < 16; ++c) s_t[(cb + c) * vstride + row] = v[c];
        } else if (EPI != kTcArgmax) {
          if (n < p.N) {
            const float lo8[8] = {v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7]};
            const float hi8[8] = {v[8], v[9], v[10], v[11], v[12], v[13], v[14], v[15]};
            tc_store8<EPI>(p, slice, t0 + cb, min(8, nt - cb), n, lo8, s_mean, s_rstd, cb, s_slot);
            tc_store8<EPI>(p, slice, t0 + cb + 8, min(8, nt - cb - 8), n, hi8, s_mean, s_rstd, cb + 8, s_slot);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c) s_t[(cb + c) * tstride + row] = (n < p.N) ? v[c] : -INFINITY;
          if (extras) {
#pragma unroll
            for (int c = 0; c < 16; ++c) {
              if (p.logits && cb + c < nt && n < p.N) p.logits[(size_t)(t0 + cb + c) * p.N + n] = v[c];
              if (cb + c < nt) count_beats(p, t0 + cb + c, n, (n < p.N) ? v[c] : -INFINITY, lane);
            }
          }
        }
      }
    } else {
      // partial tile -> workspace [split][token][128], coalesced over features
      for (int cb = 0; cb < bn; cb += 16) {
        float v[16];
        if (nchunks > 0) tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + cb, v);
        else {
#pragma unroll
          for (int c = 0; c < 16; ++c) v[c] = 0.f;
        }
#pragma unroll
        for (int c = 0; c < 16; ++c)
          if (cb + c < nt) wsz[((size_t)split * bn + cb + c) * kBM + row] = v[c];
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et == 0) {
        BPD_TC_STAMP(6);
        const unsigned prev = atom_add_acq_rel(&p.tile_counters[(size_t)u.zidx * ntiles + tile], 1u);
        ctl[1] = (prev == (unsigned)p.splits - 1) ? 1u : 0u;
        BPD_TC_STAMP(7);
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ctl[1]) {
        // Splits are added in split order.  The partial tiles sit in L2 and every load is a round trip of about a
        // microsecond, so as many as the registers hold are issued together: G tokens x SB splits = 64 per thread.
        auto emit8 = [&](const float (&acc)[8], int cg) {
          if (EPI != kTcArgmax && vec) {
#pragma unroll
            for (int c = 0; c < 8; ++c)
              if (cg + c < nt) s_t[(cg + c) * vstride + row] = acc[c];
          } else if (EPI != kTcArgmax) {
            if (n < p.N) tc_store8<EPI>(p, slice, t0 + cg, min(8, nt - cg), n, acc, s_mean, s_rstd, cg, s_slot);
          } else {
#pragma unroll
            for (int c = 0; c < 8; ++c)
              if (cg + c < nt) s_t[(cg + c) * tstride + row] = (n < p.N) ? acc[c] : -INFINITY;
            if (extras) {
#pragma unroll
              for (int c = 0; c < 8; ++c) {
                if (cg + c >= nt) break;
                if (p.logits && n < p.N) p.logits[(size_t)(t0 + cg + c) * p.N + n] = acc[c];
                count_beats(p, t0 + cg + c, n, (n < p.N) ? acc[c] : -INFINITY, lane);
              }
            }
          }
        };
        auto merge = [&](auto g_tag, auto sb_tag) {
          constexpr int G = decltype(g_tag)::value, SB = decltype(sb_tag)::value;
          for (int cg = 0; cg < nt; cg += G) {
            float acc[G];
#pragma unroll
            for (int c = 0; c < G; ++c) acc[c] = 0.f;
            for (int s0 = 0; s0 < p.splits; s0 += SB) {
              float v[SB][G];
#pragma unroll
              for (int ss = 0; ss < SB; ++ss)
#pragma unroll
                for (int c = 0; c < G; ++c)
                  v[ss][c] = (s0 + ss < p.splits && cg + c < nt)
                                 ? __ldcg(&wsz[((size_t)(s0 + ss) * bn + cg + c) * kBM + row]) : 0.f;
#pragma unroll
              for (int ss = 0; ss < SB; ++ss)
#pragma unroll
                for (int c = 0; c < G; ++c) acc[c] += v[ss][c];
            }
#pragma unroll
            for (int g8 = 0; g8 < G; g8 += 8) {
              if (cg + g8 < nt) {
                const float a8[8] = {acc[g8], acc[g8 + 1], acc[g8 + 2], acc[g8 + 3], acc[g8 + 4], acc[g8 + 5], acc[g8 + 6], acc[g8 + 7]};
                emit8(a8, cg + g8);
              }
            }
          }
        };
        if (WIDE && EPI != kTcArgmax && vec) {
          tc_merge_finish_tile<EPI, 4>(p, slice, t0, nt, tile, wsz, bn, s_slot, et, s_mean, s_rstd);
        } else if (!WIDE || nt <= 8) merge(std::integral_constant<int, 8>{}, std::integral_constant<int, 8>{});
        else if (p.splits <= 2) merge(std::integral_constant<int, 32>{}, std::integral_constant<int, 2>{});
        else if (p.splits <= 4) merge(std::integral_constant<int, 16>{}, std::integral_constant<int, 4>{});
        else merge(std::integral_constant<int, 8>{}, std::integral_constant<int, 8>{});
        if (et == 0) p.tile_counters[(size_t)u.zidx * ntiles + tile] = 0;   // ready for the next launch
      }
    }
    if (WIDE && EPI != kTcArgmax && vec && direct) {
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et == 0) BPD_TC_STAMP(8);
      tc_finish_tile<EPI>(p, slice, t0, nt, tile, s_t, vstride, s_slot, et, s_mean, s_rstd);
    }
    if (EPI == kTcArgmax && (direct || ctl[1])) {
      // The tile sits in shared memory with one row per token.  tpt threads share a token: each scans every
      // tpt-th feature in ascending order (a strict comparison keeps the lowest index among equals), then the
      // tpt partial results are merged with the same ordering.  No shuffle per token, no work for absent tokens.
      // Then the CTA that completes the last tile merges all tiles.
      asm volatile("bar.sync 1, 128;" ::: "memory");
      {
        const int token = et / tpt, part = et % tpt;            // tokens >= bn do not occur: tpt * bn <= 128
        const float* rowp = s_t + token * tstride;
        float x = -INFINITY;
        int ix = 0x7fffffff;
        if (token < nt) {
          // four independent running maxima (features part + tpt * (4j + a)), merged by (value, lower index)
          float xa[4];
          int ia[4];
#pragma unroll
          for (int a = 0; a < 4; ++a) { ia[a] = part + tpt * a; xa[a] = rowp[ia[a]]; }
          for (int f = part + 4 * tpt; f < kBM; f += 4 * tpt) {
#pragma unroll
            for (int a = 0; a < 4; ++a) {
              const float y = rowp[f + tpt * a];
              if (y > xa[a]) { xa[a] = y; ia[a] = f + tpt * a; }
            }
          }
          x = xa[0];
          ix = ia[0];
#pragma unroll
          for (int a = 1; a < 4; ++a)
            if (better(xa[a], ia[a], x, ix)) { x = xa[a]; ix = ia[a]; }
          ix = (tile * kBM + ix < p.N) ? tile * kBM + ix : 0x7fffffff;
        }
        for (int o = 1; o < tpt; o <<= 1) {                     // partners are neighbouring lanes of one warp
          const float ov = __shfl_xor_sync(0xffffffffu, x, o);
          const int oi = __shfl_xor_sync(0xffffffffu, ix, o);
          if (better(ov, oi, x, ix)) { x = ov; ix = oi; }
        }
        // one 64-bit atomic max per (tile, token): larger value wins, equal values go to the lower index;
        // max is order independent, so the result does not depend on which tile arrives first
        if (token < nt && part == 0) atomicMax(&p.best[(size_t)(t0 + token) * kBestStride], pack_best(x, ix));
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et == 0) {
        const unsigned prev = atom_add_acq_rel(p.done_counter, 1u);
        ctl[2] = (prev == (unsigned)(ntiles * u.zcount) - 1) ? 1u : 0u;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ctl[2]) {
        for (int t = et; t < p.T; t += 128) {
          const unsigned long long key = __ldcg(&p.best[(size_t)t * kBestStride]);
          p.out_idx[t] = (int)(0xffffffffu - (unsigned)(key & 0xffffffffull));
          if (p.out_val) p.out_val[t] = unpack_value(key);
          p.best[(size_t)t * kBestStride] = 0ull;                       // ready for the next launch
        }
        if (et == 0) *p.done_counter = 0;
      }
    }
  }
}

// ---------------------------------------------------------------- the kernel
// grid = (feature tiles, K splits, z), z = token tile * zslices + slice (slices: block-diagonal heads).
// tmA: weights [N, K]; tmBh / tmBl: activation planes [rows, K]; box = (64, 128) and (64, bn).
template <int EPI, bool WIDE>
__global__ void __launch_bounds__(kThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmBh,
               const __grid_constant__ CUtensorMap tmBl, TcParams p, int zslices, int a_rows_per_slice,
               int b_cols_per_slice) {
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    BPD_TC_STAMP(0);
#ifdef BPD_TC_TRACE
    if (g_tc_trace && blockIdx.x + blockIdx.y + blockIdx.z == 0) {
      unsigned long long* h = g_tc_trace + ((size_t)p.trace_id * 2048 + 2047) * 16;
      h[10] = EPI; h[11] = p.N; h[12] = p.K; h[13] = p.T; h[14] = p.splits;
      h[15] = gridDim.x | (gridDim.y << 12) | ((unsigned long long)gridDim.z << 24) | ((unsigned long long)p.bn << 40);
    }
#endif
  }
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;      // swizzled tiles need 1024-byte alignment
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const int bn = p.bn;
  const int kStages = stages_for(bn);
  const uint32_t stage_sz = (uint32_t)stage_bytes(bn);
  const uint32_t bars = base + kStages * stage_sz;                   // full[kStages], empty[kStages], accum
  volatile uint32_t* ctl = reinterpret_cast<volatile uint32_t*>(gen_base + kStages * stage_sz + 128);
  // ctl[0] = tensor-memory base, ctl[1] = "this CTA reduces the tile", ctl[2] = "this CTA merges the top-1",
  // ctl[3] = "the accumulator arrived"
  __shared__ float s_mean[WIDE ? kMaxBN : 16], s_rstd[WIDE ? kMaxBN : 16];
  __shared__ unsigned long long s_slot[kMaxBN];   // kTcQkv: cache slot (element offset) of every token of the tile

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int ttile = blockIdx.z / zslices, slice = blockIdx.z % zslices;
  const int t0 = ttile * bn;
  const int nt = min(bn, p.T - t0);                                  // live tokens in this tile
  const int total_chunks = (p.K + kBK - 1) / kBK;
  const int c0 = split * p.chunks_per_split;
  const int c1 = min(total_chunks, c0 + p.chunks_per_split);
  const int nchunks = max(0, c1 - c0);
  const uint32_t ncols = bn <= 32 ? 32u : (bn <= 64 ? 64u : 128u);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bars + 8 * s, 1);
      mbar_init(bars + 8 * (kStages + s), 1);
    }
    mbar_init(bars + 8 * 2 * kStages, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    ctl[1] = 0;
    ctl[2] = 0;
  }
  if (warp == 1) tmem_alloc(base + kStages * stage_sz + 128, ncols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl[0];
  bool ok = true;
  if (threadIdx.x == 0) BPD_TC_STAMP(1);

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer.  Weights do not depend on the preceding kernel: the first stages'
    // weight tiles are requested before waiting for it; activations only after.
    const int a_row = slice * a_rows_per_slice + tile * kBM;
    const int npre = min(nchunks, kStages);
    for (int it = 0; it < npre; ++it) {
      mbar_expect_tx(bars + 8 * it, stage_sz);
      if (p.stream_weights) tma_load_2d_hint(base + it * stage_sz, &tmA, bars + 8 * it, (c0 + it) * kBK, a_row, l2_evict_first());
      else tma_load_2d(base + it * stage_sz, &tmA, bars + 8 * it, (c0 + it) * kBK, a_row);
    }
    pdl_wait();
    BPD_TC_STAMP(2);
    const bool skip = p.all_done && *p.all_done;
    for (int it = 0; it < npre; ++it) {
      const uint32_t sa = base + it * stage_sz;
      const int kx = slice * b_cols_per_slice + (c0 + it) * kBK;
      tma_load_2d(sa + kBM * 128, &tmBh, bars + 8 * it, kx, t0);
      tma_load_2d(sa + kBM * 128 + bn * 128, &tmBl, bars + 8 * it, kx, t0);
    }
    int issued = npre;
    for (int it = npre; it < nchunks && !skip; ++it) {
      const int s = it % kStages;
      const uint32_t ph = (it / kStages) & 1;
      if (!mbar_wait(bars + 8 * (kStages + s), ph ^ 1)) { ok = false; break; }
      issued = it + 1;
      const uint32_t full = bars + 8 * s;
      const uint32_t sa = base + s * stage_sz;
      mbar_expect_tx(full, stage_sz);
      const int kx = (c0 + it) * kBK;
      if (p.stream_weights) tma_load_2d_hint(sa, &tmA, full, kx, a_row, l2_evict_first());
      else tma_load_2d(sa, &tmA, full, kx, a_row);
      tma_load_2d(sa + kBM * 128, &tmBh, full, slice * b_cols_per_slice + kx, t0);
      tma_load_2d(sa + kBM * 128 + bn * 128, &tmBl, full, slice * b_cols_per_slice + kx, t0);
    }
    if (!ok) atomicCAS(p.error, 0, 101);
    if (!ok || skip) {
      // nobody will consume what is in flight: give it a bounded chance to land before shared memory goes away
      for (int it = max(0, issued - kStages); it < issued; ++it) mbar_wait(bars + 8 * (it % kStages), (it / kStages) & 1);
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = instr_desc_bf16(bn);
    pdl_wait();
    const bool skip = p.all_done && *p.all_done;
    for (int it = 0; it < nchunks && !skip; ++it) {
      const int s = it % kStages;
      const uint32_t ph = (it / kStages) & 1;
      if (!mbar_wait(bars + 8 * s, ph)) { ok = false; break; }
      tc_fence_after();
      if (it == 0) BPD_TC_STAMP(3);
      const uint32_t sa = base + s * stage_sz;
#pragma unroll
      for (int kk = 0; kk < kBK / 16; ++kk) {
        const uint64_t ad = smem_desc_sw128(sa + kk * 32);
        const uint64_t bh = smem_desc_sw128(sa + kBM * 128 + kk * 32);
        const uint64_t bl = smem_desc_sw128(sa + kBM * 128 + bn * 128 + kk * 32);
        umma_f16(tmem, ad, bh, idesc, (it > 0 || kk > 0) ? 1u : 0u);
        umma_f16(tmem, ad, bl, idesc, 1u);
      }
      umma_commit(bars + 8 * (kStages + s));       // frees the stage once these MMAs have read it
    }
    if (!skip) umma_commit(bars + 8 * 2 * kStages);            // accumulator complete
    BPD_TC_STAMP(4);
    if (!ok) atomicCAS(p.error, 0, 102);
  } else if (warp >= 2) {
    // ---------------- epilogue: thread = one feature row, registers = tokens
    pdl_wait();
    // the stages are free once the accumulator is complete: the top-1 epilogue transposes the tile into them
    const EpiShared sh{reinterpret_cast<float*>(gen_base), s_mean, s_rstd, s_slot, ctl};
    const EpiUnit u{tmem, bars + 8 * 2 * kStages, 0u, tile, split, slice, (int)blockIdx.z, (int)gridDim.x,
                    (int)gridDim.z / zslices, t0, nt, bn, nchunks, p.all_done && *p.all_done};
    tc_epilogue<EPI, WIDE>(p, sh, u, warp, lane);
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) BPD_TC_STAMP(9);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, ncols);
  }
}

}  // namespace tc
}  // namespace bpd
