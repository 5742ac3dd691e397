// The whole decoder layer stack of a pass as ONE persistent kernel (sessions with at most 16 rows per pass).
//
// A pass over few rows is a chain of small dependent steps; what costs time is what separates them.  Here the
// launch boundaries of the layer-by-layer path become device-wide counter joins, the residual stream never
// leaves the chip between layers, and the weights of the next steps are already on their way into shared
// memory (TMA, cp.async.bulk.tensor) while the current step computes.
//
// Work split.  One thread-block cluster of 8 CTAs per attention head (the same clusters take ff / H hidden units
// of the feed-forward block).  Rank c of a cluster owns columns [c d/8, (c+1) d/8) of the residual stream x and
// the same slice of every reduction:
//
//   self-attention   x slice -> Q,K,V of the head over this rank's columns (partial sums, exchanged through
//                    distributed shared memory, added in rank order) -> cache write -> attention -> the head's
//                    share of the output projection for feature slice c -> workspace
//   cross-attention  the same with Q only and the encoder's keys / values (staged in shared memory by TMA)
//   feed-forward     the cluster's hidden units over this rank's columns -> exchange -> ReLU -> all ranks ->
//                    the hidden units times slice c of the second projection -> workspace
//
// After each of the three blocks every CTA arrives on a device-wide counter, waits for all, and then adds the
// H partial outputs of its own column slice in cluster order to its copy of x: every cluster holds the same x,
// computed by the same sums in the same order, so nothing has to be broadcast.  The layer norm that follows is
// folded into the next projection (y = rstd (acc - mean s) + c); its row statistics are merged from the eight
// slices in rank order.  All sums have an order that depends on neither the number of rows nor on timing.
//
// Weights travel as tiles through a byte ring in shared memory: one thread issues the TMA loads of the next tiles
// whenever earlier ones have been consumed; a tile is a few boxes of 64 (or 32) reduction columns in the
// swizzled layout that ldmatrix reads without bank conflicts.  The products are at most 16 columns wide and sit
// on a latency chain, so they run on mma.sync.m16n8k16 (bf16 x bf16 -> fp32, hi + lo activation planes).
//
// Every wait is bounded.  When one expires the CTA records an error, raises a device-wide flag and stops
// waiting: it (and, through the flag, every other CTA) runs the remaining steps without waits, so that all
// cluster barriers are still matched, drains its copies in flight and returns.
#pragma once
#include <cooperative_groups.h>
#include <cuda.h>

#include "fused_layer.cuh"

namespace bpd {
namespace stack {

namespace cg = cooperative_groups;
using fused::kC;
using fused::kDH;
using fused::kMaxRows;
using fused::kPartial;

constexpr int kThreads = 256;
constexpr int kWarps = 8;
constexpr int kNB = 16;                    // tiles resident or in flight at most (one mbarrier each)
constexpr int kMapsPerLayer = 8;
enum MapKind { kMapQkv = 0, kMapWo = 1, kMapCq = 2, kMapCwo = 3, kMapW1 = 4, kMapW2 = 5, kMapCk = 6, kMapCv = 7 };
constexpr unsigned long long kSpin = 2000000000ull;   // about a second
// words of the device-wide join (each on a line of its own where it matters)
constexpr int kBarCount = 0;               // arrivals, never reset while the session decodes
constexpr int kBarAbort = 1;               // non-zero: some wait expired, nobody waits any more
constexpr int kBarBase = 32;               // arrivals at the start of the next launch
constexpr int kBarWords = 64;

struct LayerPtrs {
  const bf16 *g1, *g2, *g3;                // gains of the three layer norms
  const float *s_qkv, *c_qkv, *s_cq, *c_cq, *s_f1, *c_f1;   // folded layer norms (see fold_ln_kernel)
  const bf16* b2;                          // bias of the second feed-forward projection
  bf16 *kcache, *vcache;                   // paged self-attention cache of the layer
  const float* crosskv;                    // encoder keys | values [B * max_src][2 d] fp32
};

// Byte offsets inside dynamic shared memory (the ring first, 1024-byte aligned).
struct Layout {
  int ring_bytes;
  int x, xh, xl, oh, ol, hh, hl, inbox, q, stats, attn, wst, lvl1, lvl2, pt, layers, misc, total;
};

struct StackParams {
  const CUtensorMap* maps;                 // [L][kMapsPerLayer], device memory
  const LayerPtrs* layers;                 // [L], device memory
  int L, d, H, ff, R, rows_per_b, nb;
  float eps;
  // embedding of the block (Section 6's decoder input)
  const bf16* tgt_embed; const float* pe; int npos, vocab;
  RowState st;
  const int* forced; int forced_rows, kforced;
  // attention
  int local_q, local_m, max_src;
  float scale;
  int cross_rows;                          // encoder rows staged per CTA (nb * max_src), 0: read from L2
  int long_seq;                            // 1: sequences may exceed 256 keys (buffers of the shared-key schedule exist)
  // final layer norm -> planes for the head's first projection and the fp32 residual of the heads
  const bf16 *lnf_g, *lnf_b;
  bf16* xn_hi; long long xn_plane; float* h_f32;
  float* layer_dump;                       // optional [L][R][d]: the residual stream after every layer
  // exchange between clusters
  float* ws;                               // [2][H][kMaxRows][d]
  unsigned* bar;                           // [kBarWords]
  int* error;
  const int* all_done;
  unsigned long long spin;                 // wait limit in clock cycles
  Layout lay;
};

// ------------------------------------------------------------------ small PTX helpers
__device__ __forceinline__ unsigned long long ld_acquire_u64(const void* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// Byte offset inside a swizzled tile: 16-byte pieces are permuted within 128 bytes by the row group
// (mask 7: rows of 128 bytes, TMA's 128-byte mode; mask 3: rows of 64 bytes, its 64-byte mode).
__device__ __forceinline__ uint32_t swz(uint32_t off, uint32_t mask) { return off ^ (((off >> 7) & mask) << 4); }

// acc[nt] += W(16 rows from row0 of a tile box) * X(8 tokens of tile nt), X = hi + lo planes, over one panel of
// `ksteps` * 16 reduction columns.  a_ib / b_ib: bytes per row of the weight box / of the planes' panel.
template <int NT>
__device__ __forceinline__ void mma_panel(float (&acc)[NT][4], uint32_t a_base, int a_ib, uint32_t a_mask, int row0,
                                          uint32_t bh, uint32_t bl, int b_ib, uint32_t b_mask, int ksteps, int lane) {
  const uint32_t a_row = (uint32_t)(row0 + (lane & 15)) * a_ib + (lane >> 4) * 16;
  const uint32_t b_row = (uint32_t)(lane & 7) * b_ib + ((lane >> 3) & 1) * 16;
  const uint32_t b_base = (lane & 16) ? bl : bh;           // lanes 0-15 address the hi plane, 16-31 the lo plane
  for (int kk = 0; kk < ksteps; ++kk) {
    uint32_t a0, a1, a2, a3;
    ldsm_x4(a_base + swz(a_row + kk * 32, a_mask), a0, a1, a2, a3);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      uint32_t h0, h1, l0, l1;
      ldsm_x4(b_base + swz(b_row + nt * 8 * b_ib + kk * 32, b_mask), h0, h1, l0, l1);
      fused::mma_bf16(acc[nt], a0, a1, a2, a3, h0, h1);
      fused::mma_bf16(acc[nt], a0, a1, a2, a3, l0, l1);
    }
  }
}

// ------------------------------------------------------------------ per-CTA control block in shared memory
struct Ctl {
  unsigned long long full[kNB];            // one mbarrier per tile slot
  int off[kNB];                            // ring offset of the tile in that slot
  int head, issued, freed, zombie;
  int flag;
};

struct Geo {                               // derived sizes, the same in every CTA
  int ks, PW, P, HCt, PH, UPR, ntl, staged, total_tiles;
  uint32_t xmask;                          // swizzle mask of the x planes and of the weight panels over x
};
__host__ __device__ inline Geo make_geo(int d, int H, int ff, int L, int cross_rows) {
  Geo g;
  g.ks = d / kC;
  g.PW = g.ks < 64 ? g.ks : 64;
  g.P = g.ks / g.PW;
  g.HCt = ff / H;
  g.PH = g.HCt / 64;
  g.UPR = g.HCt / kC;
  g.staged = cross_rows > 0 ? 1 : 0;
  g.ntl = 2 * g.P + g.PH + 3 + g.staged;
  g.total_tiles = g.ntl * L;
  g.xmask = g.PW == 64 ? 7u : 3u;
  return g;
}
__host__ __device__ inline int round1k(int v) { return (v + 1023) & ~1023; }
// Bytes of tile i of a layer (i in [0, ntl)), rounded to the ring's 1024-byte grain.
__host__ __device__ inline int tile_bytes(const Geo& g, int i, int cross_rows) {
  if (i < g.P) return 3 * 64 * g.PW * 2;                       // Q, K, V rows of the head, one panel
  i -= g.P;
  if (i == 0) return g.ks * 128;                               // output projection slice
  if (i == 1) return g.P * 64 * g.PW * 2;                      // cross-attention query rows, all panels
  i -= 2;
  if (g.staged) {
    if (i == 0) return 2 * round1k(cross_rows * 128) + round1k(cross_rows * 256);   // encoder keys (two halves), values
    i -= 1;
  }
  if (i == 0) return g.ks * 128;                               // cross-attention output projection slice
  i -= 1;
  if (i < g.P) return g.HCt * g.PW * 2;                        // first feed-forward projection, one panel
  return g.ks * 128;                                           // second feed-forward projection, 64 hidden units
}

struct Cta {                               // what the device functions below share
  const StackParams* p;
  Geo g;
  uint8_t* sm;
  Ctl* ctl;
  uint32_t ring;                           // shared-memory address of the ring
  int c, j, tid, warp, lane;
  unsigned long long policy;
};

// One thread: issue the TMA loads of tile `seq` into ring offset `at`.
__device__ __forceinline__ void issue_tile(const Cta& k, int seq, int at) {
  const StackParams& p = *k.p;
  const Geo& g = k.g;
  const int l = seq / g.ntl;
  int i = seq % g.ntl;
  const int slot = seq % kNB;
  const uint32_t bar = tc::smem_u32(&k.ctl->full[slot]);
  const uint32_t dst = k.ring + at;
  const CUtensorMap* maps = p.maps + (size_t)l * kMapsPerLayer;
  const int c = k.c, j = k.j, d = p.d;
  if (i < g.P) {
    tc::mbar_expect_tx(bar, 3 * 64 * g.PW * 2);
    for (int s = 0; s < 3; ++s)
      tc::tma_load_2d_hint(dst + s * 64 * g.PW * 2, maps + kMapQkv, bar, c * g.ks + i * g.PW, s * d + j * kDH, k.policy);
    return;
  }
  i -= g.P;
  if (i == 0) {
    tc::mbar_expect_tx(bar, g.ks * 128);
    tc::tma_load_2d_hint(dst, maps + kMapWo, bar, j * kDH, c * g.ks, k.policy);
    return;
  }
  if (i == 1) {
    tc::mbar_expect_tx(bar, g.P * 64 * g.PW * 2);
    for (int q = 0; q < g.P; ++q)
      tc::tma_load_2d_hint(dst + q * 64 * g.PW * 2, maps + kMapCq, bar, c * g.ks + q * g.PW, j * kDH, k.policy);
    return;
  }
  i -= 2;
  if (g.staged) {
    if (i == 0) {
      const int rows = p.cross_rows, kb = round1k(rows * 128);
      tc::mbar_expect_tx(bar, rows * 512);
      tc::tma_load_2d(dst, maps + kMapCk, bar, j * kDH, 0);
      tc::tma_load_2d(dst + kb, maps + kMapCk, bar, j * kDH + 32, 0);
      tc::tma_load_2d(dst + 2 * kb, maps + kMapCv, bar, d + j * kDH, 0);
      return;
    }
    i -= 1;
  }
  if (i == 0) {
    tc::mbar_expect_tx(bar, g.ks * 128);
    tc::tma_load_2d_hint(dst, maps + kMapCwo, bar, j * kDH, c * g.ks, k.policy);
    return;
  }
  i -= 1;
  if (i < g.P) {
    tc::mbar_expect_tx(bar, g.HCt * g.PW * 2);
    tc::tma_load_2d_hint(dst, maps + kMapW1, bar, c * g.ks + i * g.PW, j * g.HCt, k.policy);
    return;
  }
  i -= g.P;
  tc::mbar_expect_tx(bar, g.ks * 128);
  tc::tma_load_2d_hint(dst, maps + kMapW2, bar, j * g.HCt + i * 64, c * g.ks, k.policy);
}

// One thread: request as many of the next tiles as the ring has room for.  Tiles are consumed and released in
// the order they are requested; a tile never straddles the end of the ring.
__device__ __forceinline__ void pump(const Cta& k, int stop_before = 0x7fffffff) {
  Ctl* ctl = k.ctl;
  const int ring_bytes = k.p->lay.ring_bytes;
  if (ctl->zombie) return;                 // nothing new goes into flight once a wait has expired
  while (ctl->issued < k.g.total_tiles && ctl->issued < stop_before && ctl->issued - ctl->freed < kNB) {
    const int b = tile_bytes(k.g, ctl->issued % k.g.ntl, k.p->cross_rows);
    int place = -1;
    if (ctl->issued == ctl->freed) {
      if (b <= ring_bytes) place = 0;
    } else {
      const int tail = ctl->off[ctl->freed % kNB], head = ctl->head;
      if (head > tail) {
        if (head + b <= ring_bytes) place = head;
        else if (b <= tail) place = 0;
      } else if (head + b <= tail) {
        place = head;
      }
    }
    if (place < 0) break;
    ctl->off[ctl->issued % kNB] = place;
    ctl->head = place + b;
    issue_tile(k, ctl->issued, place);
    ctl->issued += 1;
  }
}
// One thread, after a barrier behind the last read of the tiles: release the n oldest tiles and refill the ring.
__device__ __forceinline__ void release_tiles(const Cta& k, int n) {
  k.ctl->freed += n;
  pump(k);
}

__device__ __forceinline__ void raise_abort(const Cta& k, int code) {
  atomicCAS(k.p->error, 0, code);
  atomicExch(k.p->bar + kBarAbort, 1u);
  *reinterpret_cast<volatile int*>(&k.ctl->zombie) = 1;
}

// All threads: wait until tile `seq` has landed; returns its shared-memory address.
__device__ __forceinline__ uint32_t tile_wait(const Cta& k, int seq) {
  const int slot = seq % kNB;
  if (!*reinterpret_cast<volatile int*>(&k.ctl->zombie)) {
    if (!tc::mbar_wait(tc::smem_u32(&k.ctl->full[slot]), (uint32_t)(seq / kNB) & 1u, k.p->spin)) raise_abort(k, 105);
  }
  return k.ring + *reinterpret_cast<volatile int*>(&k.ctl->off[slot]);
}

// All threads: the device-wide join.  Arrive (our workspace writes are released), release `nfree` consumed tiles,
// wait until `target` arrivals have been counted.
__device__ __forceinline__ void grid_join(const Cta& k, unsigned target, int nfree) {
  __syncthreads();
  if (k.tid == 0) {
    red_release_add(k.p->bar + kBarCount, 1u);
    if (nfree) release_tiles(k, nfree);
    if (!*reinterpret_cast<volatile int*>(&k.ctl->zombie)) {
      const unsigned long long t0 = clock64();
      for (unsigned spins = 0;; ++spins) {
        const unsigned long long v = ld_acquire_u64(k.p->bar + kBarCount);
        if ((int)((unsigned)v - target) >= 0) break;
        if ((unsigned)(v >> 32) != 0u) { *reinterpret_cast<volatile int*>(&k.ctl->zombie) = 1; break; }
        if ((spins & 63u) == 63u && (unsigned long long)(clock64() - t0) > k.p->spin) { raise_abort(k, 104); break; }
      }
    }
  }
  __syncthreads();
}

// ------------------------------------------------------------------ x slice: reduce, planes, statistics
// After a join: x[t][col] += bias[col] + sum over the H clusters' partial outputs, in cluster order, for this
// rank's columns.  Item = (row, four columns); rows are aligned to groups of lanes.
// Static words of a thread's (at most two) items, fetched before the join: four gains or four bias values each.
struct Words { uint2 w[2]; };
__device__ __forceinline__ Words load_words(const Cta& k, const bf16* v) {
  Words o;
  const int n4 = k.g.ks >> 2;
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int idx = k.tid + u * kThreads;
    o.w[u] = (v != nullptr && idx < k.p->R * n4) ? *reinterpret_cast<const uint2*>(v + k.c * k.g.ks + (idx % n4) * 4) : make_uint2(0u, 0u);
  }
  return o;
}
__device__ __forceinline__ void reduce_slice(const Cta& k, float* x_s, const float* ws, const Words& bias) {
  const StackParams& p = *k.p;
  const int ks = k.g.ks, n4 = ks >> 2, R = p.R, d = p.d, H = p.H;
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int idx = k.tid + it * kThreads;
    if (idx >= R * n4) break;
    const int t = idx / n4, c4 = idx % n4;
    const float4* src = reinterpret_cast<const float4*>(ws + (size_t)t * d + k.c * ks) + c4;
    const size_t step = (size_t)kMaxRows * d / 4;
    float4 acc = *reinterpret_cast<const float4*>(x_s + t * ks + c4 * 4);
    {
      const uint2 bw = bias.w[it];
      acc.x += __uint_as_float(bw.x << 16); acc.y += __uint_as_float(bw.x & 0xffff0000u);
      acc.z += __uint_as_float(bw.y << 16); acc.w += __uint_as_float(bw.y & 0xffff0000u);
    }
    for (int p0 = 0; p0 < H; p0 += 8) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = (p0 + u < H) ? __ldcg(src + (size_t)(p0 + u) * step) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (p0 + u < H) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
    }
    *reinterpret_cast<float4*>(x_s + t * ks + c4 * 4) = acc;
  }
}

// Planes (hi, lo) of x * gain for this rank's columns, and the slice's per-row (mean, sum of squared deviations),
// which go to every rank of the cluster.  A thread reads back the items it wrote itself in reduce_slice / embed
// (the same idx -> thread mapping), so no barrier is needed in between.
template <int NT>
__device__ __forceinline__ void planes_and_stats(const Cta& k, cg::cluster_group& cluster, const float* x_s, const Words& gain,
                                                 uint8_t* xh, uint8_t* xl, float* stats_in) {
  const StackParams& p = *k.p;
  const int ks = k.g.ks, n4 = ks >> 2, R = p.R, PW = k.g.PW;
  constexpr int RP = NT * 8;
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int idx = k.tid + it * kThreads;
    if (idx >= ((R * n4 + 31) & ~31)) break;                 // whole warps leave together
    const bool live = idx < R * n4;
    const int t = live ? idx / n4 : 0, c4 = live ? idx % n4 : 0;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live) {
      v = *reinterpret_cast<const float4*>(x_s + t * ks + c4 * 4);
      const uint2 gw = gain.w[it];
      const float w[4] = {v.x * __uint_as_float(gw.x << 16), v.y * __uint_as_float(gw.x & 0xffff0000u),
                          v.z * __uint_as_float(gw.y << 16), v.w * __uint_as_float(gw.y & 0xffff0000u)};
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) fused::split_bits(w[e], hi[e], lo[e]);
      const int col = c4 * 4, panel = col / PW, within = col % PW;
      const uint32_t at = panel * (RP * PW * 2) + swz((uint32_t)(t * PW * 2 + within * 2), k.g.xmask);
      *reinterpret_cast<uint2*>(xh + at) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
      *reinterpret_cast<uint2*>(xl + at) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
    }
    // the n4 lanes of a row (a power of two, at most 32, aligned) add up in a fixed butterfly
    float s = (v.x + v.y) + (v.z + v.w);
    for (int o = 1; o < n4; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mean = s / (float)ks;
    const float d0 = v.x - mean, d1 = v.y - mean, d2 = v.z - mean, d3 = v.w - mean;
    float m2 = (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
    for (int o = 1; o < n4; o <<= 1) m2 += __shfl_xor_sync(0xffffffffu, m2, o);
    if (live && c4 == 0) {
#pragma unroll
      for (int dst = 0; dst < kC; ++dst) {
        float* out = cluster.map_shared_rank(stats_in, dst) + (k.c * kMaxRows + t) * 2;
        out[0] = mean;
        out[1] = m2;
      }
    }
  }
}

// Row statistics from the eight slices, merged in rank order (threads t < R); needs a barrier afterwards.
__device__ __forceinline__ void merge_stats(const Cta& k, const float* stats_in, float* s_mean, float* s_rstd) {
  const int t = k.tid;
  if (t < k.p->R) {
    const float n1 = (float)k.g.ks;
    float mean = stats_in[t * 2], m2 = stats_in[t * 2 + 1], n = n1;
#pragma unroll
    for (int c = 1; c < kC; ++c) {
      const float mb = stats_in[(c * kMaxRows + t) * 2], qb = stats_in[(c * kMaxRows + t) * 2 + 1];
      const float delta = mb - mean, nn = n + n1;
      mean += delta * (n1 / nn);
      m2 += qb + delta * delta * (n * n1 / nn);
      n = nn;
    }
    s_mean[t] = mean;
    s_rstd[t] = rsqrtf(fmaxf(m2, 0.f) / n + k.p->eps);
  }
}

// ------------------------------------------------------------------ cross-attention over a staged tile
// Keys: two boxes [rows][32 floats] in the 128-byte swizzle (lane = key reads 16 bytes per step without bank
// conflicts); values: [rows][64 floats] as they are.  Warp w folds chunks w, w + 8, ... of 32 positions in order,
// the warps' states are merged in warp order.  Threads c < kDH return output element c.
__device__ __forceinline__ float cross_attention_tile(const uint8_t* k0, const uint8_t* k1, const uint8_t* vv, int row0,
                                                      int limit, AttnSmem<kDH, kWarps>& sm) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float m_run = -INFINITY, l_run = 0.f, a0 = 0.f, a1 = 0.f;
  for (int c0 = warp * 32; c0 < limit; c0 += kWarps * 32) {
    const int nk = min(32, limit - c0);
    float sc = -INFINITY;
    if (lane < nk) {
      const uint32_t row = (uint32_t)(row0 + c0 + lane) * 128;
      const float4* qv = reinterpret_cast<const float4*>(sm.q);
      float dot = 0.f;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float4 k4 = *reinterpret_cast<const float4*>(k0 + swz(row + u * 16, 7u)), q4 = qv[u];
        dot = fmaf(q4.x, k4.x, dot); dot = fmaf(q4.y, k4.y, dot); dot = fmaf(q4.z, k4.z, dot); dot = fmaf(q4.w, k4.w, dot);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float4 k4 = *reinterpret_cast<const float4*>(k1 + swz(row + u * 16, 7u)), q4 = qv[8 + u];
        dot = fmaf(q4.x, k4.x, dot); dot = fmaf(q4.y, k4.y, dot); dot = fmaf(q4.z, k4.z, dot); dot = fmaf(q4.w, k4.w, dot);
      }
      sc = dot;
    }
    const float m_new = fmaxf(m_run, warp_max(sc));
    const float corr = expf(m_run - m_new);
    const float pj = (lane < nk) ? expf(sc - m_new) : 0.f;
    l_run = l_run * corr + warp_sum(pj);
    a0 *= corr;
    a1 *= corr;
    for (int jj = 0; jj < nk; ++jj) {
      const float pw = __shfl_sync(0xffffffffu, pj, jj);
      const float2 v2 = *reinterpret_cast<const float2*>(vv + (size_t)(row0 + c0 + jj) * 256 + lane * 8);
      a0 = fmaf(pw, v2.x, a0);
      a1 = fmaf(pw, v2.y, a1);
    }
    m_run = m_new;
  }
  if (lane == 0) { sm.m[warp] = m_run; sm.l[warp] = l_run; }
  sm.acc[warp][2 * lane] = a0;
  sm.acc[warp][2 * lane + 1] = a1;
  __syncthreads();
  float ov = 0.f;
  if (threadIdx.x < kDH) {
    const int c = threadIdx.x;
    float M = sm.m[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) M = fmaxf(M, sm.m[w]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float e = expf(sm.m[w] - M);          // warps without keys hold -inf: weight 0
      num = fmaf(e, sm.acc[w][c], num);
      den = fmaf(e, sm.l[w], den);
    }
    ov = num / den;
  }
  return ov;
}

// Attention output element `dim` of row `token` -> planes of every rank of the cluster.
__device__ __forceinline__ void send_attn_out(cg::cluster_group& cluster, uint8_t* oh, uint8_t* ol, int token, int dim, float v) {
  uint32_t hi, lo;
  fused::split_bits(v, hi, lo);
  const uint32_t at = swz((uint32_t)(token * 128 + dim * 2), 7u);
#pragma unroll
  for (int dst = 0; dst < kC; ++dst) {
    *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(oh, dst) + at) = (unsigned short)hi;
    *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(ol, dst) + at) = (unsigned short)lo;
  }
}

// This head's (or hidden-unit group's) share of an output projection for feature slice c: rows of the tile(s) times
// the planes `ah` / `al` ([panels][RP][128 bytes]), written to the workspace of cluster j.
template <int NT>
__device__ __forceinline__ void out_share(const Cta& k, int first_seq, int npanels, const uint8_t* ah, const uint8_t* al, float* wsj) {
  const StackParams& p = *k.p;
  constexpr int RP = NT * 8;
  const int g = k.lane >> 2, t4 = k.lane & 3, ks = k.g.ks;
  for (int mt = k.warp; mt < ks / 16; mt += kWarps) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    for (int q = 0; q < npanels; ++q) {
      const uint32_t a = tile_wait(k, first_seq + q);
      mma_panel<NT>(acc, a, 128, 7u, mt * 16, tc::smem_u32(ah) + q * RP * 128, tc::smem_u32(al) + q * RP * 128, 128, 7u, 4, k.lane);
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int row = mt * 16 + g + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
        if (token < p.R) wsj[(size_t)token * p.d + k.c * ks + row] = acc[nt][e];
      }
  }
}

// ------------------------------------------------------------------ the kernel
// grid = (8, H), clusters of 8 along x.  All clusters must be resident at once (the host checks the occupancy).
template <int NT>
__global__ void __cluster_dims__(kC, 1, 1) __launch_bounds__(kThreads, 2) layer_stack_kernel(const __grid_constant__ StackParams p) {
  extern __shared__ __align__(1024) uint8_t ssm_raw[];
  // swizzled tiles need 1024-byte alignment (the launch carries 1024 bytes of slack for this)
  uint8_t* ssm = ssm_raw + ((1024u - (tc::smem_u32(ssm_raw) & 1023u)) & 1023u);
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int RP = NT * 8;
  Cta k;
  k.p = &p;
  k.g = make_geo(p.d, p.H, p.ff, p.L, p.cross_rows);
  k.sm = ssm;
  k.ctl = reinterpret_cast<Ctl*>(ssm + p.lay.misc);
  k.ring = tc::smem_u32(ssm);
  k.c = (int)cluster.block_rank();
  k.j = blockIdx.y;
  k.tid = threadIdx.x;
  k.warp = k.tid >> 5;
  k.lane = k.tid & 31;
  k.policy = tc::l2_evict_first();
  const Geo& g = k.g;
  const int c = k.c, j = k.j, tid = k.tid, warp = k.warp, lane = k.lane;
  const int d = p.d, ks = g.ks, R = p.R, nb = p.nb, rpb = p.rows_per_b;
  const int lg = lane >> 2, t4 = lane & 3;
  float* x_s = reinterpret_cast<float*>(ssm + p.lay.x);
  uint8_t* xh = ssm + p.lay.xh;
  uint8_t* xl = ssm + p.lay.xl;
  uint8_t* oh = ssm + p.lay.oh;
  uint8_t* ol = ssm + p.lay.ol;
  uint8_t* hh = ssm + p.lay.hh;
  uint8_t* hl = ssm + p.lay.hl;
  float* inbox = reinterpret_cast<float*>(ssm + p.lay.inbox);
  float* q_all = reinterpret_cast<float*>(ssm + p.lay.q);
  float* stats_in = reinterpret_cast<float*>(ssm + p.lay.stats);          // [rank][kMaxRows][2]
  float* s_mean = stats_in + kC * kMaxRows * 2;
  float* s_rstd = s_mean + kMaxRows;
  int* s_len = reinterpret_cast<int*>(s_rstd + kMaxRows);                 // [kMaxRows] cache lengths of the sequences
  int* s_src = s_len + kMaxRows;                                          // [kMaxRows] source lengths
  AttnSmem<kDH, kWarps>& sm = *reinterpret_cast<AttnSmem<kDH, kWarps>*>(ssm + p.lay.attn);
  float* wst = reinterpret_cast<float*>(ssm + p.lay.wst);                 // [warp][slot][kPartial]
  float* lvl1 = reinterpret_cast<float*>(ssm + p.lay.lvl1);
  float* lvl2 = reinterpret_cast<float*>(ssm + p.lay.lvl2);
  int* s_pt = reinterpret_cast<int*>(ssm + p.lay.pt);
  LayerPtrs* layers_s = reinterpret_cast<LayerPtrs*>(ssm + p.lay.layers);
  const unsigned G = gridDim.x * gridDim.y;

  if (tid == 0) {
    for (int i = 0; i < kNB; ++i) tc::mbar_init(tc::smem_u32(&k.ctl->full[i]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    k.ctl->head = 0; k.ctl->issued = 0; k.ctl->freed = 0; k.ctl->zombie = 0; k.ctl->flag = 0;
  }
  __syncthreads();
  // Weights and page tables do not depend on anything earlier in the stream.  The encoder's keys and values do:
  // the launches before this one (the encoder's, right after bpd_encode) may still be running, so the first
  // tile that carries them is not requested before the dependency wait.
  if (tid == 0) pump(k, g.staged ? g.P + 2 : 0x7fffffff);
  for (int i = tid; i < nb * p.st.pages_per_row; i += kThreads) s_pt[i] = p.st.page_table[i];
  for (int i = tid; i < p.L * (int)(sizeof(LayerPtrs) / 8); i += kThreads)
    reinterpret_cast<unsigned long long*>(layers_s)[i] = reinterpret_cast<const unsigned long long*>(p.layers)[i];
  // the hidden planes' rows beyond R are never written: zero them once so that no NaN pattern reaches an MMA
  for (int i = tid; i < (p.lay.inbox - p.lay.xh) / 16; i += kThreads) reinterpret_cast<uint4*>(ssm + p.lay.xh)[i] = make_uint4(0, 0, 0, 0);
  pdl_wait();
  if (p.all_done && *p.all_done) {
    // nothing to do: let what was requested land (bounded), then leave
    __syncthreads();
    if (tid == 0)
      for (int s = k.ctl->freed; s < k.ctl->issued; ++s) tc::mbar_wait(tc::smem_u32(&k.ctl->full[s % kNB]), (uint32_t)(s / kNB) & 1u, p.spin);
    return;
  }
  if (tid == 0) pump(k);
  const unsigned base = __ldcg(p.bar + kBarBase);
  if (tid < nb) { s_len[tid] = p.st.len[tid]; s_src[tid] = p.st.src_len[tid]; }
  __syncthreads();

  // ---- embedding of the block: x[t] = E[token] sqrt(d) + PE(position), this rank's columns
  {
    const int n4 = ks >> 2;
    const float scale = sqrtf((float)d);
    for (int idx = tid; idx < R * n4; idx += kThreads) {
      const int t = idx / n4, c4 = idx % n4;
      const int b = t / rpb, i = t % rpb;
      int tok = p.st.block[b * kMaxK + i];
      if (p.forced && i >= 1 && i < p.kforced) {
        const int jb = p.st.j[b];
        if (p.forced_rows == 1) tok = p.forced[(size_t)b * (p.kforced - 1) + (i - 1)];
        else if (jb < p.forced_rows) tok = p.forced[((size_t)b * p.forced_rows + jb) * (p.kforced - 1) + (i - 1)];
      }
      int pos = s_len[b] + i;
      if (j == 0 && c == 0 && c4 == 0) p.st.cur_block[b * kMaxK + i] = tok;
      if (tok < 0 || tok >= p.vocab || pos >= p.npos) {     // never index outside the tables; report instead
        atomicCAS(p.error, 0, 1);
        tok = 0;
        pos = 0;
      }
      const uint2 ew = *reinterpret_cast<const uint2*>(p.tgt_embed + (size_t)tok * d + c * ks + c4 * 4);
      const float4 pe = *reinterpret_cast<const float4*>(p.pe + (size_t)pos * d + c * ks + c4 * 4);
      float4 v;
      v.x = __uint_as_float(ew.x << 16) * scale + pe.x;
      v.y = __uint_as_float(ew.x & 0xffff0000u) * scale + pe.y;
      v.z = __uint_as_float(ew.y << 16) * scale + pe.z;
      v.w = __uint_as_float(ew.y & 0xffff0000u) * scale + pe.w;
      *reinterpret_cast<float4*>(x_s + t * ks + c4 * 4) = v;
    }
  }
  fused::cluster_arrive();
  fused::cluster_wait();                    // every CTA of the cluster runs: its shared memory may be written

  AttnParams ap;
  memset(&ap, 0, sizeof(ap));
  ap.rows = R; ap.rows_per_b = rpb; ap.H = p.H; ap.dh = kDH; ap.causal = 1; ap.local_q = p.local_q; ap.local_m = p.local_m;
  ap.ldkv = d; ap.paged = 1; ap.st = p.st; ap.st.page_table = s_pt; ap.scale = p.scale;
  bool one_chunk_per_rank = true;
  for (int b = 0; b < nb; ++b)
    one_chunk_per_rank = one_chunk_per_rank && ((s_len[b] + rpb + 31) >> 5) - (attn_first_key(ap, s_len[b]) >> 5) <= kC;

  unsigned nbar = 0;                        // joins passed so far in this launch
  int seq = 0;                              // next tile to consume
  for (int l = 0; l < p.L; ++l) {
    const LayerPtrs& LP = layers_s[l];
    // =================================================================== self-attention block
    // static words first (gains, folded layer-norm vectors, bias): their latency hides behind the join
    Words gw = load_words(k, LP.g1);
    float fs = 0.f, fc = 0.f;
    if (tid < 3 * kDH) {
      const int n = (tid / kDH) * d + j * kDH + (tid % kDH);
      fs = LP.s_qkv[n];
      fc = LP.c_qkv[n];
    }
    if (l > 0) {
      const Words bw = load_words(k, layers_s[l - 1].b2);
      grid_join(k, base + (++nbar) * G, g.PH);
      reduce_slice(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, bw);
      if (p.layer_dump && j == 0) {
        __syncthreads();
        for (int idx = tid; idx < R * ks; idx += kThreads)
          p.layer_dump[((size_t)(l - 1) * R + idx / ks) * d + c * ks + idx % ks] = x_s[idx];
      }
    }
    planes_and_stats<NT>(k, cluster, x_s, gw, xh, xl, stats_in);
    __syncthreads();
    // Q, K, V of the head over this rank's columns; token t's partial goes to rank t % 8
    for (int mt = warp; mt < 3 * kDH / 16; mt += kWarps) {
      float acc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
      for (int q = 0; q < g.P; ++q) {
        const uint32_t a = tile_wait(k, seq + q);
        mma_panel<NT>(acc, a + (mt / 4) * 64 * g.PW * 2, g.PW * 2, g.xmask, (mt % 4) * 16, tc::smem_u32(xh) + q * RP * g.PW * 2,
                      tc::smem_u32(xl) + q * RP * g.PW * 2, g.PW * 2, g.xmask, g.PW / 16, lane);
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int row = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
          if (token < R) cluster.map_shared_rank(inbox, token % kC)[(c * NT + token / kC) * 3 * kDH + row] = acc[nt][e];
        }
    }
    seq += g.P;
    cluster.sync();
    if (tid == 0) release_tiles(k, g.P);
    merge_stats(k, stats_in + 0, s_mean, s_rstd);
    __syncthreads();
    // this rank's tokens: partials in rank order, layer norm, keys / values into the cache
    for (int slot = 0; slot < NT; ++slot) {
      const int token = slot * kC + c;
      if (token < R && tid < 3 * kDH) {
        float a = 0.f;
#pragma unroll
        for (int src = 0; src < kC; ++src) a += inbox[(src * NT + slot) * 3 * kDH + tid];
        const int sect = tid / kDH, f = tid % kDH;
        const float y = s_rstd[token] * (a - s_mean[token] * fs) + fc;
        if (sect == 0) {
          if (one_chunk_per_rank) {
            q_all[token * kDH + f] = y * p.scale;
          } else {
#pragma unroll
            for (int dst = 0; dst < kC; ++dst) cluster.map_shared_rank(q_all, dst)[token * kDH + f] = y * p.scale;
          }
        } else {
          const int b = token / rpb, i = token % rpb;
          const int pos = s_len[b] + i;
          const int page = s_pt[b * p.st.pages_per_row + pos / kPage];
          const size_t at = ((size_t)page * kPage + (pos % kPage)) * d + j * kDH + f;
          (sect == 1 ? LP.kcache : LP.vcache)[at] = __float2bfloat16_rn(y);
        }
      }
    }
    __threadfence();
    cluster.sync();                         // the block's new keys and values are in the cache for every rank's rows
    {
      ap.k = LP.kcache; ap.v = LP.vcache;
      const bf16* Kc = LP.kcache;
      const bf16* Vc = LP.vcache;
      if (one_chunk_per_rank) {
        // this rank attends for its own rows; warp w folds the chunk that belongs to rank w
        for (int slot = 0; slot < NT; ++slot) {
          const int token = slot * kC + c;
          if (token < R) {                                           // uniform over the CTA
            const int b = token / rpb, i = token % rpb;
            const int len = s_len[b], lim_max = len + rpb;
            const int fk = attn_first_key(ap, len + i), ch0 = attn_first_key(ap, len) >> 5;
            const int ch = ch0 + ((warp - ch0) & (kC - 1));
            float* state = wst + (warp * NT + slot) * kPartial;
            if (lane == 0) { state[kDH] = -INFINITY; state[kDH + 1] = 0.f; }
            __syncwarp();
            if ((ch << 5) <= len + i) {
              const int c0 = ch << 5;
              const size_t kbase = ((size_t)s_pt[b * p.st.pages_per_row + c0 / kPage] * kPage + (c0 % kPage)) * d + j * kDH;
              uint4 kq[8];
              uint32_t vq[32];
              fused::chunk_fetch(Kc, Vc, kbase, min(32, lim_max - c0), d, lane, kq, vq);
              const int key = c0 + lane;
              fused::chunk_fold(kq, vq, q_all + token * kDH, key <= len + i && key >= fk, state, lane);
            }
            __syncthreads();
            if (tid < kDH) {
              float M, num, den;
              fused::states_merge(wst + slot * kPartial, NT * kPartial, tid, M, num, den);
              send_attn_out(cluster, oh, ol, token, tid, num / den);
            }
          }
        }
      } else {
        // long sequences: rank c folds its own chunks for every row (keys fetched once per sequence), the ranks'
        // states travel through distributed shared memory
        const int RL = R;
        for (int i = tid; i < 8 * RL; i += kThreads) { lvl1[i * kPartial + kDH] = -INFINITY; lvl1[i * kPartial + kDH + 1] = 0.f; }
        __syncthreads();
        for (int b = 0; b < nb; ++b) {
          const int len = s_len[b];
          const int lim_max = len + rpb;
          const int nch = (lim_max + 31) >> 5, ch0 = attn_first_key(ap, len) >> 5;
          const int first_my = ch0 + ((c - ch0) & (kC - 1));
          const int n_my = first_my < nch ? (nch - first_my + kC - 1) / kC : 0;
          const int active = min(8, n_my);
          if (active == 0) continue;
          const int S = 8 / active;
          const int a = warp / S, sub = warp % S;
          if (a >= active) continue;
          const int ch_first = first_my + kC * a;
          const int lump = (ch_first / kC) & 7;
          const int* pt = s_pt + b * p.st.pages_per_row;
          for (int ch = ch_first; ch < nch; ch += 8 * kC) {
            const int c0 = ch << 5;
            const size_t kbase = ((size_t)pt[c0 / kPage] * kPage + (c0 % kPage)) * d + j * kDH;
            uint4 kq[8];
            uint32_t vq[32];
            fused::chunk_fetch(Kc, Vc, kbase, min(32, lim_max - c0), d, lane, kq, vq);
            const int key = c0 + lane;
#pragma unroll 1
            for (int i = sub; i < rpb; i += S)
              fused::chunk_fold(kq, vq, q_all + (b * rpb + i) * kDH, key <= len + i && key >= attn_first_key(ap, len + i),
                                lvl1 + ((size_t)lump * RL + b * rpb + i) * kPartial, lane);
          }
        }
        __syncthreads();
        for (int idx = tid; idx < R * kDH; idx += kThreads) {
          const int row = idx / kDH, dim = idx % kDH;
          float M, num, den;
          fused::states_merge(lvl1 + row * kPartial, RL * kPartial, dim, M, num, den);
#pragma unroll
          for (int dst = 0; dst < kC; ++dst) {
            float* out = cluster.map_shared_rank(lvl2, dst) + (c * RL + row) * kPartial;
            out[dim] = num;
            if (dim == 0) { out[kDH] = M; out[kDH + 1] = den; }
          }
        }
        cluster.sync();
        for (int idx = tid; idx < R * kDH; idx += kThreads) {
          const int row = idx / kDH, dim = idx % kDH;
          float M, num, den;
          fused::states_merge(lvl2 + row * kPartial, RL * kPartial, dim, M, num, den);
          uint32_t hi, lo;
          fused::split_bits(num / den, hi, lo);
          const uint32_t at = swz((uint32_t)(row * 128 + dim * 2), 7u);
          *reinterpret_cast<unsigned short*>(oh + at) = (unsigned short)hi;
          *reinterpret_cast<unsigned short*>(ol + at) = (unsigned short)lo;
        }
      }
    }
    cluster.sync();
    out_share<NT>(k, seq, 1, oh, ol, p.ws + ((size_t)(nbar & 1) * p.H + j) * kMaxRows * d);
    seq += 1;

    // =================================================================== cross-attention block
    gw = load_words(k, LP.g2);
    const Words nobias = load_words(k, nullptr);
    if (tid < kDH) { fs = LP.s_cq[j * kDH + tid]; fc = LP.c_cq[j * kDH + tid]; }
    grid_join(k, base + (++nbar) * G, 1);
    reduce_slice(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, nobias);
    planes_and_stats<NT>(k, cluster, x_s, gw, xh, xl, stats_in);
    __syncthreads();
    for (int mt = warp; mt < kDH / 16; mt += kWarps) {
      float acc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
      const uint32_t a = tile_wait(k, seq);
      for (int q = 0; q < g.P; ++q)
        mma_panel<NT>(acc, a + q * 64 * g.PW * 2, g.PW * 2, g.xmask, mt * 16, tc::smem_u32(xh) + q * RP * g.PW * 2,
                      tc::smem_u32(xl) + q * RP * g.PW * 2, g.PW * 2, g.xmask, g.PW / 16, lane);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int row = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
          if (token < R) cluster.map_shared_rank(inbox, token % kC)[(c * NT + token / kC) * kDH + row] = acc[nt][e];
        }
    }
    seq += 1;
    cluster.sync();
    if (tid == 0) release_tiles(k, 1);
    merge_stats(k, stats_in, s_mean, s_rstd);
    __syncthreads();
    {
      uint32_t ckv = 0;
      if (g.staged) ckv = tile_wait(k, seq);
      const uint8_t* ckv_g = ssm + (ckv - k.ring);
      const int kb = round1k(p.cross_rows * 128);
      ap.causal = 0; ap.limit_b = s_src; ap.k = LP.crosskv; ap.v = LP.crosskv + d; ap.ldkv = 2 * d;
      ap.bstride = (long long)p.max_src * 2 * d; ap.paged = 0;
      for (int slot = 0; slot < NT; ++slot) {
        const int token = slot * kC + c;
        if (token < R) {                     // uniform over the CTA
          if (tid < kDH) {
            float a = 0.f;
#pragma unroll
            for (int src = 0; src < kC; ++src) a += inbox[(src * NT + slot) * kDH + tid];
            sm.q[tid] = (s_rstd[token] * (a - s_mean[token] * fs) + fc) * p.scale;
          }
          __syncthreads();
          const int b = token / rpb;
          const float ov = g.staged ? cross_attention_tile(ckv_g, ckv_g + kb, ckv_g + 2 * kb, b * p.max_src, s_src[b], sm)
                                    : attention_head<float, kDH, kWarps, false>(ap, b, j, 0, s_src[b], sm);
          if (tid < kDH) send_attn_out(cluster, oh, ol, token, tid, ov);
          __syncthreads();
        }
      }
      ap.causal = 1; ap.ldkv = d; ap.paged = 1;
      seq += g.staged;
    }
    cluster.sync();
    if (tid == 0 && g.staged) release_tiles(k, 1);
    out_share<NT>(k, seq, 1, oh, ol, p.ws + ((size_t)(nbar & 1) * p.H + j) * kMaxRows * d);
    seq += 1;

    // =================================================================== feed-forward block
    gw = load_words(k, LP.g3);
    float fs1[2], fc1[2];                    // folded vectors of the (at most two) hidden units this thread finishes
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int idx = tid + u * kThreads;
      const int unit = j * g.HCt + c * g.UPR + idx % g.UPR;
      fs1[u] = idx < g.UPR * R ? LP.s_f1[unit] : 0.f;
      fc1[u] = idx < g.UPR * R ? LP.c_f1[unit] : 0.f;
    }
    grid_join(k, base + (++nbar) * G, 1);
    reduce_slice(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, nobias);
    planes_and_stats<NT>(k, cluster, x_s, gw, xh, xl, stats_in);
    __syncthreads();
    // the cluster's hidden units over this rank's columns; unit f belongs to rank f / UPR
    for (int mt = warp; mt < g.HCt / 16; mt += kWarps) {
      float acc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
      for (int q = 0; q < g.P; ++q) {
        const uint32_t a = tile_wait(k, seq + q);
        mma_panel<NT>(acc, a, g.PW * 2, g.xmask, mt * 16, tc::smem_u32(xh) + q * RP * g.PW * 2, tc::smem_u32(xl) + q * RP * g.PW * 2,
                      g.PW * 2, g.xmask, g.PW / 16, lane);
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int f = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
          if (token < R) cluster.map_shared_rank(inbox, f / g.UPR)[(c * g.UPR + f % g.UPR) * RP + token] = acc[nt][e];
        }
    }
    seq += g.P;
    cluster.sync();
    if (tid == 0) release_tiles(k, g.P);
    merge_stats(k, stats_in, s_mean, s_rstd);
    __syncthreads();
    // ranks in order, layer norm, bias, ReLU; every rank of the cluster gets the planes of these hidden units
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int idx = tid + u * kThreads;
      if (idx >= g.UPR * R) break;
      const int f = idx % g.UPR, token = idx / g.UPR;
      float a = 0.f;
#pragma unroll
      for (int src = 0; src < kC; ++src) a += inbox[(src * g.UPR + f) * RP + token];
      const float y = fmaxf(s_rstd[token] * (a - s_mean[token] * fs1[u]) + fc1[u], 0.f);
      uint32_t hi, lo;
      fused::split_bits(y, hi, lo);
      const int hu = c * g.UPR + f;
      const uint32_t at = (hu / 64) * (RP * 128) + swz((uint32_t)(token * 128 + (hu % 64) * 2), 7u);
#pragma unroll
      for (int dst = 0; dst < kC; ++dst) {
        *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(hh, dst) + at) = (unsigned short)hi;
        *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(hl, dst) + at) = (unsigned short)lo;
      }
    }
    cluster.sync();
    out_share<NT>(k, seq, g.PH, hh, hl, p.ws + ((size_t)(nbar & 1) * p.H + j) * kMaxRows * d);
    seq += g.PH;
  }
  // =================================================================== final layer norm
  {
    const Words bw = load_words(k, layers_s[p.L - 1].b2), gw = load_words(k, p.lnf_g);
    grid_join(k, base + (++nbar) * G, g.PH);
    pdl_launch_dependents();
    reduce_slice(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, bw);
    if (p.layer_dump && j == 0) {
      __syncthreads();
      for (int idx = tid; idx < R * ks; idx += kThreads)
        p.layer_dump[((size_t)(p.L - 1) * R + idx / ks) * d + c * ks + idx % ks] = x_s[idx];
    }
    planes_and_stats<NT>(k, cluster, x_s, gw, xh, xl, stats_in);   // the planes are not used; the statistics are
  }
  cluster.sync();
  merge_stats(k, stats_in, s_mean, s_rstd);
  __syncthreads();
  if (j == 0) {
    const int n4 = ks >> 2;
    for (int idx = tid; idx < R * n4; idx += kThreads) {
      const int t = idx / n4, col = c * ks + (idx % n4) * 4;
      const float4 v = *reinterpret_cast<const float4*>(x_s + t * ks + (idx % n4) * 4);
      const uint2 gw = *reinterpret_cast<const uint2*>(p.lnf_g + col), bw = *reinterpret_cast<const uint2*>(p.lnf_b + col);
      const float mean = s_mean[t], rstd = s_rstd[t];
      float o[4];
      o[0] = (v.x - mean) * rstd * __uint_as_float(gw.x << 16) + __uint_as_float(bw.x << 16);
      o[1] = (v.y - mean) * rstd * __uint_as_float(gw.x & 0xffff0000u) + __uint_as_float(bw.x & 0xffff0000u);
      o[2] = (v.z - mean) * rstd * __uint_as_float(gw.y << 16) + __uint_as_float(bw.y << 16);
      o[3] = (v.w - mean) * rstd * __uint_as_float(gw.y & 0xffff0000u) + __uint_as_float(bw.y & 0xffff0000u);
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) fused::split_bits(o[e], hi[e], lo[e]);
      bf16* yp = p.xn_hi + (size_t)t * d + col;
      *reinterpret_cast<uint2*>(yp) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
      *reinterpret_cast<uint2*>(yp + p.xn_plane) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
      *reinterpret_cast<float4*>(p.h_f32 + (size_t)t * d + col) = make_float4(o[0], o[1], o[2], o[3]);
    }
    if (c == 0 && tid == 0) p.bar[kBarBase] = base + nbar * G;     // where the next launch starts counting
  }
  if (tid == 0 && k.ctl->zombie) {
    // a wait expired somewhere: tiles may still be in flight; give each slot's last request a bounded chance to land
    for (int s2 = max(0, k.ctl->issued - kNB); s2 < k.ctl->issued; ++s2)
      tc::mbar_wait(tc::smem_u32(&k.ctl->full[s2 % kNB]), (uint32_t)(s2 / kNB) & 1u, p.spin);
  }
}

}  // namespace stack
}  // namespace bpd
