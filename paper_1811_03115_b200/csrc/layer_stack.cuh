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
//   self-attention   x slice -> Q,K,V of the head over this rank's columns (partial sums, exchanged inside the
//                    cluster, added in rank order) -> cache write -> attention -> the head's share of the output
//                    projection for feature slice c -> workspace
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
// Exchanges inside a cluster are bulk copies between the CTAs' shared memories (cp.async.bulk
// shared::cta -> shared::cluster): a sender lays its contribution out contiguously, one thread per destination
// issues the copy, and the copy itself signals an mbarrier in the destination CTA, which is what the receiver
// waits on -- one transfer per destination instead of thousands of scalar remote stores, and no cluster-wide
// barrier.  The smallest exchanges (single rows) go as 16-byte asynchronous stores (st.async) counted on the same
// mbarriers.  Two mbarriers alternate between successive exchanges, so a fast sender's next exchange can never be
// counted into the one a receiver is still waiting for.
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

constexpr int kThreads = 256;
constexpr int kWarps = 8;
constexpr int kNB = 16;                    // tiles resident or in flight at most (one mbarrier each)
constexpr int kPumpThread = 32;            // the thread that requests tiles: not thread 0, which arrives on and polls the
                                           // device-wide join and sends to rank 0, so the two work side by side
constexpr int kMaps = 8;
enum MapKind { kMapQkv = 0, kMapWo = 1, kMapCq = 2, kMapCwo = 3, kMapW1 = 4, kMapW2 = 5, kMapCk = 6, kMapCv = 7 };
constexpr int kMaxTiles = 16;              // tiles per layer at most
constexpr int kState = 68;                 // floats per partial attention state: 64 outputs, maximum, weight sum, and
                                           // padding to a multiple of 16 bytes
constexpr unsigned long long kSpin = 2000000000ull;   // about a second
// words of the device-wide join
constexpr int kBarAbort = 1;               // non-zero: some wait expired, nobody waits any more
constexpr int kBarBase = 32;               // reductions done so far in this session: the next launch's tags go on from here (never reset)
constexpr int kBarWords = 64;

// Tensor maps over all decoder layers at once (the layers' tensors lie at a constant stride): dimensions
// (columns, rows, layer).  Passed as a kernel parameter, so that issuing a load never waits for a descriptor.
struct StackMaps { CUtensorMap m[kMaps]; };

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
  int x, xh, xl, oh, ol, hid, outbox, inbox, kvq, stats, attn, wst, lvl1, lvl2, pt, layers, misc, total;
};

struct StackParams {
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
  unsigned long long* ws;                  // [2][H][kMaxRows][d] words of (value bits, tag): the clusters' shares of a projection output
  unsigned long long* gather;              // [2][kMaxRows][d] words of (value bits, tag): the summed shares, models with 16 or more heads
  unsigned* bar;                           // [kBarWords]
  int* error;
  const int* all_done;
  unsigned long long spin;                 // wait limit in clock cycles
  Layout lay;
};

// ------------------------------------------------------------------ small PTX helpers
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z,
                                            unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "l"(policy) : "memory");
}
// Shared-memory address of `addr` (an address of this CTA) in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_rank(uint32_t addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// Bulk copy of `bytes` (a multiple of 16) from this CTA's shared memory into another CTA's; completion is counted
// on the mbarrier `bar_remote` of the destination CTA.
__device__ __forceinline__ void dsmem_bulk(uint32_t dst_remote, uint32_t src_local, uint32_t bytes, uint32_t bar_remote) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_remote), "r"(src_local), "r"(bytes), "r"(bar_remote) : "memory");
}
// 16 bytes from registers into another CTA's shared memory; completion (16 bytes) is counted on the mbarrier
// `bar_remote` of the destination CTA, like a bulk copy's -- but issued by the thread itself, with no staging fence.
__device__ __forceinline__ void dsmem_store16(uint32_t dst_remote, uint4 v, uint32_t bar_remote) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(dst_remote), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(bar_remote) : "memory");
}
// What this thread wrote to shared memory becomes visible to bulk copies issued after the next barrier.
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Byte offset inside a swizzled tile: 16-byte pieces are permuted within 128 bytes by the row group
// (mask 7: rows of 128 bytes, TMA's 128-byte mode; mask 3: rows of 64 bytes, its 64-byte mode; 0: none).
__device__ __forceinline__ uint32_t swz(uint32_t off, uint32_t mask) { return off ^ (((off >> 7) & mask) << 4); }

// One 16-column step of acc[nt] += W(16 rows) * X(8 tokens of tile nt), X = hi + lo planes.  a_addr: this lane's
// ldmatrix address in the weight box (row = row0 + lane % 16, second 8 columns for lanes >= 16); b_addr: this
// lane's address in the planes (token lane % 8, second 8 columns for lanes 8-15 / 24-31; lanes 0-15 the hi plane,
// 16-31 the lo plane); b_nt: bytes between token tiles.
template <int NT>
__device__ __forceinline__ void mma_step(float (&acc)[NT][4], uint32_t a_addr, uint32_t b_addr, uint32_t b_nt) {
  uint32_t a0, a1, a2, a3;
  ldsm_x4(a_addr, a0, a1, a2, a3);
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    uint32_t h0, h1, l0, l1;
    ldsm_x4(b_addr + nt * b_nt, h0, h1, l0, l1);
    fused::mma_bf16(acc[nt], a0, a1, a2, a3, h0, h1);
    fused::mma_bf16(acc[nt], a0, a1, a2, a3, l0, l1);
  }
}

// ------------------------------------------------------------------ per-CTA control block in shared memory
struct TileDesc {                          // one tile of a layer: nbox boxes of map `map`, optionally one more of map2
  int bytes, map, nbox, x, y, dx, dstep, box_bytes;
  int map2, x2, off2, bytes2;
};
struct Ctl {
  unsigned long long full[kNB];            // one mbarrier per tile slot
  unsigned long long ex[2];                // exchanges inside the cluster alternate between these two
  int off[kNB];                            // ring offset of the tile in that slot
  int head, issued, freed, zombie;
  int issue_layer, issue_idx;              // layer and index within the layer of the next tile to request
  TileDesc tiles[kMaxTiles];
#ifdef BPD_STACK_TRACE
  long long cyc_wait, cyc_pump, cyc_poll;   // thread 0: cycles spent waiting for tiles, requesting tiles, polling the join
#endif
};

struct Geo {                               // derived sizes, the same in every CTA
  int ks, PW, P, HCt, PH, UPR, ntl, staged, total_tiles;
  int lg_n4, lg_pw, lg_upr;                // log2 of ks / 4, PW, UPR (all powers of two)
  uint32_t xmask, hmask;                   // swizzle masks of the x planes (and weight panels over x), of the hidden planes
};
__host__ __device__ inline int ilog2(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }
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
  g.hmask = g.UPR == 32 ? 3u : 0u;
  g.lg_n4 = ilog2(g.ks >> 2); g.lg_pw = ilog2(g.PW); g.lg_upr = ilog2(g.UPR);
  return g;
}
__host__ __device__ inline int round1k(int v) { return (v + 1023) & ~1023; }
// Tile i of a layer (i in [0, ntl)) for rank c of cluster j.  Sizes are multiples of the ring's 1024-byte grain.
__host__ __device__ inline TileDesc make_tile(const Geo& g, int i, int cross_rows, int d, int c, int j) {
  TileDesc t;
  t.map2 = -1; t.x2 = 0; t.off2 = 0; t.bytes2 = 0; t.dx = 0; t.dstep = 0; t.nbox = 1;
  if (i < g.P) {                                               // Q, K, V rows of the head, one panel: three boxes
    t.map = kMapQkv; t.nbox = 3; t.box_bytes = 64 * g.PW * 2; t.x = c * g.ks + i * g.PW; t.y = j * kDH;
    t.dstep = t.box_bytes;                                     // the boxes differ in y (by d_model): see issue_tile
    t.bytes = 3 * t.box_bytes;
    return t;
  }
  i -= g.P;
  if (i == 0) { t.map = kMapWo; t.box_bytes = g.ks * 128; t.x = j * kDH; t.y = c * g.ks; t.bytes = t.box_bytes; return t; }
  if (i == 1) {                                                // cross-attention query rows, all panels
    t.map = kMapCq; t.nbox = g.P; t.box_bytes = 64 * g.PW * 2; t.x = c * g.ks; t.y = j * kDH; t.dx = g.PW; t.dstep = t.box_bytes;
    t.bytes = g.P * t.box_bytes;
    return t;
  }
  i -= 2;
  if (g.staged) {
    if (i == 0) {                                              // encoder keys (two halves of 32 floats), then values
      const int kb = round1k(cross_rows * 128);
      t.map = kMapCk; t.nbox = 2; t.box_bytes = cross_rows * 128; t.x = j * kDH; t.y = 0; t.dx = 32; t.dstep = kb;
      t.map2 = kMapCv; t.x2 = d + j * kDH; t.off2 = 2 * kb; t.bytes2 = cross_rows * 256;
      t.bytes = 2 * kb + round1k(cross_rows * 256);
      return t;
    }
    i -= 1;
  }
  if (i == 0) { t.map = kMapCwo; t.box_bytes = g.ks * 128; t.x = j * kDH; t.y = c * g.ks; t.bytes = t.box_bytes; return t; }
  i -= 1;
  if (i < g.P) { t.map = kMapW1; t.box_bytes = g.HCt * g.PW * 2; t.x = c * g.ks + i * g.PW; t.y = j * g.HCt; t.bytes = t.box_bytes; return t; }
  i -= g.P;
  t.map = kMapW2; t.box_bytes = g.ks * 128; t.x = j * g.HCt + i * 64; t.y = c * g.ks; t.bytes = t.box_bytes;
  return t;
}

struct Cta {                               // what the device functions below share
  const StackParams* p;
  const StackMaps* maps;
  Geo g;
  uint8_t* sm;
  Ctl* ctl;
  uint32_t ring;                           // shared-memory address of the ring
  int c, j, tid, warp, lane;
  unsigned long long policy;
};

// One thread: request as many of the next tiles as the ring has room for.  Tiles are consumed and released in
// the order they are requested; a tile never straddles the end of the ring.  The bookkeeping is copied into
// registers for the loop: this thread is on the critical path of its CTA.
__device__ __forceinline__ void pump(const Cta& k, int stop_before = 0x7fffffff) {
  Ctl* ctl = k.ctl;
  if (ctl->zombie) return;                 // nothing new goes into flight once a wait has expired
  const int ring_bytes = k.p->lay.ring_bytes, total = min(k.g.total_tiles, stop_before), ntl = k.g.ntl, dmodel = k.p->d;
  int issued = ctl->issued, head = ctl->head, idx = ctl->issue_idx, layer = ctl->issue_layer;
  const int freed = ctl->freed;
  int tail = ctl->off[freed & (kNB - 1)];
  while (issued < total && issued - freed < kNB) {
    const TileDesc t = ctl->tiles[idx];
    int place = -1;
    if (issued == freed) {
      if (t.bytes <= ring_bytes) { place = 0; tail = 0; }
    } else if (head > tail) {
      if (head + t.bytes <= ring_bytes) place = head;
      else if (t.bytes <= tail) place = 0;
    } else if (head + t.bytes <= tail) {
      place = head;
    }
    if (place < 0) break;
    const int slot = issued & (kNB - 1);
    ctl->off[slot] = place;
    head = place + t.bytes;
    const uint32_t bar = tc::smem_u32(&ctl->full[slot]);
    const uint32_t dst = k.ring + place;
    tc::mbar_expect_tx(bar, t.nbox * t.box_bytes + t.bytes2);
    const int dy = (t.map == kMapQkv) ? dmodel : 0;
    for (int b = 0; b < t.nbox; ++b)
      tma_load_3d(dst + b * t.dstep, &k.maps->m[t.map], bar, t.x + b * t.dx, t.y + b * dy, layer, k.policy);
    if (t.map2 >= 0) tma_load_3d(dst + t.off2, &k.maps->m[t.map2], bar, t.x2, 0, layer, k.policy);
    if (++idx == ntl) { idx = 0; ++layer; }
    ++issued;
  }
  ctl->issued = issued; ctl->head = head; ctl->issue_idx = idx; ctl->issue_layer = layer;
}
// One thread, after a barrier behind the last read of the tiles: release the n oldest tiles and refill the ring.
__device__ __forceinline__ void release_tiles(const Cta& k, int n) {
#ifdef BPD_STACK_TRACE
  const long long t0 = clock64();
#endif
  k.ctl->freed += n;
  pump(k);
#ifdef BPD_STACK_TRACE
  k.ctl->cyc_pump += clock64() - t0;
#endif
}

__device__ __forceinline__ void raise_abort(const Cta& k, int code) {
  atomicCAS(k.p->error, 0, code);
  atomicExch(k.p->bar + kBarAbort, 1u);
  *reinterpret_cast<volatile int*>(&k.ctl->zombie) = 1;
}
__device__ __forceinline__ bool is_zombie(const Cta& k) { return *reinterpret_cast<volatile int*>(&k.ctl->zombie) != 0; }

// All threads: wait until tile `seq` has landed; returns its shared-memory address.
__device__ __forceinline__ uint32_t tile_wait(const Cta& k, int seq) {
  const int slot = seq & (kNB - 1);
#ifdef BPD_STACK_TRACE
  const long long t0 = clock64();
#endif
  if (!is_zombie(k)) {
    if (!tc::mbar_wait(tc::smem_u32(&k.ctl->full[slot]), (uint32_t)(seq / kNB) & 1u, k.p->spin)) raise_abort(k, 105);
  }
#ifdef BPD_STACK_TRACE
  if (k.tid == 0) k.ctl->cyc_wait += clock64() - t0;
#endif
  return k.ring + *reinterpret_cast<volatile int*>(&k.ctl->off[slot]);
}

// ---- exchanges inside the cluster.  Exchange number n uses mbarrier n % 2, phase (n / 2) % 2.
// Thread 0: announce how many bytes exchange n will bring into this CTA (any time before waiting for it).
__device__ __forceinline__ void xchg_expect(const Cta& k, int n, uint32_t bytes) {
  tc::mbar_expect_tx(tc::smem_u32(&k.ctl->ex[n & 1]), bytes);
}
// One thread per destination: copy `bytes` from `src` (this CTA) to `dst_local_equiv`'s counterpart in CTA `rank`.
__device__ __forceinline__ void xchg_send(const Cta& k, int n, int rank, const void* dst_local_equiv, const void* src, uint32_t bytes) {
  if (is_zombie(k)) return;                // after an expired wait nothing new goes into flight
  dsmem_bulk(map_rank(tc::smem_u32(dst_local_equiv), rank), tc::smem_u32(src), bytes, map_rank(tc::smem_u32(&k.ctl->ex[n & 1]), rank));
}
// All threads: wait for everything exchange n brings.
__device__ __forceinline__ void xchg_wait(const Cta& k, int n) {
  if (!is_zombie(k)) {
    if (!tc::mbar_wait(tc::smem_u32(&k.ctl->ex[n & 1]), (uint32_t)(n >> 1) & 1u, k.p->spin)) raise_abort(k, 106);
  }
}

// A cluster's share of a projection output travels to the other clusters as 64-bit words (value bits, tag): the tag
// is the number of the reduction in this session (never reused), and an aligned 64-bit store is indivisible, so a
// reader that sees the tag has the value -- no fence, no counter, one trip through L2 instead of three.
__device__ __forceinline__ void ll_store(unsigned long long* at, float v, unsigned tag) {
  asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(at), "l"(((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(v)) : "memory");
}
__device__ __forceinline__ void ll_load2(const unsigned long long* at, unsigned long long& a, unsigned long long& b) {
  asm volatile("ld.volatile.global.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(at) : "memory");
}

// ------------------------------------------------------------------ x slice: reduce, planes, statistics
// Static words of a thread's (at most two) items, fetched before the join: four gains or four bias values each.
struct Words { uint2 w[2]; };
__device__ __forceinline__ Words load_words(const Cta& k, const bf16* v) {
  Words o;
  const int n4 = k.g.ks >> 2;
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int idx = k.tid + u * kThreads;
    o.w[u] = (v != nullptr && idx < k.p->R * n4) ? *reinterpret_cast<const uint2*>(v + k.c * k.g.ks + (idx & (n4 - 1)) * 4) : make_uint2(0u, 0u);
  }
  return o;
}
// After a join: x[t][col] += bias[col] + sum over the H clusters' partial outputs, in cluster order, for this
// rank's columns.  Item = (row, four columns); rows are aligned to groups of lanes.  The loads of up to 16
// partials are all in flight before the first is added.
__device__ __forceinline__ void reduce_slice(const Cta& k, float* x_s, const unsigned long long* ws, const Words& bias,
                                             unsigned tag, int nfree) {
  const StackParams& p = *k.p;
  const int ks = k.g.ks, n4 = ks >> 2, R = p.R, d = p.d, H = p.H;
  __syncthreads();                                             // every warp is done with the tiles released here
  if (k.tid == kPumpThread && nfree) release_tiles(k, nfree);
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int idx = k.tid + it * kThreads;
    if (idx >= R * n4) break;
    const int t = idx >> k.g.lg_n4, c4 = idx & (n4 - 1);
    const unsigned long long* src = ws + (size_t)t * d + k.c * ks + c4 * 4;
    const size_t step = (size_t)kMaxRows * d;
    float4 acc = *reinterpret_cast<const float4*>(x_s + t * ks + c4 * 4);
    {
      const uint2 bw = bias.w[it];
      acc.x += __uint_as_float(bw.x << 16); acc.y += __uint_as_float(bw.x & 0xffff0000u);
      acc.z += __uint_as_float(bw.y << 16); acc.w += __uint_as_float(bw.y & 0xffff0000u);
    }
    for (int p0 = 0; p0 < H; p0 += 8) {
      // eight producers per round; a round is repeated as a whole until every word carries this reduction's tag
      unsigned long long v[8][4];
      const unsigned long long t0 = clock64();
      for (unsigned spins = 0;; ++spins) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const unsigned long long* at = src + (size_t)min(p0 + u, H - 1) * step;
          ll_load2(at, v[u][0], v[u][1]);
          ll_load2(at + 2, v[u][2], v[u][3]);
        }
        bool ready = true;
#pragma unroll
        for (int u = 0; u < 8; ++u)
          ready = ready && (unsigned)(v[u][0] >> 32) == tag && (unsigned)(v[u][1] >> 32) == tag &&
                  (unsigned)(v[u][2] >> 32) == tag && (unsigned)(v[u][3] >> 32) == tag;
        if (ready || is_zombie(k)) break;
        if ((spins & 15u) == 15u) {
          if (__ldcg(p.bar + kBarAbort) != 0u) { *reinterpret_cast<volatile int*>(&k.ctl->zombie) = 1; break; }
          if ((unsigned long long)(clock64() - t0) > p.spin) { raise_abort(k, 104); break; }
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (p0 + u < H) {
          acc.x += __uint_as_float((unsigned)v[u][0]); acc.y += __uint_as_float((unsigned)v[u][1]);
          acc.z += __uint_as_float((unsigned)v[u][2]); acc.w += __uint_as_float((unsigned)v[u][3]);
        }
    }
    *reinterpret_cast<float4*>(x_s + t * ks + c4 * 4) = acc;
  }
}

// The same for models with many heads, where every CTA pulling all H shares of its slice (H * 8 KB through L2, H-fold
// redundant over the clusters) is what takes the time: cluster j sums only part j of the slice (2R of the slice's
// R * ks / 4 four-value items; one (item, producer) load per thread, the 16 producers added by a fixed butterfly)
// and publishes the sums, again as tagged words; every cluster then gathers the H parts.  Two trips through L2 but
// 16 KB per CTA instead of 128.
__device__ __forceinline__ bool ll_wait4(const Cta& k, const unsigned long long* at, unsigned tag, float4& out) {
  const StackParams& p = *k.p;
  unsigned long long a0, a1, a2, a3;
  const unsigned long long t0 = clock64();
  for (unsigned spins = 0;; ++spins) {
    ll_load2(at, a0, a1);
    ll_load2(at + 2, a2, a3);
    if (((unsigned)(a0 >> 32) == tag && (unsigned)(a1 >> 32) == tag && (unsigned)(a2 >> 32) == tag && (unsigned)(a3 >> 32) == tag) ||
        is_zombie(k))
      break;
    if ((spins & 15u) == 15u) {
      if (__ldcg(p.bar + kBarAbort) != 0u) { *reinterpret_cast<volatile int*>(&k.ctl->zombie) = 1; break; }
      if ((unsigned long long)(clock64() - t0) > p.spin) { raise_abort(k, 104); break; }
    }
  }
  out = make_float4(__uint_as_float((unsigned)a0), __uint_as_float((unsigned)a1), __uint_as_float((unsigned)a2), __uint_as_float((unsigned)a3));
  return true;
}
__device__ __forceinline__ void reduce_slice_2hop(const Cta& k, float* x_s, const unsigned long long* ws, unsigned long long* gather,
                                                  const Words& bias, unsigned tag, int nfree) {
  const StackParams& p = *k.p;
  const int ks = k.g.ks, n4 = ks >> 2, R = p.R, d = p.d, H = p.H, j = blockIdx.y;
  __syncthreads();                                             // every warp is done with the tiles released here
  if (k.tid == kPumpThread && nfree) release_tiles(k, nfree);
  const int ipp = (R * n4) / H;                                // items of a part: n4 = 2H, so 2R
  const size_t step = (size_t)kMaxRows * d;
  // hop 1: (item q of part j, producer h) per thread; H = 16, so the 16 producers of an item sit in one half-warp
  // and are added by a fixed butterfly (ipp * H = 32 R pairs: whole warps are in or out); lane 0's order is the sum
  for (int w = k.tid; w < ipp * H; w += kThreads) {
    const int q = w >> 4, h = w & 15;
    const int item = j * ipp + q, t = item >> k.g.lg_n4, c4 = item & (n4 - 1);
    float4 v;
    ll_wait4(k, ws + (size_t)h * step + (size_t)t * d + k.c * ks + c4 * 4, tag, v);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      v.x += __shfl_xor_sync(0xffffffffu, v.x, o); v.y += __shfl_xor_sync(0xffffffffu, v.y, o);
      v.z += __shfl_xor_sync(0xffffffffu, v.z, o); v.w += __shfl_xor_sync(0xffffffffu, v.w, o);
    }
    if (h == 0) {
      unsigned long long* at = gather + (size_t)t * d + k.c * ks + c4 * 4;
      ll_store(at, v.x, tag); ll_store(at + 1, v.y, tag); ll_store(at + 2, v.z, tag); ll_store(at + 3, v.w, tag);
    }
  }
  // hop 2: every cluster gathers the whole slice
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int idx = k.tid + it * kThreads;
    if (idx >= R * n4) break;
    const int t = idx >> k.g.lg_n4, c4 = idx & (n4 - 1);
    float4 acc = *reinterpret_cast<const float4*>(x_s + t * ks + c4 * 4);
    {
      const uint2 bw = bias.w[it];
      acc.x += __uint_as_float(bw.x << 16); acc.y += __uint_as_float(bw.x & 0xffff0000u);
      acc.z += __uint_as_float(bw.y << 16); acc.w += __uint_as_float(bw.y & 0xffff0000u);
    }
    float4 v;
    ll_wait4(k, gather + (size_t)t * d + k.c * ks + c4 * 4, tag, v);
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    *reinterpret_cast<float4*>(x_s + t * ks + c4 * 4) = acc;
  }
}

// Self test of the bounded wait on tagged words: one warp waits for a tag that nobody writes, gives up after
// `limit_cycles`, records the error code a real pass would (104) and raises the abort word; the kernel returns
// normally and the context stays usable.
static __device__ unsigned long long g_probe_words[4];
static __device__ unsigned g_probe_bar[kBarWords];
static __global__ void tagged_wait_probe_kernel(int* error, unsigned long long limit_cycles) {
  __shared__ Ctl ctl;
  __shared__ StackParams sp;
  if (threadIdx.x == 0) {
    ctl.zombie = 0;
    sp.error = error; sp.bar = g_probe_bar; sp.spin = limit_cycles;
    g_probe_bar[kBarAbort] = 0u;
    for (int i = 0; i < 4; ++i) g_probe_words[i] = 0ull;          // tag 0: never the tag of a reduction
  }
  __syncthreads();
  Cta k;
  k.p = &sp; k.ctl = &ctl; k.tid = threadIdx.x;
  float4 v;
  ll_wait4(k, g_probe_words, 1u, v);
  __syncthreads();
  if (threadIdx.x == 0 && (ctl.zombie == 0 || g_probe_bar[kBarAbort] == 0u)) atomicExch(error, -1);   // the wait ended some other way
}

// Planes (hi, lo) of x * gain for this rank's columns, and the slice's per-row (mean, sum of squared deviations)
// into this rank's block of the statistics table (sent to the other ranks with the next exchange).  A thread
// reads back the items it wrote itself in reduce_slice / the embedding (same idx -> thread mapping): no barrier
// is needed in between.
template <int NT>
__device__ __forceinline__ void planes_and_stats(const Cta& k, const float* x_s, const Words& gain, uint8_t* xh, uint8_t* xl,
                                                 float* stats_mine) {
  const StackParams& p = *k.p;
  const int ks = k.g.ks, n4 = ks >> 2, R = p.R, PW = k.g.PW;
  constexpr int RP = NT * 8;
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int idx = k.tid + it * kThreads;
    if (idx >= ((R * n4 + 31) & ~31)) break;                 // whole warps leave together
    const bool live = idx < R * n4;
    const int t = live ? idx >> k.g.lg_n4 : 0, c4 = live ? idx & (n4 - 1) : 0;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live) {
      v = *reinterpret_cast<const float4*>(x_s + t * ks + c4 * 4);
      const uint2 gw = gain.w[it];
      const float w[4] = {v.x * __uint_as_float(gw.x << 16), v.y * __uint_as_float(gw.x & 0xffff0000u),
                          v.z * __uint_as_float(gw.y << 16), v.w * __uint_as_float(gw.y & 0xffff0000u)};
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) fused::split_bits(w[e], hi[e], lo[e]);
      const int col = c4 * 4, panel = col >> k.g.lg_pw, within = col & (PW - 1);
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
    if (live && c4 == 0) { stats_mine[t * 2] = mean; stats_mine[t * 2 + 1] = m2; }
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

// Attention output element `dim` of row `token` into this CTA's planes (the row goes to the other ranks by bulk copy).
__device__ __forceinline__ void store_attn_out(uint8_t* oh, uint8_t* ol, int token, int dim, float v) {
  uint32_t hi, lo;
  fused::split_bits(v, hi, lo);
  const uint32_t at = swz((uint32_t)(token * 128 + dim * 2), 7u);
  *reinterpret_cast<unsigned short*>(oh + at) = (unsigned short)hi;
  *reinterpret_cast<unsigned short*>(ol + at) = (unsigned short)lo;
}

// Partial sums in `outbox` ([destination][chunk_bytes]) to every rank (the receiver finds sender c's chunk at
// inbox[c]) and this rank's block of the statistics table to every other rank: exchange n.
__device__ __forceinline__ void send_partials(const Cta& k, int n, const float* outbox, float* inbox, uint32_t chunk_bytes, float* stats_in,
                                              int nfree) {
  fence_async_smem();
  __syncthreads();
  if (k.tid == kPumpThread && nfree) release_tiles(k, nfree);   // behind the barrier: every warp is done with those tiles
  if (k.tid == 0) xchg_expect(k, n, kC * chunk_bytes + (kC - 1) * kMaxRows * 8u);
  if (k.tid < kC) {
    xchg_send(k, n, k.tid, reinterpret_cast<const uint8_t*>(inbox) + k.c * chunk_bytes,
              reinterpret_cast<const uint8_t*>(outbox) + k.tid * chunk_bytes, chunk_bytes);
    if (k.tid != k.c) xchg_send(k, n, k.tid, stats_in + k.c * kMaxRows * 2, stats_in + k.c * kMaxRows * 2, kMaxRows * 8u);
  }
  xchg_wait(k, n);
}

// One chunk of 32 key / value rows for fused::chunk_fold, like fused::chunk_fetch, except that rows of the block
// being scored (chunk rows >= first_new) come from shared memory, where every rank holds all rows of the block
// (new_rows: the row of the sequence's first block position; 512 bytes per row: key, value, scaled query), and
// only committed positions come from the cache.
__device__ __forceinline__ void chunk_fetch_mixed(const bf16* Kc, const bf16* Vc, size_t base, int nk, long long ldkv, int lane,
                                                  uint4 (&kq)[8], uint32_t (&vq)[32], const uint8_t* new_rows, int first_new) {
  const int grp = lane >> 3, seg = lane & 7;
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int r = min(4 * u + grp, nk - 1);
    if (r >= first_new) kq[u] = *reinterpret_cast<const uint4*>(new_rows + (r - first_new) * 512 + seg * 16);
    else kq[u] = __ldcg(reinterpret_cast<const uint4*>(Kc + base + (size_t)r * ldkv) + seg);
  }
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int r = min(j, nk - 1);
    if (r >= first_new) vq[j] = *reinterpret_cast<const uint32_t*>(new_rows + (r - first_new) * 512 + 128 + lane * 4);
    else vq[j] = __ldcg(reinterpret_cast<const uint32_t*>(Vc + base + (size_t)r * ldkv) + lane);
  }
}

// This rank's rows of `buf` (tokens slot * 8 + c, `row_bytes` each, one or two pieces `piece_stride` apart) to every
// other rank of the cluster: exchange n.
// The rows are a few hundred bytes per destination: the threads' own 16-byte asynchronous stores (one or two per
// thread, straight out of this CTA's rows, no staging fence) arrive sooner than bulk copies set up for so little --
// measured on the headline shape: 0.3-0.5 us per exchange.  The larger exchanges (partial sums, hidden units: up to
// a kilobyte per destination) stay bulk copies: as per-thread stores they measured slower.
template <int NT>
__device__ __forceinline__ void send_rows(const Cta& k, int n, uint8_t* buf0, uint8_t* buf1, uint32_t row_bytes, int nfree) {
  __syncthreads();
  if (k.tid == kPumpThread && nfree) release_tiles(k, nfree);   // behind the barrier: every warp is done with those tiles
  int mine = 0;
#pragma unroll
  for (int slot = 0; slot < NT; ++slot) mine += (slot * kC + k.c < k.p->R) ? 1 : 0;
  if (k.tid == 0) xchg_expect(k, n, (uint32_t)(k.p->R - mine) * row_bytes * (buf1 ? 2u : 1u));
  if (!is_zombie(k)) {                     // after an expired wait nothing new goes into flight
    const int ppr = (int)(row_bytes >> 4), per_dst = mine * ppr * (buf1 ? 2 : 1);
    const uint32_t bar = tc::smem_u32(&k.ctl->ex[n & 1]);
    for (int idx = k.tid; idx < (kC - 1) * per_dst; idx += kThreads) {
      const int di = idx / per_dst, piece = idx - di * per_dst, rank = di < k.c ? di : di + 1;
      const int pb = piece / ppr, off = (piece - pb * ppr) << 4;           // (row, buffer) pair and byte offset in the row
      const int slot = buf1 ? pb >> 1 : pb;
      uint8_t* at = ((buf1 && (pb & 1)) ? buf1 : buf0) + (slot * kC + k.c) * row_bytes + off;
      dsmem_store16(map_rank(tc::smem_u32(at), rank), *reinterpret_cast<const uint4*>(at), map_rank(bar, rank));
    }
  }
  xchg_wait(k, n);
}

// ------------------------------------------------------------------ development trace
#ifdef BPD_STACK_TRACE
__device__ unsigned long long* g_stack_trace = nullptr;
constexpr int kTracePts = 256;
#define BPD_TR() do { if (g_stack_trace && tid == 0 && tp < kTracePts - 4) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); \
                        g_stack_trace[(size_t)(blockIdx.y * kC + c) * kTracePts + tp] = t_; } ++tp; } while (0)
#else
#define BPD_TR() do { } while (0)
#endif

// ------------------------------------------------------------------ the kernel
// grid = (8, H), clusters of 8 along x.  All clusters must be resident at once (the host checks the occupancy).
// MINB: CTAs per SM the kernel is compiled for.  Models with at most 15 heads have an SM to themselves per CTA (no
// register limit to speak of); 16 clusters only fit with two CTAs on some SMs, which caps the registers at 128.
// LEAN: sessions whose cache holds at most 256 positions and whose encoder rows are staged by TMA carry only that
// path (the short self-attention schedule, the staged cross-attention); the general kernel needs far more than the
// 128 registers a thread has when two CTAs share an SM.
template <int NT, int KS, int MINB, bool LEAN>
__global__ void __cluster_dims__(kC, 1, 1) __launch_bounds__(kThreads, MINB)
layer_stack_kernel(const __grid_constant__ StackMaps maps, const __grid_constant__ StackParams p) {
  extern __shared__ __align__(1024) uint8_t ssm_raw[];
  // swizzled tiles need 1024-byte alignment (the launch carries 1024 bytes of slack for this)
  uint8_t* ssm = ssm_raw + ((1024u - (tc::smem_u32(ssm_raw) & 1023u)) & 1023u);
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int RP = NT * 8;
  Cta k;
  k.p = &p;
  k.maps = &maps;
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
  uint8_t* hid = ssm + p.lay.hid;                                         // [rank][plane][RP][UPR * 2 bytes]
  float* outbox = reinterpret_cast<float*>(ssm + p.lay.outbox);           // [destination][chunk]
  float* inbox = reinterpret_cast<float*>(ssm + p.lay.inbox);             // [source][chunk]
  uint8_t* kvq = ssm + p.lay.kvq;                                         // [RP][key 128 B | value 128 B | scaled query 256 B]
  float* stats_in = reinterpret_cast<float*>(ssm + p.lay.stats);          // [rank][kMaxRows][2]
  float* s_mean = stats_in + kC * kMaxRows * 2;
  float* s_rstd = s_mean + kMaxRows;
  int* s_len = reinterpret_cast<int*>(s_rstd + kMaxRows);                 // [kMaxRows] cache lengths of the sequences
  int* s_src = s_len + kMaxRows;                                          // [kMaxRows] source lengths
  AttnSmem<kDH, kWarps>& sm = *reinterpret_cast<AttnSmem<kDH, kWarps>*>(ssm + p.lay.attn);
  float* wst = reinterpret_cast<float*>(ssm + p.lay.wst);                 // [warp][slot][kState]
  float* lvl1 = reinterpret_cast<float*>(ssm + p.lay.lvl1);
  float* lvl2 = reinterpret_cast<float*>(ssm + p.lay.lvl2);
  int* s_pt = reinterpret_cast<int*>(ssm + p.lay.pt);
  LayerPtrs* layers_s = reinterpret_cast<LayerPtrs*>(ssm + p.lay.layers);
  float* stats_mine = stats_in + c * kMaxRows * 2;
  const int hrow = g.UPR * 2;                                             // bytes per row of a rank's hidden planes
  const int hblock = 2 * RP * hrow;                                       // bytes of a rank's hidden planes (hi, lo)

  if (tid == 0) {
    for (int i = 0; i < kNB; ++i) tc::mbar_init(tc::smem_u32(&k.ctl->full[i]), 1);
    tc::mbar_init(tc::smem_u32(&k.ctl->ex[0]), 1);
    tc::mbar_init(tc::smem_u32(&k.ctl->ex[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    k.ctl->head = 0; k.ctl->issued = 0; k.ctl->freed = 0; k.ctl->zombie = 0; k.ctl->issue_layer = 0; k.ctl->issue_idx = 0;
#ifdef BPD_STACK_TRACE
    k.ctl->cyc_wait = 0; k.ctl->cyc_pump = 0; k.ctl->cyc_poll = 0;
#endif
  }
  if (tid < g.ntl) k.ctl->tiles[tid] = make_tile(g, tid, p.cross_rows, d, c, j);
  __syncthreads();
  // Weights and page tables do not depend on anything earlier in the stream.  The encoder's keys and values do:
  // the launches before this one (the encoder's, right after bpd_encode) may still be running, so the first
  // tile that carries them is not requested before the dependency wait.
  if (tid == kPumpThread) pump(k, g.staged ? g.P + 2 : 0x7fffffff);
  for (int i = tid; i < nb * p.st.pages_per_row; i += kThreads) s_pt[i] = p.st.page_table[i];
  for (int i = tid; i < p.L * (int)(sizeof(LayerPtrs) / 8); i += kThreads)
    reinterpret_cast<unsigned long long*>(layers_s)[i] = reinterpret_cast<const unsigned long long*>(p.layers)[i];
  // rows beyond R of the planes are never written: zero them once so that no NaN pattern reaches an MMA
  for (int i = tid; i < (p.lay.outbox - p.lay.xh) / 16; i += kThreads) reinterpret_cast<uint4*>(ssm + p.lay.xh)[i] = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < kC * kMaxRows * 2; i += kThreads) stats_in[i] = 0.f;
  pdl_wait();
  if (p.all_done && *p.all_done) {
    // nothing to do: let what was requested land (bounded), then leave
    __syncthreads();
    if (tid == kPumpThread)
      for (int s = k.ctl->freed; s < k.ctl->issued; ++s) tc::mbar_wait(tc::smem_u32(&k.ctl->full[s % kNB]), (uint32_t)(s / kNB) & 1u, p.spin);
    return;
  }
  if (tid == kPumpThread) pump(k);
  const unsigned base = __ldcg(p.bar + kBarBase);
  if (tid < nb) { s_len[tid] = p.st.len[tid]; s_src[tid] = p.st.src_len[tid]; }
  __syncthreads();

  // ---- embedding of the block: x[t] = E[token] sqrt(d) + PE(position), this rank's columns
  {
    const int n4 = ks >> 2;
    const float scale = sqrtf((float)d);
    for (int idx = tid; idx < R * n4; idx += kThreads) {
      const int t = idx >> g.lg_n4, c4 = idx & (n4 - 1);
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
  fused::cluster_wait();                    // every CTA of the cluster runs: its shared memory and mbarriers may be written

  AttnParams ap;
  memset(&ap, 0, sizeof(ap));
  ap.rows = R; ap.rows_per_b = rpb; ap.H = p.H; ap.dh = kDH; ap.causal = 1; ap.local_q = p.local_q; ap.local_m = p.local_m;
  ap.ldkv = d; ap.paged = 1; ap.st = p.st; ap.st.page_table = s_pt; ap.scale = p.scale;
  bool one_chunk_per_rank = true;
  if (!LEAN) {
    for (int b = 0; b < nb; ++b)
      one_chunk_per_rank = one_chunk_per_rank && ((s_len[b] + rpb + 31) >> 5) - (attn_first_key(ap, s_len[b]) >> 5) <= kC;
  }

  unsigned nbar = 0;                        // joins passed so far in this launch
  int seq = 0;                              // next tile to consume
  int xn = 0;                               // exchanges inside the cluster so far
#ifdef BPD_STACK_TRACE
  int tp = 0;
  if (g_stack_trace && tid == 0) {
    unsigned smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    g_stack_trace[(size_t)(blockIdx.y * kC + c) * kTracePts + kTracePts - 1] = smid;
  }
#endif
  BPD_TR();
  // this lane's ldmatrix offsets: weight boxes (row lane % 16, second half of the step for lanes >= 16) and planes
  // (token lane % 8, second half for lanes 8-15 and 24-31; lanes >= 16 address the lo plane)
  const uint32_t a_lane_row = (uint32_t)(lane & 15), a_lane_half = (uint32_t)(lane >> 4) * 16;
  const uint32_t b_lane_row = (uint32_t)(lane & 7), b_lane_half = (uint32_t)((lane >> 3) & 1) * 16;
  const bool b_lo = (lane & 16) != 0;
  constexpr uint32_t xrow = KS * 32;                                      // bytes per row of an x panel (KS steps of 16 columns)
  const uint32_t x_plane = b_lo ? tc::smem_u32(xl) : tc::smem_u32(xh);
  const uint32_t o_plane = b_lo ? tc::smem_u32(ol) : tc::smem_u32(oh);
  // swizzled once: a step of 16 columns further only flips bits 5-6 of these (all bases are 128-byte aligned)
  const uint32_t ax_pre = swz(a_lane_row * xrow + a_lane_half, g.xmask), bx_pre = swz(b_lane_row * xrow + b_lane_half, g.xmask);
  const uint32_t ao_pre = swz(a_lane_row * 128 + a_lane_half, 7u), bo_pre = swz(b_lane_row * 128 + b_lane_half, 7u);

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
      ++nbar;
      BPD_TR();
      if (p.H == 16) reduce_slice_2hop(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, p.gather + (size_t)((nbar - 1) & 1) * kMaxRows * d, bw, base + nbar, g.PH);
      else reduce_slice(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, bw, base + nbar, g.PH);
      BPD_TR();
      if (p.layer_dump && j == 0) {
        __syncthreads();
        for (int idx = tid; idx < R * ks; idx += kThreads)
          p.layer_dump[((size_t)(l - 1) * R + idx / ks) * d + c * ks + idx % ks] = x_s[idx];
      }
    }
    planes_and_stats<NT>(k, x_s, gw, xh, xl, stats_mine);
    __syncthreads();
    BPD_TR();
    // Q, K, V of the head over this rank's columns; token t's partial goes to rank t % 8
    for (int mt = warp; mt < 3 * kDH / 16; mt += kWarps) {
      float acc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
      for (int q = 0; q < g.P; ++q) {
        const uint32_t a = tile_wait(k, seq + q) + ((mt / 4) * 64 + (mt % 4) * 16) * xrow, b = x_plane + q * RP * xrow;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) mma_step<NT>(acc, a + (ax_pre ^ (kk << 5)), b + (bx_pre ^ (kk << 5)), 8 * xrow);
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int row = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
          if (token < R) outbox[((token % kC) * NT + token / kC) * 3 * kDH + row] = acc[nt][e];
        }
    }
    seq += g.P;
    BPD_TR();
    send_partials(k, xn, outbox, inbox, NT * 3 * kDH * 4, stats_in, g.P);
    ++xn;
    BPD_TR();
    merge_stats(k, stats_in, s_mean, s_rstd);
    __syncthreads();
    // this rank's tokens: partials in rank order, layer norm; the row's key and value (rounded as the cache holds
    // them) go into the cache for later passes and, with the scaled query, into this rank's copy of the block's rows
    for (int slot = 0; slot < NT; ++slot) {
      const int token = slot * kC + c;
      if (token < R && tid < 3 * kDH) {
        float a = 0.f;
#pragma unroll
        for (int src = 0; src < kC; ++src) a += inbox[(src * NT + slot) * 3 * kDH + tid];
        const int sect = tid / kDH, f = tid % kDH;
        const float y = s_rstd[token] * (a - s_mean[token] * fs) + fc;
        uint8_t* row = kvq + token * 512;
        if (sect == 0) {
          reinterpret_cast<float*>(row + 256)[f] = y * p.scale;
        } else {
          const int b = token / rpb, i = token % rpb;
          const int pos = s_len[b] + i;
          const int page = s_pt[b * p.st.pages_per_row + pos / kPage];
          const size_t at = ((size_t)page * kPage + (pos % kPage)) * d + j * kDH + f;
          const bf16 yb = __float2bfloat16_rn(y);
          (sect == 1 ? LP.kcache : LP.vcache)[at] = yb;
          reinterpret_cast<bf16*>(row + (sect - 1) * 128)[f] = yb;
        }
      }
    }
    send_rows<NT>(k, xn, kvq, nullptr, 512, 0);  // every rank now holds the keys, values and queries of all block rows
    ++xn;
    BPD_TR();
    {
      ap.k = LP.kcache; ap.v = LP.vcache;
      const bf16* Kc = LP.kcache;
      const bf16* Vc = LP.vcache;
      if (LEAN || one_chunk_per_rank) {
        // this rank attends for its own rows; warp w folds the chunk that belongs to rank w
        for (int slot = 0; slot < NT; ++slot) {
          const int token = slot * kC + c;
          if (token < R) {                                           // uniform over the CTA
            const int b = token / rpb, i = token % rpb;
            const int len = s_len[b], lim_max = len + rpb;
            const int fk = attn_first_key(ap, len + i), ch0 = attn_first_key(ap, len) >> 5;
            const int ch = ch0 + ((warp - ch0) & (kC - 1));
            float* state = wst + (warp * NT + slot) * kState;
            if (lane == 0) { state[kDH] = -INFINITY; state[kDH + 1] = 0.f; }
            __syncwarp();
            if ((ch << 5) <= len + i) {
              const int c0 = ch << 5;
              const size_t kbase = ((size_t)s_pt[b * p.st.pages_per_row + c0 / kPage] * kPage + (c0 % kPage)) * d + j * kDH;
              uint4 kq[8];
              uint32_t vq[32];
              chunk_fetch_mixed(Kc, Vc, kbase, min(32, lim_max - c0), d, lane, kq, vq, kvq + (b * rpb) * 512, len - c0);
              const int key = c0 + lane;
              fused::chunk_fold(kq, vq, reinterpret_cast<const float*>(kvq + token * 512 + 256), key <= len + i && key >= fk, state, lane);
            }
            __syncthreads();
            if (tid < kDH) {
              float M, num, den;
              fused::states_merge(wst + slot * kState, NT * kState, tid, M, num, den);
              store_attn_out(oh, ol, token, tid, num / den);
            }
          }
        }
        send_rows<NT>(k, xn, oh, ol, 128, 0);
        ++xn;
      } else {
        // long sequences: rank c folds its own chunks for every row (keys fetched once per sequence), the ranks'
        // states travel through distributed shared memory
        const int RL = R;
        for (int i = tid; i < 8 * RL; i += kThreads) { lvl1[i * kState + kDH] = -INFINITY; lvl1[i * kState + kDH + 1] = 0.f; }
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
            chunk_fetch_mixed(Kc, Vc, kbase, min(32, lim_max - c0), d, lane, kq, vq, kvq + (b * rpb) * 512, len - c0);
            const int key = c0 + lane;
#pragma unroll 1
            for (int i = sub; i < rpb; i += S)
              fused::chunk_fold(kq, vq, reinterpret_cast<const float*>(kvq + (b * rpb + i) * 512 + 256), key <= len + i && key >= attn_first_key(ap, len + i),
                                lvl1 + ((size_t)lump * RL + b * rpb + i) * kState, lane);
          }
        }
        __syncthreads();
        // this rank's state per row (its lumps in lump order) into its block of the table, then to every other rank
        for (int idx = tid; idx < R * kDH; idx += kThreads) {
          const int row = idx / kDH, dim = idx % kDH;
          float M, num, den;
          fused::states_merge(lvl1 + row * kState, RL * kState, dim, M, num, den);
          float* out = lvl2 + (c * RL + row) * kState;
          out[dim] = num;
          if (dim == 0) { out[kDH] = M; out[kDH + 1] = den; }
        }
        fence_async_smem();
        __syncthreads();
        if (tid == 0) xchg_expect(k, xn, (uint32_t)((kC - 1) * RL * kState * 4));
        if (tid < kC && tid != c) xchg_send(k, xn, tid, lvl2 + c * RL * kState, lvl2 + c * RL * kState, (uint32_t)(RL * kState * 4));
        xchg_wait(k, xn);
        ++xn;
        for (int idx = tid; idx < R * kDH; idx += kThreads) {
          const int row = idx / kDH, dim = idx % kDH;
          float M, num, den;
          fused::states_merge(lvl2 + row * kState, RL * kState, dim, M, num, den);
          store_attn_out(oh, ol, row, dim, num / den);
        }
        __syncthreads();
      }
    }
    BPD_TR();
    // this head's share of the output projection for feature slice c
    {
      unsigned long long* wsj = p.ws + ((size_t)(nbar & 1) * p.H + j) * kMaxRows * d;
      const unsigned tag_out = base + nbar + 1;            // the reduction that consumes these shares
      for (int mt = warp; mt < ks / 16; mt += kWarps) {
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
        const uint32_t a = tile_wait(k, seq) + mt * 16 * 128;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) mma_step<NT>(acc, a + (ao_pre ^ (kk << 5)), o_plane + (bo_pre ^ (kk << 5)), 8 * 128);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int row = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
            if (token < R) ll_store(wsj + (size_t)token * d + c * ks + row, acc[nt][e], tag_out);
          }
      }
      seq += 1;
    }
    BPD_TR();

    // =================================================================== cross-attention block
    gw = load_words(k, LP.g2);
    const Words nobias = load_words(k, nullptr);
    if (tid < kDH) { fs = LP.s_cq[j * kDH + tid]; fc = LP.c_cq[j * kDH + tid]; }
    ++nbar;
    BPD_TR();
    if (p.H == 16) reduce_slice_2hop(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, p.gather + (size_t)((nbar - 1) & 1) * kMaxRows * d, nobias, base + nbar, 1);
      else reduce_slice(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, nobias, base + nbar, 1);
    BPD_TR();
    planes_and_stats<NT>(k, x_s, gw, xh, xl, stats_mine);
    __syncthreads();
    BPD_TR();
    for (int mt = warp; mt < kDH / 16; mt += kWarps) {
      float acc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
      const uint32_t a0 = tile_wait(k, seq);
      for (int q = 0; q < g.P; ++q) {
        const uint32_t a = a0 + (q * 64 + mt * 16) * xrow, b = x_plane + q * RP * xrow;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) mma_step<NT>(acc, a + (ax_pre ^ (kk << 5)), b + (bx_pre ^ (kk << 5)), 8 * xrow);
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int row = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
          if (token < R) outbox[((token % kC) * NT + token / kC) * kDH + row] = acc[nt][e];
        }
    }
    seq += 1;
    BPD_TR();
    send_partials(k, xn, outbox, inbox, NT * kDH * 4, stats_in, 1);
    ++xn;
    BPD_TR();
    merge_stats(k, stats_in, s_mean, s_rstd);
    __syncthreads();
    {
      uint32_t ckv = k.ring;
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
          float ov;
          if (LEAN || g.staged) ov = cross_attention_tile(ckv_g, ckv_g + kb, ckv_g + 2 * kb, b * p.max_src, s_src[b], sm);
          else ov = attention_head<float, kDH, kWarps, false>(ap, b, j, 0, s_src[b], sm);
          if (tid < kDH) store_attn_out(oh, ol, token, tid, ov);
          __syncthreads();
        }
      }
      ap.causal = 1; ap.ldkv = d; ap.paged = 1;
      seq += g.staged;
    }
    send_rows<NT>(k, xn, oh, ol, 128, g.staged);
    ++xn;
    BPD_TR();
    {
      unsigned long long* wsj = p.ws + ((size_t)(nbar & 1) * p.H + j) * kMaxRows * d;
      const unsigned tag_out = base + nbar + 1;            // the reduction that consumes these shares
      for (int mt = warp; mt < ks / 16; mt += kWarps) {
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
        const uint32_t a = tile_wait(k, seq) + mt * 16 * 128;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) mma_step<NT>(acc, a + (ao_pre ^ (kk << 5)), o_plane + (bo_pre ^ (kk << 5)), 8 * 128);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int row = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
            if (token < R) ll_store(wsj + (size_t)token * d + c * ks + row, acc[nt][e], tag_out);
          }
      }
      seq += 1;
    }
    BPD_TR();

    // =================================================================== feed-forward block
    gw = load_words(k, LP.g3);
    float fs1[2], fc1[2];                    // folded vectors of the (at most two) hidden units this thread finishes
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int idx = tid + u * kThreads;
      const int unit = j * g.HCt + c * g.UPR + (idx & (g.UPR - 1));
      fs1[u] = idx < g.UPR * R ? LP.s_f1[unit] : 0.f;
      fc1[u] = idx < g.UPR * R ? LP.c_f1[unit] : 0.f;
    }
    ++nbar;
    BPD_TR();
    if (p.H == 16) reduce_slice_2hop(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, p.gather + (size_t)((nbar - 1) & 1) * kMaxRows * d, nobias, base + nbar, 1);
      else reduce_slice(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, nobias, base + nbar, 1);
    BPD_TR();
    planes_and_stats<NT>(k, x_s, gw, xh, xl, stats_mine);
    __syncthreads();
    BPD_TR();
    // the cluster's hidden units over this rank's columns; unit f belongs to rank f / UPR
    for (int mt = warp; mt < g.HCt / 16; mt += kWarps) {
      float acc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
      for (int q = 0; q < g.P; ++q) {
        const uint32_t a = tile_wait(k, seq + q) + mt * 16 * xrow, b = x_plane + q * RP * xrow;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) mma_step<NT>(acc, a + (ax_pre ^ (kk << 5)), b + (bx_pre ^ (kk << 5)), 8 * xrow);
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int f = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
          if (token < R) outbox[f * RP + token] = acc[nt][e];      // destination rank f / UPR, chunks of UPR * RP floats
        }
    }
    seq += g.P;
    BPD_TR();
    send_partials(k, xn, outbox, inbox, g.UPR * RP * 4, stats_in, g.P);
    ++xn;
    BPD_TR();
    merge_stats(k, stats_in, s_mean, s_rstd);
    __syncthreads();
    // ranks in order, layer norm, bias, ReLU -> this rank's block of the hidden planes, which goes to every rank
    {
      uint8_t* mine = hid + c * hblock;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int idx = tid + u * kThreads;
        if (idx >= g.UPR * R) break;
        const int f = idx & (g.UPR - 1), token = idx >> g.lg_upr;
        float a = 0.f;
#pragma unroll
        for (int src = 0; src < kC; ++src) a += inbox[(src * g.UPR + f) * RP + token];
        const float y = fmaxf(s_rstd[token] * (a - s_mean[token] * fs1[u]) + fc1[u], 0.f);
        uint32_t hi, lo;
        fused::split_bits(y, hi, lo);
        const uint32_t at = swz((uint32_t)(token * hrow + f * 2), g.hmask);
        *reinterpret_cast<unsigned short*>(mine + at) = (unsigned short)hi;
        *reinterpret_cast<unsigned short*>(mine + RP * hrow + at) = (unsigned short)lo;
      }
      fence_async_smem();
      __syncthreads();
      if (tid == 0) xchg_expect(k, xn, (uint32_t)((kC - 1) * hblock));
      if (tid < kC && tid != c) xchg_send(k, xn, tid, mine, mine, (uint32_t)hblock);
      xchg_wait(k, xn);
      ++xn;
    }
    BPD_TR();
    // the hidden units times slice c of the second projection: this cluster's share of the block's output
    {
      unsigned long long* wsj = p.ws + ((size_t)(nbar & 1) * p.H + j) * kMaxRows * d;
      const unsigned tag_out = base + nbar + 1;            // the reduction that consumes these shares
      for (int mt = warp; mt < ks / 16; mt += kWarps) {
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
        // step kk of panel q covers hidden units q * 64 + kk * 16 ..: rank (q * 64 + kk * 16) / UPR, offset within its rows
        const uint32_t hb = tc::smem_u32(hid) + (b_lo ? RP * hrow : 0);
        const uint32_t bh_pre = swz(b_lane_row * hrow + b_lane_half, g.hmask);
        for (int q = 0; q < g.PH; ++q) {
          const uint32_t a = tile_wait(k, seq + q) + mt * 16 * 128;
          if (g.UPR == 32) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              mma_step<NT>(acc, a + (ao_pre ^ (kk << 5)), hb + (q * 2 + (kk >> 1)) * hblock + (bh_pre ^ ((kk & 1) << 5)), 8 * hrow);
          } else {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) mma_step<NT>(acc, a + (ao_pre ^ (kk << 5)), hb + (q * 4 + kk) * hblock + bh_pre, 8 * hrow);
          }
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int row = mt * 16 + lg + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
            if (token < R) ll_store(wsj + (size_t)token * d + c * ks + row, acc[nt][e], tag_out);
          }
      }
      seq += g.PH;
    }
    BPD_TR();
  }
  // =================================================================== final layer norm
  {
    const Words bw = load_words(k, layers_s[p.L - 1].b2), gw = load_words(k, p.lnf_g);
    ++nbar;
    BPD_TR();
    pdl_launch_dependents();
    if (p.H == 16) reduce_slice_2hop(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, p.gather + (size_t)((nbar - 1) & 1) * kMaxRows * d, bw, base + nbar, g.PH);
      else reduce_slice(k, x_s, p.ws + (size_t)((nbar - 1) & 1) * p.H * kMaxRows * d, bw, base + nbar, g.PH);
    BPD_TR();
    if (p.layer_dump && j == 0) {
      __syncthreads();
      for (int idx = tid; idx < R * ks; idx += kThreads)
        p.layer_dump[((size_t)(p.L - 1) * R + idx / ks) * d + c * ks + idx % ks] = x_s[idx];
    }
    planes_and_stats<NT>(k, x_s, gw, xh, xl, stats_mine);   // the planes are not used; the statistics are
    BPD_TR();
  }
  fence_async_smem();
  __syncthreads();
  if (tid == 0) xchg_expect(k, xn, (kC - 1) * kMaxRows * 8u);
  if (tid < kC && tid != c) xchg_send(k, xn, tid, stats_mine, stats_mine, kMaxRows * 8u);
  xchg_wait(k, xn);
  ++xn;
  BPD_TR();
  merge_stats(k, stats_in, s_mean, s_rstd);
  __syncthreads();
  if (j == 0) {
    const int n4 = ks >> 2;
    for (int idx = tid; idx < R * n4; idx += kThreads) {
      const int t = idx >> g.lg_n4, col = c * ks + (idx & (n4 - 1)) * 4;
      const float4 v = *reinterpret_cast<const float4*>(x_s + t * ks + (idx & (n4 - 1)) * 4);
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
    if (c == 0 && tid == 0) p.bar[kBarBase] = base + nbar;         // tags of the next launch go on from here
  }
#ifdef BPD_STACK_TRACE
  if (g_stack_trace && tid == 0) {
    unsigned long long* tr = g_stack_trace + (size_t)(blockIdx.y * kC + c) * kTracePts;
    tr[kTracePts - 2] = k.ctl->cyc_wait; tr[kTracePts - 3] = k.ctl->cyc_pump; tr[kTracePts - 4] = k.ctl->cyc_poll;
  }
#endif
  if (tid == kPumpThread && k.ctl->zombie) {
    // a wait expired somewhere: tiles may still be in flight; give each slot's last request a bounded chance to land
    for (int s2 = max(0, k.ctl->issued - kNB); s2 < k.ctl->issued; ++s2)
      tc::mbar_wait(tc::smem_u32(&k.ctl->full[s2 % kNB]), (uint32_t)(s2 / kNB) & 1u, p.spin);
  }
  // nobody leaves while a copy out of (or into) its shared memory may still be under way: every CTA of the cluster
  // has seen its last exchange complete by the time this barrier opens
  cluster.sync();
}

}  // namespace stack
}  // namespace bpd
