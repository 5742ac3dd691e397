// Decoder layers for sessions with few rows per pass (batch 1, at most 16 rows): three launches per layer
// instead of eight.
//
// With so few rows a decoder layer is a chain of eight small dependent steps, and the time goes to what separates
// them (launch, a trip to L2 and back, a device-wide join), not to the 29 MB of weights.  Most of those joins are
// not needed: a head's attention only needs that head's 3 x 64 query/key/value features, and the output
// projection is a sum over heads.  So
//
//   attn_block_kernel<SELF>   layer norm -> Q,K,V of one head -> cache write -> attention -> that head's share of
//                             the output projection -> sum over heads + residual
//   attn_block_kernel<CROSS>  layer norm -> Q of one head -> attention over the encoder keys -> same tail
//   ffn_block_kernel          layer norm -> the cluster's 128 hidden units, each CTA over its part of the reduction
//                             -> 16 of them finished per CTA (ReLU) and shared with the cluster -> the 128 hidden
//                             units times this CTA's slice of the second projection -> sum over clusters + bias
//                             + residual
//
// One thread-block cluster of kC CTAs works on a head (or on kC * 16 hidden units).  In the attention blocks the
// reduction length of the input projection is split over the CTAs and partial sums travel through distributed
// shared memory, always added in rank order; in the feed-forward block the CTAs exchange their hidden units.  Across clusters the partial outputs go through a small workspace and the last cluster to arrive adds
// them in cluster order, so every element is the same sum in the same order however many rows a pass carries.
// Weights are static: every CTA starts copying its slice into shared memory before it waits for the previous
// launch (programmatic dependent launch), which takes HBM latency off the chain.
//
// The products are tiny (at most 16 columns), so they run on mma.sync (m16n8k16, bf16 in, fp32 out) straight
// from shared memory; activations are two bf16 planes (hi + lo) as everywhere else on the tensor-core path.
#pragma once
#include <cooperative_groups.h>

#include "gemm_tc.cuh"
#include "kernels_simt.cuh"

namespace bpd {
namespace fused {

namespace cg = cooperative_groups;

constexpr int kC = 8;            // CTAs per cluster
constexpr int kThreads = 256;
constexpr int kWarps = 8;
constexpr int kDH = 64;          // head width this path is built for
constexpr int kHS = 16;          // hidden units per CTA in the feed-forward block
constexpr int kMaxRows = 16;
constexpr int kCrossKeyPitch = kDH * 4 + 16;   // bytes per staged encoder key row (fp32): 16-byte reads of 8 lanes hit all banks
constexpr int kCrossRowBytes = kCrossKeyPitch + kDH * 4;   // key row + value row
constexpr int kCrossStageMax = 24 * 1024;      // more encoder rows than fit here are read from L2 instead
constexpr int kPartial = kDH + 2;   // a partial attention state: weighted value sum [kDH], running maximum, weight sum

// Byte offset of (row, byte) in a shared-memory matrix with rb bytes per row (a multiple of 64).  When rb is a
// multiple of 128 the two 64-byte halves of every 128 bytes trade places in odd rows, so that the 16-byte
// fragment loads of eight lanes (two rows x four quarters) cover all 32 banks once; 64-byte rows do so as they are.
__host__ __device__ inline int sw(int row, int byte, int rb) { return row * rb + ((rb & 127) ? byte : (byte ^ ((row & 1) << 6))); }

// 16 bytes of weights, global -> shared, marked "evict first" in L2 (they are read once per pass).
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, unsigned long long policy) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(tc::smem_u32(smem)), "l"(gmem), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async16_keep(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(tc::smem_u32(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
// Cluster barrier in two halves (all threads of the CTA execute both).  The first pair of a kernel only makes
// sure that every CTA of the cluster is running before anybody writes into its shared memory.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// v = hi + lo with hi, lo bf16 (as 16-bit patterns).
__device__ __forceinline__ void split_bits(float v, uint32_t& hi, uint32_t& lo) {
  bf16 h, l;
  tc::split_bf16(v, h, l);
  hi = __bfloat16_as_ushort(h);
  lo = __bfloat16_as_ushort(l);
}

// acc[nt] += W(16 rows x K) * X(K x 8 tokens of tile nt), X = hi + lo planes, over columns [kb0/2, kb0/2 + K).
// w: first of 16 weight rows (an even row of a matrix laid out by sw() with sw_ bytes per row); xh / xl: planes,
// one row per token (sx bytes per row, same lay-out).  K is a multiple of 32.  The contraction index is permuted
// inside each group of 32 so that a lane's fragments are 16 contiguous bytes: lane (g, t) takes k = 8t..8t+7 of
// rows g and g+8 and of token g, and uses them as slots {2t, 2t+1, 2t+8, 2t+9} of two successive MMAs -- the same
// permutation on both operands.
// acc[nt][0..3] = (row g, token 2t), (row g, token 2t+1), (row g+8, token 2t), (row g+8, token 2t+1).
template <int NT>
__device__ __forceinline__ void mma_rows16(float (&acc)[NT][4], const uint8_t* w, int sw_, const uint8_t* xh, const uint8_t* xl,
                                           int sx, int K, int lane, int kb0 = 0) {
  const int g = lane >> 2, t = lane & 3;
  const int flip_w = (sw_ & 127) ? 0 : ((g & 1) << 6), flip_x = (sx & 127) ? 0 : ((g & 1) << 6);
  const uint8_t* w0 = w + g * sw_;
  const uint8_t* w1 = w0 + 8 * sw_;
  for (int k0 = 0; k0 < K; k0 += 32) {
    const int kb = kb0 + k0 * 2 + t * 16;
    const uint4 a = *reinterpret_cast<const uint4*>(w0 + (kb ^ flip_w));
    const uint4 b = *reinterpret_cast<const uint4*>(w1 + (kb ^ flip_w));
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const uint4 h = *reinterpret_cast<const uint4*>(xh + (nt * 8 + g) * sx + (kb ^ flip_x));
      const uint4 l = *reinterpret_cast<const uint4*>(xl + (nt * 8 + g) * sx + (kb ^ flip_x));
      mma_bf16(acc[nt], a.x, b.x, a.y, b.y, h.x, h.y);
      mma_bf16(acc[nt], a.x, b.x, a.y, b.y, l.x, l.y);
      mma_bf16(acc[nt], a.z, b.z, a.w, b.w, h.z, h.w);
      mma_bf16(acc[nt], a.z, b.z, a.w, b.w, l.z, l.w);
    }
  }
}

// Per-token mean and 1/std of the rows of the residual stream.  One warp per token (tokens w, w+8), every lane
// the same fixed share of the row (d is a multiple of 128), one pass: each lane sums its share about its own
// first element, then the 32 partial (mean, M2) pairs -- all over equally many elements -- are merged pairwise in
// a fixed order: mean = (mean_a + mean_b) / 2, M2 = M2_a + M2_b + (mean_b - mean_a)^2 * n / 2 with n elements on
// each side.  Rows come from L2 (another launch wrote them), eight loads per lane in flight.
__device__ __forceinline__ void rows_stats(const float* __restrict__ x, int R, int d, float eps, float* s_mean, float* s_rstd) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nv = d >> 2;
  constexpr int kBatch = 8;
  const float per_lane = (float)(d >> 5), inv_per_lane = 1.0f / per_lane;
  for (int tk = warp; tk < R; tk += kWarps) {
    const float4* xr = reinterpret_cast<const float4*>(x + (size_t)tk * d);
    float shift = 0.f, a1 = 0.f, a2 = 0.f;
    for (int i0 = lane; i0 < nv; i0 += 32 * kBatch) {
      float4 buf[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) buf[u] = (i0 + 32 * u < nv) ? __ldcg(&xr[i0 + 32 * u]) : make_float4(0.f, 0.f, 0.f, 0.f);
      if (i0 == lane) shift = buf[0].x;
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        if (i0 + 32 * u < nv) {
          const float4 a = buf[u];
          const float d0 = a.x - shift, d1 = a.y - shift, d2 = a.z - shift, d3 = a.w - shift;
          a1 += (d0 + d1) + (d2 + d3);
          a2 += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
        }
      }
    }
    float mu = shift + a1 * inv_per_lane;
    float m2 = a2 - a1 * a1 * inv_per_lane;
    float half_n = 0.5f * per_lane;                  // half the elements behind each side of the next merge
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const float mb = __shfl_xor_sync(0xffffffffu, mu, off);
      const float qb = __shfl_xor_sync(0xffffffffu, m2, off);
      const float delta = mb - mu;
      m2 = (m2 + qb) + delta * delta * half_n;       // symmetric in the two lanes: both hold the same result
      mu = 0.5f * (mu + mb);
      half_n *= 2.f;
    }
    if (lane == 0) {
      s_mean[tk] = mu;
      s_rstd[tk] = rsqrtf(fmaxf(m2, 0.f) / (float)d + eps);
    }
  }
}

// Planes (hi, lo) of x * gain for columns [k_lo, k_lo + ks) of all R rows: item idx = (row, group of four columns),
// thread t takes items t and t + kThreads (R * ks / 4 <= 512).  The gain words are static and fetched ahead
// (planes_gain, before the wait on the previous launch), the rows are fetched by planes_fetch right after it.
__device__ __forceinline__ void planes_gain(const bf16* __restrict__ gain, int R, int k_lo, int ks, uint2 (&g)[2]) {
  const int k4 = ks >> 2;
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int idx = threadIdx.x + j * kThreads;
    g[j] = (idx < R * k4) ? *reinterpret_cast<const uint2*>(gain + k_lo + (idx % k4) * 4) : make_uint2(0u, 0u);
  }
}
__device__ __forceinline__ void planes_fetch(const float* __restrict__ x, int R, int d, int k_lo, int ks, float4 (&v)[2]) {
  const int k4 = ks >> 2;
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int idx = threadIdx.x + j * kThreads;
    v[j] = (idx < R * k4) ? __ldcg(reinterpret_cast<const float4*>(x + (size_t)(idx / k4) * d + k_lo + (idx % k4) * 4))
                          : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}
__device__ __forceinline__ void planes_store(const float4 (&v)[2], const uint2 (&g)[2], int R, int ks, uint8_t* xh, uint8_t* xl, int sx) {
  const int k4 = ks >> 2;
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int idx = threadIdx.x + j * kThreads;
    if (idx < R * k4) {
      const float w[4] = {v[j].x * __uint_as_float(g[j].x << 16), v[j].y * __uint_as_float(g[j].x & 0xffff0000u),
                          v[j].z * __uint_as_float(g[j].y << 16), v[j].w * __uint_as_float(g[j].y & 0xffff0000u)};
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) split_bits(w[e], hi[e], lo[e]);
      const int at = sw(idx / k4, (idx % k4) * 8, sx);
      *reinterpret_cast<uint2*>(xh + at) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
      *reinterpret_cast<uint2*>(xl + at) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
    }
  }
}

// Sum over `np` partial outputs + residual (+ bias) for the feature slice [col0, col0 + width) of all R rows, by
// the CTA that completed the slice: x[t][f] += bias[f] + ws[0][t][f] + ws[1][t][f] + ... in that order.
template <int kBatch>
__device__ __forceinline__ void merge_slice(float* x, const float* ws, const bf16* bias, int np, int R, int d, int col0, int width) {
  const int w4 = width >> 2;
  for (int idx = threadIdx.x; idx < R * w4; idx += kThreads) {
    const int t = idx / w4, col = col0 + (idx % w4) * 4;
    float4 acc = __ldcg(reinterpret_cast<const float4*>(x + (size_t)t * d + col));
    uint2 bw = make_uint2(0u, 0u);
    if (bias) bw = *reinterpret_cast<const uint2*>(bias + col);
    const float4* wp = reinterpret_cast<const float4*>(ws + (size_t)t * d + col);
    const size_t step = (size_t)R * d / 4;
    float4 v[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) v[u] = (u < np) ? __ldcg(wp + u * step) : make_float4(0.f, 0.f, 0.f, 0.f);
    acc.x += __uint_as_float(bw.x << 16); acc.y += __uint_as_float(bw.x & 0xffff0000u);
    acc.z += __uint_as_float(bw.y << 16); acc.w += __uint_as_float(bw.y & 0xffff0000u);
    for (int p0 = 0; p0 < np; p0 += kBatch) {
      if (p0 > 0) {
#pragma unroll
        for (int u = 0; u < kBatch; ++u) v[u] = (p0 + u < np) ? __ldcg(wp + (p0 + u) * step) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        if (p0 + u < np) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
      }
    }
    *reinterpret_cast<float4*>(x + (size_t)t * d + col) = acc;
  }
}

// ------------------------------------------------------------------ self-attention over the paged cache
// Keys are taken in chunks of 32 absolute positions.  Chunk ch belongs to rank ch % kC and, there, to lump
// (ch / kC) % 8.  A lump's chunks are folded in position order into one state per query row (running maximum,
// weight sum, weighted values), the eight lumps of a rank are merged in lump order, the ranks in rank order.
// The grouping depends on key positions only, so a row's result depends neither on the other rows of the pass
// nor on which CTA or warp did the arithmetic: the two schedules below (one CTA per row while every rank has at
// most one chunk; keys shared by all rows of a sequence otherwise) give the same bits.

// One chunk: the 32 key rows and the 32 value rows, 128 contiguous bytes per row and load.  For the keys a lane
// holds 16 bytes (dimensions 8 seg .. 8 seg + 7, seg = lane % 8) of rows 4 u + lane / 8, u = 0..7; for the
// values its two output dimensions of every row.  Rows beyond the chunk's last repeat it (their weight is 0).
// Every load is in flight before the first is used; they go to L2 (other SMs wrote the newest rows in this launch).
__device__ __forceinline__ void chunk_fetch(const bf16* Kc, const bf16* Vc, size_t base, int nk, long long ldkv, int lane,
                                            uint4 (&kq)[8], uint32_t (&vq)[32]) {
  const int grp = lane >> 3, seg = lane & 7;
#pragma unroll
  for (int u = 0; u < 8; ++u)
    kq[u] = __ldcg(reinterpret_cast<const uint4*>(Kc + base + (size_t)min(4 * u + grp, nk - 1) * ldkv) + seg);
#pragma unroll
  for (int j = 0; j < 32; ++j)
    vq[j] = __ldcg(reinterpret_cast<const uint32_t*>(Vc + base + (size_t)min(j, nk - 1) * ldkv) + lane);
}

// Folds a chunk into the state of one query row (q_row: kDH scaled floats in shared memory; state: kPartial
// floats in shared memory that only this warp touches; vis: may this lane's key be seen by the row).
__device__ __forceinline__ void chunk_fold(const uint4 (&kq)[8], const uint32_t (&vq)[32], const float* q_row, bool vis,
                                           float* state, int lane) {
  const int seg = lane & 7;
  const float4* qr = reinterpret_cast<const float4*>(q_row);
  const float4 qa = qr[2 * seg], qb = qr[2 * seg + 1];
  // this lane's share (8 dimensions) of the scores of keys 4 u + lane / 8
  float v[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    float t = qa.x * __uint_as_float(kq[u].x << 16);
    t = fmaf(qa.y, __uint_as_float(kq[u].x & 0xffff0000u), t);
    t = fmaf(qa.z, __uint_as_float(kq[u].y << 16), t);
    t = fmaf(qa.w, __uint_as_float(kq[u].y & 0xffff0000u), t);
    t = fmaf(qb.x, __uint_as_float(kq[u].z << 16), t);
    t = fmaf(qb.y, __uint_as_float(kq[u].z & 0xffff0000u), t);
    t = fmaf(qb.z, __uint_as_float(kq[u].w << 16), t);
    v[u] = fmaf(qb.w, __uint_as_float(kq[u].w & 0xffff0000u), t);
  }
  // sum over the 8 lanes of a group, scattering the 8 sums: lane seg ends with the score of key 4 seg + lane / 8
  // (a fixed tree over the dimensions)
  float w4[4], w2[2];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float send = (seg & 4) ? v[j] : v[j + 4], keep = (seg & 4) ? v[j + 4] : v[j];
    w4[j] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
  }
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const float send = (seg & 2) ? w4[j] : w4[j + 2], keep = (seg & 2) ? w4[j + 2] : w4[j];
    w2[j] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
  }
  const float send1 = (seg & 1) ? w2[0] : w2[1], keep1 = (seg & 1) ? w2[1] : w2[0];
  const float mine = keep1 + __shfl_xor_sync(0xffffffffu, send1, 1);
  // lane = key: key 4 (lane / 4) + lane % 4 of the chunk sits in group lane % 4, lane lane / 4 of it
  const float dot = __shfl_sync(0xffffffffu, mine, 8 * (lane & 3) + (lane >> 2));
  const float sc = vis ? dot : -INFINITY;
  const float m_old = state[kDH], l_old = state[kDH + 1];
  const float m_new = fmaxf(m_old, warp_max(sc));
  if (m_new == -INFINITY) return;                                 // no key of this chunk is visible to the row yet
  // a row that has seen no key before starts from an empty state (whatever the slot holds)
  const float corr = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
  const float pj = vis ? expf(sc - m_new) : 0.f;
  const float l_new = l_old * corr + warp_sum(pj);
  float2 acc = (m_old == -INFINITY) ? make_float2(0.f, 0.f) : *reinterpret_cast<const float2*>(state + 2 * lane);
  acc.x *= corr;
  acc.y *= corr;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const float pw = __shfl_sync(0xffffffffu, pj, j);
    acc.x = fmaf(pw, __uint_as_float(vq[j] << 16), acc.x);
    acc.y = fmaf(pw, __uint_as_float(vq[j] & 0xffff0000u), acc.y);
  }
  __syncwarp();                                                   // every lane has read the old maximum and sum
  *reinterpret_cast<float2*>(state + 2 * lane) = acc;
  if (lane == 0) { state[kDH] = m_new; state[kDH + 1] = l_new; }
  __syncwarp();
}

// Merges eight states, `stride` floats apart, in order, for output dimension dim: states without a visible key
// (maximum -inf) weigh nothing.
__device__ __forceinline__ void states_merge(const float* first, int stride, int dim, float& M, float& num, float& den) {
  M = -INFINITY;
#pragma unroll
  for (int j = 0; j < 8; ++j) M = fmaxf(M, first[j * stride + kDH]);
  num = 0.f;
  den = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float* src = first + j * stride;
    const float mj = src[kDH];
    if (mj > -INFINITY) {
      const float e = expf(mj - M);
      num = fmaf(e, src[dim], num);
      den = fmaf(e, src[kDH + 1], den);
    }
  }
}

// ------------------------------------------------------------------ cross-attention over staged encoder rows
// Attention of one query row (sm.q, scaled) over `limit` encoder positions whose keys and values of this head lie
// in shared memory (rows of kCrossRowBytes: key, padding, value; fp32).  Warp w folds the chunks w, w + 8, ... of
// 32 positions in order (lane = key for the scores, lane = two output dimensions for the values); the warps'
// states are merged in warp order.  Threads c < kDH return output element c.
__device__ __forceinline__ float cross_attention_staged(const uint8_t* kv, int limit, AttnSmem<kDH, kWarps>& sm) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float m_run = -INFINITY, l_run = 0.f, a0 = 0.f, a1 = 0.f;
  for (int c0 = warp * 32; c0 < limit; c0 += kWarps * 32) {
    const int nk = min(32, limit - c0);
    float sc = -INFINITY;
    if (lane < nk) {
      const float4* kr = reinterpret_cast<const float4*>(kv + (size_t)(c0 + lane) * kCrossRowBytes);
      const float4* qv = reinterpret_cast<const float4*>(sm.q);
      float dot = 0.f;
#pragma unroll
      for (int u = 0; u < kDH / 4; ++u) {
        const float4 k4 = kr[u], q4 = qv[u];
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
    for (int j = 0; j < nk; ++j) {
      const float pw = __shfl_sync(0xffffffffu, pj, j);
      const float2 v2 = *reinterpret_cast<const float2*>(kv + (size_t)(c0 + j) * kCrossRowBytes + kCrossKeyPitch + lane * 8);
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

// ------------------------------------------------------------------ attention block (self or cross)
struct AttnBlockParams {
  float* x;                       // residual stream [R, d], updated in place
  const bf16* gain;               // layer-norm gain [d]
  const float* fold_s;            // layer norm folded into the input projection: y = rstd (acc - mean s[n]) + c[n]
  const float* fold_c;
  const bf16* w_in;               // [3d, d] (self: Q, K, V stacked) or [d, d] (cross: Q)
  const bf16* w_out;              // [d, d]
  int d, H, R, rows_per_b;
  float eps;
  bf16* kcache; bf16* vcache;     // self: paged cache of this layer, new rows are written here
  AttnParams attn;                // keys / values, paging, lengths, scale (q and out are not used)
  int cross_smax;                 // cross: encoder rows per sequence staged in shared memory (0: read from L2)
  float* ws;                      // [H][R][d] per-head shares of the output projection
  unsigned* counters;             // [kC], zero between launches
  const int* all_done;
};

struct AttnLayout {
  int s_in, s_out, s_x;           // row strides (bytes)
  int w_in, w_out, xh, xl, oh, ol, part, q, mean, rstd, attn, flag, len, pt, total;   // offsets (bytes)
  int qall, lvl1, lvl2;           // self-attention: every row's query, partial attention states (two levels)
  int ckv;                        // cross-attention: the sequences' encoder keys and values of this head
  int zero_begin, zero_end;       // planes that must start at zero
};
template <bool SELF>
__host__ __device__ inline AttnLayout attn_layout(int d, int NT, int pt_ints, int cross_rows = 0) {
  AttnLayout L;
  const int ks = d / kC, rows_in = SELF ? 3 * kDH : kDH;
  L.s_in = ks * 2; L.s_out = kDH * 2; L.s_x = ks * 2;
  int off = 0;
  L.w_in = off; off += rows_in * L.s_in;
  L.w_out = off; off += (d / kC) * L.s_out;
  L.zero_begin = off;
  L.xh = off; off += NT * 8 * L.s_x;
  L.xl = off; off += NT * 8 * L.s_x;
  L.oh = off; off += NT * 8 * L.s_out;
  L.ol = off; off += NT * 8 * L.s_out;
  L.zero_end = off;
  L.part = off; off += kC * NT * rows_in * 4;
  L.q = off; off += NT * kDH * 4;
  L.mean = off; off += kMaxRows * 4;
  L.rstd = off; off += kMaxRows * 4;
  L.attn = off; off += (int)((sizeof(AttnSmem<kDH, kWarps>) + 15) / 16 * 16);
  L.flag = off; off += 16;
  L.len = off; off += kMaxRows * 4;
  L.pt = off; off += (pt_ints * 4 + 15) / 16 * 16;
  L.qall = L.lvl1 = L.lvl2 = 0;
  L.ckv = off;
  if (!SELF) off += cross_rows * kCrossRowBytes;
  if (SELF) {
    // Buffers of the attention step reuse what is dead by then where it is large enough: the planes of x (read
    // by the input projection only) hold every row's query, the input projection's weights hold the partial
    // attention states.  Other CTAs write into them only after a cluster barrier that follows the projection.
    const int rp = NT * 8, q_bytes = rp * kDH * 4, lvl_bytes = kC * rp * kPartial * 4;
    if (2 * NT * 8 * L.s_x >= q_bytes) L.qall = L.xh; else { L.qall = off; off += q_bytes; }
    if (2 * lvl_bytes <= rows_in * L.s_in) { L.lvl1 = L.w_in; L.lvl2 = L.w_in + lvl_bytes; }
    else { L.lvl1 = off; off += lvl_bytes; L.lvl2 = off; off += lvl_bytes; }
  }
  L.total = off;
  return L;
}

// LEAN variants carry only the path their session takes -- the general kernels run out of registers under the
// 128-per-thread budget that keeps two CTAs on an SM (ptxas: 184 bytes of spills in the self-attention block) and
// are 1.5-2 us per launch slower.  Self-attention: the cache never holds more than kC chunks of keys per row, so
// only the short schedule is compiled in (sessions of up to 256 positions: the machine-translation shapes).
// Cross-attention: the encoder's rows are staged in shared memory (cross_smax > 0).
// Self-attention, LEAN = 2: only the long schedule (rank c folds its own chunks for all rows), which is correct at
// any length and the same arithmetic; sessions whose cache can exceed 256 positions use it from the start.
// MINB = 1 lifts the register budget to 255 per thread for models whose attention launches occupy at most half the
// SMs (the next launch's CTAs find free SMs anyway): the long schedule then keeps its chunk in registers.
template <bool SELF, int NT, int LEAN = 0, int MINB = 2>
__global__ void __cluster_dims__(kC, 1, 1) __launch_bounds__(kThreads, MINB) attn_block_kernel(AttnBlockParams p) {
  extern __shared__ __align__(16) uint8_t fsm[];
  cg::cluster_group cluster = cg::this_cluster();
  const int c = (int)cluster.block_rank(), h = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const int d = p.d, ks = d / kC, slice = d / kC;
  constexpr int ROWS_IN = SELF ? 3 * kDH : kDH;
  const int nb = p.R / p.rows_per_b;                                   // sequences in this pass
  const int pt_ints = SELF ? nb * p.attn.st.pages_per_row : 0;
  const AttnLayout L = attn_layout<SELF>(d, NT, pt_ints, SELF ? 0 : nb * p.cross_smax);
  uint8_t* w_in_s = fsm + L.w_in;
  uint8_t* ckv_s = fsm + L.ckv;                        // cross: [sequence][row][key | value] of this head
  uint8_t* w_out_s = fsm + L.w_out;
  uint8_t* xh_s = fsm + L.xh;
  uint8_t* xl_s = fsm + L.xl;
  uint8_t* oh_s = fsm + L.oh;
  uint8_t* ol_s = fsm + L.ol;
  float* part_s = reinterpret_cast<float*>(fsm + L.part);
  float* q_s = reinterpret_cast<float*>(fsm + L.q);
  float* s_mean = reinterpret_cast<float*>(fsm + L.mean);
  float* s_rstd = reinterpret_cast<float*>(fsm + L.rstd);
  AttnSmem<kDH, kWarps>& sm = *reinterpret_cast<AttnSmem<kDH, kWarps>*>(fsm + L.attn);
  volatile int* flag = reinterpret_cast<volatile int*>(fsm + L.flag);
  int* s_len = reinterpret_cast<int*>(fsm + L.len);    // per sequence: tokens in the cache (self) or source length (cross)
  int* s_pt = reinterpret_cast<int*>(fsm + L.pt);      // self: the sequences' page-table rows
  float* q_all = reinterpret_cast<float*>(fsm + L.qall);   // self: scaled query of every row [rows][kDH]
  float* lvl1 = reinterpret_cast<float*>(fsm + L.lvl1);    // self: [lump][row][kPartial] states of this CTA's key lumps
  float* lvl2 = reinterpret_cast<float*>(fsm + L.lvl2);    // self: [rank][row][kPartial] states of the cluster's CTAs

  pdl_launch_dependents();
  const unsigned long long stream = tc::l2_evict_first();
  // Everything that does not depend on the previous launch starts now.  This CTA's weights: ROWS_IN rows x ks
  // columns of the input projection, `slice` rows x 64 columns of the output projection.
  {
    const int cpr = ks * 2 / 16;
    for (int idx = tid; idx < ROWS_IN * cpr; idx += kThreads) {
      const int row = idx / cpr, c16 = idx % cpr;
      const int grow = (row / kDH) * d + h * kDH + (row % kDH);
      cp_async16(w_in_s + sw(row, c16 * 16, L.s_in), p.w_in + (size_t)grow * d + c * ks + c16 * 8, stream);
    }
    for (int idx = tid; idx < slice * 8; idx += kThreads) {
      const int row = idx >> 3, c16 = idx & 7;
      cp_async16(w_out_s + sw(row, c16 * 16, L.s_out), p.w_out + (size_t)(c * slice + row) * d + h * kDH + c16 * 8, stream);
    }
    if (!SELF && (LEAN != 0 || p.cross_smax > 0)) {
      // the encoder's keys and values of this head do not change after the encoder ran: they come along
      const float* Kg = reinterpret_cast<const float*>(p.attn.k);
      const float* Vg = reinterpret_cast<const float*>(p.attn.v);
      for (int idx = tid; idx < nb * p.cross_smax * 32; idx += kThreads) {
        const int row = idx >> 5, piece = idx & 31, b = row / p.cross_smax, sidx = row % p.cross_smax;
        const size_t at = (size_t)b * p.attn.bstride + (size_t)sidx * p.attn.ldkv + h * kDH + (piece & 15) * 4;
        if (piece < 16) cp_async16_keep(ckv_s + row * kCrossRowBytes + piece * 16, Kg + at);
        else cp_async16_keep(ckv_s + row * kCrossRowBytes + kCrossKeyPitch + (piece - 16) * 16, Vg + at);
      }
    }
    cp_async_commit();
  }
  for (int i = L.zero_begin / 16 + tid; i < L.zero_end / 16; i += kThreads) reinterpret_cast<uint4*>(fsm)[i] = make_uint4(0, 0, 0, 0);
  // the folded layer-norm vectors of the feature this thread finishes, page tables, source lengths: all static
  float fs = 0.f, fc = 0.f;
  if (tid < ROWS_IN) {
    const int n = (tid / kDH) * d + h * kDH + (tid % kDH);
    fs = p.fold_s[n];
    fc = p.fold_c[n];
  }
  if (SELF) {
    for (int i = tid; i < pt_ints; i += kThreads) s_pt[i] = p.attn.st.page_table[i];
  } else if (tid < nb) {
    s_len[tid] = p.attn.limit_b[tid];
  }
  uint2 gwords[2];
  planes_gain(p.gain, p.R, c * ks, ks, gwords);
  __syncthreads();
  cluster_arrive();            // this CTA's shared memory is set up; matched by cluster_wait() below
  pdl_wait();
  const int ended = p.all_done ? *p.all_done : 0;      // the same answer in every CTA
  // a warp issues in order: every load goes out before the first value is used
  int len_v = 0;
  if (SELF && tid < nb) len_v = p.attn.st.len[tid];
  float4 xrow[2];
  planes_fetch(p.x, p.R, d, c * ks, ks, xrow);
  rows_stats(p.x, p.R, d, p.eps, s_mean, s_rstd);
  if (SELF && tid < nb) s_len[tid] = len_v;
  planes_store(xrow, gwords, p.R, ks, xh_s, xl_s, L.s_x);
  cp_async_wait_all();
  __syncthreads();
  cluster_wait();                                      // every CTA of the cluster is running: its shared memory may be written
  if (ended) return;

  // ---- input projection over this CTA's part of the reduction; token t's partial goes to rank t % kC
  for (int mt = warp; mt < ROWS_IN / 16; mt += kWarps) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    mma_rows16<NT>(acc, w_in_s + mt * 16 * L.s_in, L.s_in, xh_s, xl_s, L.s_x, ks, lane);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int row = mt * 16 + g + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
        if (token < p.R) {
          float* remote = cluster.map_shared_rank(part_s, token % kC);
          remote[(c * NT + token / kC) * ROWS_IN + row] = acc[nt][e];
        }
      }
  }
  cluster.sync();

  // self-attention: does every rank have at most one chunk of keys?  (the same answer in every CTA of the grid)
  bool one_chunk_per_rank = true;
  if (SELF && LEAN == 0) {
    for (int b = 0; b < nb; ++b)
      one_chunk_per_rank = one_chunk_per_rank &&
          ((s_len[b] + p.rows_per_b + 31) >> 5) - (attn_first_key(p.attn, s_len[b]) >> 5) <= kC;
  }
  // ---- this rank's tokens: add the partials in rank order, finish the layer norm, write keys / values
  for (int slot = 0; slot < NT; ++slot) {
    const int token = slot * kC + c;
    if (token < p.R && tid < ROWS_IN) {
      float a = 0.f;
#pragma unroll
      for (int src = 0; src < kC; ++src) a += part_s[(src * NT + slot) * ROWS_IN + tid];
      const int sect = tid / kDH, f = tid % kDH;
      const float y = s_rstd[token] * (a - s_mean[token] * fs) + fc;
      if (sect == 0) {
        if (SELF) {
          if (LEAN == 1 || (LEAN == 0 && one_chunk_per_rank)) {
            q_all[token * kDH + f] = y * p.attn.scale;             // this rank attends for its own rows
          } else {
#pragma unroll
            for (int dst = 0; dst < kC; ++dst) cluster.map_shared_rank(q_all, dst)[token * kDH + f] = y * p.attn.scale;
          }
        } else {
          q_s[slot * kDH + f] = y * p.attn.scale;
        }
      } else {
        const int b = token / p.rows_per_b, i = token % p.rows_per_b;
        const int pos = s_len[b] + i;
        const int page = s_pt[b * p.attn.st.pages_per_row + pos / kPage];
        const size_t at = ((size_t)page * kPage + (pos % kPage)) * d + h * kDH + f;
        (sect == 1 ? p.kcache : p.vcache)[at] = __float2bfloat16_rn(y);
      }
    }
  }
  if (SELF) {
    __threadfence();
    cluster.sync();                      // the block's new keys and values are in the cache for every rank's rows
  } else {
    __syncthreads();
  }

  AttnParams ap = p.attn;
  if (SELF) {
    // ---- self-attention (see chunk_fetch / chunk_fold / states_merge above)
    ap.st.page_table = s_pt;
    constexpr int RP = NT * 8;
    const bf16* Kc = reinterpret_cast<const bf16*>(ap.k);
    const bf16* Vc = reinterpret_cast<const bf16*>(ap.v);
    const int rpb = p.rows_per_b;
    if (LEAN == 1 || (LEAN == 0 && one_chunk_per_rank)) {
      // Short sequences: this rank takes its own rows (as the projection handed them out), warp w stands in for
      // rank w and folds that rank's only chunk; a rank's single lump is its state (merging one lump multiplies
      // by exp(0) = 1), so the eight warp states are merged like the ranks' states.  The result goes to every
      // rank as planes.
      for (int slot = 0; slot < NT; ++slot) {
        const int token = slot * kC + c;
        if (token < p.R) {                                         // uniform over the CTA
          const int b = token / rpb, i = token % rpb;
          const int len = s_len[b], lim_max = len + rpb;
          const int fk = attn_first_key(ap, len + i), ch0 = attn_first_key(ap, len) >> 5;
          const int ch = ch0 + ((warp - ch0) & (kC - 1));          // chunk of rank `warp` at or after ch0
          float* state = lvl2 + (warp * RP + token) * kPartial;
          if (lane == 0) { state[kDH] = -INFINITY; state[kDH + 1] = 0.f; }
          __syncwarp();
          if ((ch << 5) <= len + i) {                              // the row sees at least the chunk's first key
            const int c0 = ch << 5;
            const size_t base = ((size_t)s_pt[b * ap.st.pages_per_row + c0 / kPage] * kPage + (c0 % kPage)) * ap.ldkv + h * kDH;
            uint4 kq[8];
            uint32_t vq[32];
            chunk_fetch(Kc, Vc, base, min(32, lim_max - c0), ap.ldkv, lane, kq, vq);
            const int key = c0 + lane;
            chunk_fold(kq, vq, q_all + token * kDH, key <= len + i && key >= fk, state, lane);
          }
          __syncthreads();
          if (tid < kDH) {
            float M, num, den;
            states_merge(lvl2 + token * kPartial, RP * kPartial, tid, M, num, den);
            uint32_t hi, lo;
            split_bits(num / den, hi, lo);
#pragma unroll
            for (int dst = 0; dst < kC; ++dst) {
              *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(oh_s, dst) + sw(token, tid * 2, L.s_out)) = (unsigned short)hi;
              *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(ol_s, dst) + sw(token, tid * 2, L.s_out)) = (unsigned short)lo;
            }
          }
        }
      }
      cluster.sync();
    } else {
      // Long sequences: rank c folds its own chunks for every row, so that a chunk's keys and values are fetched
      // once for all rows of the sequence.  Which warp takes which (lump, rows) is free: with few lumps the rows
      // are spread over the warps, with many a warp takes one lump for all rows.
      for (int i = tid; i < 8 * RP; i += kThreads) { lvl1[i * kPartial + kDH] = -INFINITY; lvl1[i * kPartial + kDH + 1] = 0.f; }
      __syncthreads();
      for (int b = 0; b < nb; ++b) {
        const int len = s_len[b];
        const int lim_max = len + rpb;                              // keys in the cache once the block is written
        const int nch = (lim_max + 31) >> 5, ch0 = attn_first_key(ap, len) >> 5;
        const int first_my = ch0 + ((c - ch0) & (kC - 1));          // this rank's first chunk at or after ch0
        const int n_my = first_my < nch ? (nch - first_my + kC - 1) / kC : 0;
        const int active = min(8, n_my);
        if (active == 0) continue;                                  // uniform over the CTA
        const int S = 8 / active;                                   // row subsets per lump
        const int a = warp / S, sub = warp % S;
        if (a >= active) continue;                                  // uniform over the warp; no CTA barrier below
        const int ch_first = first_my + kC * a;
        const int lump = (ch_first / kC) & 7;
        const int* pt = s_pt + b * ap.st.pages_per_row;
        for (int ch = ch_first; ch < nch; ch += 8 * kC) {
          const int c0 = ch << 5;
          const size_t base = ((size_t)pt[c0 / kPage] * kPage + (c0 % kPage)) * ap.ldkv + h * kDH;
          uint4 kq[8];
          uint32_t vq[32];
          chunk_fetch(Kc, Vc, base, min(32, lim_max - c0), ap.ldkv, lane, kq, vq);
          const int key = c0 + lane;
#pragma unroll 1
          for (int i = sub; i < rpb; i += S)
            chunk_fold(kq, vq, q_all + (b * rpb + i) * kDH, key <= len + i && key >= attn_first_key(ap, len + i),
                       lvl1 + ((size_t)lump * RP + b * rpb + i) * kPartial, lane);
        }
      }
      __syncthreads();
      // this rank's state per row: its lumps in lump order; sent to every rank
      for (int idx = tid; idx < p.R * kDH; idx += kThreads) {
        const int row = idx / kDH, dim = idx % kDH;
        float M, num, den;
        states_merge(lvl1 + row * kPartial, RP * kPartial, dim, M, num, den);
#pragma unroll
        for (int dst = 0; dst < kC; ++dst) {
          float* out = cluster.map_shared_rank(lvl2, dst) + (c * RP + row) * kPartial;
          out[dim] = num;
          if (dim == 0) { out[kDH] = M; out[kDH + 1] = den; }
        }
      }
      cluster.sync();
      // every rank merges the ranks' states in rank order and keeps the result as planes for the output projection
      for (int idx = tid; idx < p.R * kDH; idx += kThreads) {
        const int row = idx / kDH, dim = idx % kDH;
        float M, num, den;
        states_merge(lvl2 + row * kPartial, RP * kPartial, dim, M, num, den);
        uint32_t hi, lo;
        split_bits(num / den, hi, lo);
        *reinterpret_cast<unsigned short*>(oh_s + sw(row, dim * 2, L.s_out)) = (unsigned short)hi;
        *reinterpret_cast<unsigned short*>(ol_s + sw(row, dim * 2, L.s_out)) = (unsigned short)lo;
      }
      __syncthreads();
    }
  } else {
  // ---- attention of this rank's rows; the result goes to every rank as planes
  for (int slot = 0; slot < NT; ++slot) {
    const int token = slot * kC + c;
    if (token < p.R) {                   // uniform over the CTA
      if (tid < kDH) sm.q[tid] = q_s[slot * kDH + tid];
      __syncthreads();
      const int b = token / p.rows_per_b;
      float ov;
      if (LEAN != 0 || p.cross_smax > 0) ov = cross_attention_staged(ckv_s + (size_t)b * p.cross_smax * kCrossRowBytes, s_len[b], sm);
      else ov = attention_head<float, kDH, kWarps, false>(ap, b, h, 0, s_len[b], sm);
      if (tid < kDH) {
        uint32_t hi, lo;
        split_bits(ov, hi, lo);
#pragma unroll
        for (int dst = 0; dst < kC; ++dst) {
          *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(oh_s, dst) + sw(token, tid * 2, L.s_out)) = (unsigned short)hi;
          *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(ol_s, dst) + sw(token, tid * 2, L.s_out)) = (unsigned short)lo;
        }
      }
      __syncthreads();
    }
  }
  cluster.sync();
  }

  // ---- this head's share of the output projection for the features of slice c
  float* wsh = p.ws + (size_t)h * p.R * d;
  for (int mt = warp; mt < slice / 16; mt += kWarps) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    mma_rows16<NT>(acc, w_out_s + mt * 16 * L.s_out, L.s_out, oh_s, ol_s, L.s_out, kDH, lane);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int row = mt * 16 + g + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
        if (token < p.R) wsh[(size_t)token * d + c * slice + row] = acc[nt][e];
      }
  }
  __syncthreads();
  if (tid == 0) *flag = (tc::atom_add_acq_rel(&p.counters[c], 1u) == (unsigned)p.H - 1) ? 1 : 0;
  __syncthreads();
  if (*flag) {                           // last head to arrive at this slice: heads are added in head order
    merge_slice<16>(p.x, p.ws, nullptr, p.H, p.R, d, c * slice, slice);
    if (tid == 0) p.counters[c] = 0;
  }
}

// ------------------------------------------------------------------ feed-forward block
struct FfnBlockParams {
  float* x;                       // residual stream [R, d], updated in place
  const bf16* gain;
  const float* fold_s;            // layer norm folded into the first projection (c also holds its bias)
  const float* fold_c;
  const bf16* w1;                 // [ff, d]
  const bf16* w2;                 // [d, ff]
  const bf16* b2;                 // [d]
  int d, ff, R, NJ;               // NJ clusters, each kC * kHS hidden units
  float eps;
  float* ws;                      // [NJ][R][d] per-cluster shares of the second projection
  unsigned* counters;             // [kC], zero between launches
  const int* all_done;
};

struct FfnLayout {
  int s1, s2, s_x, s_h;           // bytes per row
  int w1, w2, xh, xl, hh, hl, part, mean, rstd, flag, total;
  int zero_begin, zero_end;
};
__host__ __device__ inline FfnLayout ffn_layout(int d, int NT) {
  FfnLayout L;
  const int ks = d / kC;
  L.s1 = ks * 2; L.s2 = kC * kHS * 2; L.s_x = ks * 2; L.s_h = kC * kHS * 2;
  int off = 0;
  L.w1 = off; off += kC * kHS * L.s1;
  L.w2 = off; off += (d / kC) * L.s2;
  // The planes of the hidden units take the place of the planes of x: they are written (by the whole cluster)
  // only after every rank has finished its first projection.  Rows of tokens beyond R hold left-overs; a token's
  // column of a product depends on that token's row only, and those columns are never stored.
  const int x_bytes = NT * 8 * L.s_x, h_bytes = NT * 8 * L.s_h, pl = x_bytes > h_bytes ? x_bytes : h_bytes;
  L.zero_begin = off;
  L.xh = off; L.hh = off; off += pl;
  L.xl = off; L.hl = off; off += pl;
  L.zero_end = off;
  L.part = off; off += kC * kHS * NT * 8 * 4;
  L.mean = off; off += kMaxRows * 4;
  L.rstd = off; off += kMaxRows * 4;
  L.flag = off; off += 16;
  L.total = off;
  return L;
}

// MINB = 3 (80 registers) lets all 32 clusters of a wide feed-forward layer be resident at once; launches of at
// most 148 CTAs take MINB = 2 (128 registers).
template <int NT, int MINB = 3>
__global__ void __cluster_dims__(kC, 1, 1) __launch_bounds__(kThreads, MINB) ffn_block_kernel(FfnBlockParams p) {
  extern __shared__ __align__(16) uint8_t fsm[];
  cg::cluster_group cluster = cg::this_cluster();
  const int c = (int)cluster.block_rank(), j = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const int d = p.d, ks = d / kC, slice = d / kC;
  constexpr int HC = kC * kHS;                       // hidden units of a cluster
  const int hid_cluster = j * HC, hid0 = hid_cluster + c * kHS;
  const FfnLayout L = ffn_layout(d, NT);
  uint8_t* w1_s = fsm + L.w1;
  uint8_t* w2_s = fsm + L.w2;
  uint8_t* xh_s = fsm + L.xh;
  uint8_t* xl_s = fsm + L.xl;
  uint8_t* hh_s = fsm + L.hh;
  uint8_t* hl_s = fsm + L.hl;
  float* part_s = reinterpret_cast<float*>(fsm + L.part);
  float* s_mean = reinterpret_cast<float*>(fsm + L.mean);
  float* s_rstd = reinterpret_cast<float*>(fsm + L.rstd);
  volatile int* flag = reinterpret_cast<volatile int*>(fsm + L.flag);

  pdl_launch_dependents();
  const unsigned long long stream = tc::l2_evict_first();
  // Static weights of this CTA: the cluster's HC rows of the first projection restricted to this rank's ks
  // columns and, of the second projection, the rows of feature slice c restricted to the cluster's HC hidden units.
  {
    const int cpr = ks * 2 / 16;
    for (int idx = tid; idx < HC * cpr; idx += kThreads) {
      const int row = idx / cpr, c16 = idx % cpr;
      cp_async16(w1_s + sw(row, c16 * 16, L.s1), p.w1 + (size_t)(hid_cluster + row) * d + c * ks + c16 * 8, stream);
    }
    constexpr int cpr2 = HC * 2 / 16;
    for (int idx = tid; idx < slice * cpr2; idx += kThreads) {
      const int row = idx / cpr2, c16 = idx % cpr2;
      cp_async16(w2_s + sw(row, c16 * 16, L.s2), p.w2 + (size_t)(c * slice + row) * p.ff + hid_cluster + c16 * 8, stream);
    }
    cp_async_commit();
  }
  for (int i = L.zero_begin / 16 + tid; i < L.zero_end / 16; i += kThreads) reinterpret_cast<uint4*>(fsm)[i] = make_uint4(0, 0, 0, 0);
  // the folded layer-norm vectors of the hidden unit this thread finishes (kHS * R <= 256 items, one per thread)
  const float fs = p.fold_s[hid0 + tid % kHS], fc = p.fold_c[hid0 + tid % kHS];
  uint2 gwords[2];
  planes_gain(p.gain, p.R, c * ks, ks, gwords);
  __syncthreads();
  cluster_arrive();            // this CTA's shared memory is set up; matched by cluster_wait() below
  pdl_wait();
  const int ended = p.all_done ? *p.all_done : 0;      // the same answer in every CTA
  float4 xrow[2];
  planes_fetch(p.x, p.R, d, c * ks, ks, xrow);
  rows_stats(p.x, p.R, d, p.eps, s_mean, s_rstd);
  planes_store(xrow, gwords, p.R, ks, xh_s, xl_s, L.s_x);
  cp_async_wait_all();
  __syncthreads();
  cluster_wait();                                      // every CTA of the cluster is running
  if (ended) return;

  // ---- first projection of the cluster's hidden units over this rank's columns; unit f belongs to rank f / kHS
  for (int mt = warp; mt < HC / 16; mt += kWarps) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    mma_rows16<NT>(acc, w1_s + mt * 16 * L.s1, L.s1, xh_s, xl_s, L.s_x, ks, lane);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int f = mt * 16 + g + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
        if (token < p.R) {
          float* remote = cluster.map_shared_rank(part_s, f / kHS);
          remote[(c * kHS + f % kHS) * (NT * 8) + token] = acc[nt][e];
        }
      }
  }
  cluster.sync();
  // ranks in order, layer norm, bias, ReLU; every rank of the cluster gets the planes of these hidden units
  if (tid < kHS * p.R) {
    const int f = tid % kHS, token = tid / kHS;
    float a = 0.f;
#pragma unroll
    for (int src = 0; src < kC; ++src) a += part_s[(src * kHS + f) * (NT * 8) + token];
    const float y = fmaxf(s_rstd[token] * (a - s_mean[token] * fs) + fc, 0.f);
    uint32_t hi, lo;
    split_bits(y, hi, lo);
    const int at = sw(token, (c * kHS + f) * 2, L.s_h);
#pragma unroll
    for (int dst = 0; dst < kC; ++dst) {
      *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(hh_s, dst) + at) = (unsigned short)hi;
      *reinterpret_cast<unsigned short*>(cluster.map_shared_rank(hl_s, dst) + at) = (unsigned short)lo;
    }
  }
  cluster.sync();

  // ---- second projection: feature slice c, over the cluster's hidden units: the cluster's share of the output
  float* wsj = p.ws + (size_t)j * p.R * d;
  for (int mt = warp; mt < slice / 16; mt += kWarps) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    mma_rows16<NT>(acc, w2_s + mt * 16 * L.s2, L.s2, hh_s, hl_s, L.s_h, HC, lane);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int row = mt * 16 + g + ((e & 2) ? 8 : 0), token = nt * 8 + 2 * t4 + (e & 1);
        if (token < p.R) wsj[(size_t)token * d + c * slice + row] = acc[nt][e];
      }
  }
  __syncthreads();
  if (tid == 0) *flag = (tc::atom_add_acq_rel(&p.counters[c], 1u) == (unsigned)p.NJ - 1) ? 1 : 0;
  __syncthreads();
  if (*flag) {               // last cluster to arrive at this slice: clusters are added in cluster order
    merge_slice<12>(p.x, p.ws, p.b2, p.NJ, p.R, d, c * slice, slice);
    if (tid == 0) p.counters[c] = 0;
  }
}

// Shapes this path is built for.
__host__ inline bool supported(int d, int H, int ff, int rows) {
  return H > 0 && d == H * kDH && d % (kC * 32) == 0 && d % 128 == 0 && ff % (kC * kHS) == 0 && rows >= 1 && rows <= kMaxRows &&
         rows * (d / kC) <= 8 * kThreads;   // planes: at most two groups of four columns per thread
}

}  // namespace fused
}  // namespace bpd
