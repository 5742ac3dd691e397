// CUDA-core kernels of the decoding pass: embedding, layer norm, skinny
// projections with fused epilogues, attention over the paged cache, the
// vocabulary projection with a fused top-1, and verify/accept/commit.
// Every reduction has a fixed order that does not depend on how many rows a
// launch carries, so a position scored alone (greedy) and the same position
// scored inside a block give bit-identical results.
#pragma once
#include "common.cuh"
#include "host.hpp"

namespace bpd {

// ------------------------------------------------------------------ embedding (decoder and encoder)
struct EmbedParams {
  const void* table;       // [V, d] weight dtype
  const float* pe;         // [npos, d] sinusoidal position signal, tabulated on the host in double precision
  int npos;
  float* x;                // [rows, d] residual stream
  int rows, rows_per_b, d, vocab;
  // decoder: token = block[b][i] (or a forced proposal), position = len[b] + i
  RowState st;
  const int* forced;       // [B][forced_rows][kforced-1] or null
  int forced_rows;         // 1: one tail per row; >1: indexed by tokens emitted so far
  int kforced;
  // encoder: token = src[b][s], position = s
  const int* src;          // [B][rows_per_b] or null (decoder mode)
  const bf16* gain;        // optional: also write planes (hi, lo) of x * gain for a projection with a folded layer norm
  bf16* xg_hi; long long xg_plane;
  float* stat_out; int stat_T;   // optional: mean and squared deviations of every 128 consecutive features of a row, [d / 128][stat_T][2]
  const int* all_done;
};

// One row of the embedding (all threads of the CTA).
template <typename WT>
__device__ __forceinline__ void embed_row(const EmbedParams& p, int r) {
  const int b = r / p.rows_per_b, i = r % p.rows_per_b;
  int tok, pos;
  if (p.src) {
    tok = p.src[r];
    pos = i;
  } else {
    tok = p.st.block[b * kMaxK + i];
    if (p.forced && i >= 1 && i < p.kforced) {
      const int jb = p.st.j[b];
      if (p.forced_rows == 1)
        tok = p.forced[(size_t)b * (p.kforced - 1) + (i - 1)];
      else if (jb < p.forced_rows)
        tok = p.forced[((size_t)b * p.forced_rows + jb) * (p.kforced - 1) + (i - 1)];
    }
    pos = p.st.len[b] + i;
    if (threadIdx.x == 0) p.st.cur_block[b * kMaxK + i] = tok;
  }
  if (tok < 0 || tok >= p.vocab || pos >= p.npos) {   // never index outside the tables; report instead
    if (threadIdx.x == 0) atomicCAS(p.st.error, 0, 1);
    tok = 0;
    pos = 0;
  }
  const WT* row = reinterpret_cast<const WT*>(p.table) + (size_t)tok * p.d;
  const float* pe = p.pe + (size_t)pos * p.d;
  const float scale = sqrtf((float)p.d);
  for (int c = threadIdx.x * 8; c < p.d; c += blockDim.x * 8) {
    float w[8], e[8];
    load8(row + c, w);
    load8(pe + c, e);
    float4* out = reinterpret_cast<float4*>(p.x + (size_t)r * p.d + c);
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = w[i] * scale + e[i];
    out[0] = make_float4(v[0], v[1], v[2], v[3]);
    out[1] = make_float4(v[4], v[5], v[6], v[7]);
    if (p.stat_out) {
      // 16 consecutive lanes hold 128 consecutive features (d is a multiple of 128 here, so half-warps are whole)
      float sum = ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float mean = sum * (1.0f / 128.0f);
      float sq = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) sq += (v[i] - mean) * (v[i] - mean);
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if ((threadIdx.x & 15) == 0) reinterpret_cast<float2*>(p.stat_out)[(size_t)(c >> 7) * p.stat_T + r] = make_float2(mean, sq);
    }
    if (p.gain) {
      float g[8];
      load8(p.gain + c, g);
      bf16 hi[8], lo[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float xg = v[i] * g[i];
        hi[i] = __float2bfloat16_rn(xg);
        lo[i] = __float2bfloat16_rn(xg - __bfloat162float(hi[i]));
      }
      bf16* dst = p.xg_hi + (size_t)r * p.d + c;
      *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(hi);
      *reinterpret_cast<uint4*>(dst + p.xg_plane) = *reinterpret_cast<const uint4*>(lo);
    }
  }
}

template <typename WT>
__global__ void embed_kernel(EmbedParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  embed_row<WT>(p, blockIdx.x);
}

// ------------------------------------------------------------------ folding a layer norm into the projection after it
// LN(x) w^T = rstd * (x*gain) w^T - rstd * mean * s + c   with   s[n] = sum_c gain[c] w[n][c],
// c[n] = sum_c shift[c] w[n][c] + bias[n].  One warp per output feature, accumulated in double (load time only).
struct FoldParams {
  const bf16* w; const bf16* gain; const bf16* shift; const bf16* bias;
  float* s; float* c;
  int N, K;
};
static __global__ void __launch_bounds__(128) fold_ln_kernel(FoldParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = blockIdx.x * 4 + warp;
  if (n >= p.N) return;
  double ss = 0.0, cc = 0.0;
  for (int k = lane * 8; k < p.K; k += 256) {
    float w[8], g[8], b[8];
    load8(p.w + (size_t)n * p.K + k, w);
    load8(p.gain + k, g);
    load8(p.shift + k, b);
#pragma unroll
    for (int e = 0; e < 8; ++e) { ss += (double)g[e] * (double)w[e]; cc += (double)b[e] * (double)w[e]; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ss += __shfl_xor_sync(0xffffffffu, ss, o);
    cc += __shfl_xor_sync(0xffffffffu, cc, o);
  }
  if (lane == 0) {
    p.s[n] = (float)ss;
    p.c[n] = (float)(cc + (p.bias ? (double)__bfloat162float(p.bias[n]) : 0.0));
  }
}

// ------------------------------------------------------------------ layer norm (one warp per row)
struct LnParams {
  const float* x;   // [rows, d]
  const void* g;    // [d] weight dtype
  const void* b;
  void* y;          // [rows, d] activation dtype, or two bf16 planes (hi, lo) when plane > 0
  long long plane;  // elements between the hi and the lo plane; 0 = single array
  float* y_f32;     // optional fp32 copy
  int rows, d;
  float eps;
  const int* all_done;
};

constexpr int kLnMaxD = 1024;   // the row is held in registers: 8 float4 per lane

template <typename WT, typename AT>
__global__ void __launch_bounds__(128) layernorm_kernel(LnParams p) {
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * 4 + warp;
  const int nv = p.d >> 2;                 // float4 per row (d is a multiple of 8)
  // gain and shift do not depend on the preceding launch: they are fetched before the wait
  const WT* g = reinterpret_cast<const WT*>(p.g);
  const WT* bb = reinterpret_cast<const WT*>(p.b);
  float gv[kLnMaxD / 128][4], bv[kLnMaxD / 128][4];
#pragma unroll
  for (int i = 0; i < kLnMaxD / 128; ++i) {
    const int idx = i * 32 + lane;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      gv[i][e] = (idx < nv) ? to_f(g[idx * 4 + e]) : 0.f;
      bv[i][e] = (idx < nv) ? to_f(bb[idx * 4 + e]) : 0.f;
    }
  }
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  if (r >= p.rows) return;
  const float4* x4 = reinterpret_cast<const float4*>(p.x + (size_t)r * p.d);
  float4 v[kLnMaxD / 128];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < kLnMaxD / 128; ++i) {
    const int idx = i * 32 + lane;
    v[i] = (idx < nv) ? x4[idx] : make_float4(0.f, 0.f, 0.f, 0.f);
    s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  }
  const float mean = warp_sum(s) / (float)p.d;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < kLnMaxD / 128; ++i) {
    if (i * 32 + lane < nv) {
      const float a = v[i].x - mean, b = v[i].y - mean, c = v[i].z - mean, d = v[i].w - mean;
      q += (a * a + b * b) + (c * c + d * d);
    }
  }
  const float rstd = rsqrtf(warp_sum(q) / (float)p.d + p.eps);
#pragma unroll
  for (int i = 0; i < kLnMaxD / 128; ++i) {
    const int idx = i * 32 + lane;
    if (idx < nv) {
      const int c = idx * 4;
      const float in[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
      float o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) o[e] = (in[e] - mean) * rstd * gv[i][e] + bv[i][e];
      if (p.plane) {
        bf16* yp = reinterpret_cast<bf16*>(p.y) + (size_t)r * p.d + c;
        bf16 hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          hi[e] = __float2bfloat16_rn(o[e]);
          lo[e] = __float2bfloat16_rn(o[e] - __bfloat162float(hi[e]));
        }
        *reinterpret_cast<uint2*>(yp) = *reinterpret_cast<const uint2*>(hi);
        *reinterpret_cast<uint2*>(yp + p.plane) = *reinterpret_cast<const uint2*>(lo);
      } else {
        AT* y = reinterpret_cast<AT*>(p.y) + (size_t)r * p.d + c;
#pragma unroll
        for (int e = 0; e < 4; ++e) y[e] = from_f<AT>(o[e]);
      }
      if (p.y_f32) *reinterpret_cast<float4*>(p.y_f32 + (size_t)r * p.d + c) = make_float4(o[0], o[1], o[2], o[3]);
    }
  }
}

// ------------------------------------------------------------------ skinny projection y = x W^T (+ epilogue)
enum Epilogue {
  kEpiStoreAct = 0,  // y_act[r][n] = act(v + bias)
  kEpiStoreF32 = 1,  // y_f32[r][n] = act(v + bias)
  kEpiResidual = 2,  // x_f32[r][n] += v + bias
  kEpiQkv = 3,       // n < d: q[r][n]; else key / value into the paged cache at position len[b] + i
  kEpiHeadOut = 4    // o[r][n] = v + bias + h[r][n mod d]   (residual to each of the k outputs)
};

struct LinearParams {
  const void* x; long long ldx;   // activations [rows, K]
  const void* w; long long ldw;   // weights [N, K]
  const void* bias;               // [N] or null
  int rows, K, N;
  long long xz, wz, bz, yz;       // element offsets per blockIdx.z
  int relu;
  void* y; long long ldy;
  const float* h; int d;          // kEpiHeadOut: residual source; kEpiQkv: model width
  int head_identity;              // kEpiHeadOut: first d outputs are h itself
  void* kcache; void* vcache;     // kEpiQkv
  RowState st; int rows_per_b;
  const int* all_done;
};

constexpr int kRC = 8;      // rows per CTA pass
constexpr int kFPW = 4;     // output features per warp
constexpr int kKT = 512;    // K tile staged in shared memory
constexpr int kLinWarps = 8;

template <typename WT, typename AT, int EPI>
__device__ __forceinline__ void linear_epilogue(const LinearParams& p, int z, int r, int n, float v) {
  if (p.bias) v += to_f(reinterpret_cast<const WT*>(p.bias)[z * p.bz + n]);
  if (p.relu) v = fmaxf(v, 0.f);
  if (EPI == kEpiStoreAct) {
    reinterpret_cast<AT*>(p.y)[z * p.yz + (long long)r * p.ldy + n] = from_f<AT>(v);
  } else if (EPI == kEpiStoreF32) {
    reinterpret_cast<float*>(p.y)[z * p.yz + (long long)r * p.ldy + n] = v;
  } else if (EPI == kEpiResidual) {
    reinterpret_cast<float*>(p.y)[(long long)r * p.ldy + n] += v;
  } else if (EPI == kEpiHeadOut) {
    const int c = n % p.d;
    const float hv = p.h[(size_t)r * p.d + c];
    const int nz = z * (int)(p.yz) + n;   // output column within the row of k*d
    v = (p.head_identity && nz < p.d) ? hv : v + hv;
    reinterpret_cast<AT*>(p.y)[z * p.yz + (long long)r * p.ldy + n] = from_f<AT>(v);
  } else if (EPI == kEpiQkv) {
    const int d = p.d;
    if (n < d) {
      reinterpret_cast<AT*>(p.y)[(long long)r * p.ldy + n] = from_f<AT>(v);
    } else {
      const int b = r / p.rows_per_b, i = r % p.rows_per_b;
      const int pos = p.st.len[b] + i;
      const int page = p.st.page_table[b * p.st.pages_per_row + pos / kPage];
      const size_t slot = ((size_t)page * kPage + (pos % kPage)) * d;
      // the cache is stored in the weights' element type
      if (n < 2 * d) reinterpret_cast<WT*>(p.kcache)[slot + (n - d)] = from_f<WT>(v);
      else reinterpret_cast<WT*>(p.vcache)[slot + (n - 2 * d)] = from_f<WT>(v);
    }
  }
}

// One warp owns kFPW output features and kRC rows; its lanes split K, each
// accumulating in increasing-k order, then a butterfly sum.  The order depends
// only on K, never on the number of rows.
template <typename WT, typename AT, int EPI>
__global__ void __launch_bounds__(kLinWarps * 32) linear_kernel(LinearParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  __shared__ __align__(16) float xs[kRC][kKT];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int z = blockIdx.z;
  const AT* X = reinterpret_cast<const AT*>(p.x) + z * p.xz;
  const WT* W = reinterpret_cast<const WT*>(p.w) + z * p.wz;
  const int r0 = blockIdx.y * kRC;
  const int nr = min(kRC, p.rows - r0);
  const int n0 = blockIdx.x * (kLinWarps * kFPW) + warp * kFPW;
  float acc[kFPW][kRC];
#pragma unroll
  for (int f = 0; f < kFPW; ++f)
#pragma unroll
    for (int r = 0; r < kRC; ++r) acc[f][r] = 0.f;

  for (int kt = 0; kt < p.K; kt += kKT) {
    __syncthreads();
    for (int v = threadIdx.x; v < kRC * kKT / 8; v += kLinWarps * 32) {
      const int r = v / (kKT / 8), kk = (v % (kKT / 8)) * 8;
      float t[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (r < nr && kt + kk < p.K) load8(X + (long long)(r0 + r) * p.ldx + kt + kk, t);
      *reinterpret_cast<float4*>(&xs[r][kk]) = make_float4(t[0], t[1], t[2], t[3]);
      *reinterpret_cast<float4*>(&xs[r][kk + 4]) = make_float4(t[4], t[5], t[6], t[7]);
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < kKT / 256; ++c) {
      const int kk = c * 256 + lane * 8;
      if (kt + kk < p.K) {
        float wv[kFPW][8];
#pragma unroll
        for (int f = 0; f < kFPW; ++f) {
          if (n0 + f < p.N) {
            load8_stream(W + (long long)(n0 + f) * p.ldw + kt + kk, wv[f]);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) wv[f][e] = 0.f;
          }
        }
#pragma unroll
        for (int r = 0; r < kRC; ++r) {
          const float4 a = *reinterpret_cast<const float4*>(&xs[r][kk]);
          const float4 b = *reinterpret_cast<const float4*>(&xs[r][kk + 4]);
          const float xv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
          for (int f = 0; f < kFPW; ++f)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[f][r] = fmaf(wv[f][e], xv[e], acc[f][r]);
        }
      }
    }
  }
#pragma unroll
  for (int f = 0; f < kFPW; ++f)
#pragma unroll
    for (int r = 0; r < kRC; ++r) {
      const float v = warp_sum(acc[f][r]);
      if (lane == f * kRC + r && r < nr && n0 + f < p.N) linear_epilogue<WT, AT, EPI>(p, z, r0 + r, n0 + f, v);
    }
}

// ------------------------------------------------------------------ attention (one warp per (row, head))
struct AttnParams {
  const void* q; long long ldq;    // query of row r, head h at q + r*ldq + h*dh
  void* out; long long ldo;
  long long out_plane;             // > 0: output as two bf16 planes (hi, lo) this many elements apart
  int rows, rows_per_b, H, dh;
  int by_rows;                     // 1: one CTA per (sequence, head) instead of per (row, head)
  int causal;                      // 1: keys 0 .. len[b]+i ; 0: keys 0 .. limit_b[b]-1
  int local_q, local_m;            // causal only, local_q > 0: 1D local attention -- a query at position t sees keys
                                   // from (t / local_q) * local_q - local_m (not below 0) to t
  const int* limit_b;
  const void* k; const void* v;    // linear: row s of batch b at base + b*bstride + s*ldkv ; paged: page pool
  long long ldkv, bstride;
  int paged;
  RowState st;
  float scale;
  const int* all_done;
};

// First key a causal query at position pos may see (0 unless the model uses 1D local attention).
__device__ __forceinline__ int attn_first_key(const AttnParams& p, int pos) {
  if (!p.causal || p.local_q <= 0) return 0;
  return max(0, (pos / p.local_q) * p.local_q - p.local_m);
}

// Keys are taken in chunks of 32 absolute positions, lane = key; running
// max / sum are merged chunk by chunk in position order (fixed order).
template <typename QT, typename CT>
__global__ void __launch_bounds__(128) attention_kernel(AttnParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  __shared__ float qs[4][128];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int item = blockIdx.x * 4 + warp;
  if (item >= p.rows * p.H) return;
  const int r = item / p.H, h = item % p.H;
  const int b = r / p.rows_per_b, i = r % p.rows_per_b;
  const int dh = p.dh;
  const int limit = p.causal ? (p.st.len[b] + i + 1) : p.limit_b[b];
  const int first = attn_first_key(p, limit - 1);
  const QT* q = reinterpret_cast<const QT*>(p.q) + (long long)r * p.ldq + h * dh;
  for (int c = lane; c < dh; c += 32) qs[warp][c] = to_f(q[c]) * p.scale;
  __syncwarp();
  const CT* K = reinterpret_cast<const CT*>(p.k);
  const CT* V = reinterpret_cast<const CT*>(p.v);
  const int* pt = p.st.page_table + b * p.st.pages_per_row;
  auto row_off = [&](int pos) -> size_t {
    if (p.paged) return ((size_t)pt[pos / kPage] * kPage + (pos % kPage)) * p.ldkv + h * dh;
    return (size_t)b * p.bstride + (size_t)pos * p.ldkv + h * dh;
  };
  float m_run = -INFINITY, l_run = 0.f;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};   // output dims lane, lane+32, lane+64, lane+96
  for (int c0 = first & ~31; c0 < limit; c0 += 32) {
    const int pos = c0 + lane;
    float s = -INFINITY;
    if (pos >= first && pos < limit) {
      const CT* kr = K + row_off(pos);
      float dot = 0.f;
      for (int c = 0; c < dh; c += 8) {
        float kv[8];
        load8(kr + c, kv);
#pragma unroll
        for (int e = 0; e < 8; ++e) dot = fmaf(qs[warp][c + e], kv[e], dot);
      }
      s = dot;
    }
    const float m_new = fmaxf(m_run, warp_max(s));
    const float corr = expf(m_run - m_new);      // exp(-inf) = 0 on the first chunk
    const float pj = (pos >= first && pos < limit) ? expf(s - m_new) : 0.f;
    l_run = l_run * corr + warp_sum(pj);
#pragma unroll
    for (int t = 0; t < 4; ++t) acc[t] *= corr;
    const int nk = min(32, limit - c0);
    for (int jj = 0; jj < nk; ++jj) {
      const float pw = __shfl_sync(0xffffffffu, pj, jj);
      const CT* vr = V + row_off(c0 + jj);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int c = lane + 32 * t;
        if (c < dh) acc[t] = fmaf(pw, to_f(vr[c]), acc[t]);
      }
    }
    m_run = m_new;
  }
  QT* o = reinterpret_cast<QT*>(p.out) + (long long)r * p.ldo + h * dh;
  const float inv = 1.f / l_run;
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int c = lane + 32 * t;
    if (c < dh) {
      const float ov = acc[t] * inv;
      if (p.out_plane) {
        bf16* op = reinterpret_cast<bf16*>(p.out) + (long long)r * p.ldo + h * dh + c;
        const bf16 hi = __float2bfloat16_rn(ov);
        op[0] = hi;
        op[p.out_plane] = __float2bfloat16_rn(ov - __bfloat162float(hi));
      } else {
        o[c] = from_f<QT>(ov);
      }
    }
  }
}

// Attention with the keys of one (row, head) spread over the 8 warps of a CTA: warp w takes the 32-key
// chunks w, w+8, ... in increasing position order, then the 8 partial (max, sum, output) states are
// merged in warp order.  The partition depends only on key positions, so the result for a position does
// not depend on how many rows the launch carries.  DH = head width (16, 32, 64 or 128).
constexpr int kAttnWarps = 8;

template <int N> __device__ __forceinline__ void load_n(const float* p, float (&o)[N]) {
#pragma unroll
  for (int i = 0; i < N; ++i) o[i] = p[i];
}
template <> __device__ __forceinline__ void load_n<2>(const float* p, float (&o)[2]) {
  const float2 v = *reinterpret_cast<const float2*>(p); o[0] = v.x; o[1] = v.y;
}
template <> __device__ __forceinline__ void load_n<4>(const float* p, float (&o)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(p); o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
}
template <int N> __device__ __forceinline__ void load_n(const bf16* p, float (&o)[N]) {
#pragma unroll
  for (int i = 0; i < N; ++i) o[i] = __bfloat162float(p[i]);
}
template <> __device__ __forceinline__ void load_n<2>(const bf16* p, float (&o)[2]) {
  const uint32_t v = *reinterpret_cast<const uint32_t*>(p);
  o[0] = __uint_as_float(v << 16); o[1] = __uint_as_float(v & 0xffff0000u);
}
template <> __device__ __forceinline__ void load_n<4>(const bf16* p, float (&o)[4]) {
  const uint2 v = *reinterpret_cast<const uint2*>(p);
  o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
  o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
}

template <int DH, int NW> struct AttnSmem {
  float q[DH];
  float m[NW], l[NW];
  float acc[NW][DH];
};
// Variants of load_n that read from L2 (see COHERENT below).
template <int N> __device__ __forceinline__ void load_n_cg(const float* p, float (&o)[N]) {
#pragma unroll
  for (int i = 0; i < N; ++i) o[i] = __ldcg(p + i);
}
template <> __device__ __forceinline__ void load_n_cg<2>(const float* p, float (&o)[2]) {
  const float2 v = __ldcg(reinterpret_cast<const float2*>(p)); o[0] = v.x; o[1] = v.y;
}
template <> __device__ __forceinline__ void load_n_cg<4>(const float* p, float (&o)[4]) {
  const float4 v = __ldcg(reinterpret_cast<const float4*>(p)); o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
}
template <int N> __device__ __forceinline__ void load_n_cg(const bf16* p, float (&o)[N]) {
#pragma unroll
  for (int i = 0; i < N; ++i) o[i] = __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short*>(p + i)) << 16);
}
template <> __device__ __forceinline__ void load_n_cg<2>(const bf16* p, float (&o)[2]) {
  const uint32_t v = __ldcg(reinterpret_cast<const uint32_t*>(p));
  o[0] = __uint_as_float(v << 16); o[1] = __uint_as_float(v & 0xffff0000u);
}
template <> __device__ __forceinline__ void load_n_cg<4>(const bf16* p, float (&o)[4]) {
  const uint2 v = __ldcg(reinterpret_cast<const uint2*>(p));
  o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
  o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
}

// Attention of one query row and one head by a CTA of NW warps (see the comment above).  sm.q holds the scaled
// query and a __syncthreads() lies between its writes and this call.  Threads c < DH return output element c.
// COHERENT: keys and values may have been written by other SMs earlier in the same launch, so they are read
// from L2 rather than through L1.
template <typename CT, int DH, int NW, bool COHERENT>
__device__ __forceinline__ float attention_head(const AttnParams& p, int b, int h, int first, int limit, AttnSmem<DH, NW>& sm) {
  constexpr int DPL = (DH >= 32) ? DH / 32 : 1;       // output dims per lane (contiguous)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const CT* K = reinterpret_cast<const CT*>(p.k);
  const CT* V = reinterpret_cast<const CT*>(p.v);
  const int* pt = p.st.page_table + b * p.st.pages_per_row;
  float m_run = -INFINITY, l_run = 0.f;
  float acc[DPL];
#pragma unroll
  for (int t = 0; t < DPL; ++t) acc[t] = 0.f;
  const int nchunks = (limit + 31) >> 5;
  const bool owns = (DH >= 32) || (lane < DH);
  const int dim0 = (DH >= 32) ? lane * DPL : lane;
  for (int ch = (first >> 5) + warp; ch < nchunks; ch += NW) {
    const int c0 = ch << 5;
    const int lo = first - c0;                       // lanes below it hold keys before the first visible one
    // a 32-key chunk never straddles a 64-position page
    const size_t base = p.paged ? ((size_t)pt[c0 / kPage] * kPage + (c0 % kPage)) * p.ldkv + h * DH
                                : (size_t)b * p.bstride + (size_t)c0 * p.ldkv + h * DH;
    const int nk = min(32, limit - c0);
    // key row of this lane and the first batch of value rows are fetched together (a warp issues in order: all
    // loads go out before the first one is used).  Value rows are taken VB at a time; rows beyond the chunk's
    // last key repeat it with weight 0 (pj is 0 in those lanes), which leaves the sum unchanged.
    constexpr int VB0 = ((sizeof(CT) == 2) ? 64 : 32) / DPL, VB = VB0 > 32 ? 32 : (VB0 < 8 ? 8 : VB0);
    const CT* vb = V + base + dim0;
    float kv[DH / 8][8];
    if (lane < nk) {
      const CT* kr = K + base + (size_t)lane * p.ldkv;
#pragma unroll
      for (int c = 0; c < DH; c += 8) {
        if (COHERENT) load8_cg(kr + c, kv[c / 8]); else load8(kr + c, kv[c / 8]);
      }
    }
    float vv[VB][DPL];
    if (owns) {
#pragma unroll
      for (int jj = 0; jj < VB; ++jj) {
        const int jc = min(jj, nk - 1);
        if (COHERENT) load_n_cg<DPL>(vb + (size_t)jc * p.ldkv, vv[jj]); else load_n<DPL>(vb + (size_t)jc * p.ldkv, vv[jj]);
      }
    }
    float sc = -INFINITY;
    if (lane >= lo && lane < nk) {
      float dot = 0.f;
#pragma unroll
      for (int c = 0; c < DH; c += 8) {
#pragma unroll
        for (int e = 0; e < 8; ++e) dot = fmaf(sm.q[c + e], kv[c / 8][e], dot);
      }
      sc = dot;
    }
    const float m_new = fmaxf(m_run, warp_max(sc));
    const float corr = expf(m_run - m_new);
    const float pj = (lane >= lo && lane < nk) ? expf(sc - m_new) : 0.f;
    l_run = l_run * corr + warp_sum(pj);
#pragma unroll
    for (int t = 0; t < DPL; ++t) acc[t] *= corr;
#pragma unroll
    for (int j0 = 0; j0 < 32; j0 += VB) {
      if (j0 < nk) {
        if (j0 > 0 && owns) {
#pragma unroll
          for (int jj = 0; jj < VB; ++jj) {
            const int jc = min(j0 + jj, nk - 1);
            if (COHERENT) load_n_cg<DPL>(vb + (size_t)jc * p.ldkv, vv[jj]); else load_n<DPL>(vb + (size_t)jc * p.ldkv, vv[jj]);
          }
        }
#pragma unroll
        for (int jj = 0; jj < VB; ++jj) {
          const float pw = __shfl_sync(0xffffffffu, pj, j0 + jj);
          if (owns) {
#pragma unroll
            for (int t = 0; t < DPL; ++t) acc[t] = fmaf(pw, vv[jj][t], acc[t]);
          }
        }
      }
    }
    m_run = m_new;
  }
  if (lane == 0) { sm.m[warp] = m_run; sm.l[warp] = l_run; }
  if (owns) {
#pragma unroll
    for (int t = 0; t < DPL; ++t) sm.acc[warp][dim0 + t] = acc[t];
  }
  __syncthreads();
  float ov = 0.f;
  if (threadIdx.x < DH) {
    const int c = threadIdx.x;
    float M = sm.m[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) M = fmaxf(M, sm.m[w]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float e = expf(sm.m[w] - M);          // warps without keys hold -inf: weight 0
      num = fmaf(e, sm.acc[w][c], num);
      den = fmaf(e, sm.l[w], den);
    }
    ov = num / den;
  }
  return ov;
}

// One (row, head) item of a launch: query from p.q, output to p.out; callers separate items with __syncthreads().
template <typename QT, typename CT, int DH, int NW>
__device__ __forceinline__ void attention_item(const AttnParams& p, int item, AttnSmem<DH, NW>& sm) {
  const int r = item / p.H, h = item % p.H;
  const int b = r / p.rows_per_b, i = r % p.rows_per_b;
  const int limit = p.causal ? (p.st.len[b] + i + 1) : p.limit_b[b];
  const QT* q = reinterpret_cast<const QT*>(p.q) + (long long)r * p.ldq + h * DH;
  if (threadIdx.x < DH) sm.q[threadIdx.x] = to_f(q[threadIdx.x]) * p.scale;
  __syncthreads();
  const float ov = attention_head<CT, DH, NW, false>(p, b, h, attn_first_key(p, limit - 1), limit, sm);
  if (threadIdx.x < DH) {
    const int c = threadIdx.x;
    if (p.out_plane) {
      bf16* op = reinterpret_cast<bf16*>(p.out) + (long long)r * p.ldo + h * DH + c;
      const bf16 hi = __float2bfloat16_rn(ov);
      op[0] = hi;
      op[p.out_plane] = __float2bfloat16_rn(ov - __bfloat162float(hi));
    } else {
      reinterpret_cast<QT*>(p.out)[(long long)r * p.ldo + h * DH + c] = from_f<QT>(ov);
    }
  }
}

template <typename QT, typename CT, int DH>
__global__ void __launch_bounds__(kAttnWarps * 32) attention_split_kernel(AttnParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  __shared__ AttnSmem<DH, kAttnWarps> sm;
  attention_item<QT, CT, DH, kAttnWarps>(p, blockIdx.x, sm);
}

// Attention for sessions with many rows: one CTA per (sequence, head), one warp per query row (rows beyond
// 8 wrap around).  A warp walks the 32-key chunks of its row in position order with a running max / sum, so
// the order again depends only on key positions; the rows of a sequence share its keys through L1/L2.
template <typename QT, typename CT, int DH>
__global__ void __launch_bounds__(kAttnWarps * 32) attention_rows_kernel(AttnParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  constexpr int DPL = (DH >= 32) ? DH / 32 : 1;
  __shared__ float s_q[kAttnWarps][DH];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / p.H, h = blockIdx.x % p.H;
  const CT* K = reinterpret_cast<const CT*>(p.k);
  const CT* V = reinterpret_cast<const CT*>(p.v);
  const int* pt = p.st.page_table + b * p.st.pages_per_row;
  const bool owns = (DH >= 32) || (lane < DH);
  const int dim0 = (DH >= 32) ? lane * DPL : lane;
  for (int i = warp; i < p.rows_per_b; i += kAttnWarps) {
    const int r = b * p.rows_per_b + i;
    const int limit = p.causal ? (p.st.len[b] + i + 1) : p.limit_b[b];
    const int first = attn_first_key(p, limit - 1);
    const QT* q = reinterpret_cast<const QT*>(p.q) + (long long)r * p.ldq + h * DH;
    __syncwarp();
    for (int c = lane; c < DH; c += 32) s_q[warp][c] = to_f(q[c]) * p.scale;
    __syncwarp();
    float m_run = -INFINITY, l_run = 0.f;
    float acc[DPL];
#pragma unroll
    for (int t = 0; t < DPL; ++t) acc[t] = 0.f;
    for (int c0 = first & ~31; c0 < limit; c0 += 32) {
      const size_t base = p.paged ? ((size_t)pt[c0 / kPage] * kPage + (c0 % kPage)) * p.ldkv + h * DH
                                  : (size_t)b * p.bstride + (size_t)c0 * p.ldkv + h * DH;
      const int nk = min(32, limit - c0);
      const int lo = first - c0;
      float sc = -INFINITY;
      if (lane >= lo && lane < nk) {
        const CT* kr = K + base + (size_t)lane * p.ldkv;
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < DH; c += 8) {
          float kv[8];
          load8(kr + c, kv);
#pragma unroll
          for (int e = 0; e < 8; ++e) dot = fmaf(s_q[warp][c + e], kv[e], dot);
        }
        sc = dot;
      }
      const float m_new = fmaxf(m_run, warp_max(sc));
      const float corr = expf(m_run - m_new);
      const float pj = (lane >= lo && lane < nk) ? expf(sc - m_new) : 0.f;
      l_run = l_run * corr + warp_sum(pj);
#pragma unroll
      for (int t = 0; t < DPL; ++t) acc[t] *= corr;
      const CT* vb = V + base + dim0;
#pragma unroll 8
      for (int jj = 0; jj < nk; ++jj) {
        const float pw = __shfl_sync(0xffffffffu, pj, jj);
        if (owns) {
          float vv[DPL];
          load_n<DPL>(vb + (size_t)jj * p.ldkv, vv);
#pragma unroll
          for (int t = 0; t < DPL; ++t) acc[t] = fmaf(pw, vv[t], acc[t]);
        }
      }
      m_run = m_new;
    }
    if (owns) {
      const float inv = 1.f / l_run;
#pragma unroll
      for (int t = 0; t < DPL; ++t) {
        const float ov = acc[t] * inv;
        const long long o = (long long)r * p.ldo + h * DH + dim0 + t;
        if (p.out_plane) {
          bf16* op = reinterpret_cast<bf16*>(p.out) + o;
          const bf16 hi = __float2bfloat16_rn(ov);
          op[0] = hi;
          op[p.out_plane] = __float2bfloat16_rn(ov - __bfloat162float(hi));
        } else {
          reinterpret_cast<QT*>(p.out)[o] = from_f<QT>(ov);
        }
      }
    }
  }
}

// Same job for blocks of at most 16 query rows per sequence (the decoder's passes): the CTA stages each
// 32-key chunk of K and V in shared memory once (coalesced), every warp then serves its one or two query rows
// from there.  Per row the chunks are folded in position order with a running max / sum.
template <typename QT, typename CT, int DH>
__global__ void __launch_bounds__(kAttnWarps * 32) attention_seq_kernel(AttnParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  constexpr int DPL = (DH >= 32) ? DH / 32 : 1;
  constexpr int RPW = 2;                                  // rows per warp: 8 warps x 2 = 16 rows
  __shared__ float s_q[kAttnWarps * RPW][DH];
  __shared__ float s_k[32][DH + 1];
  __shared__ float s_v[32][DH];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / p.H, h = blockIdx.x % p.H;
  const CT* K = reinterpret_cast<const CT*>(p.k);
  const CT* V = reinterpret_cast<const CT*>(p.v);
  const int* pt = p.st.page_table + b * p.st.pages_per_row;
  const bool owns = (DH >= 32) || (lane < DH);
  const int dim0 = (DH >= 32) ? lane * DPL : lane;
  const int nrows = p.rows_per_b;
  const int base_limit = p.causal ? p.st.len[b] + 1 : p.limit_b[b];
  const int limit_max = p.causal ? base_limit + nrows - 1 : base_limit;
  const int first_min = attn_first_key(p, base_limit - 1);   // the first row's window starts earliest
  for (int idx = threadIdx.x; idx < nrows * DH; idx += blockDim.x) {
    const int i = idx / DH, c = idx % DH;
    s_q[i][c] = to_f(reinterpret_cast<const QT*>(p.q)[(long long)(b * nrows + i) * p.ldq + h * DH + c]) * p.scale;
  }
  float m_run[RPW], l_run[RPW], acc[RPW][DPL];
#pragma unroll
  for (int r = 0; r < RPW; ++r) {
    m_run[r] = -INFINITY; l_run[r] = 0.f;
#pragma unroll
    for (int t = 0; t < DPL; ++t) acc[r][t] = 0.f;
  }
  for (int c0 = first_min & ~31; c0 < limit_max; c0 += 32) {
    const size_t base = p.paged ? ((size_t)pt[c0 / kPage] * kPage + (c0 % kPage)) * p.ldkv + h * DH
                                : (size_t)b * p.bstride + (size_t)c0 * p.ldkv + h * DH;
    const int nk = min(32, limit_max - c0);
    __syncthreads();                                       // the previous chunk is no longer needed
    for (int v8 = threadIdx.x; v8 < 32 * DH / 8; v8 += blockDim.x) {
      const int j = v8 / (DH / 8), c = (v8 % (DH / 8)) * 8;
      float kv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, vv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (j < nk) {
        load8(K + base + (size_t)j * p.ldkv + c, kv);
        load8(V + base + (size_t)j * p.ldkv + c, vv);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) { s_k[j][c + e] = kv[e]; s_v[j][c + e] = vv[e]; }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      const int i = warp + r * kAttnWarps;
      if (i >= nrows) continue;                            // uniform over the warp
      const int limit = p.causal ? base_limit + i : base_limit;
      const int live = min(32, limit - c0);                // keys of this chunk the row may see
      const int lo = attn_first_key(p, limit - 1) - c0;    // ... and lanes below lo hold keys before its window
      if (live <= 0 || lo >= live) continue;
      float sc = -INFINITY;
      if (lane >= lo && lane < live) {
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < DH; ++c) dot = fmaf(s_q[i][c], s_k[lane][c], dot);
        sc = dot;
      }
      const float m_new = fmaxf(m_run[r], warp_max(sc));
      const float corr = expf(m_run[r] - m_new);
      const float pj = (lane >= lo && lane < live) ? expf(sc - m_new) : 0.f;
      l_run[r] = l_run[r] * corr + warp_sum(pj);
#pragma unroll
      for (int t = 0; t < DPL; ++t) acc[r][t] *= corr;
      for (int jj = 0; jj < live; ++jj) {
        const float pw = __shfl_sync(0xffffffffu, pj, jj);
        if (owns) {
#pragma unroll
          for (int t = 0; t < DPL; ++t) acc[r][t] = fmaf(pw, s_v[jj][dim0 + t], acc[r][t]);
        }
      }
      m_run[r] = m_new;
    }
  }
#pragma unroll
  for (int r = 0; r < RPW; ++r) {
    const int i = warp + r * kAttnWarps;
    if (i >= nrows || !owns) continue;
    const float inv = 1.f / l_run[r];
#pragma unroll
    for (int t = 0; t < DPL; ++t) {
      const float ov = acc[r][t] * inv;
      const long long o = (long long)(b * nrows + i) * p.ldo + h * DH + dim0 + t;
      if (p.out_plane) {
        bf16* op = reinterpret_cast<bf16*>(p.out) + o;
        const bf16 hi = __float2bfloat16_rn(ov);
        op[0] = hi;
        op[p.out_plane] = __float2bfloat16_rn(ov - __bfloat162float(hi));
      } else {
        reinterpret_cast<QT*>(p.out)[o] = from_f<QT>(ov);
      }
    }
  }
}

// Decoder cross-attention for sessions with many sequences: a CTA per (sequence, head), head width 64, fp32 keys
// and values.  The encoder's keys and values do not change during a decode, so the CTA copies its head's rows
// (all positions below the source length) into shared memory before it waits for the preceding launch; only the
// queries depend on that.  Rows of kXKeyPitch + 256 bytes: lane-per-key 16-byte reads of 8 lanes hit all banks.
// A warp serves query rows warp, warp + 8 and folds the 32-key chunks of a row in position order with a running
// maximum / sum, the same arithmetic per row as attention_seq_kernel.
constexpr int kXKeyPitch = 64 * 4 + 16;
constexpr int kXRowBytes = kXKeyPitch + 64 * 4;
__host__ __device__ inline size_t cross_staged_smem(int max_src) { return (size_t)max_src * kXRowBytes + 16 * 64 * sizeof(float); }
// kv_static = 0: the keys and values come from the preceding launch (encoder self-attention); they are copied
// after the wait.  Query rows are taken 16 at a time.
template <typename QT>
__global__ void __launch_bounds__(kAttnWarps * 32) cross_attention_staged_kernel(AttnParams p, int max_src, int kv_static) {
  extern __shared__ __align__(16) uint8_t xs[];
  uint8_t* kv = xs;
  float* s_q = reinterpret_cast<float*>(xs + (size_t)max_src * kXRowBytes);   // [16][64]
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / p.H, h = blockIdx.x % p.H;
  const int limit = min(p.limit_b[b], max_src);
  if (!kv_static) pdl_wait();
  {
    const float* Kg = reinterpret_cast<const float*>(p.k) + (size_t)b * p.bstride + h * 64;
    const float* Vg = reinterpret_cast<const float*>(p.v) + (size_t)b * p.bstride + h * 64;
    for (int idx = threadIdx.x; idx < limit * 32; idx += blockDim.x) {
      const int row = idx >> 5, piece = idx & 31;
      const float* src = (piece < 16 ? Kg : Vg) + (size_t)row * p.ldkv + (piece & 15) * 4;
      uint8_t* dst = kv + (size_t)row * kXRowBytes + (piece < 16 ? piece * 16 : kXKeyPitch + (piece - 16) * 16);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  if (kv_static) pdl_wait();
  const bool ended = p.all_done && *p.all_done;
  const int nrows = p.rows_per_b;
  for (int row0 = 0; row0 < nrows; row0 += 16) {
  const int ngroup = min(16, nrows - row0);
  if (row0 > 0) __syncthreads();                       // the previous group's queries have been read
  if (!ended) {
    for (int idx = threadIdx.x; idx < ngroup * 64; idx += blockDim.x) {
      const int i = row0 + (idx >> 6), c = idx & 63;
      s_q[idx] = to_f(reinterpret_cast<const QT*>(p.q)[(long long)(b * nrows + i) * p.ldq + h * 64 + c]) * p.scale;
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  if (ended) return;
  for (int i = row0 + warp; i < row0 + ngroup; i += kAttnWarps) {
    float m_run = -INFINITY, l_run = 0.f, a0 = 0.f, a1 = 0.f;
    const float4* qv = reinterpret_cast<const float4*>(s_q + (i - row0) * 64);
    for (int c0 = 0; c0 < limit; c0 += 32) {
      const int nk = min(32, limit - c0);
      float sc = -INFINITY;
      if (lane < nk) {
        const float4* kr = reinterpret_cast<const float4*>(kv + (size_t)(c0 + lane) * kXRowBytes);
        float dot = 0.f;
#pragma unroll
        for (int u = 0; u < 16; ++u) {
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
        const float2 v2 = *reinterpret_cast<const float2*>(kv + (size_t)(c0 + j) * kXRowBytes + kXKeyPitch + lane * 8);
        a0 = fmaf(pw, v2.x, a0);
        a1 = fmaf(pw, v2.y, a1);
      }
      m_run = m_new;
    }
    const float inv = 1.f / l_run;
    const float o2[2] = {a0 * inv, a1 * inv};
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const long long o = (long long)(b * nrows + i) * p.ldo + h * 64 + lane * 2 + t;
      if (p.out_plane) {
        bf16* op = reinterpret_cast<bf16*>(p.out) + o;
        const bf16 hi = __float2bfloat16_rn(o2[t]);
        op[0] = hi;
        op[p.out_plane] = __float2bfloat16_rn(o2[t] - __bfloat162float(hi));
      } else {
        reinterpret_cast<QT*>(p.out)[o] = from_f<QT>(o2[t]);
      }
    }
  }
  }
}

// Picks the split kernel for the common head widths, the generic one-warp kernel otherwise.
template <typename QT, typename CT>
static void launch_attention(const AttnParams& p, cudaStream_t st, bool pdl = false) {
  const int items = p.rows * p.H;
  const dim3 g(items), b(kAttnWarps * 32);
  if (p.by_rows) {   // many sequences: a CTA per (sequence, head); a property of the session, not of the pass
    const dim3 gr((p.rows / p.rows_per_b) * p.H);
    if (p.rows_per_b <= 16) {
      switch (p.dh) {
        case 16: launch_k(attention_seq_kernel<QT, CT, 16>, gr, b, 0, st, pdl, p); return;
        case 32: launch_k(attention_seq_kernel<QT, CT, 32>, gr, b, 0, st, pdl, p); return;
        case 64: launch_k(attention_seq_kernel<QT, CT, 64>, gr, b, 0, st, pdl, p); return;
        default: break;
      }
    }
    switch (p.dh) {
      case 16: launch_k(attention_rows_kernel<QT, CT, 16>, gr, b, 0, st, pdl, p); return;
      case 32: launch_k(attention_rows_kernel<QT, CT, 32>, gr, b, 0, st, pdl, p); return;
      case 64: launch_k(attention_rows_kernel<QT, CT, 64>, gr, b, 0, st, pdl, p); return;
      case 128: launch_k(attention_rows_kernel<QT, CT, 128>, gr, b, 0, st, pdl, p); return;
      default: break;
    }
  }
  switch (p.dh) {
    case 16: launch_k(attention_split_kernel<QT, CT, 16>, g, b, 0, st, pdl, p); break;
    case 32: launch_k(attention_split_kernel<QT, CT, 32>, g, b, 0, st, pdl, p); break;
    case 64: launch_k(attention_split_kernel<QT, CT, 64>, g, b, 0, st, pdl, p); break;
    case 128: launch_k(attention_split_kernel<QT, CT, 128>, g, b, 0, st, pdl, p); break;
    default: launch_k(attention_kernel<QT, CT>, dim3((items + 3) / 4), dim3(128), 0, st, pdl, p); break;
  }
}

// ------------------------------------------------------------------ logit of each proposal under p_1 (top-n acceptance)
struct ProposalLogitParams {
  const void* o; long long o_plane;   // head outputs [B*kcur*kh, d]: activation dtype, or bf16 planes when o_plane > 0
  const void* w;                      // [V, d]
  RowState st;
  RankState rank;
  int B, kcur, kh, d;
  const int* all_done;
};
// One warp per block position: thr = o[position, head 1] . w[proposal after it].
template <typename WT>
__global__ void __launch_bounds__(128) proposal_logit_kernel(ProposalLogitParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pr = blockIdx.x * 4 + warp;
  if (pr >= p.B * p.kcur) return;
  const int b = pr / p.kcur, r = pr % p.kcur;
  int tok = -1;
  float thr = 0.f;
  if (r + 1 < p.kcur) {
    tok = p.st.cur_block[b * kMaxK + r + 1];
    const WT* wr = reinterpret_cast<const WT*>(p.w) + (size_t)tok * p.d;
    const size_t row = (size_t)pr * p.kh * p.d;
    float acc = 0.f;
    for (int c = lane * 8; c < p.d; c += 256) {
      float wv[8], ov[8];
      load8(wr + c, wv);
      if (p.o_plane) {
        float lo[8];
        load8(reinterpret_cast<const bf16*>(p.o) + row + c, ov);
        load8(reinterpret_cast<const bf16*>(p.o) + row + c + p.o_plane, lo);
#pragma unroll
        for (int e = 0; e < 8; ++e) ov[e] += lo[e];
      } else {
        load8(reinterpret_cast<const float*>(p.o) + row + c, ov);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) acc = fmaf(wv[e], ov[e], acc);
    }
    thr = warp_sum(acc);
  }
  if (lane == 0) { p.rank.tok[pr] = tok; p.rank.thr[pr] = thr; p.rank.cnt[pr] = 0; }
}

// ------------------------------------------------------------------ vocabulary projection + top-1
struct ArgmaxParams {
  const void* x; long long ldx;   // [rows, d] activations
  const void* w;                  // [V, d]
  int rows, d, V;
  float* part_val; int* part_idx; // [tiles][rows] workspace
  unsigned* counters;             // [row chunks], zero between launches
  int* out_idx; float* out_val;   // [rows]
  float* logits;                  // optional dump [rows, V]
  const int* all_done;
  RankState rank; int rank_kh;    // top-n acceptance: count entries beating each proposal (rank.cnt null = off)
};
constexpr int kVocTile = 256;     // vocabulary rows per CTA
constexpr int kArgmaxMaxD = 1024;

template <typename WT, typename AT>
__global__ void __launch_bounds__(kLinWarps * 32) vocab_argmax_kernel(ArgmaxParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  extern __shared__ __align__(16) float xs_dyn[];   // [kRC][d]
  __shared__ float sv[kLinWarps][kRC];
  __shared__ int si[kLinWarps][kRC];
  __shared__ unsigned ticket;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = blockIdx.y * kRC;
  const int nr = min(kRC, p.rows - r0);
  const int d = p.d;
  const AT* X = reinterpret_cast<const AT*>(p.x);
  const WT* W = reinterpret_cast<const WT*>(p.w);
  for (int v = threadIdx.x; v < kRC * d / 8; v += kLinWarps * 32) {
    const int r = v / (d / 8), kk = (v % (d / 8)) * 8;
    float t[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (r < nr) load8(X + (long long)(r0 + r) * p.ldx + kk, t);
    *reinterpret_cast<float4*>(&xs_dyn[r * d + kk]) = make_float4(t[0], t[1], t[2], t[3]);
    *reinterpret_cast<float4*>(&xs_dyn[r * d + kk + 4]) = make_float4(t[4], t[5], t[6], t[7]);
  }
  __syncthreads();
  float bv[kRC];
  int bi[kRC];
#pragma unroll
  for (int r = 0; r < kRC; ++r) { bv[r] = -INFINITY; bi[r] = 0x7fffffff; }
  const int tile0 = blockIdx.x * kVocTile;
  for (int g = 0; g < kVocTile / (kLinWarps * kFPW); ++g) {
    const int n0 = tile0 + g * (kLinWarps * kFPW) + warp * kFPW;   // ascending over g for a given warp
    if (n0 >= p.V) break;
    float acc[kFPW][kRC];
#pragma unroll
    for (int f = 0; f < kFPW; ++f)
#pragma unroll
      for (int r = 0; r < kRC; ++r) acc[f][r] = 0.f;
    for (int kk = lane * 8; kk < d; kk += 256) {
      float wv[kFPW][8];
#pragma unroll
      for (int f = 0; f < kFPW; ++f) {
        if (n0 + f < p.V) {
          load8_stream(W + (size_t)(n0 + f) * d + kk, wv[f]);
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) wv[f][e] = 0.f;
        }
      }
#pragma unroll
      for (int r = 0; r < kRC; ++r) {
        const float4 a = *reinterpret_cast<const float4*>(&xs_dyn[r * d + kk]);
        const float4 b = *reinterpret_cast<const float4*>(&xs_dyn[r * d + kk + 4]);
        const float xv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int f = 0; f < kFPW; ++f)
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[f][r] = fmaf(wv[f][e], xv[e], acc[f][r]);
      }
    }
#pragma unroll
    for (int f = 0; f < kFPW; ++f)
#pragma unroll
      for (int r = 0; r < kRC; ++r) {
        const float v = warp_sum(acc[f][r]);
        if (n0 + f < p.V) {
          if (p.rank.cnt && lane == 0 && r < nr && (r0 + r) % p.rank_kh == 0) {
            const int pr = (r0 + r) / p.rank_kh, tok = p.rank.tok[pr];
            if (tok >= 0 && tok != n0 + f && better(v, n0 + f, p.rank.thr[pr], tok)) atomicAdd(&p.rank.cnt[pr], 1);
          }
          if (better(v, n0 + f, bv[r], bi[r])) { bv[r] = v; bi[r] = n0 + f; }
          if (p.logits && lane == f * kRC + r && r < nr) p.logits[(size_t)(r0 + r) * p.V + n0 + f] = v;
        }
      }
  }
  if (lane == 0) {
#pragma unroll
    for (int r = 0; r < kRC; ++r) { sv[warp][r] = bv[r]; si[warp][r] = bi[r]; }
  }
  __syncthreads();
  if (threadIdx.x < nr) {
    const int r = threadIdx.x;
    float v = sv[0][r];
    int ix = si[0][r];
    for (int w2 = 1; w2 < kLinWarps; ++w2)
      if (better(sv[w2][r], si[w2][r], v, ix)) { v = sv[w2][r]; ix = si[w2][r]; }
    p.part_val[(size_t)blockIdx.x * p.rows + r0 + r] = v;
    p.part_idx[(size_t)blockIdx.x * p.rows + r0 + r] = ix;
  }
  // The CTA that finishes last for this row chunk merges all tiles (no waiting on anyone).
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) ticket = atomicAdd(&p.counters[blockIdx.y], 1u);
  __syncthreads();
  if (ticket != gridDim.x - 1) return;
  __threadfence();
  for (int r = warp; r < nr; r += kLinWarps) {
    float v = -INFINITY;
    int ix = 0x7fffffff;
    for (int t = lane; t < (int)gridDim.x; t += 32) {
      const float tv = __ldcg(&p.part_val[(size_t)t * p.rows + r0 + r]);
      const int ti = __ldcg(&p.part_idx[(size_t)t * p.rows + r0 + r]);
      if (better(tv, ti, v, ix)) { v = tv; ix = ti; }
    }
    warp_argmax(v, ix);
    if (lane == 0) {
      p.out_idx[r0 + r] = ix;
      if (p.out_val) p.out_val[r0 + r] = v;
    }
  }
  if (threadIdx.x == 0) p.counters[blockIdx.y] = 0;
}

// ------------------------------------------------------------------ verify / accept / commit / select next
struct VerifyParams {
  RowState st;
  int B, kcur, kh, knext;   // positions scored per row, heads per position, width of the next block
  int mode;
  int max_new, eos;
  int accept_kind, accept_param, min_block;   // exact / top-n (n) / distance (eps); forced minimum block size
  RankState rank;                             // top-n only
};

// Tells the host that one more pass has been verified, and whether every row is finished.
__device__ __forceinline__ void signal_host(const RowState& st, int done) {
  const int seq = st.signal[1];
  st.signal[1] = seq + 1;
  // a plain store: the host only needs to see it some time before it enqueues the pass after the next, and no
  // other data rides on it (a system-wide fence here cost 3 us per pass)
  *reinterpret_cast<volatile int*>(st.host_flags + (seq & 7)) = (st.signal[0] << 2) | (done ? 2 : 1);
}

static __global__ void verify_commit_kernel(VerifyParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (*p.st.all_done) {
    if (threadIdx.x == 0) signal_host(p.st, 1);
    return;
  }
  __shared__ int any_open;
  if (threadIdx.x == 0) any_open = 0;
  __syncthreads();
  const int b = threadIdx.x;
  if (b < p.B) {
    int* blk = p.st.block + b * kMaxK;
    const int* cur = p.st.cur_block + b * kMaxK;
    const int* A = p.st.table + (size_t)b * p.kcur * p.kh;
    if (p.st.finished[b]) {
      p.st.khat[b] = 0;
    } else if (p.mode != kModePrime && p.mode != kModePredict && p.st.j[b] >= p.max_new) {
      // the caller lowered max_new below what the row already holds (bpd_iteration takes it per call): the row
      // is complete, nothing is appended or committed
      p.st.khat[b] = 0;
      p.st.finished[b] = 1;
    } else if (p.mode == kModePrime || p.mode == kModePredict) {
      // priming: the start token becomes part of the prefix; its row of predictions is the first block.
      // Predict call of the two-call form: the row of the last accepted token (the length was stepped back onto
      // it) is part of the prefix again; its predictions are the next block.  The accepted count stays.
      p.st.len[b] += 1;
      if (p.mode == kModePrime) p.st.khat[b] = 0;
      for (int i = 0; i < p.knext; ++i) blk[i] = A[i];
      atomicOr(&any_open, 1);
    } else if (p.mode == kModeGreedy) {
      const int tok = A[0];
      const int j = p.st.j[b];
      p.st.out_ids[(size_t)b * p.st.max_tgt + j] = tok;
      p.st.j[b] = j + 1;
      p.st.len[b] += 1;
      p.st.khat[b] = 1;
      blk[0] = tok;
      const int fin = (j + 1 >= p.max_new) || (p.eos >= 0 && tok == p.eos);
      p.st.finished[b] = fin;
      if (!fin) atomicOr(&any_open, 1);
      atomicAdd((unsigned long long*)&p.st.stats[0], 1ull);
      atomicAdd((unsigned long long*)&p.st.stats[1], 1ull);
      atomicAdd((unsigned long long*)&p.st.stats[4 + 1], 1ull);
    } else {
      // longest prefix of the block that the base model would have produced itself:
      // proposal i+1 is checked against head 1 at the position of proposal i
      int khat = 1;
      while (khat < p.kcur) {
        const int top1 = A[(khat - 1) * p.kh];
        bool okay;
        if (p.accept_kind == kAcceptTopN) okay = p.rank.cnt[b * p.kcur + khat - 1] < p.accept_param;
        else if (p.accept_kind == kAcceptDistance) okay = abs(cur[khat] - top1) <= p.accept_param;
        else okay = (cur[khat] == top1);
        if (!okay && khat >= p.min_block) break;
        ++khat;
      }
      const int j = p.st.j[b];
      khat = min(khat, p.max_new - j);
      int fin = (j + khat >= p.max_new);
      if (p.eos >= 0) {
        for (int i = 0; i < khat; ++i)
          if (cur[i] == p.eos) { khat = i + 1; fin = 1; break; }
      }
      for (int i = 0; i < khat; ++i) p.st.out_ids[(size_t)b * p.st.max_tgt + j + i] = cur[i];
      p.st.j[b] = j + khat;
      p.st.len[b] += khat;      // keys/values of rejected positions stay behind the length and get overwritten
      p.st.khat[b] = khat;
      for (int i = 0; i < p.knext; ++i) blk[i] = A[(khat - 1) * p.kh + i];
      p.st.finished[b] = fin;
      if (!fin) atomicOr(&any_open, 1);
      atomicAdd((unsigned long long*)&p.st.stats[0], 1ull);
      atomicAdd((unsigned long long*)&p.st.stats[1], (unsigned long long)khat);
      atomicAdd((unsigned long long*)&p.st.stats[4 + khat], 1ull);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    p.st.stats[(p.mode == kModePrime || p.mode == kModePredict) ? 3 : 2] += 1;
    if (!any_open) *p.st.all_done = 1;
    signal_host(p.st, !any_open);
  }
}

// Before a Predict call of the two-call form (Section 3): the single row it scores is the last accepted token, which
// already sits in the cache at position len - 1.  Step the length back onto it and make it the block's first entry;
// the pass recomputes that position and the verify kernel (kModePredict) moves the length forward again.
struct StepBackParams { RowState st; int B; };
static __global__ void step_back_kernel(StepBackParams p) {
  if (*p.st.all_done) return;
  const int b = threadIdx.x;
  if (b >= p.B || p.st.finished[b]) return;
  const int khat = p.st.khat[b];
  if (khat < 1 || p.st.len[b] < 2) return;       // nothing accepted since the last Predict: the block stands
  p.st.len[b] -= 1;
  p.st.block[b * kMaxK] = p.st.cur_block[b * kMaxK + khat - 1];
}

// ------------------------------------------------------------------ lazy heads (two-stage evaluation)
// Stage 1 scores p_1 at every block position and verifies; stage 2 evaluates all k heads only at the last
// accepted position of each row.  These two small kernels move the selected rows into a compact buffer and
// then assemble the next block and the (partly filled) k x k table.
struct GatherParams {
  const bf16* u; long long pl_u; long long ldu;   // head hidden activations, planes [rows, ldu]
  bf16* u2; long long pl_u2;                      // compact planes [B, ldu]
  const float* h; float* h2; int d;               // decoder outputs [rows, d] -> [B, d]
  RowState st;
  int B, kcur;
  const int* all_done;
};
static __global__ void __launch_bounds__(256) gather_selected_kernel(GatherParams p) {
  pdl_launch_dependents();
  pdl_wait();
  if (p.all_done && *p.all_done) return;
  // grid = (sequences, column parts): a row of hidden activations is some hundred KB, one CTA per row copied it
  // in tens of dependent steps
  const int b = blockIdx.x;
  const int row = b * p.kcur + max(p.st.khat[b], 1) - 1;     // last accepted position (first one for idle rows)
  const uint4* s_hi = reinterpret_cast<const uint4*>(p.u + (size_t)row * p.ldu);
  const uint4* s_lo = reinterpret_cast<const uint4*>(p.u + (size_t)row * p.ldu + p.pl_u);
  uint4* d_hi = reinterpret_cast<uint4*>(p.u2 + (size_t)b * p.ldu);
  uint4* d_lo = reinterpret_cast<uint4*>(p.u2 + (size_t)b * p.ldu + p.pl_u2);
  const int step = blockDim.x * gridDim.y, first = blockIdx.y * blockDim.x + threadIdx.x;
  for (int i = first; i < p.ldu / 8; i += step) { d_hi[i] = s_hi[i]; d_lo[i] = s_lo[i]; }
  for (int c = first; c < p.d; c += step) p.h2[(size_t)b * p.d + c] = p.h[(size_t)row * p.d + c];
}

struct SelectParams {
  RowState st;
  const int* table1;   // [B, kcur]      p_1 at every block position
  const int* table2;   // [B, kh]        all heads at the selected position
  int* table_full;     // [B, kcur, kh]  what is known of the k x k table, -1 elsewhere
  int B, kcur, kh, knext;
  const int* all_done;
};
static __global__ void select_next_kernel(SelectParams p) {
  pdl_launch_dependents();
  pdl_wait();
  // When the decode ended in this very pass, stage 2 did not run: the table still reports p_1, the rest is unknown.
  const bool ended = p.all_done && *p.all_done;
  const int b = threadIdx.x;
  if (b >= p.B) return;
  const int khat = p.st.khat[b];
  const int sel = max(khat, 1) - 1;
  int* full = p.table_full + (size_t)b * p.kcur * p.kh;
  for (int r = 0; r < p.kcur; ++r)
    for (int i = 0; i < p.kh; ++i)
      full[r * p.kh + i] = (i == 0) ? p.table1[b * p.kcur + r] : ((r == sel && !ended) ? p.table2[b * p.kh + i] : -1);
  if (khat > 0 && !ended)
    for (int i = 1; i < p.knext; ++i) p.st.block[b * kMaxK + i] = p.table2[b * p.kh + i];
}

struct ResetParams {
  RowState st;
  int B, ppr;
  const int* src_len;
  unsigned* join_words;   // control words of the persistent layer kernel (64), or null
};
static __global__ void reset_rows_kernel(ResetParams p) {
  const int b = threadIdx.x;
  if (b < p.B) {
    p.st.len[b] = 0;
    p.st.j[b] = 0;
    p.st.finished[b] = 0;
    p.st.khat[b] = 0;
    p.st.src_len[b] = p.src_len[b];
    for (int i = 0; i < kMaxK; ++i) { p.st.block[b * kMaxK + i] = 0; p.st.cur_block[b * kMaxK + i] = 0; }
  }
  if (threadIdx.x == 0) {
    *p.st.all_done = 0;
    *p.st.error = 0;
    for (int i = 0; i < 4 + kMaxK + 1; ++i) p.st.stats[i] = 0;
  }
  // the abort word is cleared; word 32 numbers the kernel's reductions over the whole life of the session (its
  // workspace keeps the tags of earlier decodes) and stays
  if (p.join_words)
    for (int i = threadIdx.x; i < 64; i += blockDim.x)
      if (i != 32) p.join_words[i] = 0u;
}

}  // namespace bpd
