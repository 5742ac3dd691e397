// C ABI of the blockwise-parallel-decoding library: blob parsing, buffer
// planning, the encoder, the decoder pass and the decode loops.
#include <chrono>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <map>
#include <mutex>
#include <new>
#include <utility>

#include "host.hpp"
#include "kernels_simt.cuh"
#include "tc_host.hpp"
#include "fused_layer.cuh"
#include "layer_stack.cuh"

namespace bpd {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

int ensure_smem_limit(const void* kernel, size_t bytes) {
  static std::mutex mu;
  static std::map<std::pair<int, const void*>, size_t> most;
  int dev = 0;
  BPD_CUDA(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lock(mu);
  size_t& cur = most[std::make_pair(dev, kernel)];
  if (bytes > cur) {
    BPD_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    cur = bytes;
  }
  return BPD_OK;
}

static inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }
static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ------------------------------------------------------------------ blob
static const char kMagic[8] = {'B', 'P', 'D', 'W', '0', '0', '0', '1'};

int parse_blob(const void* blob, size_t n, ParsedBlob* out) {
  if (!blob) return fail(BPD_E_INVALID, "blob is null");
  if (n < 128) return fail(BPD_E_FORMAT, "blob shorter than its header (%zu bytes)", n);
  const unsigned char* p = static_cast<const unsigned char*>(blob);
  if (memcmp(p, kMagic, 8) != 0) return fail(BPD_E_FORMAT, "bad magic");
  int32_t f[12];
  memcpy(f, p + 8, sizeof(f));
  float eps;
  memcpy(&eps, p + 56, 4);
  int32_t n_tensors;
  memcpy(&n_tensors, p + 60, 4);
  uint64_t dir_off, data_off, total;
  memcpy(&dir_off, p + 64, 8);
  memcpy(&data_off, p + 72, 8);
  memcpy(&total, p + 80, 8);
  if (f[0] != 1) return fail(BPD_E_FORMAT, "unsupported blob version %d", f[0]);
  if (total != n) return fail(BPD_E_FORMAT, "blob size %zu does not match header %llu", n, (unsigned long long)total);
  Config& c = out->cfg;
  c.dtype = f[1]; c.n_enc = f[2]; c.n_dec = f[3]; c.d = f[4]; c.H = f[5]; c.d_ff = f[6]; c.V = f[7];
  c.k_model = f[8]; c.d_hidden = f[9]; c.head_layout = f[10]; c.p1_identity = f[11]; c.eps = eps;
  int32_t local[2];
  memcpy(local, p + 88, sizeof(local));      // 1D local self-attention in the decoder: query block length, memory length
  c.local_q = local[0]; c.local_m = local[1];
  if (c.local_q < 0 || c.local_m < 0) return fail(BPD_E_FORMAT, "bad local-attention lengths %d/%d", c.local_q, c.local_m);
  if (c.dtype != 0 && c.dtype != 1) return fail(BPD_E_FORMAT, "unknown dtype %d", c.dtype);
  if (c.n_enc < 1 || c.n_dec < 1 || c.n_enc > 64 || c.n_dec > 64) return fail(BPD_E_FORMAT, "bad layer counts");
  if (c.d < 8 || c.d % 8 || c.H < 1 || c.d % c.H) return fail(BPD_E_FORMAT, "bad d_model/heads %d/%d", c.d, c.H);
  const int dh = c.d / c.H;
  if (dh % 8 || dh > 128) return fail(BPD_E_UNSUPPORTED, "head width %d (need a multiple of 8, at most 128)", dh);
  if (c.d > kArgmaxMaxD) return fail(BPD_E_UNSUPPORTED, "d_model %d above %d", c.d, kArgmaxMaxD);
  if (c.d_ff < 8 || c.d_ff % 8 || c.d_hidden < 8 || c.d_hidden % 8) return fail(BPD_E_FORMAT, "bad FFN widths");
  if (c.V < 2) return fail(BPD_E_FORMAT, "bad vocabulary size %d", c.V);
  if (c.k_model < 1 || c.k_model > kMaxK) return fail(BPD_E_UNSUPPORTED, "k_model %d outside 1..%d", c.k_model, kMaxK);
  if (c.head_layout != 0 && c.head_layout != 1) return fail(BPD_E_FORMAT, "unknown head layout %d", c.head_layout);
  if (!(eps > 0.f)) return fail(BPD_E_FORMAT, "bad layer-norm eps");
  if (n_tensors < 1 || dir_off != 128 || dir_off + 96ull * n_tensors > n || data_off > n)
    return fail(BPD_E_FORMAT, "bad directory");
  for (int t = 0; t < n_tensors; ++t) {
    const unsigned char* e = p + dir_off + 96ull * t;
    char name[65];
    memcpy(name, e, 64);
    name[64] = 0;
    TensorEntry te;
    memcpy(&te.ndim, e + 64, 4);
    memcpy(te.dims, e + 68, 12);
    memcpy(&te.offset, e + 80, 8);
    memcpy(&te.nbytes, e + 88, 8);
    if (te.ndim < 1 || te.ndim > 3) return fail(BPD_E_FORMAT, "tensor %s: bad rank", name);
    uint64_t cnt = 1;
    for (int i = 0; i < te.ndim; ++i) {
      if (te.dims[i] < 1) return fail(BPD_E_FORMAT, "tensor %s: bad dimension", name);
      cnt *= (uint64_t)te.dims[i];
    }
    if (cnt * c.elem() != te.nbytes || te.offset % 256 || te.offset < data_off || te.offset + te.nbytes > n)
      return fail(BPD_E_FORMAT, "tensor %s: bad extent", name);
    out->t[name] = te;
  }
  out->total = total;
  return BPD_OK;
}

static int find(const ParsedBlob& pb, char* base, const std::string& name, std::initializer_list<int> shape,
                const void** out) {
  auto it = pb.t.find(name);
  if (it == pb.t.end()) return fail(BPD_E_FORMAT, "tensor %s missing", name.c_str());
  const TensorEntry& te = it->second;
  if (te.ndim != (int)shape.size()) return fail(BPD_E_FORMAT, "tensor %s: rank %d", name.c_str(), te.ndim);
  int i = 0;
  for (int s : shape)
    if (te.dims[i++] != s) return fail(BPD_E_FORMAT, "tensor %s: dimension %d is %d, want %d", name.c_str(), i - 1, te.dims[i - 1], s);
  *out = base + te.offset;
  return BPD_OK;
}

// ------------------------------------------------------------------ session planning
struct Arena {
  size_t off = 0;
  char* base = nullptr;
  template <typename T> T* take(size_t count) {
    off = align_up(off);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
  void* take_bytes(size_t n) { return take<char>(n); }
};

static int pages_per_row(const Config& c, int max_tgt) { return ceil_div(max_tgt + 1 + c.k_model, kPage); }

// Sessions whose widest pass has more than 64 rows plan their projections for full token tiles.
static int session_wide_ttiles(const Config& c, int B) {
  const int rmax = B * c.k_model;
  return rmax > 64 ? tc::token_tiles(rmax) : 0;
}

// Lays the session out; with base == nullptr only measures.
static size_t plan_session(const Config& c, int B, int max_src, int max_tgt, char* base, bpd_session* s) {
  Arena a;
  a.base = base;
  const size_t ea = sizeof(float);   // activations stay fp32 between kernels; only weights and the cache are narrow
  const size_t ec = c.elem();
  const size_t Rmax = (size_t)B * c.k_model, E = (size_t)B * max_src, Rall = std::max(Rmax, E);
  const size_t R2 = Rmax * c.k_model;
  const int ppr = pages_per_row(c, max_tgt);
  const size_t d = c.d;
  float* x = a.take<float>(Rall * d);
  float* h_f32 = a.take<float>(Rmax * d);
  void* xn = a.take_bytes(Rall * d * ea);
  void* qbuf = a.take_bytes(std::max(E * 3 * d, Rmax * d) * ea);
  void* attn = a.take_bytes(Rall * d * ea);
  void* ffh = a.take_bytes(Rall * c.d_ff * ea);
  void* u = a.take_bytes(Rmax * c.k_model * c.d_hidden * ea);
  void* o = a.take_bytes(R2 * d * ea);
  std::vector<void*> crosskv(c.n_dec), kc(c.n_dec), vc(c.n_dec);
  for (int l = 0; l < c.n_dec; ++l) crosskv[l] = a.take_bytes(E * 2 * d * ea);
  for (int l = 0; l < c.n_dec; ++l) {
    kc[l] = a.take_bytes((size_t)B * ppr * kPage * d * ec);
    vc[l] = a.take_bytes((size_t)B * ppr * kPage * d * ec);
  }
  const size_t npos = std::max<size_t>(max_src, (size_t)max_tgt + 1 + c.k_model);
  float* pe = a.take<float>(npos * d);
  int* page_table = a.take<int>((size_t)B * ppr);
  RowState st;
  st.len = a.take<int>(B); st.j = a.take<int>(B); st.finished = a.take<int>(B); st.src_len = a.take<int>(B);
  st.block = a.take<int>((size_t)B * kMaxK); st.cur_block = a.take<int>((size_t)B * kMaxK);
  st.khat = a.take<int>(B);
  st.table = a.take<int>((size_t)B * kMaxK * kMaxK);
  st.out_ids = a.take<int>((size_t)B * max_tgt);
  st.all_done = a.take<int>(1); st.error = a.take<int>(1);
  st.signal = a.take<int>(2); st.host_flags = nullptr;
  st.stats = a.take<long long>(4 + kMaxK + 1);
  st.page_table = page_table; st.pages_per_row = ppr; st.max_tgt = max_tgt;
  void* u2 = a.take_bytes((size_t)B * c.k_model * c.d_hidden * ea);
  float* h2 = a.take<float>((size_t)B * d);
  int* table2 = a.take<int>((size_t)B * kMaxK);
  int* table_full = a.take<int>((size_t)B * kMaxK * kMaxK);
  RankState rank;
  rank.thr = a.take<float>(Rmax); rank.tok = a.take<int>(Rmax); rank.cnt = a.take<int>(Rmax);
  int* src_dev = a.take<int>(E);
  int* tail_dev = a.take<int>((size_t)B * kMaxK);
  int* plan_dev = a.take<int>((size_t)B * max_tgt * (kMaxK - 1));
  const size_t tiles = std::max(ceil_div(c.V, kVocTile), ceil_div(c.V, tc::kBM));
  float* part_val = a.take<float>(tiles * R2);
  int* part_idx = a.take<int>(tiles * R2);
  unsigned* counters = a.take<unsigned>(ceil_div((int)R2, kRC) + 1);
  // split-K workspace of the tensor-core projections: the largest any launch of this session can need
  size_t ws = 0, ncnt = 1;
  if (c.dtype == 1) {
    const int wide = session_wide_ttiles(c, B);
    auto need = [&](int N, int K, size_t T, int z) {
      ws = std::max(ws, tc::ws_floats(N, K, (int)T, z, wide));
      ncnt = std::max(ncnt, tc::counters_needed(N, (int)T, z));
    };
    const int dd = c.d, ff = c.d_ff, fh = c.d_hidden, km = c.k_model;
    for (size_t T : {Rmax, E}) {
      need(3 * dd, dd, T, 1); need(dd, dd, T, 1); need(ff, dd, T, 1); need(dd, ff, T, 1); need(2 * dd, dd, T, 1);
    }
    for (int kh = 1; kh <= km; ++kh) {
      need(kh * fh, dd, Rmax, 1); need(km * fh, dd, Rmax, 1);
      need(kh * dd, km * fh, Rmax, 1);
      if (wide) ws = std::max(ws, tc::ws_floats(kh * dd, km * fh, B, 1, 1, tc::kSlots));   // stage 2 of the lazy heads
      need(dd, fh, Rmax, kh);
    }
    need(c.V, dd, R2, 1);
  }
  float* tc_ws = a.take<float>(ws);
  unsigned* tc_counters = a.take<unsigned>(ncnt);
  unsigned* tc_done = a.take<unsigned>(1);
  unsigned long long* tc_best = a.take<unsigned long long>(R2 * tc::kBestStride);
  // fused decoder layers (few rows per pass): per-head / per-cluster shares of the output projections, slice counters
  const bool fused_ok = c.dtype == 1 && fused::supported(c.d, c.H, c.d_ff, (int)Rmax);
  const size_t fused_parts = std::max<size_t>(c.H, c.d_ff / (fused::kC * fused::kHS));
  float* fused_ws = a.take<float>(fused_ok ? fused_parts * Rmax * d : 0);
  unsigned* fused_counters = a.take<unsigned>(fused::kC);
  // persistent layer stack: tensor maps, per-layer pointers, the clusters' partial outputs, the join's words
  void* stack_layers = a.take_bytes(fused_ok ? (size_t)c.n_dec * sizeof(stack::LayerPtrs) : 0);
  unsigned long long* stack_ws = a.take<unsigned long long>(fused_ok ? (size_t)2 * (c.H + 1) * fused::kMaxRows * d : 0);
  unsigned* stack_bar = a.take<unsigned>(stack::kBarWords);
  float* ln_stats = a.take<float>((size_t)ceil_div(d, 128) * Rall * 2);
  if (s) {
    s->ln_stats = ln_stats;
    s->stack_layers = stack_layers; s->stack_ws = stack_ws; s->stack_bar = stack_bar;
    s->fused_ws = fused_ws; s->fused_counters = fused_counters;
    s->x = x; s->h_f32 = h_f32; s->xn = xn; s->qbuf = qbuf; s->attn = attn; s->ffh = ffh; s->u = u; s->o = o;
    s->crosskv = crosskv; s->kcache = kc; s->vcache = vc; s->st = st; s->src_dev = src_dev;
    s->tail_dev = tail_dev; s->plan_dev = plan_dev; s->part_val = part_val; s->part_idx = part_idx;
    s->rank = rank;
    s->u2 = u2; s->pl_u2 = (long long)B * c.k_model * c.d_hidden; s->h2 = h2; s->table2 = table2; s->table_full = table_full;
    s->counters = counters; s->ppr = ppr; s->part_elems = tiles * R2; s->pe = pe; s->npos = (int)npos;
    s->tc_ws = tc_ws; s->tc_ws_floats = ws; s->tc_counters = tc_counters; s->tc_n_counters = ncnt; s->tc_done = tc_done; s->tc_best = tc_best; s->tc_best_elems = R2;
    s->pl_xn = (long long)(Rall * d); s->pl_attn = (long long)(Rall * d); s->pl_ffh = (long long)(Rall * c.d_ff);
    s->pl_u = (long long)(Rmax * c.k_model * c.d_hidden); s->pl_o = (long long)(R2 * d);
    s->rows_all = (int)Rall; s->rows_dec = (int)Rmax; s->rows_head = (int)R2;
  }
  return align_up(a.off);
}

static size_t fold_floats(const Config& c) { return c.dtype == 1 ? (size_t)c.n_dec * 2 * (3 * c.d + c.d + c.d_ff) : 0; }
static size_t weight_bytes_for(const ParsedBlob& pb) { return align_up(pb.total) + align_up(fold_floats(pb.cfg) * sizeof(float)); }

// ------------------------------------------------------------------ launches
std::atomic<long long> g_launches{0};
template <typename WT, typename AT, int EPI>
static void launch_linear(const LinearParams& p, int zcount, cudaStream_t st) {
  dim3 grid(ceil_div(p.N, kLinWarps * kFPW), ceil_div(p.rows, kRC), zcount);
  linear_kernel<WT, AT, EPI><<<grid, kLinWarps * 32, 0, st>>>(p);
  ++g_launches;
}

static LinearParams lin(const void* x, long long ldx, const void* w, int K, int N, const void* bias, int rows,
                        void* y, long long ldy, int relu, const int* all_done) {
  LinearParams p;
  memset(&p, 0, sizeof(p));
  p.x = x; p.ldx = ldx; p.w = w; p.ldw = K; p.bias = bias; p.rows = rows; p.K = K; p.N = N;
  p.relu = relu; p.y = y; p.ldy = ldy; p.all_done = all_done;
  return p;
}

template <typename WT, typename AT>
static void launch_ln(const float* x, const void* g, const void* b, void* y, float* y32, int rows, int d, float eps,
                      const int* all_done, cudaStream_t st, long long plane = 0, bool pdl = false) {
  LnParams p{x, g, b, y, plane, y32, rows, d, eps, all_done};
  launch_k(layernorm_kernel<WT, AT>, dim3(ceil_div(rows, 4)), dim3(128), 0, st, pdl, p);
  ++g_launches;
}

template <typename WT, typename AT>
static void launch_vocab_argmax(const void* x, const void* w, int rows, int d, int V, float* part_val, int* part_idx,
                                unsigned* counters, int* out_idx, float* out_val, float* logits, const int* all_done,
                                cudaStream_t st, const RankState* rank = nullptr, int rank_kh = 1) {
  ArgmaxParams p{x, (long long)d, w, rows, d, V, part_val, part_idx, counters, out_idx, out_val, logits, all_done};
  if (rank) { p.rank = *rank; p.rank_kh = rank_kh; }
  dim3 grid(ceil_div(V, kVocTile), ceil_div(rows, kRC));
  vocab_argmax_kernel<WT, AT><<<grid, kLinWarps * 32, (size_t)kRC * d * sizeof(float), st>>>(p);
  ++g_launches;
}

// Optional per-phase timing: pairs of events around a phase of the pass, on the session's stream.
static void prof_mark(bpd_session* s, int slot, int end) {
  if (!s->profiling) return;
  cudaEvent_t ev;
  if (cudaEventCreate(&ev) != cudaSuccess) return;
  cudaEventRecord(ev, s->stream);
  (end ? s->prof_end : s->prof_begin)[slot].push_back(ev);
}

static void prof_clear(bpd_session* s) {
  for (int i = 0; i < kProfSlots; ++i) {
    for (cudaEvent_t e : s->prof_begin[i]) cudaEventDestroy(e);
    for (cudaEvent_t e : s->prof_end[i]) cudaEventDestroy(e);
    s->prof_begin[i].clear();
    s->prof_end[i].clear();
  }
}

// ------------------------------------------------------------------ encoder
template <typename WT>
static int run_encoder(bpd_session* s) {
  const bpd_model* m = s->m;
  const Config& c = m->cfg;
  cudaStream_t st = s->stream;
  const int E = s->B * s->max_src, d = c.d;
  EmbedParams ep;
  memset(&ep, 0, sizeof(ep));
  ep.table = m->src_embed; ep.pe = s->pe; ep.npos = s->npos; ep.x = s->x; ep.rows = E; ep.rows_per_b = s->max_src;
  ep.d = d; ep.vocab = c.V; ep.st = s->st; ep.src = s->src_dev;
  embed_kernel<WT><<<E, 128, 0, st>>>(ep);
  ++g_launches;
  for (int l = 0; l < c.n_enc; ++l) {
    const EncLayer& L = m->enc[l];
    launch_ln<WT, float>(s->x, L.ln1g, L.ln1b, s->xn, nullptr, E, d, c.eps, nullptr, st);
    launch_linear<WT, float, kEpiStoreAct>(lin(s->xn, d, L.wqkv, d, 3 * d, nullptr, E, s->qbuf, 3 * d, 0, nullptr), 1, st);
    AttnParams ap;
    memset(&ap, 0, sizeof(ap));
    ap.q = s->qbuf; ap.ldq = 3 * d; ap.out = s->attn; ap.ldo = d; ap.rows = E; ap.rows_per_b = s->max_src;
    ap.H = c.H; ap.dh = d / c.H; ap.causal = 0; ap.limit_b = s->st.src_len;
    ap.k = static_cast<float*>(s->qbuf) + d; ap.v = static_cast<float*>(s->qbuf) + 2 * d;
    ap.ldkv = 3 * d; ap.bstride = (long long)s->max_src * 3 * d; ap.paged = 0; ap.st = s->st;
    ap.scale = 1.0f / sqrtf((float)ap.dh); ap.by_rows = (s->B >= 8) ? 1 : 0;
    launch_attention<float, float>(ap, st);
    ++g_launches;
    LinearParams po = lin(s->attn, d, L.wo, d, d, nullptr, E, s->x, d, 0, nullptr);
    launch_linear<WT, float, kEpiResidual>(po, 1, st);
    launch_ln<WT, float>(s->x, L.ln2g, L.ln2b, s->xn, nullptr, E, d, c.eps, nullptr, st);
    launch_linear<WT, float, kEpiStoreAct>(lin(s->xn, d, L.w1, d, c.d_ff, L.b1, E, s->ffh, c.d_ff, 1, nullptr), 1, st);
    launch_linear<WT, float, kEpiResidual>(lin(s->ffh, c.d_ff, L.w2, c.d_ff, d, L.b2, E, s->x, d, 0, nullptr), 1, st);
  }
  launch_ln<WT, float>(s->x, m->enc_lnf_g, m->enc_lnf_b, s->xn, nullptr, E, d, c.eps, nullptr, st);
  for (int l = 0; l < c.n_dec; ++l)
    launch_linear<WT, float, kEpiStoreAct>(lin(s->xn, d, m->dec[l].cwkv, d, 2 * d, nullptr, E, s->crosskv[l], 2 * d, 0, nullptr), 1, st);
  BPD_CUDA(cudaGetLastError());
  return BPD_OK;
}

// ------------------------------------------------------------------ one decoder pass + heads + top-1 + verify
struct PassArgs {
  int mode;          // PassMode
  int kcur;          // positions scored per row
  int kh;            // heads evaluated per position
  int knext;         // width of the block selected for the next pass
  const int* forced; // device, or null
  int forced_rows, kforced;
  int max_new, eos;
  float* logits_dump;   // device [B*kcur*kh, V] or null
  int accept_kind = kAcceptExact;   // Verify criterion, its parameter (n or eps), forced minimum block size
  int accept_param = 0;
  int min_block = 1;
  float* layer_dump = nullptr;   // device [n_dec, B*kcur, d] or null: the residual stream after every decoder layer
};

// accept_mode of the public calls: bits 0-7 parameter, bits 8-15 criterion, bits 16-23 minimum block size
static int decode_accept(int accept_mode, int k, PassArgs* a) {
  const int param = accept_mode & 0xff, kind = (accept_mode >> 8) & 0xff, minb = (accept_mode >> 16) & 0xff;
  if (accept_mode < 0 || (accept_mode >> 24)) return fail(BPD_E_INVALID, "acceptance mode 0x%x", accept_mode);
  if (kind == kAcceptExact) {
    if (param) return fail(BPD_E_INVALID, "exact acceptance takes no parameter");
  } else if (kind == kAcceptTopN) {
    if (param < 1) return fail(BPD_E_INVALID, "top-n acceptance needs n >= 1");
  } else if (kind != kAcceptDistance) {
    return fail(BPD_E_UNSUPPORTED, "acceptance criterion %d", kind);
  }
  if (minb > k) return fail(BPD_E_INVALID, "minimum block size %d above k = %d", minb, k);
  a->accept_kind = kind; a->accept_param = param; a->min_block = std::max(1, minb);
  return BPD_OK;
}

static VerifyParams verify_params(bpd_session* s, const PassArgs& a) {
  VerifyParams vp{s->st, s->B, a.kcur, a.kh, a.knext, a.mode, a.max_new, a.eos, a.accept_kind, a.accept_param, a.min_block, s->rank};
  return vp;
}
static bool pass_is_lazy(const bpd_session* s, const PassArgs& a) {
  return s->tc && s->lazy_heads && a.mode == kModeBlock && a.kcur > 1 && a.kh > 1 && !a.logits_dump;
}
static bool wants_rank(const PassArgs& a) { return a.mode == kModeBlock && a.accept_kind == kAcceptTopN && a.kcur > 1; }

template <typename WT>
static int run_pass(bpd_session* s, const PassArgs& a) {
  const bpd_model* m = s->m;
  const Config& c = m->cfg;
  cudaStream_t st = s->stream;
  const int d = c.d, R = s->B * a.kcur, R2 = R * a.kh;
  const int* done = s->st.all_done;
  EmbedParams ep;
  memset(&ep, 0, sizeof(ep));
  ep.table = m->tgt_embed; ep.pe = s->pe; ep.npos = s->npos; ep.x = s->x; ep.rows = R; ep.rows_per_b = a.kcur;
  ep.d = d; ep.vocab = c.V; ep.st = s->st; ep.forced = a.forced; ep.forced_rows = a.forced_rows;
  ep.kforced = a.kforced; ep.src = nullptr; ep.all_done = done;
  prof_mark(s, kProfLayers, 0);
  embed_kernel<WT><<<R, 128, 0, st>>>(ep);
  ++g_launches;
  for (int l = 0; l < c.n_dec; ++l) {
    const DecLayer& L = m->dec[l];
    // self-attention over the cache plus the causal part of the block
    launch_ln<WT, float>(s->x, L.ln1g, L.ln1b, s->xn, nullptr, R, d, c.eps, done, st);
    LinearParams pq = lin(s->xn, d, L.wqkv, d, 3 * d, nullptr, R, s->qbuf, d, 0, done);
    pq.d = d; pq.kcache = s->kcache[l]; pq.vcache = s->vcache[l]; pq.st = s->st; pq.rows_per_b = a.kcur;
    launch_linear<WT, float, kEpiQkv>(pq, 1, st);
    AttnParams ap;
    memset(&ap, 0, sizeof(ap));
    ap.q = s->qbuf; ap.ldq = d; ap.out = s->attn; ap.ldo = d; ap.rows = R; ap.rows_per_b = a.kcur;
    ap.H = c.H; ap.dh = d / c.H; ap.causal = 1; ap.local_q = c.local_q; ap.local_m = c.local_m;
    ap.k = s->kcache[l]; ap.v = s->vcache[l]; ap.ldkv = d;
    ap.paged = 1; ap.st = s->st; ap.scale = 1.0f / sqrtf((float)ap.dh); ap.by_rows = (s->B >= 8) ? 1 : 0; ap.all_done = done;
    launch_attention<float, WT>(ap, st);
    ++g_launches;
    launch_linear<WT, float, kEpiResidual>(lin(s->attn, d, L.wo, d, d, nullptr, R, s->x, d, 0, done), 1, st);
    // cross-attention over the encoder memory
    launch_ln<WT, float>(s->x, L.ln2g, L.ln2b, s->xn, nullptr, R, d, c.eps, done, st);
    launch_linear<WT, float, kEpiStoreAct>(lin(s->xn, d, L.cwq, d, d, nullptr, R, s->qbuf, d, 0, done), 1, st);
    ap.causal = 0; ap.limit_b = s->st.src_len; ap.k = s->crosskv[l]; ap.v = static_cast<float*>(s->crosskv[l]) + d;
    ap.ldkv = 2 * d; ap.bstride = (long long)s->max_src * 2 * d; ap.paged = 0;
    launch_attention<float, float>(ap, st);
    ++g_launches;
    launch_linear<WT, float, kEpiResidual>(lin(s->attn, d, L.cwo, d, d, nullptr, R, s->x, d, 0, done), 1, st);
    // feed-forward
    launch_ln<WT, float>(s->x, L.ln3g, L.ln3b, s->xn, nullptr, R, d, c.eps, done, st);
    launch_linear<WT, float, kEpiStoreAct>(lin(s->xn, d, L.w1, d, c.d_ff, L.b1, R, s->ffh, c.d_ff, 1, done), 1, st);
    launch_linear<WT, float, kEpiResidual>(lin(s->ffh, c.d_ff, L.w2, c.d_ff, d, L.b2, R, s->x, d, 0, done), 1, st);
    if (a.layer_dump)
      BPD_CUDA(cudaMemcpyAsync(a.layer_dump + (size_t)l * R * d, s->x, sizeof(float) * R * d, cudaMemcpyDeviceToDevice, st));
  }
  launch_ln<WT, float>(s->x, m->dec_lnf_g, m->dec_lnf_b, s->xn, s->h_f32, R, d, c.eps, done, st);
  prof_mark(s, kProfLayers, 1);
  // proposal heads: hidden layer, k output layers with a residual from the decoder output
  const int fh = c.d_hidden;
  const long long ldu = (long long)c.k_model * fh;
  const int hid = (c.head_layout == 0) ? c.k_model * fh : a.kh * fh;
  prof_mark(s, kProfHeadW1, 0);
  launch_linear<WT, float, kEpiStoreAct>(lin(s->xn, d, m->head_w1, d, hid, m->head_b1, R, s->u, ldu, 1, done), 1, st);
  prof_mark(s, kProfHeadW1, 1);
  prof_mark(s, kProfHeadW2, 0);
  if (c.head_layout == 0) {
    LinearParams ph = lin(s->u, ldu, m->head_w2, c.k_model * fh, a.kh * d, m->head_b2, R, s->o, (long long)a.kh * d, 0, done);
    ph.h = s->h_f32; ph.d = d; ph.head_identity = c.p1_identity;
    launch_linear<WT, float, kEpiHeadOut>(ph, 1, st);
  } else {
    LinearParams ph = lin(s->u, ldu, m->head_w2, fh, d, m->head_b2, R, s->o, (long long)a.kh * d, 0, done);
    ph.xz = fh; ph.wz = (long long)d * fh; ph.bz = d; ph.yz = d;
    ph.h = s->h_f32; ph.d = d; ph.head_identity = c.p1_identity;
    launch_linear<WT, float, kEpiHeadOut>(ph, a.kh, st);
  }
  prof_mark(s, kProfHeadW2, 1);
  // shared vocabulary projection with a fused top-1: table[b][r][i]
  prof_mark(s, kProfVocab, 0);
  if (wants_rank(a)) {
    ProposalLogitParams pl{s->o, 0, m->out_proj, s->st, s->rank, s->B, a.kcur, a.kh, d, done};
    proposal_logit_kernel<WT><<<ceil_div(R, 4), 128, 0, st>>>(pl);
    ++g_launches;
  }
  launch_vocab_argmax<WT, float>(s->o, m->out_proj, R2, d, c.V, s->part_val, s->part_idx, s->counters, s->st.table,
                              nullptr, a.logits_dump, done, st, wants_rank(a) ? &s->rank : nullptr, a.kh);
  prof_mark(s, kProfVocab, 1);
  VerifyParams vp = verify_params(s, a);
  verify_commit_kernel<<<1, 32 * ceil_div(s->B, 32), 0, st>>>(vp);
  ++g_launches;
  BPD_CUDA(cudaGetLastError());
  s->invocations += 1;
  return BPD_OK;
}

// ------------------------------------------------------------------ tensor-core path (bf16 models)
static tc::Scratch tc_scratch(bpd_session* s) {
  tc::Scratch sc;
  sc.ws = s->tc_ws; sc.ws_floats = s->tc_ws_floats; sc.tile_counters = s->tc_counters; sc.n_counters = s->tc_n_counters;
  sc.done_counter = s->tc_done; sc.best = s->tc_best; sc.best_elems = s->tc_best_elems;
  sc.error = s->st.error;
  sc.wide_ttiles = session_wide_ttiles(s->m->cfg, s->B);
  sc.l2_hints = s->opt.l2_stream_hints;
  return sc;
}

static tc::TcParams tc_params(const void* bias, int relu, const int* all_done) {
  tc::TcParams p;
  memset(&p, 0, sizeof(p));
  p.bias = static_cast<const bf16*>(bias); p.relu = relu; p.all_done = all_done;
  return p;
}

#define BPD_TRY(expr) do { int rc__ = (expr); if (rc__) return rc__; } while (0)

// The opt-in shared-memory limit of the staged attention kernel grows with the longest source seen so far.
static int cross_staged_attr(size_t smem) {
  return ensure_smem_limit(reinterpret_cast<const void*>(cross_attention_staged_kernel<float>), smem);
}

static int run_encoder_tc(bpd_session* s) {
  const bpd_model* m = s->m;
  const Config& c = m->cfg;
  cudaStream_t st = s->stream;
  const int E = s->B * s->max_src, d = c.d, f = c.d_ff;
  const tc::Scratch sc = tc_scratch(s);
  const bool pdl = s->use_pdl != 0;   // every kernel after the first may start while its predecessor ends
  EmbedParams ep;
  memset(&ep, 0, sizeof(ep));
  ep.table = m->src_embed; ep.pe = s->pe; ep.npos = s->npos; ep.x = s->x; ep.rows = E; ep.rows_per_b = s->max_src;
  ep.d = d; ep.vocab = c.V; ep.st = s->st; ep.src = s->src_dev;
  embed_kernel<bf16><<<E, 128, 0, st>>>(ep);
  ++g_launches;
  const tc::Operands xn{nullptr, 0, s->xn, s->pl_xn, d, s->rows_all, d};
  const tc::Operands at{nullptr, 0, s->attn, s->pl_attn, d, s->rows_all, d};
  const tc::Operands fh{nullptr, 0, s->ffh, s->pl_ffh, f, s->rows_all, f};
  auto with_w = [](tc::Operands o, const void* w, int rows) { o.w = w; o.w_rows = rows; return o; };
  for (int l = 0; l < c.n_enc; ++l) {
    const EncLayer& L = m->enc[l];
    launch_ln<bf16, float>(s->x, L.ln1g, L.ln1b, s->xn, nullptr, E, d, c.eps, nullptr, st, s->pl_xn, pdl);
    tc::TcParams pq = tc_params(nullptr, 0, nullptr);
    pq.out_f32 = static_cast<float*>(s->qbuf); pq.ldo = 3 * d;
    BPD_TRY(tc::launch<tc::kTcF32>(with_w(xn, L.wqkv, 3 * d), 3 * d, d, E, pq, sc, st, 1, 0, 0, pdl)); ++g_launches;
    AttnParams ap;
    memset(&ap, 0, sizeof(ap));
    ap.q = s->qbuf; ap.ldq = 3 * d; ap.out = s->attn; ap.ldo = d; ap.out_plane = s->pl_attn; ap.rows = E;
    ap.rows_per_b = s->max_src; ap.H = c.H; ap.dh = d / c.H; ap.causal = 0; ap.limit_b = s->st.src_len;
    ap.k = static_cast<float*>(s->qbuf) + d; ap.v = static_cast<float*>(s->qbuf) + 2 * d;
    ap.ldkv = 3 * d; ap.bstride = (long long)s->max_src * 3 * d; ap.paged = 0; ap.st = s->st;
    ap.scale = 1.0f / sqrtf((float)ap.dh); ap.by_rows = (s->B >= 8) ? 1 : 0;
    // many sequences, head width 64: a CTA per (sequence, head) with the sequence's keys and values in shared memory
    if (ap.by_rows && ap.dh == 64 && cross_staged_smem(s->max_src) <= 160 * 1024 && s->opt.stage_encoder_rows) {
      const size_t smem = cross_staged_smem(s->max_src);
      BPD_TRY(cross_staged_attr(smem));
      BPD_CUDA(launch_k(cross_attention_staged_kernel<float>, dim3(s->B * c.H), dim3(kAttnWarps * 32), smem, st, pdl, ap, s->max_src, 0));
    } else {
      launch_attention<float, float>(ap, st, pdl);
    }
    ++g_launches;
    tc::TcParams po = tc_params(nullptr, 0, nullptr);
    po.out_f32 = s->x; po.ldo = d;
    BPD_TRY(tc::launch<tc::kTcResidual>(with_w(at, L.wo, d), d, d, E, po, sc, st, 1, 0, 0, pdl)); ++g_launches;
    launch_ln<bf16, float>(s->x, L.ln2g, L.ln2b, s->xn, nullptr, E, d, c.eps, nullptr, st, s->pl_xn, pdl);
    tc::TcParams p1 = tc_params(L.b1, 1, nullptr);
    p1.out_hi = static_cast<bf16*>(s->ffh); p1.plane = s->pl_ffh; p1.ldo = f;
    BPD_TRY(tc::launch<tc::kTcPlanes>(with_w(xn, L.w1, f), f, d, E, p1, sc, st, 1, 0, 0, pdl)); ++g_launches;
    tc::TcParams p2 = tc_params(L.b2, 0, nullptr);
    p2.out_f32 = s->x; p2.ldo = d;
    BPD_TRY(tc::launch<tc::kTcResidual>(with_w(fh, L.w2, d), d, f, E, p2, sc, st, 1, 0, 0, pdl)); ++g_launches;
  }
  launch_ln<bf16, float>(s->x, m->enc_lnf_g, m->enc_lnf_b, s->xn, nullptr, E, d, c.eps, nullptr, st, s->pl_xn, pdl);
  for (int l = 0; l < c.n_dec; ++l) {
    tc::TcParams pk = tc_params(nullptr, 0, nullptr);
    pk.out_f32 = static_cast<float*>(s->crosskv[l]); pk.ldo = 2 * d;
    BPD_TRY(tc::launch<tc::kTcF32>(with_w(xn, m->dec[l].cwkv, 2 * d), 2 * d, d, E, pk, sc, st, 1, 0, 0, pdl)); ++g_launches;
  }
  BPD_CUDA(cudaGetLastError());
  return BPD_OK;
}

// ------------------------------------------------------------------ fused decoder layers (few rows per pass)
template <typename P>
static int fused_attr(void (*kernel)(P), size_t smem) {
  return ensure_smem_limit(reinterpret_cast<const void*>(kernel), smem);
}

// Embedding, then three launches per decoder layer (self-attention block, cross-attention block, feed-forward
// block); leaves the residual stream in s->x like the kernel-per-projection path.
static int run_layers_fused(bpd_session* s, const PassArgs& a) {
  const bpd_model* m = s->m;
  const Config& c = m->cfg;
  cudaStream_t st = s->stream;
  const int d = c.d, R = s->B * a.kcur;
  const int* done = s->st.all_done;
  const bool pdl = s->use_pdl != 0;
  const int nt = (R + 7) / 8;
  // encoder keys / values of a head are staged in shared memory when all sequences' rows fit a small budget
  // (24 KB keep the three kernels of a big model co-resident on an SM; a model whose attention launches leave half
  // the SMs free may take up to 160 KB for it)
  const size_t cross_bytes = (size_t)s->B * s->max_src * fused::kCrossRowBytes;
  const bool cross_fits = cross_bytes <= (size_t)fused::kCrossStageMax ||
                          (c.H * fused::kC <= 74 && cross_bytes + fused::attn_layout<false>(d, nt, 0, 0).total <= 160 * 1024);
  const int cross_smax = (cross_fits && s->opt.stage_encoder_rows) ? s->max_src : 0;
  const size_t smem_self = fused::attn_layout<true>(d, nt, s->B * s->ppr).total;
  const size_t smem_cross = fused::attn_layout<false>(d, nt, 0, s->B * cross_smax).total;
  const size_t smem_ffn = fused::ffn_layout(d, nt).total;
  // the opt-in shared-memory limit of each kernel grows with the widest model seen so far
  {
    BPD_TRY(fused_attr(fused::attn_block_kernel<true, 1, 1>, smem_self));
    BPD_TRY(fused_attr(fused::attn_block_kernel<true, 2, 1>, smem_self));
    BPD_TRY(fused_attr(fused::attn_block_kernel<true, 1, 2>, smem_self));
    BPD_TRY(fused_attr(fused::attn_block_kernel<true, 2, 2>, smem_self));
    BPD_TRY(fused_attr(fused::attn_block_kernel<true, 1, 2, 1>, smem_self));
    BPD_TRY(fused_attr(fused::attn_block_kernel<true, 2, 2, 1>, smem_self));
    BPD_TRY(fused_attr(fused::attn_block_kernel<false, 1, 1>, smem_cross));
    BPD_TRY(fused_attr(fused::attn_block_kernel<false, 2, 1>, smem_cross));
    if (nt == 1) {
      BPD_TRY(fused_attr(fused::attn_block_kernel<false, 1>, smem_cross));
      BPD_TRY(fused_attr(fused::ffn_block_kernel<1>, smem_ffn));
      BPD_TRY(fused_attr(fused::ffn_block_kernel<1, 2>, smem_ffn));
    } else {
      BPD_TRY(fused_attr(fused::attn_block_kernel<false, 2>, smem_cross));
      BPD_TRY(fused_attr(fused::ffn_block_kernel<2>, smem_ffn));
      BPD_TRY(fused_attr(fused::ffn_block_kernel<2, 2>, smem_ffn));
    }
  }
  EmbedParams ep;
  memset(&ep, 0, sizeof(ep));
  ep.table = m->tgt_embed; ep.pe = s->pe; ep.npos = s->npos; ep.x = s->x; ep.rows = R; ep.rows_per_b = a.kcur;
  ep.d = d; ep.vocab = c.V; ep.st = s->st; ep.forced = a.forced; ep.forced_rows = a.forced_rows;
  ep.kforced = a.kforced; ep.src = nullptr; ep.all_done = done;
  embed_kernel<bf16><<<R, 128, 0, st>>>(ep);
  ++g_launches;
  const dim3 block(fused::kThreads), grid_attn(fused::kC, c.H), grid_ffn(fused::kC, c.d_ff / (fused::kC * fused::kHS));
  for (int l = 0; l < c.n_dec; ++l) {
    const DecLayer& L = m->dec[l];
    fused::AttnBlockParams ps;
    memset(&ps, 0, sizeof(ps));
    ps.x = s->x; ps.gain = static_cast<const bf16*>(L.ln1g); ps.fold_s = L.s_qkv; ps.fold_c = L.c_qkv;
    ps.w_in = static_cast<const bf16*>(L.wqkv); ps.w_out = static_cast<const bf16*>(L.wo);
    ps.d = d; ps.H = c.H; ps.R = R; ps.rows_per_b = a.kcur; ps.eps = c.eps;
    ps.kcache = static_cast<bf16*>(s->kcache[l]); ps.vcache = static_cast<bf16*>(s->vcache[l]);
    ps.attn.rows = R; ps.attn.rows_per_b = a.kcur; ps.attn.H = c.H; ps.attn.dh = fused::kDH; ps.attn.causal = 1;
    ps.attn.local_q = c.local_q; ps.attn.local_m = c.local_m;
    ps.attn.k = s->kcache[l]; ps.attn.v = s->vcache[l]; ps.attn.ldkv = d; ps.attn.paged = 1; ps.attn.st = s->st;
    ps.attn.scale = 1.0f / sqrtf((float)fused::kDH);
    ps.ws = s->fused_ws; ps.counters = s->fused_counters; ps.all_done = done;
    fused::AttnBlockParams pc = ps;
    pc.gain = static_cast<const bf16*>(L.ln2g); pc.fold_s = L.s_cq; pc.fold_c = L.c_cq;
    pc.w_in = static_cast<const bf16*>(L.cwq); pc.w_out = static_cast<const bf16*>(L.cwo);
    pc.kcache = nullptr; pc.vcache = nullptr; pc.cross_smax = cross_smax;
    pc.attn.causal = 0; pc.attn.limit_b = s->st.src_len; pc.attn.k = s->crosskv[l];
    pc.attn.v = static_cast<float*>(s->crosskv[l]) + d; pc.attn.ldkv = 2 * d;
    pc.attn.bstride = (long long)s->max_src * 2 * d; pc.attn.paged = 0;
    fused::FfnBlockParams pf;
    memset(&pf, 0, sizeof(pf));
    pf.x = s->x; pf.gain = static_cast<const bf16*>(L.ln3g); pf.fold_s = L.s_f1; pf.fold_c = L.c_f1;
    pf.w1 = static_cast<const bf16*>(L.w1); pf.w2 = static_cast<const bf16*>(L.w2); pf.b2 = static_cast<const bf16*>(L.b2);
    pf.d = d; pf.ff = c.d_ff; pf.R = R; pf.NJ = (int)grid_ffn.y; pf.eps = c.eps;
    pf.ws = s->fused_ws; pf.counters = s->fused_counters; pf.all_done = done;
    // every position the cache can hold (max_tgt + k + 1 of them) within kC chunks of 32: the short schedule only
    const bool short_only = s->max_tgt + c.k_model + 1 <= fused::kC * 32;
    const bool roomy = c.H * fused::kC <= 74;      // an attention launch leaves half the SMs free
    const bool ffn_small = grid_ffn.x * grid_ffn.y <= 148;   // one CTA per SM is enough for the feed-forward launch
    if (nt == 1) {
      if (short_only) BPD_CUDA(launch_k(fused::attn_block_kernel<true, 1, 1>, grid_attn, block, smem_self, st, pdl, ps));
      else if (roomy) BPD_CUDA(launch_k(fused::attn_block_kernel<true, 1, 2, 1>, grid_attn, block, smem_self, st, pdl, ps));
      else BPD_CUDA(launch_k(fused::attn_block_kernel<true, 1, 2>, grid_attn, block, smem_self, st, pdl, ps));
      if (cross_smax > 0) BPD_CUDA(launch_k(fused::attn_block_kernel<false, 1, 1>, grid_attn, block, smem_cross, st, pdl, pc));
      else
      BPD_CUDA(launch_k(fused::attn_block_kernel<false, 1>, grid_attn, block, smem_cross, st, pdl, pc));
      if (ffn_small) BPD_CUDA(launch_k(fused::ffn_block_kernel<1, 2>, grid_ffn, block, smem_ffn, st, pdl, pf));
      else BPD_CUDA(launch_k(fused::ffn_block_kernel<1>, grid_ffn, block, smem_ffn, st, pdl, pf));
    } else {
      if (short_only) BPD_CUDA(launch_k(fused::attn_block_kernel<true, 2, 1>, grid_attn, block, smem_self, st, pdl, ps));
      else if (roomy) BPD_CUDA(launch_k(fused::attn_block_kernel<true, 2, 2, 1>, grid_attn, block, smem_self, st, pdl, ps));
      else BPD_CUDA(launch_k(fused::attn_block_kernel<true, 2, 2>, grid_attn, block, smem_self, st, pdl, ps));
      if (cross_smax > 0) BPD_CUDA(launch_k(fused::attn_block_kernel<false, 2, 1>, grid_attn, block, smem_cross, st, pdl, pc));
      else
      BPD_CUDA(launch_k(fused::attn_block_kernel<false, 2>, grid_attn, block, smem_cross, st, pdl, pc));
      if (ffn_small) BPD_CUDA(launch_k(fused::ffn_block_kernel<2, 2>, grid_ffn, block, smem_ffn, st, pdl, pf));
      else BPD_CUDA(launch_k(fused::ffn_block_kernel<2>, grid_ffn, block, smem_ffn, st, pdl, pf));
    }
    g_launches += 3;
    if (a.layer_dump)
      BPD_CUDA(cudaMemcpyAsync(a.layer_dump + (size_t)l * R * d, s->x, sizeof(float) * R * d, cudaMemcpyDeviceToDevice, st));
  }
  return BPD_OK;
}

// ------------------------------------------------------------------ persistent layer stack (few rows per pass)
// Shared-memory plan of the persistent kernel for a session whose widest pass has `rows` rows; `budget` bytes per
// CTA.  Returns false when the working buffers and a ring that holds at least the two largest tiles do not fit.
static bool stack_plan(const Config& c, int rows, int nb, int ppr, int cross_rows, bool long_seq, size_t budget,
                       stack::Layout* out) {
  const int NT = rows > 8 ? 2 : 1, RP = NT * 8;
  const stack::Geo g = stack::make_geo(c.d, c.H, c.d_ff, c.n_dec, cross_rows);
  auto up = [](size_t v, size_t a) { return (v + a - 1) / a * a; };
  size_t off = 0;
  stack::Layout L;
  memset(&L, 0, sizeof(L));
  auto take = [&](size_t bytes) { const size_t at = off; off = up(off + bytes, 128); return (int)at; };
  L.x = take((size_t)RP * g.ks * 4);
  L.xh = take((size_t)RP * g.ks * 2);
  L.xl = take((size_t)RP * g.ks * 2);
  L.oh = take((size_t)RP * 128);
  L.ol = take((size_t)RP * 128);
  L.hid = take((size_t)fused::kC * 2 * RP * g.UPR * 2);
  const size_t chunk = std::max((size_t)NT * 3 * fused::kDH * 4, (size_t)g.UPR * RP * 4);
  L.outbox = take(fused::kC * chunk);
  L.inbox = take(fused::kC * chunk);
  L.kvq = take((size_t)RP * 512);
  L.stats = take((size_t)fused::kC * fused::kMaxRows * 2 * 4 + 4 * fused::kMaxRows * 4);
  L.attn = take(sizeof(AttnSmem<fused::kDH, stack::kWarps>));
  L.wst = take((size_t)stack::kWarps * NT * stack::kState * 4);
  const size_t lvl = long_seq ? (size_t)fused::kC * rows * stack::kState * 4 : 0;
  L.lvl1 = take(lvl);
  L.lvl2 = take(lvl);
  L.pt = take((size_t)nb * ppr * 4);
  L.layers = take((size_t)c.n_dec * sizeof(stack::LayerPtrs));
  L.misc = take(sizeof(stack::Ctl));
  const size_t work = off;
  int largest = 0, second = 0, per_layer = 0;
  if (g.ntl > stack::kMaxTiles) return false;
  for (int i = 0; i < g.ntl; ++i) {
    const int b = stack::make_tile(g, i, cross_rows, c.d, 0, 0).bytes;
    per_layer += b;
    if (b > largest) { second = largest; largest = b; } else if (b > second) second = b;
  }
  if (work + 1024 > budget) return false;
  size_t ring = std::min((budget - work) / 1024 * 1024, (size_t)per_layer * c.n_dec);
  if (ring < (size_t)largest + second) return false;
  L.ring_bytes = (int)ring;
  int* fields[] = {&L.x, &L.xh, &L.xl, &L.oh, &L.ol, &L.hid, &L.outbox, &L.inbox, &L.kvq, &L.stats, &L.attn, &L.wst, &L.lvl1,
                   &L.lvl2, &L.pt, &L.layers, &L.misc};
  for (int* f : fields) *f += (int)ring;
  L.total = (int)(ring + work);
  *out = L;
  return true;
}

// The persistent kernel's instantiations: token tiles (1 or 2 of 8 rows), reduction steps per panel (2: d_model 256,
// else 4), CTAs per SM (1 or 2), lean (short sequences and staged encoder rows only).  `f` gets the kernel.
template <typename F>
static int stack_variant(int nt, int ksteps, int minb, bool lean, F&& f) {
#define BPD_V(NT, KS, MB, LN) if (nt == NT && ksteps == KS && minb == MB && lean == LN) return f(stack::layer_stack_kernel<NT, KS, MB, LN>)
  BPD_V(1, 2, 1, false); BPD_V(2, 2, 1, false); BPD_V(1, 4, 1, false); BPD_V(2, 4, 1, false);
  BPD_V(1, 2, 2, false); BPD_V(2, 2, 2, false); BPD_V(1, 4, 2, false); BPD_V(2, 4, 2, false);
  BPD_V(1, 2, 1, true); BPD_V(2, 2, 1, true); BPD_V(1, 4, 1, true); BPD_V(2, 4, 1, true);
  BPD_V(1, 2, 2, true); BPD_V(2, 2, 2, true); BPD_V(1, 4, 2, true); BPD_V(2, 4, 2, true);
#undef BPD_V
  return fail(BPD_E_UNSUPPORTED, "no persistent layer kernel for %d token tiles, %d steps, %d CTAs per SM", nt, ksteps, minb);
}

template <typename K>
static int stack_clusters(K kernel, size_t smem, int H, int* out) {
  BPD_TRY(ensure_smem_limit(reinterpret_cast<const void*>(kernel), smem));
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(fused::kC, H); cfg.blockDim = dim3(stack::kThreads); cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = fused::kC; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  BPD_CUDA(cudaOccupancyMaxActiveClusters(out, kernel, &cfg));
  return BPD_OK;
}

// Shapes the persistent kernel is built for.
static bool stack_shapes_ok(const Config& c, int rows) {
  const int d = c.d, H = c.H;
  if (c.dtype != 1 || H < 1 || d != H * fused::kDH || (d != 256 && d != 512 && d != 1024)) return false;
  if (c.d_ff % H || (c.d_ff / H != 128 && c.d_ff / H != 256)) return false;   // hidden units per cluster
  if (rows < 1 || rows > fused::kMaxRows || c.n_dec > 64) return false;
  return true;
}

// Live sessions per device whose decoder layers run in the persistent kernel.  Two such kernels on one GPU at the
// same time can starve each other of SMs (each waits for clusters the other keeps from being scheduled) until their
// bounded waits expire, so the library's own choice gives the persistent kernel to one session per device at a time;
// a session that asks for it explicitly (persistent_layers = 1) gets it regardless.
static std::mutex g_stack_mu;
static std::map<int, int> g_stack_live;
static int stack_live(int dev, int delta) {
  std::lock_guard<std::mutex> lock(g_stack_mu);
  int& n = g_stack_live[dev];
  n += delta;
  return n;
}

// Decides whether the session runs its decoder layers in the persistent kernel and prepares what it needs:
// a shared-memory plan under which all H clusters are resident at once, tensor maps and per-layer pointers.
static int stack_setup(bpd_session* s) {
  const bpd_model* m = s->m;
  const Config& c = m->cfg;
  s->stack = 0;
  const int rows = s->B * c.k_model;
  if (!s->tc || !s->opt.persistent_layers || !stack_shapes_ok(c, rows)) return BPD_OK;
  const bool long_seq = s->max_tgt + 1 + c.k_model > 32 * fused::kC;
  const bool only_lean = s->opt.persistent_layers < 0;   // the library's own choice: sessions the lean kernel takes
  if (only_lean && (long_seq || !s->opt.stage_encoder_rows || s->B * s->max_src > 256)) return BPD_OK;
  cudaDeviceProp prop;
  int dev = 0;
  BPD_CUDA(cudaGetDevice(&dev));
  if (only_lean && stack_live(dev, 0) > 0) return BPD_OK;   // another session of this device has it: see stack_live
  BPD_CUDA(cudaGetDeviceProperties(&prop, dev));
  const size_t optin = prop.sharedMemPerBlockOptin, per_sm = prop.sharedMemPerMultiprocessor;
  // one CTA per SM, or two (each block also reserves 1 KB of the SM's shared memory)
  const size_t budgets[2] = {optin, std::min(optin, per_sm / 2 - 1024)};
  stack::Layout lay;
  bool ok = false;
  int cross_rows = 0;
  int minb = 0;
  for (size_t budget : budgets) {
    ++minb;                                    // first one CTA per SM, then two
    for (int staged = s->opt.stage_encoder_rows ? 1 : 0; staged >= (only_lean ? 1 : 0) && !ok; --staged) {
      cross_rows = (staged && s->B * s->max_src <= 256) ? s->B * s->max_src : 0;
      if (staged && !cross_rows) continue;
      if (budget <= 1024 || !stack_plan(c, rows, s->B, s->ppr, cross_rows, long_seq, budget - 1024, &lay)) continue;
      lay.total += 1024;                       // slack for aligning the ring to 1024 bytes
      int n1 = 0, n2 = 0;
      const size_t sm = (size_t)lay.total;
      const bool lean = !long_seq && cross_rows > 0;
      const int ksteps = c.d == 256 ? 2 : 4, H = c.H;
      BPD_TRY(stack_variant(1, ksteps, minb, lean, [&](auto kernel) { return stack_clusters(kernel, sm, H, &n1); }));
      BPD_TRY(stack_variant(2, ksteps, minb, lean, [&](auto kernel) { return stack_clusters(kernel, sm, H, &n2); }));
      ok = n1 >= c.H && n2 >= c.H;
    }
    if (ok) break;
  }
  if (!ok) return BPD_OK;
  // tensor maps over all layers at once: weight slices as boxes of 64 (32 for d_model 256) reduction columns,
  // encoder keys / values.  The layers' tensors must lie at a constant stride (they do in a blob written tensor
  // by tensor, layer after layer; the session's encoder keys / values are laid out the same way).
  const stack::Geo g = stack::make_geo(c.d, c.H, c.d_ff, c.n_dec, cross_rows);
  std::vector<stack::LayerPtrs> lp(c.n_dec);
  const int d = c.d, f = c.d_ff, nl = c.n_dec;
  auto stride_of = [&](auto get, long long* out) {
    *out = nl > 1 ? (const char*)get(1) - (const char*)get(0) : 0;
    for (int l = 1; l + 1 < nl; ++l)
      if ((const char*)get(l + 1) - (const char*)get(l) != *out) return false;
    return *out >= 0;
  };
  long long st_qkv, st_wo, st_cq, st_cwo, st_w1, st_w2, st_ckv;
  const bool regular = stride_of([&](int l) { return m->dec[l].wqkv; }, &st_qkv) && stride_of([&](int l) { return m->dec[l].wo; }, &st_wo) &&
                       stride_of([&](int l) { return m->dec[l].cwq; }, &st_cq) && stride_of([&](int l) { return m->dec[l].cwo; }, &st_cwo) &&
                       stride_of([&](int l) { return m->dec[l].w1; }, &st_w1) && stride_of([&](int l) { return m->dec[l].w2; }, &st_w2) &&
                       stride_of([&](int l) { return (const void*)s->crosskv[l]; }, &st_ckv);
  if (!regular) return BPD_OK;
  stack::StackMaps maps;
  memset(&maps, 0, sizeof(maps));
  {
    const DecLayer& L0 = m->dec[0];
    const int er = std::max(cross_rows, 1);
    BPD_TRY(tc::make_map_3d(L0.wqkv, 2, nl, st_qkv, 3 * d, d, d, g.PW, 64, true, &maps.m[stack::kMapQkv]));
    BPD_TRY(tc::make_map_3d(L0.wo, 2, nl, st_wo, d, d, d, 64, g.ks, true, &maps.m[stack::kMapWo]));
    BPD_TRY(tc::make_map_3d(L0.cwq, 2, nl, st_cq, d, d, d, g.PW, 64, true, &maps.m[stack::kMapCq]));
    BPD_TRY(tc::make_map_3d(L0.cwo, 2, nl, st_cwo, d, d, d, 64, g.ks, true, &maps.m[stack::kMapCwo]));
    BPD_TRY(tc::make_map_3d(L0.w1, 2, nl, st_w1, f, d, d, g.PW, g.HCt, true, &maps.m[stack::kMapW1]));
    BPD_TRY(tc::make_map_3d(L0.w2, 2, nl, st_w2, d, f, f, 64, g.ks, true, &maps.m[stack::kMapW2]));
    BPD_TRY(tc::make_map_3d(s->crosskv[0], 4, nl, st_ckv, (uint64_t)s->B * s->max_src, 2 * d, 2 * d, 32, er, true, &maps.m[stack::kMapCk]));
    BPD_TRY(tc::make_map_3d(s->crosskv[0], 4, nl, st_ckv, (uint64_t)s->B * s->max_src, 2 * d, 2 * d, 64, er, false, &maps.m[stack::kMapCv]));
  }
  for (int l = 0; l < nl; ++l) {
    const DecLayer& L = m->dec[l];
    stack::LayerPtrs& P = lp[l];
    P.g1 = static_cast<const bf16*>(L.ln1g); P.g2 = static_cast<const bf16*>(L.ln2g); P.g3 = static_cast<const bf16*>(L.ln3g);
    P.s_qkv = L.s_qkv; P.c_qkv = L.c_qkv; P.s_cq = L.s_cq; P.c_cq = L.c_cq; P.s_f1 = L.s_f1; P.c_f1 = L.c_f1;
    P.b2 = static_cast<const bf16*>(L.b2);
    P.kcache = static_cast<bf16*>(s->kcache[l]); P.vcache = static_cast<bf16*>(s->vcache[l]);
    P.crosskv = static_cast<const float*>(s->crosskv[l]);
  }
  static_assert(sizeof(stack::StackMaps) == sizeof(s->stack_maps), "tensor maps do not fit their opaque copy");
  memcpy(s->stack_maps, &maps, sizeof(maps));
  BPD_CUDA(cudaMemcpyAsync(s->stack_layers, lp.data(), lp.size() * sizeof(stack::LayerPtrs), cudaMemcpyHostToDevice, s->stream));
  BPD_CUDA(cudaStreamSynchronize(s->stream));
  static_assert(sizeof(stack::Layout) <= sizeof(s->stack_layout), "layout does not fit its opaque copy");
  memcpy(s->stack_layout, &lay, sizeof(lay));
  s->stack_cross_rows = cross_rows; s->stack_long = long_seq ? 1 : 0; s->stack_minb = minb;
  s->stack = 1;
  s->stack_dev = dev;
  stack_live(dev, +1);
  return BPD_OK;
}

// Embedding, all decoder layers and the final layer norm in one launch; leaves the planes of the decoder output in
// s->xn and its fp32 copy in s->h_f32 like the layer-by-layer paths followed by the layer-norm kernel.
static int run_layers_stack(bpd_session* s, const PassArgs& a) {
  const bpd_model* m = s->m;
  const Config& c = m->cfg;
  stack::StackParams p;
  memset(&p, 0, sizeof(p));
  p.layers = static_cast<const stack::LayerPtrs*>(s->stack_layers);
  p.L = c.n_dec; p.d = c.d; p.H = c.H; p.ff = c.d_ff; p.R = s->B * a.kcur; p.rows_per_b = a.kcur; p.nb = s->B; p.eps = c.eps;
  p.tgt_embed = static_cast<const bf16*>(m->tgt_embed); p.pe = s->pe; p.npos = s->npos; p.vocab = c.V;
  p.st = s->st; p.forced = a.forced; p.forced_rows = a.forced_rows; p.kforced = a.kforced;
  p.local_q = c.local_q; p.local_m = c.local_m; p.max_src = s->max_src; p.scale = 1.0f / sqrtf((float)fused::kDH);
  p.cross_rows = s->stack_cross_rows; p.long_seq = s->stack_long;
  p.lnf_g = static_cast<const bf16*>(m->dec_lnf_g); p.lnf_b = static_cast<const bf16*>(m->dec_lnf_b);
  p.xn_hi = static_cast<bf16*>(s->xn); p.xn_plane = s->pl_xn; p.h_f32 = s->h_f32;
  p.layer_dump = a.layer_dump;
  p.ws = s->stack_ws; p.gather = s->stack_ws + (size_t)2 * c.H * fused::kMaxRows * c.d; p.bar = s->stack_bar; p.error = s->st.error; p.all_done = s->st.all_done;
  p.spin = stack::kSpin;
  memcpy(&p.lay, s->stack_layout, sizeof(p.lay));
  const dim3 grid(fused::kC, c.H), block(stack::kThreads);
  const bool pdl = s->use_pdl != 0;
  stack::StackMaps maps;
  memcpy(&maps, s->stack_maps, sizeof(maps));
  const size_t smem = (size_t)p.lay.total;
  // reduction panels of 32 columns (two steps of 16) for d_model 256, else 64 (four steps); one or two CTAs per SM
  const int nt = p.R > 8 ? 2 : 1, ksteps = c.d == 256 ? 2 : 4;
  const bool lean = !s->stack_long && s->stack_cross_rows > 0;
  cudaStream_t stream = s->stream;
  BPD_TRY(stack_variant(nt, ksteps, s->stack_minb, lean, [&](auto kernel) {
    BPD_CUDA(launch_k(kernel, grid, block, smem, stream, pdl, maps, p));
    return (int)BPD_OK;
  }));
  ++g_launches;
  return BPD_OK;
}

#define PROF(slot, ...) do { prof_mark(s, slot, 0); __VA_ARGS__; prof_mark(s, slot, 1); } while (0)
static int run_pass_tc(bpd_session* s, const PassArgs& a) {
  const bpd_model* m = s->m;
  const Config& c = m->cfg;
  cudaStream_t st = s->stream;
  const int d = c.d, f = c.d_ff, R = s->B * a.kcur;
  const int* done = s->st.all_done;
  const tc::Scratch sc = tc_scratch(s);
  const bool pdl = s->use_pdl != 0;
  const bool fold = s->fold_ln != 0;   // every kernel after the first may overlap its predecessor's tail
  const tc::Operands xn{nullptr, 0, s->xn, s->pl_xn, d, s->rows_all, d};
  auto with_w = [](tc::Operands o, const void* w, int rows) { o.w = w; o.w_rows = rows; return o; };
  prof_mark(s, kProfLayers, 0);
  if (s->stack) BPD_TRY(run_layers_stack(s, a));
  else if (s->fused) BPD_TRY(run_layers_fused(s, a));
  else {
  EmbedParams ep;
  memset(&ep, 0, sizeof(ep));
  ep.table = m->tgt_embed; ep.pe = s->pe; ep.npos = s->npos; ep.x = s->x; ep.rows = R; ep.rows_per_b = a.kcur;
  ep.d = d; ep.vocab = c.V; ep.st = s->st; ep.forced = a.forced; ep.forced_rows = a.forced_rows;
  ep.kforced = a.kforced; ep.src = nullptr; ep.all_done = done;
  if (fold) { ep.gain = static_cast<const bf16*>(m->dec[0].ln1g); ep.xg_hi = static_cast<bf16*>(s->xn); ep.xg_plane = s->pl_xn; }
  // passes of more than 16 rows: layer-norm statistics travel as per-tile partial results (see TcParams::stat_out)
  const bool wide = fold && R > 16;
  const int parts = d / 128;
  if (wide) { ep.stat_out = s->ln_stats; ep.stat_T = R; }
  auto stats_from = [&](tc::TcParams& q) { if (wide) { q.ln_x = nullptr; q.stat_in = s->ln_stats; q.stat_parts = parts; q.stat_T = R; } };
  auto stats_to = [&](tc::TcParams& q) { if (wide && q.g_next) { q.stat_out = s->ln_stats; q.stat_T = R; } };
  PROF(kProfEmbed, embed_kernel<bf16><<<R, 128, 0, st>>>(ep););
  ++g_launches;
  const tc::Operands at{nullptr, 0, s->attn, s->pl_attn, d, s->rows_all, d};
  const tc::Operands fx{nullptr, 0, s->ffh, s->pl_ffh, f, s->rows_all, f};
  for (int l = 0; l < c.n_dec; ++l) {
    const DecLayer& L = m->dec[l];
    if (!fold) PROF(kProfLn, launch_ln<bf16, float>(s->x, L.ln1g, L.ln1b, s->xn, nullptr, R, d, c.eps, done, st, s->pl_xn, pdl););
    tc::TcParams pq = tc_params(nullptr, 0, done);
    pq.out_f32 = static_cast<float*>(s->qbuf); pq.ldo = d; pq.d = d;
    pq.kcache = static_cast<bf16*>(s->kcache[l]); pq.vcache = static_cast<bf16*>(s->vcache[l]);
    pq.st = s->st; pq.rows_per_b = a.kcur;
    if (fold) { pq.ln_x = s->x; pq.ln_d = d; pq.ln_eps = c.eps; pq.ln_s = L.s_qkv; pq.ln_c = L.c_qkv; stats_from(pq); }
    PROF(kProfQkv, BPD_TRY(tc::launch<tc::kTcQkv>(with_w(xn, L.wqkv, 3 * d), 3 * d, d, R, pq, sc, st, 1, 0, 0, pdl)); ++g_launches);
    AttnParams ap;
    memset(&ap, 0, sizeof(ap));
    ap.q = s->qbuf; ap.ldq = d; ap.out = s->attn; ap.ldo = d; ap.out_plane = s->pl_attn; ap.rows = R;
    ap.rows_per_b = a.kcur; ap.H = c.H; ap.dh = d / c.H; ap.causal = 1; ap.local_q = c.local_q; ap.local_m = c.local_m;
    ap.k = s->kcache[l]; ap.v = s->vcache[l];
    ap.ldkv = d; ap.paged = 1; ap.st = s->st; ap.scale = 1.0f / sqrtf((float)ap.dh); ap.by_rows = (s->B >= 8) ? 1 : 0; ap.all_done = done;
    PROF(kProfSelfAttn, launch_attention<float, bf16>(ap, st, pdl););
    ++g_launches;
    tc::TcParams po = tc_params(nullptr, 0, done);
    po.out_f32 = s->x; po.ldo = d;
    if (fold) { po.g_next = static_cast<const bf16*>(L.ln2g); po.xg_hi = static_cast<bf16*>(s->xn); po.xg_plane = s->pl_xn; stats_to(po); }
    PROF(kProfOproj, BPD_TRY(tc::launch<tc::kTcResidual>(with_w(at, L.wo, d), d, d, R, po, sc, st, 1, 0, 0, pdl)); ++g_launches);
    if (!fold) PROF(kProfLn, launch_ln<bf16, float>(s->x, L.ln2g, L.ln2b, s->xn, nullptr, R, d, c.eps, done, st, s->pl_xn, pdl););
    tc::TcParams pc = tc_params(nullptr, 0, done);
    pc.out_f32 = static_cast<float*>(s->qbuf); pc.ldo = d;
    if (fold) { pc.ln_x = s->x; pc.ln_d = d; pc.ln_eps = c.eps; pc.ln_s = L.s_cq; pc.ln_c = L.c_cq; stats_from(pc); }
    PROF(kProfCrossQ, BPD_TRY(tc::launch<tc::kTcF32>(with_w(xn, L.cwq, d), d, d, R, pc, sc, st, 1, 0, 0, pdl)); ++g_launches);
    ap.causal = 0; ap.limit_b = s->st.src_len; ap.k = s->crosskv[l]; ap.v = static_cast<float*>(s->crosskv[l]) + d;
    ap.ldkv = 2 * d; ap.bstride = (long long)s->max_src * 2 * d; ap.paged = 0;
    // many sequences, head width 64: the encoder's keys and values are staged before the dependency wait
    const bool staged_cross = ap.by_rows && ap.dh == 64 && a.kcur <= 16 && cross_staged_smem(s->max_src) <= 160 * 1024 &&
                              s->opt.stage_encoder_rows;
    if (staged_cross) {
      const size_t smem = cross_staged_smem(s->max_src);
      BPD_TRY(cross_staged_attr(smem));
      PROF(kProfCrossAttn, BPD_CUDA(launch_k(cross_attention_staged_kernel<float>, dim3(s->B * c.H), dim3(kAttnWarps * 32), smem, st, pdl, ap, s->max_src, 1)););
    } else {
      PROF(kProfCrossAttn, launch_attention<float, float>(ap, st, pdl););
    }
    ++g_launches;
    if (fold) { po.g_next = static_cast<const bf16*>(L.ln3g); stats_to(po); }
    PROF(kProfCrossO, BPD_TRY(tc::launch<tc::kTcResidual>(with_w(at, L.cwo, d), d, d, R, po, sc, st, 1, 0, 0, pdl)); ++g_launches);
    if (!fold) PROF(kProfLn, launch_ln<bf16, float>(s->x, L.ln3g, L.ln3b, s->xn, nullptr, R, d, c.eps, done, st, s->pl_xn, pdl););
    tc::TcParams p1 = tc_params(L.b1, 1, done);
    p1.out_hi = static_cast<bf16*>(s->ffh); p1.plane = s->pl_ffh; p1.ldo = f;
    if (fold) { p1.ln_x = s->x; p1.ln_d = d; p1.ln_eps = c.eps; p1.ln_s = L.s_f1; p1.ln_c = L.c_f1; stats_from(p1); }
    PROF(kProfFfn1, BPD_TRY(tc::launch<tc::kTcPlanes>(with_w(xn, L.w1, f), f, d, R, p1, sc, st, 1, 0, 0, pdl)); ++g_launches);
    tc::TcParams p2 = tc_params(L.b2, 0, done);
    p2.out_f32 = s->x; p2.ldo = d;
    if (fold && l + 1 < c.n_dec) { p2.g_next = static_cast<const bf16*>(m->dec[l + 1].ln1g); p2.xg_hi = static_cast<bf16*>(s->xn); p2.xg_plane = s->pl_xn; stats_to(p2); }
    PROF(kProfFfn2, BPD_TRY(tc::launch<tc::kTcResidual>(with_w(fx, L.w2, d), d, f, R, p2, sc, st, 1, 0, 0, pdl)); ++g_launches);
    if (a.layer_dump)
      BPD_CUDA(cudaMemcpyAsync(a.layer_dump + (size_t)l * R * d, s->x, sizeof(float) * R * d, cudaMemcpyDeviceToDevice, st));
  }
  }
  if (!s->stack) PROF(kProfLn, launch_ln<bf16, float>(s->x, m->dec_lnf_g, m->dec_lnf_b, s->xn, s->h_f32, R, d, c.eps, done, st, s->pl_xn, pdl););
  prof_mark(s, kProfLayers, 1);
  // proposal heads
  const int fhd = c.d_hidden, km = c.k_model;
  const int ldu = km * fhd;
  const int hid = (c.head_layout == 0) ? km * fhd : a.kh * fhd;
  prof_mark(s, kProfHeadW1, 0);
  tc::TcParams pu = tc_params(m->head_b1, 1, done);
  pu.out_hi = static_cast<bf16*>(s->u); pu.plane = s->pl_u; pu.ldo = ldu;
  BPD_TRY(tc::launch<tc::kTcPlanes>(with_w(xn, m->head_w1, km * fhd), hid, d, R, pu, sc, st, 1, 0, 0, pdl, km * fhd)); ++g_launches;
  prof_mark(s, kProfHeadW1, 1);
  // output layers + shared vocabulary projection with a fused top-1 for T rows and kh heads
  // Sessions that evaluate the heads lazily never use head 1 of a launch over all heads, so there the output
  // layers of head 1 alone (greedy passes, stage 1) are planned for their own size, and stage 2 (plan_tt = 1:
  // one token tile) for its own; everywhere else every launch is planned for the full matrix, so that head 1
  // is the same sum whether it is evaluated alone or with the others.
  const bool own_plan = s->lazy_heads != 0 && tc_scratch(s).wide_ttiles > 0;
  auto heads = [&](const void* u_planes, long long u_plane, int u_rows, const float* hres, int T, int kh, int* table_out,
                   bool rank, float* logits, int plan_tt) -> int {
    prof_mark(s, kProfHeadW2, 0);
    tc::Operands uo{m->head_w2, km * d, u_planes, u_plane, ldu, u_rows, ldu};
    tc::TcParams ph = tc_params(m->head_b2, 0, done);
    ph.out_hi = static_cast<bf16*>(s->o); ph.plane = s->pl_o; ph.ldo = (long long)kh * d;
    ph.h = hres; ph.d = d; ph.head_identity = c.p1_identity;
    if (c.head_layout == 0) {
      BPD_TRY(tc::launch<tc::kTcHeadOut>(uo, kh * d, km * fhd, T, ph, sc, st, 1, 0, 0, pdl, own_plan ? kh * d : km * d,
                                         own_plan ? plan_tt : 0));
    } else {
      ph.zofs_n = d;
      BPD_TRY(tc::launch<tc::kTcHeadOut>(uo, d, fhd, T, ph, sc, st, kh, d, fhd, pdl));
    }
    ++g_launches;
    prof_mark(s, kProfHeadW2, 1);
    prof_mark(s, kProfVocab, 0);
    tc::Operands oo{m->out_proj, c.V, s->o, s->pl_o, d, s->rows_head, d};
    tc::TcParams pv = tc_params(nullptr, 0, done);
    pv.out_idx = table_out; pv.logits = logits;
    if (rank) {
      ProposalLogitParams pl{s->o, s->pl_o, m->out_proj, s->st, s->rank, s->B, a.kcur, kh, d, done};
      launch_k(proposal_logit_kernel<bf16>, dim3(ceil_div(R, 4)), dim3(128), 0, st, pdl, pl);
      ++g_launches;
      pv.rank = s->rank; pv.rank_kh = kh;
    }
    BPD_TRY(tc::launch<tc::kTcArgmax>(oo, c.V, d, T * kh, pv, sc, st, 1, 0, 0, pdl)); ++g_launches;
    prof_mark(s, kProfVocab, 1);
    return BPD_OK;
  };
  const bool lazy = pass_is_lazy(s, a);
  if (lazy) {
    // stage 1: p_1 at every block position, verification and commit
    BPD_TRY(heads(s->u, s->pl_u, s->rows_dec, s->h_f32, R, 1, s->st.table, wants_rank(a), nullptr, 0));
    PassArgs a1 = a;
    a1.kh = 1; a1.knext = 1;
    VerifyParams v1 = verify_params(s, a1);
    launch_k(verify_commit_kernel, dim3(1), dim3(32 * ceil_div(s->B, 32)), 0, st, pdl, v1);
    ++g_launches;
    // stage 2: all heads at the last accepted position of every row
    GatherParams gp{static_cast<const bf16*>(s->u), s->pl_u, ldu, static_cast<bf16*>(s->u2), s->pl_u2, s->h_f32, s->h2, d,
                    s->st, s->B, a.kcur, done};
    launch_k(gather_selected_kernel, dim3(s->B, 16), dim3(256), 0, st, pdl, gp);
    ++g_launches;
    BPD_TRY(heads(s->u2, s->pl_u2, s->B, s->h2, s->B, a.kh, s->table2, false, nullptr, 1));
    SelectParams sp{s->st, s->st.table, s->table2, s->table_full, s->B, a.kcur, a.kh, a.knext, done};
    launch_k(select_next_kernel, dim3(1), dim3(32 * ceil_div(s->B, 32)), 0, st, pdl, sp);
    ++g_launches;
    BPD_CUDA(cudaGetLastError());
    s->invocations += 1;
    return BPD_OK;
  }
  BPD_TRY(heads(s->u, s->pl_u, s->rows_dec, s->h_f32, R, a.kh, s->st.table, wants_rank(a), a.logits_dump, 0));
  VerifyParams vp = verify_params(s, a);
  PROF(kProfVerify, launch_k(verify_commit_kernel, dim3(1), dim3(32 * ceil_div(s->B, 32)), 0, st, pdl, vp););
  ++g_launches;
  BPD_CUDA(cudaGetLastError());
  s->invocations += 1;
  return BPD_OK;
}

#undef PROF
static int dispatch_eager(bpd_session* s, const PassArgs& a) {
  if (a.mode == kModePredict) {
    StepBackParams sp{s->st, s->B};
    step_back_kernel<<<1, 32 * ceil_div(s->B, 32), 0, s->stream>>>(sp);
    ++g_launches;
    BPD_CUDA(cudaGetLastError());
  }
  if (s->tc) return run_pass_tc(s, a);
  return s->m->cfg.dtype == 0 ? run_pass<float>(s, a) : run_pass<bf16>(s, a);
}

// A pass is a fixed sequence of launches for given arguments: the first use runs it eagerly (which also
// creates tensor maps and sets kernel attributes), the second captures it into a CUDA graph, later uses replay it.
static int dispatch_pass(bpd_session* s, const PassArgs& a) {
  s->last_pass_lazy = pass_is_lazy(s, a) ? 1 : 0;
  if (s->profiling || !s->use_graphs || a.logits_dump || a.layer_dump) return dispatch_eager(s, a);
  const GraphKey key(a.mode, a.kcur, a.kh, a.knext, (const void*)a.forced, a.forced_rows, a.kforced, a.max_new, a.eos,
                     (const void*)a.logits_dump, (a.accept_kind << 16) | (a.accept_param << 8) | a.min_block);
  GraphEntry& ge = s->graphs[key];
  if (ge.exec) {
    BPD_CUDA(cudaGraphLaunch(ge.exec, s->stream));
    g_launches += ge.launches;
    s->invocations += 1;
    return BPD_OK;
  }
  if (ge.uses++ == 0) return dispatch_eager(s, a);
  const long long before = g_launches.load();
  BPD_CUDA(cudaStreamBeginCapture(s->stream, cudaStreamCaptureModeThreadLocal));
  const int rc = dispatch_eager(s, a);
  cudaGraph_t graph = nullptr;
  const cudaError_t e = cudaStreamEndCapture(s->stream, &graph);
  if (rc) { if (graph) cudaGraphDestroy(graph); return rc; }
  if (e != cudaSuccess || !graph) return fail(BPD_E_CUDA, "stream capture of the decoder pass failed: %s", cudaGetErrorString(e));
  ge.launches = g_launches.load() - before;
  s->invocations -= 1;                       // the captured call only recorded the work
  g_launches -= ge.launches;
  const cudaError_t e2 = cudaGraphInstantiate(&ge.exec, graph, 0);
  cudaGraphDestroy(graph);
  if (e2 != cudaSuccess) { ge.exec = nullptr; return fail(BPD_E_CUDA, "cudaGraphInstantiate failed: %s", cudaGetErrorString(e2)); }
  BPD_CUDA(cudaGraphLaunch(ge.exec, s->stream));
  g_launches += ge.launches;
  s->invocations += 1;
  return BPD_OK;
}

static int check_device_error(bpd_session* s) {
  int err = 0;
  BPD_CUDA(cudaMemcpyAsync(&s->pinned[64], s->st.error, sizeof(int), cudaMemcpyDeviceToHost, s->stream));
  BPD_CUDA(cudaStreamSynchronize(s->stream));
  err = s->pinned[64];
  if (err == 1) return fail(BPD_E_INVALID, "a token id outside the vocabulary reached the decoder");
  if (err >= 101 && err <= 103) return fail(BPD_E_TIMEOUT, "a bounded wait inside the projection kernel expired (code %d)", err);
  if (err >= 104 && err <= 106) {
    const char* what[] = {"device-wide join", "weight tile", "exchange inside the cluster"};
    return fail(BPD_E_TIMEOUT, "a bounded wait inside the persistent layer kernel expired (code %d: %s)", err, what[err - 104]);
  }
  if (err != 0) return fail(BPD_E_CUDA, "device-side error word %d", err);
  return BPD_OK;
}

static int fetch(bpd_session* s, int max_new, int32_t* out_ids, int32_t* out_len, bpd_stats* stats, float ms) {
  const int B = s->B;
  std::vector<int> ids, jj(B);
  std::vector<long long> sv(4 + kMaxK + 1);
  if (out_ids) {
    ids.resize((size_t)B * s->max_tgt);
    BPD_CUDA(cudaMemcpyAsync(ids.data(), s->st.out_ids, ids.size() * sizeof(int), cudaMemcpyDeviceToHost, s->stream));
  }
  BPD_CUDA(cudaMemcpyAsync(jj.data(), s->st.j, B * sizeof(int), cudaMemcpyDeviceToHost, s->stream));
  BPD_CUDA(cudaMemcpyAsync(sv.data(), s->st.stats, sv.size() * sizeof(long long), cudaMemcpyDeviceToHost, s->stream));
  BPD_CUDA(cudaStreamSynchronize(s->stream));
  for (int b = 0; b < B; ++b) {
    const int n = std::min(jj[b], max_new);
    if (out_len) out_len[b] = n;
    if (out_ids) {
      for (int t = 0; t < max_new; ++t) out_ids[(size_t)b * max_new + t] = (t < n) ? ids[(size_t)b * s->max_tgt + t] : -1;
    }
  }
  if (stats) {
    memset(stats, 0, sizeof(*stats));
    stats->row_iterations = sv[0]; stats->tokens = sv[1]; stats->iterations = sv[2];
    for (int i = 0; i <= kMaxK; ++i) stats->khat_hist[i] = sv[4 + i];
    stats->invocations = sv[2] + sv[3];   // passes that did work (passes issued after the end return at once)
    stats->device_ms = ms;
  }
  return BPD_OK;
}

}  // namespace bpd

using namespace bpd;

// =================================================================== C ABI
extern "C" {

const char* bpd_last_error(void) { return g_err; }

int bpd_query_sizes(const void* blob, size_t blob_bytes, int batch, int max_src, int max_tgt, size_t* weight_bytes,
                    size_t* session_bytes) {
  ParsedBlob pb;
  int rc = parse_blob(blob, blob_bytes, &pb);
  if (rc) return rc;
  if (batch < 1 || batch > 1024 || max_src < 1 || max_tgt < 1) return fail(BPD_E_INVALID, "batch/max_src/max_tgt out of range");
  if (weight_bytes) *weight_bytes = weight_bytes_for(pb);
  if (session_bytes) *session_bytes = plan_session(pb.cfg, batch, max_src, max_tgt, nullptr, nullptr);
  return BPD_OK;
}

int bpd_session_layer_path(const bpd_session* s) {
  if (!s) return fail(BPD_E_INVALID, "session is null");
  return s->stack ? 2 : (s->fused ? 1 : 0);
}

int bpd_session_bytes(const bpd_model* model, int batch, int max_src, int max_tgt, size_t* session_bytes) {
  if (!model || !session_bytes) return fail(BPD_E_INVALID, "null argument");
  if (batch < 1 || batch > 1024 || max_src < 1 || max_tgt < 1) return fail(BPD_E_INVALID, "batch/max_src/max_tgt out of range");
  *session_bytes = plan_session(model->cfg, batch, max_src, max_tgt, nullptr, nullptr);
  return BPD_OK;
}

int bpd_load_weights(const void* blob, size_t blob_bytes, void* dev_weight_buf, size_t dev_bytes, void* cuda_stream,
                     bpd_model** out) {
  if (!out) return fail(BPD_E_INVALID, "out is null");
  *out = nullptr;
  ParsedBlob pb;
  int rc = parse_blob(blob, blob_bytes, &pb);
  if (rc) return rc;
  if (!dev_weight_buf) return fail(BPD_E_INVALID, "device weight buffer is null");
  if ((uintptr_t)dev_weight_buf % 256) return fail(BPD_E_INVALID, "device weight buffer is not 256-byte aligned");
  if (dev_bytes < weight_bytes_for(pb)) return fail(BPD_E_NOMEM, "device weight buffer has %zu bytes, need %zu", dev_bytes, weight_bytes_for(pb));
  bpd_model* m = new (std::nothrow) bpd_model();
  if (!m) return fail(BPD_E_NOMEM, "host allocation failed");
  const Config& c = pb.cfg;
  m->cfg = c; m->base = static_cast<char*>(dev_weight_buf); m->bytes = dev_bytes; m->stream = (cudaStream_t)cuda_stream;
  char* B = m->base;
  const int d = c.d, f = c.d_ff, V = c.V, k = c.k_model, fh = c.d_hidden;
#define T(name, out, ...) if ((rc = find(pb, B, name, {__VA_ARGS__}, &(out)))) { delete m; return rc; }
  T("src_embed", m->src_embed, V, d) T("tgt_embed", m->tgt_embed, V, d) T("out_proj", m->out_proj, V, d)
  m->enc.resize(c.n_enc); m->dec.resize(c.n_dec);
  for (int l = 0; l < c.n_enc; ++l) {
    const std::string p = "enc." + std::to_string(l);
    EncLayer& L = m->enc[l];
    T(p + ".ln1.g", L.ln1g, d) T(p + ".ln1.b", L.ln1b, d) T(p + ".attn.wqkv", L.wqkv, 3 * d, d) T(p + ".attn.wo", L.wo, d, d)
    T(p + ".ln2.g", L.ln2g, d) T(p + ".ln2.b", L.ln2b, d)
    T(p + ".ffn.w1", L.w1, f, d) T(p + ".ffn.b1", L.b1, f) T(p + ".ffn.w2", L.w2, d, f) T(p + ".ffn.b2", L.b2, d)
  }
  T("enc.lnf.g", m->enc_lnf_g, d) T("enc.lnf.b", m->enc_lnf_b, d)
  for (int l = 0; l < c.n_dec; ++l) {
    const std::string p = "dec." + std::to_string(l);
    DecLayer& L = m->dec[l];
    T(p + ".ln1.g", L.ln1g, d) T(p + ".ln1.b", L.ln1b, d) T(p + ".self.wqkv", L.wqkv, 3 * d, d) T(p + ".self.wo", L.wo, d, d)
    T(p + ".ln2.g", L.ln2g, d) T(p + ".ln2.b", L.ln2b, d)
    T(p + ".cross.wq", L.cwq, d, d) T(p + ".cross.wkv", L.cwkv, 2 * d, d) T(p + ".cross.wo", L.cwo, d, d)
    T(p + ".ln3.g", L.ln3g, d) T(p + ".ln3.b", L.ln3b, d)
    T(p + ".ffn.w1", L.w1, f, d) T(p + ".ffn.b1", L.b1, f) T(p + ".ffn.w2", L.w2, d, f) T(p + ".ffn.b2", L.b2, d)
  }
  T("dec.lnf.g", m->dec_lnf_g, d) T("dec.lnf.b", m->dec_lnf_b, d)
  T("head.w1", m->head_w1, k * fh, d) T("head.b1", m->head_b1, k * fh)
  if (c.head_layout == 0) { T("head.w2", m->head_w2, k * d, k * fh) } else { T("head.w2", m->head_w2, k, d, fh) }
  T("head.b2", m->head_b2, k * d)
#undef T
  cudaError_t e = cudaMemcpyAsync(m->base, blob, pb.total, cudaMemcpyHostToDevice, m->stream);
  if (c.dtype == 1 && e == cudaSuccess) {
    float* fp = reinterpret_cast<float*>(m->base + align_up(pb.total));
    auto fold = [&](const void* w, const void* g, const void* b, const void* bias, int N, float** s_out, float** c_out) {
      *s_out = fp; fp += N;
      *c_out = fp; fp += N;
      FoldParams p{static_cast<const bf16*>(w), static_cast<const bf16*>(g), static_cast<const bf16*>(b),
                   static_cast<const bf16*>(bias), *s_out, *c_out, N, d};
      fold_ln_kernel<<<ceil_div(N, 4), 128, 0, m->stream>>>(p);
    };
    for (int l = 0; l < c.n_dec; ++l) {
      DecLayer& L = m->dec[l];
      fold(L.wqkv, L.ln1g, L.ln1b, nullptr, 3 * d, &L.s_qkv, &L.c_qkv);
      fold(L.cwq, L.ln2g, L.ln2b, nullptr, d, &L.s_cq, &L.c_cq);
      fold(L.w1, L.ln3g, L.ln3b, L.b1, f, &L.s_f1, &L.c_f1);
    }
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(m->stream);
  if (e != cudaSuccess) { delete m; return fail(BPD_E_CUDA, "weight upload failed: %s", cudaGetErrorString(e)); }
  *out = m;
  return BPD_OK;
}

int bpd_model_destroy(bpd_model* m) {
  delete m;
  return BPD_OK;
}

void bpd_session_options_init(bpd_session_options* o) {
  if (!o) return;
  o->struct_bytes = (int32_t)sizeof(*o);
  o->tensor_cores = o->cuda_graphs = o->dependent_launch = o->lazy_heads = o->fold_layer_norms = -1;
  o->cluster_layers = o->persistent_layers = o->stage_encoder_rows = o->l2_stream_hints = -1;
}

int bpd_session_create(const bpd_model* model, int batch, int max_src, int max_tgt, void* dev_session_buf,
                       size_t dev_bytes, void* cuda_stream, bpd_session** out) {
  return bpd_session_create_opt(model, batch, max_src, max_tgt, dev_session_buf, dev_bytes, cuda_stream, nullptr, out);
}

int bpd_session_create_opt(const bpd_model* model, int batch, int max_src, int max_tgt, void* dev_session_buf,
                           size_t dev_bytes, void* cuda_stream, const bpd_session_options* options, bpd_session** out) {
  if (!out) return fail(BPD_E_INVALID, "out is null");
  bpd_session_options o;
  bpd_session_options_init(&o);
  if (options) {
    if (options->struct_bytes != (int32_t)sizeof(o)) return fail(BPD_E_INVALID, "bpd_session_options.struct_bytes = %d, this library expects %zu", options->struct_bytes, sizeof(o));
    o = *options;
    const int32_t* f = &o.tensor_cores;
    for (int i = 0; i < 9; ++i)
      if (f[i] < -1 || f[i] > 1) return fail(BPD_E_INVALID, "session option %d has value %d (want -1, 0 or 1)", i, f[i]);
  }
  *out = nullptr;
  if (!model || !dev_session_buf) return fail(BPD_E_INVALID, "model or session buffer is null");
  if (batch < 1 || batch > 1024 || max_src < 1 || max_tgt < 1) return fail(BPD_E_INVALID, "batch/max_src/max_tgt out of range");
  if ((uintptr_t)dev_session_buf % 256) return fail(BPD_E_INVALID, "session buffer is not 256-byte aligned");
  const size_t need = plan_session(model->cfg, batch, max_src, max_tgt, nullptr, nullptr);
  if (dev_bytes < need) return fail(BPD_E_NOMEM, "session buffer has %zu bytes, need %zu", dev_bytes, need);
  bpd_session* s = new (std::nothrow) bpd_session();
  if (!s) return fail(BPD_E_NOMEM, "host allocation failed");
  s->m = model; s->B = batch; s->max_src = max_src; s->max_tgt = max_tgt;
  s->base = static_cast<char*>(dev_session_buf); s->bytes = dev_bytes; s->stream = (cudaStream_t)cuda_stream;
  s->profiling = 0;
  // options: -1 takes the library's choice for this model and batch; 0 / 1 force a strategy off / on (on only
  // where the shapes allow it)
  s->tc = (model->cfg.dtype == 1 && o.tensor_cores != 0) ? 1 : 0;
  // the default streams cannot be captured: graphs need a stream of the caller's own
  const bool own_stream = s->stream != nullptr && s->stream != cudaStreamLegacy && s->stream != cudaStreamPerThread;
  s->use_graphs = (own_stream && o.cuda_graphs != 0) ? 1 : 0;
  s->use_pdl = o.dependent_launch != 0 ? 1 : 0;
  s->lazy_heads = s->tc && (o.lazy_heads >= 0 ? o.lazy_heads != 0 : batch * model->cfg.k_model >= 64);
  s->last_pass_lazy = 0;
  // with at most 16 rows per pass every projection CTA can afford the row statistics itself
  // passes of at most 16 rows take the statistics from the stream itself; wider ones need whole 128-feature tiles (and
  // the embedding kernel whole warps: d_model a multiple of 256)
  s->fold_ln = (s->tc && o.fold_layer_norms != 0 && (batch * model->cfg.k_model <= 16 || model->cfg.d % 256 == 0)) ? 1 : 0;
  s->fused = (s->tc && fused::supported(model->cfg.d, model->cfg.H, model->cfg.d_ff, batch * model->cfg.k_model) &&
              o.cluster_layers != 0) ? 1 : 0;
  s->opt.persistent_layers = o.persistent_layers;   // -1: where its lean variant applies (measured faster there), 0: never, 1: wherever it runs
  s->opt.stage_encoder_rows = o.stage_encoder_rows != 0 ? 1 : 0;
  s->opt.l2_stream_hints = o.l2_stream_hints != 0 ? 1 : 0;
  s->stack = 0; s->stack_dump = nullptr;
  s->timed = 0;
  s->phase = kPhaseCreated; s->plan_len = 0; s->plan_k = 0; s->invocations = 0; s->pinned = nullptr;
  plan_session(model->cfg, batch, max_src, max_tgt, s->base, s);
  // page table: row b's p-th page is physical page p*B + b (rows interleaved in the pool)
  std::vector<int> pt((size_t)batch * s->ppr);
  for (int b = 0; b < batch; ++b)
    for (int p = 0; p < s->ppr; ++p) pt[(size_t)b * s->ppr + p] = p * batch + b;
  // sinusoidal positions: PE(p, 2i) = sin(p / 10000^(2i/d)), PE(p, 2i+1) = cos(same), evaluated in double
  std::vector<float> pe((size_t)s->npos * model->cfg.d);
  for (int pos = 0; pos < s->npos; ++pos)
    for (int i = 0; i < model->cfg.d / 2; ++i) {
      const double ang = (double)pos / pow(10000.0, 2.0 * i / model->cfg.d);
      pe[(size_t)pos * model->cfg.d + 2 * i] = (float)sin(ang);
      pe[(size_t)pos * model->cfg.d + 2 * i + 1] = (float)cos(ang);
    }
  cudaError_t e = cudaMallocHost(reinterpret_cast<void**>(&s->pinned), (256 + (size_t)batch * kMaxK) * sizeof(int));
  if (e == cudaSuccess) {
    memset(s->pinned, 0, (256 + (size_t)batch * kMaxK) * sizeof(int));
    void* dev_view = nullptr;
    e = cudaHostGetDevicePointer(&dev_view, s->pinned, 0);
    s->st.host_flags = static_cast<int*>(dev_view);
    s->epoch = 0;
  }
  for (int i = 0; i < 8 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&s->ev_flag[i], cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreate(&s->ev0);
  if (e == cudaSuccess) e = cudaEventCreate(&s->ev1);
  if (e == cudaSuccess) e = cudaMemsetAsync(s->base, 0, need, s->stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(const_cast<int*>(s->st.page_table), pt.data(), pt.size() * sizeof(int), cudaMemcpyHostToDevice, s->stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(s->pe, pe.data(), pe.size() * sizeof(float), cudaMemcpyHostToDevice, s->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s->stream);
  if (e != cudaSuccess) {
    delete s;
    return fail(BPD_E_CUDA, "session set-up failed: %s", cudaGetErrorString(e));
  }
  const int rc_stack = stack_setup(s);
  if (rc_stack) { bpd_session_destroy(s); return rc_stack; }
  *out = s;
  return BPD_OK;
}

int bpd_session_destroy(bpd_session* s) {
  if (!s) return BPD_OK;
  cudaStreamSynchronize(s->stream);
  if (s->stack) { stack_live(s->stack_dev, -1); s->stack = 0; }
  prof_clear(s);
  for (auto& kv : s->graphs)
    if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
  if (s->enc_graph.exec) cudaGraphExecDestroy(s->enc_graph.exec);
  if (s->pinned) cudaFreeHost(s->pinned);
  for (int i = 0; i < 8; ++i) cudaEventDestroy(s->ev_flag[i]);
  cudaEventDestroy(s->ev0);
  cudaEventDestroy(s->ev1);
  delete s;
  return BPD_OK;
}

int bpd_encode(bpd_session* s, const int32_t* src_ids, const int32_t* src_len) {
  if (!s || !src_ids || !src_len) return fail(BPD_E_INVALID, "null argument");
  const Config& c = s->m->cfg;
  const int B = s->B, S = s->max_src;
  std::vector<int> ids((size_t)B * S, 0), lens(B);
  for (int b = 0; b < B; ++b) {
    if (src_len[b] < 1 || src_len[b] > S) return fail(BPD_E_SHAPE, "src_len[%d] = %d outside 1..%d", b, src_len[b], S);
    lens[b] = src_len[b];
    for (int t = 0; t < src_len[b]; ++t) {
      const int id = src_ids[(size_t)b * S + t];
      if (id < 0 || id >= c.V) return fail(BPD_E_INVALID, "source id %d at row %d position %d outside the vocabulary", id, b, t);
      ids[(size_t)b * S + t] = id;
    }
  }
  // staging through pinned memory keeps the copies asynchronous and ordered on the stream
  BPD_CUDA(cudaStreamSynchronize(s->stream));
  BPD_CUDA(cudaMemcpyAsync(s->src_dev, ids.data(), ids.size() * sizeof(int), cudaMemcpyHostToDevice, s->stream));
  BPD_CUDA(cudaMemcpyAsync(s->tail_dev, lens.data(), B * sizeof(int), cudaMemcpyHostToDevice, s->stream));
  ResetParams rp{s->st, B, s->ppr, s->tail_dev, s->stack_bar};
  reset_rows_kernel<<<1, 32 * ceil_div(B, 32), 0, s->stream>>>(rp);
  ++g_launches;
  BPD_CUDA(cudaStreamSynchronize(s->stream));   // host vectors go out of scope
  int rc = BPD_OK;
  auto eager = [&]() { return s->tc ? run_encoder_tc(s) : ((c.dtype == 0) ? run_encoder<float>(s) : run_encoder<bf16>(s)); };
  GraphEntry& ge = s->enc_graph;
  if (s->profiling || !s->use_graphs || !s->tc) {
    rc = eager();
  } else if (ge.exec) {
    BPD_CUDA(cudaGraphLaunch(ge.exec, s->stream));
    g_launches += ge.launches;
  } else if (ge.uses++ == 0) {
    rc = eager();                              // also creates tensor maps and sets kernel attributes
  } else {
    const long long before = g_launches.load();
    BPD_CUDA(cudaStreamBeginCapture(s->stream, cudaStreamCaptureModeThreadLocal));
    rc = eager();
    cudaGraph_t graph = nullptr;
    const cudaError_t e = cudaStreamEndCapture(s->stream, &graph);
    if (rc) { if (graph) cudaGraphDestroy(graph); return rc; }
    if (e != cudaSuccess || !graph) return fail(BPD_E_CUDA, "stream capture of the encoder failed: %s", cudaGetErrorString(e));
    ge.launches = g_launches.load() - before;
    g_launches -= ge.launches;
    const cudaError_t e2 = cudaGraphInstantiate(&ge.exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e2 != cudaSuccess) { ge.exec = nullptr; return fail(BPD_E_CUDA, "cudaGraphInstantiate failed: %s", cudaGetErrorString(e2)); }
    BPD_CUDA(cudaGraphLaunch(ge.exec, s->stream));
    g_launches += ge.launches;
  }
  if (rc) return rc;
  s->phase = kPhaseEncoded; s->plan_len = 0; s->plan_k = 0; s->invocations = 0; s->timed = 0;
  return BPD_OK;
}

int bpd_rewind(bpd_session* s) {
  if (!s) return fail(BPD_E_INVALID, "session is null");
  if (s->phase < kPhaseEncoded) return fail(BPD_E_STATE, "nothing encoded yet");
  ResetParams rp{s->st, s->B, s->ppr, s->st.src_len, s->stack_bar};
  reset_rows_kernel<<<1, 32 * ceil_div(s->B, 32), 0, s->stream>>>(rp);
  ++g_launches;
  BPD_CUDA(cudaGetLastError());
  s->phase = kPhaseEncoded; s->invocations = 0; s->timed = 0;
  return BPD_OK;
}

long long bpd_kernel_launches(void) { return g_launches.load(); }

int bpd_profile(bpd_session* s, int enable) {
  if (!s) return fail(BPD_E_INVALID, "session is null");
  BPD_CUDA(cudaStreamSynchronize(s->stream));
  prof_clear(s);
  s->profiling = enable ? 1 : 0;
  return BPD_OK;
}

int bpd_profile_read(bpd_session* s, int phase, int64_t* launches, double* total_ms) {
  if (!s || !launches || !total_ms) return fail(BPD_E_INVALID, "null argument");
  if (phase < 0 || phase >= kProfSlots) return fail(BPD_E_INVALID, "phase %d outside 0..%d", phase, kProfSlots - 1);
  BPD_CUDA(cudaStreamSynchronize(s->stream));
  const size_t n = std::min(s->prof_begin[phase].size(), s->prof_end[phase].size());
  double sum = 0;
  for (size_t i = 0; i < n; ++i) {
    float ms = 0.f;
    BPD_CUDA(cudaEventElapsedTime(&ms, s->prof_begin[phase][i], s->prof_end[phase][i]));
    sum += ms;
  }
  *launches = (int64_t)n;
  *total_ms = sum;
  return BPD_OK;
}

int bpd_set_forced_plan(bpd_session* s, const int32_t* plan, int plan_len, int k) {
  if (!s) return fail(BPD_E_INVALID, "session is null");
  if (!plan) { s->plan_len = 0; s->plan_k = 0; return BPD_OK; }
  if (k < 2 || k > s->m->cfg.k_model) return fail(BPD_E_INVALID, "k = %d outside 2..%d", k, s->m->cfg.k_model);
  if (plan_len < 1 || plan_len > s->max_tgt) return fail(BPD_E_SHAPE, "plan_len = %d outside 1..%d", plan_len, s->max_tgt);
  const size_t n = (size_t)s->B * plan_len * (k - 1);
  for (size_t i = 0; i < n; ++i)
    if (plan[i] < 0 || plan[i] >= s->m->cfg.V) return fail(BPD_E_INVALID, "plan entry %zu = %d outside the vocabulary", i, plan[i]);
  BPD_CUDA(cudaMemcpyAsync(s->plan_dev, plan, n * sizeof(int), cudaMemcpyHostToDevice, s->stream));
  BPD_CUDA(cudaStreamSynchronize(s->stream));
  s->plan_len = plan_len; s->plan_k = k;
  return BPD_OK;
}

static int check_decode_args(bpd_session* s, int max_new, int eos) {
  if (!s) return fail(BPD_E_INVALID, "session is null");
  if (max_new < 1 || max_new > s->max_tgt) return fail(BPD_E_SHAPE, "max_new = %d outside 1..%d", max_new, s->max_tgt);
  if (eos < -1 || eos >= s->m->cfg.V) return fail(BPD_E_INVALID, "eos_id = %d outside the vocabulary", eos);
  return BPD_OK;
}

// Launch passes until the device reports every row finished.  The flag of pass
// t is read back asynchronously and looked at two passes later, so the host
// never stalls the stream; passes issued after the end return at once.
// The verify kernel of pass t writes (epoch, finished?) straight into slot t mod 8 of the pinned flags; nothing is
// enqueued between two passes.  Returns 1 / 2 (open / all rows finished) once the slot carries this decode's epoch.
static int wait_pass_flag(bpd_session* s, int slot, int* finished) {
  volatile int* flags = s->pinned;
  const auto t0 = std::chrono::steady_clock::now();
  for (unsigned spins = 0;; ++spins) {
    const int v = flags[slot];
    if ((v >> 2) == s->epoch) {
      flags[slot] = 0;              // the slot's next report (eight passes on) must not be mistaken for this one
      *finished = (v & 3) == 2;
      return BPD_OK;
    }
    if ((spins & 0x3ff) == 0x3ff) {
      const cudaError_t q = cudaStreamQuery(s->stream);
      if (q != cudaSuccess && q != cudaErrorNotReady) return fail(BPD_E_CUDA, "decoder pass failed: %s", cudaGetErrorString(q));
      if (q == cudaSuccess && (flags[slot] >> 2) != s->epoch) return fail(BPD_E_CUDA, "a pass ended without reporting its state");
      if (std::chrono::steady_clock::now() - t0 > std::chrono::seconds(30)) return fail(BPD_E_TIMEOUT, "no pass reported its state for 30 s");
    }
  }
}
static int decode_loop(bpd_session* s, const PassArgs* cycle, int n_cycle, int max_passes) {
  // a new epoch and pass counter for this decode, ordered on the stream behind whatever the previous one left
  s->epoch = (s->epoch % 0x0fffffff) + 1;
  int* stage = &s->pinned[200 + 2 * (s->epoch & 1)];
  stage[0] = s->epoch; stage[1] = 0;
  BPD_CUDA(cudaMemcpyAsync(s->st.signal, stage, 2 * sizeof(int), cudaMemcpyHostToDevice, s->stream));
  for (int it = 0; it < max_passes; ++it) {
    if (it >= 2) {
      int finished = 0;
      int rc = wait_pass_flag(s, (it - 2) % 8, &finished);
      if (rc) return rc;
      if (finished) break;
    }
    int rc = dispatch_pass(s, cycle[it % n_cycle]);
    if (rc) return rc;
  }
  return BPD_OK;
}

static int finish_decode(bpd_session* s, int max_new, int32_t* out_ids, int32_t* out_len, bpd_stats* stats) {
  BPD_CUDA(cudaEventRecord(s->ev1, s->stream));
  s->timed = 1;
  if (!out_ids && !out_len && !stats) return BPD_OK;
  BPD_CUDA(cudaEventSynchronize(s->ev1));
  float ms = 0.f;
  BPD_CUDA(cudaEventElapsedTime(&ms, s->ev0, s->ev1));
  int rc = check_device_error(s);
  if (rc) return rc;
  return fetch(s, max_new, out_ids, out_len, stats, ms);
}

int bpd_decode_greedy(bpd_session* s, int max_new, int32_t eos_id, int32_t* out_ids, int32_t* out_len, bpd_stats* stats) {
  int rc = check_decode_args(s, max_new, eos_id);
  if (rc) return rc;
  if (s->phase != kPhaseEncoded) return fail(BPD_E_STATE, "bpd_decode_greedy needs a freshly encoded session");
  s->phase = kPhaseGreedy;
  BPD_CUDA(cudaEventRecord(s->ev0, s->stream));
  PassArgs a{kModeGreedy, 1, 1, 1, nullptr, 0, 0, max_new, eos_id, nullptr};
  rc = decode_loop(s, &a, 1, max_new);
  if (rc) return rc;
  return finish_decode(s, max_new, out_ids, out_len, stats);
}

int bpd_decode_blockwise(bpd_session* s, int k, int accept_mode, int max_new, int32_t eos_id, int32_t* out_ids,
                         int32_t* out_len, bpd_stats* stats) {
  int rc = check_decode_args(s, max_new, eos_id);
  if (rc) return rc;
  if (k < 1 || k > s->m->cfg.k_model) return fail(BPD_E_INVALID, "k = %d outside 1..%d", k, s->m->cfg.k_model);
  PassArgs acc{};
  if ((rc = decode_accept(accept_mode, k, &acc))) return rc;
  if (s->phase != kPhaseEncoded) return fail(BPD_E_STATE, "bpd_decode_blockwise needs a freshly encoded session");
  if (s->plan_len && s->plan_k != k) return fail(BPD_E_SHAPE, "forced plan was installed for k = %d", s->plan_k);
  s->phase = kPhaseBlockwise;
  BPD_CUDA(cudaEventRecord(s->ev0, s->stream));
  PassArgs prime{kModePrime, 1, k, k, nullptr, 0, 0, max_new, eos_id, nullptr};
  rc = dispatch_pass(s, prime);
  if (rc) return rc;
  PassArgs a{kModeBlock, k, k, k, s->plan_len ? s->plan_dev : nullptr, s->plan_len, k, max_new, eos_id, nullptr,
             acc.accept_kind, acc.accept_param, acc.min_block};
  rc = decode_loop(s, &a, 1, max_new);
  if (rc) return rc;
  return finish_decode(s, max_new, out_ids, out_len, stats);
}

int bpd_decode_blockwise_twocall(bpd_session* s, int k, int accept_mode, int max_new, int32_t eos_id, int32_t* out_ids,
                                 int32_t* out_len, bpd_stats* stats) {
  int rc = check_decode_args(s, max_new, eos_id);
  if (rc) return rc;
  if (k < 1 || k > s->m->cfg.k_model) return fail(BPD_E_INVALID, "k = %d outside 1..%d", k, s->m->cfg.k_model);
  PassArgs acc{};
  if ((rc = decode_accept(accept_mode, k, &acc))) return rc;
  if (s->phase != kPhaseEncoded) return fail(BPD_E_STATE, "bpd_decode_blockwise_twocall needs a freshly encoded session");
  if (s->plan_len && s->plan_k != k) return fail(BPD_E_SHAPE, "forced plan was installed for k = %d", s->plan_k);
  s->phase = kPhaseBlockwise;
  BPD_CUDA(cudaEventRecord(s->ev0, s->stream));
  // the first Predict scores the start token: the priming pass
  PassArgs prime{kModePrime, 1, k, k, nullptr, 0, 0, max_new, eos_id, nullptr};
  rc = dispatch_pass(s, prime);
  if (rc) return rc;
  // Verify: p_1 alone at the k block positions, then accept; Predict: all k heads at the last accepted token
  PassArgs cycle[2] = {
      PassArgs{kModeBlock, k, 1, 1, s->plan_len ? s->plan_dev : nullptr, s->plan_len, k, max_new, eos_id, nullptr,
               acc.accept_kind, acc.accept_param, acc.min_block},
      PassArgs{kModePredict, 1, k, k, nullptr, 0, 0, max_new, eos_id, nullptr}};
  rc = decode_loop(s, cycle, 2, 2 * max_new);
  if (rc) return rc;
  return finish_decode(s, max_new, out_ids, out_len, stats);
}

int bpd_iteration(bpd_session* s, int k, int accept_mode, int max_new, int32_t eos_id, const int32_t* forced_tail,
                  bpd_iter_out* out) {
  int rc = check_decode_args(s, max_new, eos_id);
  if (rc) return rc;
  if (k < 1 || k > s->m->cfg.k_model) return fail(BPD_E_INVALID, "k = %d outside 1..%d", k, s->m->cfg.k_model);
  PassArgs acc{};
  if ((rc = decode_accept(accept_mode, k, &acc))) return rc;
  if (s->phase != kPhaseEncoded && s->phase != kPhaseBlockwise) return fail(BPD_E_STATE, "bpd_iteration needs an encoded session that is not decoding greedily");
  const int B = s->B, V = s->m->cfg.V;
  if (forced_tail && k > 1) {
    for (int i = 0; i < B * (k - 1); ++i)
      if (forced_tail[i] < 0 || forced_tail[i] >= V) return fail(BPD_E_INVALID, "forced_tail[%d] = %d outside the vocabulary", i, forced_tail[i]);
  }
  if (s->phase == kPhaseEncoded) {
    PassArgs prime{kModePrime, 1, k, k, nullptr, 0, 0, max_new, eos_id, nullptr};
    rc = dispatch_pass(s, prime);
    if (rc) return rc;
    s->phase = kPhaseBlockwise;
  }
  PassArgs a{kModeBlock, k, k, k, nullptr, 0, 0, max_new, eos_id, out ? out->logits_dev : nullptr,
             acc.accept_kind, acc.accept_param, acc.min_block, out ? out->layers_dev : nullptr};
  if (forced_tail && k > 1) {
    BPD_CUDA(cudaStreamSynchronize(s->stream));   // the staging slots may still be in flight
    memcpy(&s->pinned[128], forced_tail, sizeof(int) * B * (k - 1));
    BPD_CUDA(cudaMemcpyAsync(s->tail_dev, &s->pinned[128], sizeof(int) * B * (k - 1), cudaMemcpyHostToDevice, s->stream));
    a.forced = s->tail_dev; a.forced_rows = 1; a.kforced = k;
  } else if (s->plan_len) {
    if (s->plan_k != k) return fail(BPD_E_SHAPE, "forced plan was installed for k = %d", s->plan_k);
    a.forced = s->plan_dev; a.forced_rows = s->plan_len; a.kforced = k;
  }
  rc = dispatch_pass(s, a);
  if (rc) return rc;
  if (!out) return BPD_OK;
  if (out->hidden_dev)
    BPD_CUDA(cudaMemcpyAsync(out->hidden_dev, s->h_f32, sizeof(float) * B * k * s->m->cfg.d, cudaMemcpyDeviceToDevice, s->stream));
  std::vector<int> khat(B), table((size_t)B * k * k), blk((size_t)B * kMaxK), cur((size_t)B * kMaxK);
  BPD_CUDA(cudaMemcpyAsync(khat.data(), s->st.khat, B * sizeof(int), cudaMemcpyDeviceToHost, s->stream));
  BPD_CUDA(cudaMemcpyAsync(table.data(), s->last_pass_lazy ? s->table_full : s->st.table, table.size() * sizeof(int),
                           cudaMemcpyDeviceToHost, s->stream));
  BPD_CUDA(cudaMemcpyAsync(blk.data(), s->st.block, blk.size() * sizeof(int), cudaMemcpyDeviceToHost, s->stream));
  BPD_CUDA(cudaMemcpyAsync(cur.data(), s->st.cur_block, cur.size() * sizeof(int), cudaMemcpyDeviceToHost, s->stream));
  BPD_CUDA(cudaStreamSynchronize(s->stream));
  rc = check_device_error(s);
  if (rc) return rc;
  for (int b = 0; b < B; ++b) {
    if (out->khat) out->khat[b] = khat[b];
    for (int i = 0; i < k; ++i) {
      if (out->accepted) out->accepted[b * k + i] = (i < khat[b]) ? cur[b * kMaxK + i] : -1;
      if (out->next_block) out->next_block[b * k + i] = blk[b * kMaxK + i];
      if (out->block) out->block[b * k + i] = cur[b * kMaxK + i];
    }
  }
  if (out->table) memcpy(out->table, table.data(), table.size() * sizeof(int));
  return BPD_OK;
}

int bpd_fetch_output(bpd_session* s, int max_new, int32_t* out_ids, int32_t* out_len, bpd_stats* stats) {
  if (!s) return fail(BPD_E_INVALID, "session is null");
  if (max_new < 1 || max_new > s->max_tgt) return fail(BPD_E_SHAPE, "max_new = %d outside 1..%d", max_new, s->max_tgt);
  if (s->phase < kPhaseEncoded) return fail(BPD_E_STATE, "nothing encoded yet");
  float ms = 0.f;
  if (s->phase != kPhaseEncoded && s->timed) {   // a decode call bracketed its loop with events; bpd_iteration does not
    BPD_CUDA(cudaEventSynchronize(s->ev1));
    BPD_CUDA(cudaEventElapsedTime(&ms, s->ev0, s->ev1));
  }
  int rc = check_device_error(s);
  if (rc) return rc;
  return fetch(s, max_new, out_ids, out_len, stats, ms);
}

#ifdef BPD_STACK_TRACE
// Development builds only: where the persistent layer kernel writes its per-CTA step timestamps (device memory,
// clusters * 8 * 256 unsigned 64-bit words), or null to stop.
int bpd_debug_set_stack_trace(void* dev_buffer) {
  unsigned long long* ptr = static_cast<unsigned long long*>(dev_buffer);
  BPD_CUDA(cudaMemcpyToSymbol(stack::g_stack_trace, &ptr, sizeof(ptr)));

  return BPD_OK;
}
#endif

#ifdef BPD_TC_TRACE
// Development builds only: where the projection kernel writes its per-CTA step timestamps (4096 * 16 unsigned 64-bit
// words of device memory), or null to stop.
int bpd_debug_set_tc_trace(void* dev_buffer) {
  unsigned long long* ptr = static_cast<unsigned long long*>(dev_buffer);
  BPD_CUDA(cudaMemcpyToSymbol(tc::g_tc_trace, &ptr, sizeof(ptr)));
  return BPD_OK;
}
#endif

// ------------------------------------------------------------------ self test of the bounded waits
int bpd_debug_wait_timeout(int32_t* dev_word, int limit_us, void* cuda_stream) {
  if (!dev_word) return fail(BPD_E_INVALID, "device word is null");
  if (limit_us < 1 || limit_us > 2000000) return fail(BPD_E_INVALID, "limit_us = %d outside 1..2000000", limit_us);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int khz = 0, dev = 0;
  BPD_CUDA(cudaGetDevice(&dev));
  BPD_CUDA(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
  BPD_CUDA(cudaMemsetAsync(dev_word, 0, sizeof(int), st));
  tc::wait_probe_kernel<<<1, 32, 0, st>>>(dev_word, (unsigned long long)limit_us * (unsigned long long)khz / 1000ull);
  ++g_launches;
  int word = 0;
  BPD_CUDA(cudaMemcpyAsync(&word, dev_word, sizeof(int), cudaMemcpyDeviceToHost, st));
  BPD_CUDA(cudaStreamSynchronize(st));
  if (!word) return BPD_OK;
  // the same for the tagged words the persistent layer kernel's reductions wait on
  const int first = word;
  BPD_CUDA(cudaMemsetAsync(dev_word, 0, sizeof(int), st));
  stack::tagged_wait_probe_kernel<<<1, 32, 0, st>>>(dev_word, (unsigned long long)limit_us * (unsigned long long)khz / 1000ull);
  ++g_launches;
  BPD_CUDA(cudaGetLastError());
  BPD_CUDA(cudaMemcpyAsync(&word, dev_word, sizeof(int), cudaMemcpyDeviceToHost, st));
  BPD_CUDA(cudaStreamSynchronize(st));
  if (word != 104) return fail(BPD_E_CUDA, "the wait on tagged words did not expire as it should (word %d)", word);
  return fail(BPD_E_TIMEOUT, "the bounded waits inside the probe kernels expired (codes %d and %d), as they should", first, word);
}

// ------------------------------------------------------------------ single operators
// Scratch layout of the bf16 (tensor-core) operators: a zero "lo" plane for the caller's single-plane bf16
// activations, the split-K workspace, tile counters, the top-1 merge counter and partials, an error word.
struct OpScratch {
  size_t zero_off, ws_off, cnt_off, done_off, pv_off, pi_off, err_off, total;
  size_t ws_floats, n_counters, part_elems;
};
static OpScratch op_scratch_layout(int rows, int in_f, int out_f) {
  OpScratch o;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes); return at; };
  o.ws_floats = tc::ws_floats(out_f, in_f, rows, 1);
  o.n_counters = tc::counters_needed(out_f, rows, 1);
  o.part_elems = (size_t)rows;
  o.zero_off = take((size_t)rows * in_f * sizeof(bf16));
  o.ws_off = take(o.ws_floats * sizeof(float));
  o.cnt_off = take(o.n_counters * sizeof(unsigned));
  o.done_off = take(sizeof(unsigned));
  o.pv_off = take(o.part_elems * tc::kBestStride * sizeof(unsigned long long));
  o.pi_off = o.pv_off;
  o.err_off = take(sizeof(int));
  o.total = off;
  return o;
}
static bool op_use_tc(int dtype) { return dtype == 1; }

static int op_tc_finish(char* scratch, const OpScratch& L, cudaStream_t st) {
  int err = 0;
  BPD_CUDA(cudaMemcpyAsync(&err, scratch + L.err_off, sizeof(int), cudaMemcpyDeviceToHost, st));
  BPD_CUDA(cudaStreamSynchronize(st));
  if (err) return fail(BPD_E_TIMEOUT, "a bounded wait inside the projection kernel expired (code %d)", err);
  return BPD_OK;
}

size_t bpd_op_vocab_argmax_scratch_bytes(int rows, int d, int vocab, int dtype) {
  if (rows < 1 || vocab < 1 || d < 1) return 0;
  if (op_use_tc(dtype)) return op_scratch_layout(rows, d, vocab).total;
  const size_t tiles = ceil_div(vocab, kVocTile);
  return align_up(tiles * rows * sizeof(float)) + align_up(tiles * rows * sizeof(int)) +
         align_up((ceil_div(rows, kRC) + 1) * sizeof(unsigned));
}

int bpd_op_vocab_argmax(const void* x, const void* w, int rows, int d, int vocab, int dtype, void* scratch,
                        size_t scratch_bytes, int32_t* out_idx, float* out_val, void* cuda_stream) {
  if (!x || !w || !scratch || !out_idx) return fail(BPD_E_INVALID, "null argument");
  if (rows < 1 || vocab < 1 || d < 8 || d % 8 || d > kArgmaxMaxD) return fail(BPD_E_SHAPE, "rows/d/vocab out of range (d must be a multiple of 8, at most %d)", kArgmaxMaxD);
  if (dtype != 0 && dtype != 1) return fail(BPD_E_INVALID, "unknown dtype %d", dtype);
  if ((uintptr_t)x % 16 || (uintptr_t)w % 16 || (uintptr_t)scratch % 256) return fail(BPD_E_INVALID, "misaligned pointer");
  if (scratch_bytes < bpd_op_vocab_argmax_scratch_bytes(rows, d, vocab, dtype)) return fail(BPD_E_NOMEM, "scratch too small");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* p = static_cast<char*>(scratch);
  if (op_use_tc(dtype)) {
    const OpScratch L = op_scratch_layout(rows, d, vocab);
    BPD_CUDA(cudaMemsetAsync(p, 0, L.total, st));
    tc::Scratch sc{reinterpret_cast<float*>(p + L.ws_off), L.ws_floats, reinterpret_cast<unsigned*>(p + L.cnt_off),
                   L.n_counters, reinterpret_cast<unsigned*>(p + L.done_off),
                   reinterpret_cast<unsigned long long*>(p + L.pv_off), L.part_elems, reinterpret_cast<int*>(p + L.err_off), 0, 1};
    tc::Operands op{w, vocab, x, 0, d, rows, d, p + L.zero_off};   // the lo plane is the scratch's zero block
    tc::TcParams tp;
    memset(&tp, 0, sizeof(tp));
    tp.out_idx = out_idx; tp.out_val = out_val;
    int rc = tc::launch<tc::kTcArgmax>(op, vocab, d, rows, tp, sc, st);
    if (rc) return rc;
    ++g_launches;
    return op_tc_finish(p, L, st);
  }
  const size_t tiles = ceil_div(vocab, kVocTile);
  float* pv = reinterpret_cast<float*>(p);
  p += align_up(tiles * rows * sizeof(float));
  int* pi = reinterpret_cast<int*>(p);
  p += align_up(tiles * rows * sizeof(int));
  unsigned* cnt = reinterpret_cast<unsigned*>(p);
  BPD_CUDA(cudaMemsetAsync(cnt, 0, (ceil_div(rows, kRC) + 1) * sizeof(unsigned), st));
  if (dtype == 0) launch_vocab_argmax<float, float>(x, w, rows, d, vocab, pv, pi, cnt, out_idx, out_val, nullptr, nullptr, st);
  else launch_vocab_argmax<bf16, bf16>(x, w, rows, d, vocab, pv, pi, cnt, out_idx, out_val, nullptr, nullptr, st);
  BPD_CUDA(cudaGetLastError());
  return BPD_OK;
}

size_t bpd_op_linear_scratch_bytes(int rows, int in_f, int out_f, int dtype) {
  if (rows < 1 || in_f < 1 || out_f < 1) return 0;
  if (op_use_tc(dtype)) return op_scratch_layout(rows, in_f, out_f).total;
  return 256;
}

int bpd_op_linear(const void* x, const void* w, const void* bias, int rows, int in_f, int out_f, int dtype, int relu,
                  void* scratch, size_t scratch_bytes, float* y, void* cuda_stream) {
  if (!x || !w || !y) return fail(BPD_E_INVALID, "null argument");
  if (rows < 1 || out_f < 1 || in_f < 8 || in_f % 8) return fail(BPD_E_SHAPE, "rows/in_f/out_f out of range (in_f must be a multiple of 8)");
  if (dtype != 0 && dtype != 1) return fail(BPD_E_INVALID, "unknown dtype %d", dtype);
  if ((uintptr_t)x % 16 || (uintptr_t)w % 16) return fail(BPD_E_INVALID, "misaligned pointer");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (op_use_tc(dtype)) {
    if (!scratch || (uintptr_t)scratch % 256) return fail(BPD_E_INVALID, "scratch is null or misaligned");
    const OpScratch L = op_scratch_layout(rows, in_f, out_f);
    if (scratch_bytes < L.total) return fail(BPD_E_NOMEM, "scratch too small");
    char* p = static_cast<char*>(scratch);
    BPD_CUDA(cudaMemsetAsync(p, 0, L.total, st));
    tc::Scratch sc{reinterpret_cast<float*>(p + L.ws_off), L.ws_floats, reinterpret_cast<unsigned*>(p + L.cnt_off),
                   L.n_counters, reinterpret_cast<unsigned*>(p + L.done_off),
                   reinterpret_cast<unsigned long long*>(p + L.pv_off), L.part_elems, reinterpret_cast<int*>(p + L.err_off), 0, 1};
    tc::Operands op{w, out_f, x, 0, in_f, rows, in_f, p + L.zero_off};   // the lo plane is the scratch's zero block
    tc::TcParams tp;
    memset(&tp, 0, sizeof(tp));
    tp.bias = static_cast<const bf16*>(bias); tp.relu = relu; tp.out_f32 = y; tp.ldo = out_f;
    int rc = tc::launch<tc::kTcF32>(op, out_f, in_f, rows, tp, sc, st);
    if (rc) return rc;
    ++g_launches;
    return op_tc_finish(p, L, st);
  }
  LinearParams p = lin(x, in_f, w, in_f, out_f, bias, rows, y, out_f, relu, nullptr);
  if (dtype == 0) launch_linear<float, float, kEpiStoreF32>(p, 1, st);
  else launch_linear<bf16, bf16, kEpiStoreF32>(p, 1, st);
  BPD_CUDA(cudaGetLastError());
  return BPD_OK;
}

}  // extern "C"
