// Host-side structures behind the opaque handles of bpd.h.
#pragma once
#include <cuda_runtime.h>
#include <stdarg.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <map>
#include <string>
#include <tuple>
#include <vector>

#include "../../include/bpd.h"
#include "common.cuh"

namespace bpd {

extern thread_local char g_err[512];
extern std::atomic<long long> g_launches;   // kernels launched by this library in this process
int fail(int code, const char* fmt, ...);

#define BPD_CUDA(expr)                                                                   \
  do {                                                                                   \
    cudaError_t e__ = (expr);                                                            \
    if (e__ != cudaSuccess)                                                              \
      return bpd::fail(BPD_E_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), \
                       __FILE__, __LINE__);                                              \
  } while (0)

// Launch with (pdl = true) or without the programmatic-stream-serialization attribute: with it the kernel
// may begin while its predecessor in the stream is still running (it must call pdl_wait() on the device
// before touching anything the predecessor produces).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                            Args&&... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Opt-in dynamic shared-memory limit of a kernel: only ever raised, tracked per (device, kernel), so that
// sessions of different models and several devices in one process cannot lower or miss each other's limit.
int ensure_smem_limit(const void* kernel, size_t bytes);

struct Config {
  int dtype, n_enc, n_dec, d, H, d_ff, V, k_model, d_hidden, head_layout, p1_identity;
  int local_q, local_m;    // decoder self-attention: 0 = all earlier positions; else 1D local attention
  float eps;
  int elem() const { return dtype == 0 ? 4 : 2; }
};

struct TensorEntry {
  int ndim;
  int dims[3];
  uint64_t offset, nbytes;
};

struct ParsedBlob {
  Config cfg;
  std::map<std::string, TensorEntry> t;
  uint64_t total;
};
int parse_blob(const void* blob, size_t n, ParsedBlob* out);

struct EncLayer {
  const void *ln1g, *ln1b, *wqkv, *wo, *ln2g, *ln2b, *w1, *b1, *w2, *b2;
};
struct DecLayer {
  const void *ln1g, *ln1b, *wqkv, *wo, *ln2g, *ln2b, *cwq, *cwkv, *cwo, *ln3g, *ln3b, *w1, *b1, *w2, *b2;
  // layer norms folded into the projections that follow them (bf16 models): per-feature s and c vectors
  float *s_qkv, *c_qkv, *s_cq, *c_cq, *s_f1, *c_f1;
};

}  // namespace bpd

struct bpd_model {
  bpd::Config cfg;
  char* base;            // device weight buffer
  size_t bytes;
  cudaStream_t stream;
  const void *src_embed, *tgt_embed, *out_proj;
  std::vector<bpd::EncLayer> enc;
  std::vector<bpd::DecLayer> dec;
  const void *enc_lnf_g, *enc_lnf_b, *dec_lnf_g, *dec_lnf_b;
  const void *head_w1, *head_b1, *head_w2, *head_b2;
};

typedef std::tuple<int, int, int, int, const void*, int, int, int, int, const void*, int> GraphKey;
struct GraphEntry {
  int uses = 0;
  long long launches = 0;
  cudaGraphExec_t exec = nullptr;
};

enum ProfSlot { kProfLayers = 0, kProfHeadW1 = 1, kProfHeadW2 = 2, kProfVocab = 3,
                kProfEmbed = 4, kProfLn = 5, kProfQkv = 6, kProfSelfAttn = 7, kProfOproj = 8, kProfCrossQ = 9,
                kProfCrossAttn = 10, kProfCrossO = 11, kProfFfn1 = 12, kProfFfn2 = 13, kProfVerify = 14, kProfSlots = 15 };

enum SessionPhase { kPhaseCreated = 0, kPhaseEncoded = 1, kPhaseBlockwise = 2, kPhaseGreedy = 3 };

struct bpd_session {
  const bpd_model* m;
  int B, max_src, max_tgt, ppr;
  char* base;
  size_t bytes;
  cudaStream_t stream;
  int phase;
  // activations
  float *x, *h_f32, *pe;
  int npos;
  void *xn, *qbuf, *attn, *ffh, *u, *o;
  std::vector<void*> crosskv, kcache, vcache;
  // integers
  bpd::RowState st;
  bpd::RankState rank;
  int *src_dev, *tail_dev, *plan_dev;
  int plan_len, plan_k;    // 0 when no plan installed
  // vocabulary top-1 workspace
  float* part_val;
  int* part_idx;
  size_t part_elems;
  unsigned* counters;
  // tensor-core path (bf16 models): activations feeding a projection are two bf16 planes (hi + lo)
  int tc;
  long long pl_xn, pl_attn, pl_ffh, pl_u, pl_o;   // elements between the planes of each buffer
  int rows_all, rows_dec, rows_head;              // allocated rows of xn/attn/ffh, of u, of o
  float* tc_ws; size_t tc_ws_floats;
  unsigned* tc_counters; size_t tc_n_counters;
  unsigned* tc_done;
  unsigned long long* tc_best; size_t tc_best_elems;
  // host side
  int* pinned;             // pinned ring of all_done flags + staging
  cudaEvent_t ev_flag[8];
  int epoch;               // decodes started on this session (the verify kernel tags its reports with it)
  cudaEvent_t ev0, ev1;
  int timed;               // ev0 / ev1 bracket a finished decode loop
  int64_t invocations;
  int profiling;
  int use_graphs;
  int use_pdl;
  int lazy_heads;          // two-stage head evaluation (p_1 everywhere, all heads only at the accepted position)
  int last_pass_lazy;
  void* u2; long long pl_u2; float* h2; int *table2, *table_full;
  int fold_ln;             // decoder layer norms are folded into the projections that follow them
  float* ln_stats;         // [d / 128][rows][2]: per-tile mean and squared deviations of the residual stream (passes of more than 16 rows)
  int fused;               // decoder layers as three launches each (clusters; at most 16 rows per pass)
  float* fused_ws;
  unsigned* fused_counters;
  // the whole layer stack as one persistent kernel (see layer_stack.cuh); 0 when the shapes or the device's
  // cluster occupancy do not allow it
  struct { int persistent_layers, stage_encoder_rows, l2_stream_hints; } opt;   // resolved session options
  int stack;
  unsigned char stack_maps[8 * 128] __attribute__((aligned(64)));   // stack::StackMaps (eight tensor maps over all layers)
  void* stack_layers;      // device: stack::LayerPtrs [n_dec]
  unsigned long long* stack_ws;   // device: [2][H][16][d] words (value, tag): the clusters' shares of the projection outputs
  unsigned* stack_bar;     // device: words of the device-wide join
  float* stack_dump;       // device: [n_dec][rows][d] residual stream after every layer (debug dump), or null
  int stack_cross_rows, stack_long, stack_minb, stack_dev;
  int stack_layout[24];    // stack::Layout, kept opaque here
  std::map<GraphKey, GraphEntry> graphs;
  GraphEntry enc_graph;    // the encoder's launch sequence (fixed for a session), captured on its second use
  std::vector<cudaEvent_t> prof_begin[kProfSlots], prof_end[kProfSlots];
};
