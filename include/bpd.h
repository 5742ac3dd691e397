/*
 * bpd.h -- C ABI of the blockwise-parallel-decoding library for NVIDIA B200 (sm_100a).
 *
 * The library runs the merged score-and-propose iteration of blockwise parallel
 * decoding (Stern, Shazeer, Uszkoreit 2018, Sections 3, 4 and 6) on one GPU:
 * a KV-cached Transformer decoder pass over the k proposed positions, the k
 * proposal heads at every position, a fused top-1 over the vocabulary, the
 * longest-prefix verification and the cache commit.
 *
 * Conventions
 *  - Every function returns BPD_OK (0) or a negative bpd_status.  Nothing throws,
 *    aborts or exits.  bpd_last_error() returns a thread-local message for the
 *    last failing call on this thread.
 *  - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global
 *    memory of the current device.  The caller owns every buffer it passes and
 *    keeps it alive as long as the model / session that was given it.
 *  - The library allocates no device memory.  Weights live in a caller-provided
 *    device buffer (bpd_load_weights), all per-session state (encoder memory,
 *    paged KV cache, activations, reduction workspace) in another one
 *    (bpd_session_create); bpd_query_sizes tells how large they must be.
 *  - `cuda_stream` arguments are a cudaStream_t passed as void*; all work of a
 *    model / session is issued on the stream given at creation.
 *  - Token ids are int32.  Decoder input u_0 is id 0 (start); positions count
 *    from 0.  eos_id = -1 selects fixed-length termination (Section 2: language
 *    tasks stop at an end-of-sequence token, image tasks after a fixed number of
 *    steps).
 *  - Argmax ties go to the lowest id.
 */
#ifndef BPD_H_
#define BPD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BPD_OK = 0,
  BPD_E_INVALID = -1,     /* null pointer or argument out of range              */
  BPD_E_SHAPE = -2,       /* sizes inconsistent with the model / session         */
  BPD_E_FORMAT = -3,      /* malformed weight blob                               */
  BPD_E_NOMEM = -4,       /* a caller-provided buffer is too small               */
  BPD_E_STATE = -5,       /* call out of order (e.g. decode before encode)       */
  BPD_E_CUDA = -6,        /* a CUDA runtime call failed; message has the detail  */
  BPD_E_TIMEOUT = -7,     /* a bounded device-side wait expired                  */
  BPD_E_UNSUPPORTED = -8  /* valid request this build does not implement         */
} bpd_status;

typedef struct bpd_model bpd_model;     /* opaque: parsed config + device weight pointers  */
typedef struct bpd_session bpd_session; /* opaque: B rows of decode state in device memory */

/* Acceptance criteria for the Verify substep (the accept_mode argument).
 * Whatever the criterion, the token that is kept is the proposal (Section 3,
 * Accept).  BPD_ACCEPT_MIN_BLOCK(l) may be OR-ed in: at least l proposals are
 * taken per iteration regardless of the criterion (Section 5.3). */
enum {
  BPD_ACCEPT_EXACT = 0     /* Section 3: proposal == argmax p_1; the output equals greedy decoding */
};
#define BPD_ACCEPT_TOPN(n)       ((1 << 8) | ((n) & 0xff))    /* Section 5.1: proposal among the n best of p_1, 1 <= n <= 255 */
#define BPD_ACCEPT_DISTANCE(eps) ((2 << 8) | ((eps) & 0xff))  /* Section 5.2: |proposal - argmax p_1| <= eps (intensities)  */
#define BPD_ACCEPT_MIN_BLOCK(l)  (((l) & 0xff) << 16)         /* Section 5.3: 1 <= l <= k                                   */

#define BPD_MAX_K 16       /* largest block size / number of proposal heads */

/* Decode statistics.  "iterations" are score-and-propose passes (the priming
 * pass is not one); "invocations" = iterations + priming passes, the paper's
 * model-invocation count (Section 4: m/k + 1 in the best case).  Mean accepted
 * block size = tokens / iterations, summed over rows. */
typedef struct {
  int64_t tokens;                  /* tokens emitted, all rows                          */
  int64_t iterations;              /* passes of the slowest row                         */
  int64_t invocations;             /* model passes launched                             */
  int64_t row_iterations;          /* sum over rows of iterations that row took part in */
  int64_t khat_hist[BPD_MAX_K + 1];/* khat_hist[c] = (row, iteration) pairs accepting c */
  double  device_ms;               /* CUDA-event time of the decode loop                */
} bpd_stats;

/* Result of one bpd_iteration call.  Host arrays are filled when non-NULL
 * (the call then synchronises); device dumps are written when non-NULL. */
typedef struct {
  int32_t* khat;         /* host [B]       accepted block size (0 for finished rows)             */
  int32_t* accepted;     /* host [B,k]     accepted tokens, -1 beyond khat                       */
  int32_t* table;        /* host [B,k,k]   table[b][r][i] = argmax of head i+1 at block position r */
  int32_t* next_block;   /* host [B,k]     proposals for the next iteration (row khat of table)  */
  int32_t* block;        /* host [B,k]     the proposals this iteration scored                   */
  float*   logits_dev;   /* device [B,k,k,V] fp32 logits of every head at every position, or NULL */
  float*   hidden_dev;   /* device [B,k,d]   fp32 decoder outputs (after the final norm), or NULL  */
  float*   layers_dev;   /* device [n_dec,B,k,d] fp32 residual stream after every decoder layer
                            (before the final norm), or NULL; for parity debugging             */
} bpd_iter_out;

/* Execution strategies a session may use.  They change how the passes are
 * scheduled on the GPU, never what is computed: every combination decodes the
 * same tokens (sums are split differently, so hidden states agree to fp32
 * rounding).  Each field: -1 = the library's choice for this model and batch,
 * 0 = off, 1 = on where the shapes allow it.  Initialise with
 * bpd_session_options_init and change what you need. */
typedef struct {
  int32_t struct_bytes;       /* sizeof(bpd_session_options), set by bpd_session_options_init              */
  int32_t tensor_cores;       /* bf16 models: tcgen05 / TMA projection kernels (0: CUDA-core kernels)       */
  int32_t cuda_graphs;        /* replay each pass as a CUDA graph (needs a non-default stream)              */
  int32_t dependent_launch;   /* programmatic dependent launch between the kernels of a pass               */
  int32_t lazy_heads;         /* two-stage heads: p_1 at all k positions, all heads only at the accepted
                                 one (default: on when batch * k_model >= 64)                              */
  int32_t fold_layer_norms;   /* decoder layer norms folded into the projections after them (<= 16 rows)   */
  int32_t cluster_layers;     /* decoder layers as three cluster launches each (<= 16 rows per pass)        */
  int32_t persistent_layers;  /* all decoder layers of a pass in one persistent TMA-fed kernel (<= 16 rows
                                 per pass, d_model 256 / 512 / 1024; takes precedence over cluster_layers).
                                 Default: on for sessions of at most 256 positions whose encoder rows fit
                                 the staging tile (measured faster there) while no other live session of
                                 the device has it, off elsewhere; 1 asks for it wherever it runs.  See
                                 bpd_session_create_opt for what it needs                                  */
  int32_t stage_encoder_rows; /* encoder keys / values staged in shared memory for cross-attention          */
  int32_t l2_stream_hints;    /* weights read once per pass are loaded "evict first"                        */
} bpd_session_options;

/* ---- set-up ------------------------------------------------------------- */

/* Sizes of the two device buffers the caller must provide.
 * blob: host, the weight container (self-describing header, then tensors).
 * weight_bytes / session_bytes: host outputs, either may be NULL. */
int bpd_query_sizes(const void* blob, size_t blob_bytes, int batch, int max_src, int max_tgt,
                    size_t* weight_bytes, size_t* session_bytes);

/* session_bytes for an already loaded model (same value bpd_query_sizes gives). */
int bpd_session_bytes(const bpd_model* model, int batch, int max_src, int max_tgt, size_t* session_bytes);

/* Which form the session's decoder layers take: 0 = one kernel per projection, 1 = three cluster launches per
 * layer, 2 = one persistent kernel per pass.  The options of bpd_session_create_opt are requests: a shape or a
 * device that a form does not take falls back to the next one, and this call tells.  Negative on a null handle. */
int bpd_session_layer_path(const bpd_session* s);

/* Copy the blob's tensors into dev_weight_buf (device, 256-byte aligned,
 * >= weight_bytes) and return a model handle.  The blob may be freed after the
 * call returns (the call synchronises the stream). */
int bpd_load_weights(const void* blob, size_t blob_bytes, void* dev_weight_buf, size_t dev_bytes,
                     void* cuda_stream, bpd_model** out);

/* Lay a session of `batch` rows out in dev_session_buf (device, 256-byte
 * aligned, >= session_bytes for these arguments).  max_src bounds the source
 * length, max_tgt the number of decoded tokens per row. */
int bpd_session_create(const bpd_model* model, int batch, int max_src, int max_tgt,
                       void* dev_session_buf, size_t dev_bytes, void* cuda_stream, bpd_session** out);

/* The same with explicit options (NULL = all defaults).  A session that runs
 * its decoder layers in the persistent kernel (persistent_layers; see
 * bpd_session_layer_path) occupies most of the GPU with CTAs that wait for
 * one another: passes of two such sessions must not overlap on one GPU (keep
 * them on one stream, or finish one decode before starting another); if they
 * do, their bounded waits expire after about a second and the calls return
 * BPD_E_TIMEOUT.  Left to the library (the default), at most one live session
 * per device gets the persistent kernel -- a session created while another
 * holds it runs the cluster launches, which may overlap with anything -- so
 * only sessions that ask for it with persistent_layers = 1 can meet this. */
void bpd_session_options_init(bpd_session_options* options);
int bpd_session_create_opt(const bpd_model* model, int batch, int max_src, int max_tgt,
                           void* dev_session_buf, size_t dev_bytes, void* cuda_stream,
                           const bpd_session_options* options, bpd_session** out);

int bpd_session_destroy(bpd_session* s);
int bpd_model_destroy(bpd_model* m);
const char* bpd_last_error(void);

/* ---- the decoding path (Sections 2-4) ------------------------------------ */

/* Run the encoder over the source rows, fill the cross-attention keys/values
 * of every decoder layer, and reset all rows to "nothing decoded".
 * src_ids: host [batch, max_src] (row b valid in [0, src_len[b]), rest ignored);
 * src_len: host [batch], 1 <= src_len[b] <= max_src. */
int bpd_encode(bpd_session* s, const int32_t* src_ids, const int32_t* src_len);

/* Greedy decoding (Section 2): one decoder pass per token, head p_1 only.
 * out_ids: host [batch, max_new] or NULL; out_len: host [batch] or NULL.  When
 * out_ids is NULL the call only enqueues the work and results stay on the
 * device (bpd_fetch_output reads them).  stats may be NULL. */
int bpd_decode_greedy(bpd_session* s, int max_new, int32_t eos_id,
                      int32_t* out_ids, int32_t* out_len, bpd_stats* stats);

/* Blockwise parallel decoding with the combined model (Sections 3 and 4): a
 * priming pass, then merged verify+predict iterations until every row has
 * max_new tokens or has accepted eos_id.  1 <= k <= k_model uses the first k
 * heads.  Output arguments as for bpd_decode_greedy. */
int bpd_decode_blockwise(bpd_session* s, int k, int accept_mode, int max_new, int32_t eos_id,
                         int32_t* out_ids, int32_t* out_len, bpd_stats* stats);

/* Blockwise parallel decoding in its two-call form (Section 3: predict,
 * verify, accept), kept for comparison with the merged form of Section 4:
 * every iteration is a Verify invocation (p_1 alone at the k block positions,
 * followed by acceptance and the cache commit) and a Predict invocation (all
 * k heads at the last accepted token, whose position is recomputed).  The
 * ids and accepted block sizes are those of bpd_decode_blockwise; the number
 * of model invocations is 2 per iteration instead of 1 per iteration + 1
 * (stats->invocations), which is why the merged form is the product path.
 * Arguments, outputs, forced plans and error behaviour as for
 * bpd_decode_blockwise. */
int bpd_decode_blockwise_twocall(bpd_session* s, int k, int accept_mode, int max_new, int32_t eos_id,
                                 int32_t* out_ids, int32_t* out_len, bpd_stats* stats);

/* One merged score-and-propose iteration (Section 4) on the session's current
 * state; on a freshly encoded session the priming pass runs first.
 * forced_tail: host [batch, k-1] replacing proposals 2..k of every row, or
 * NULL.  Proposal 1 is never replaced: it is p_1's own argmax (Section 3, the
 * remark that khat >= 1).  max_new / eos_id bound acceptance as in the decode
 * calls.  out may be NULL (no synchronisation then). */
int bpd_iteration(bpd_session* s, int k, int accept_mode, int max_new, int32_t eos_id,
                  const int32_t* forced_tail, bpd_iter_out* out);

/* Controlled acceptance: install (plan != NULL) or clear (NULL) a table of
 * forced proposal tails, host [batch, plan_len, k-1]: an iteration of row b
 * that starts with j tokens accepted (j < plan_len) replaces its proposals
 * 2..k by plan[b][j][:].  Stays in force for bpd_decode_blockwise and
 * bpd_iteration (when that is given no forced_tail) until cleared or until
 * the next bpd_encode.  Needs plan_len <= max_tgt and k <= k_model. */
int bpd_set_forced_plan(bpd_session* s, const int32_t* plan, int plan_len, int k);

/* Forget everything decoded (rows back to "nothing decoded") but keep the
 * encoder memory and any forced plan: the state bpd_encode leaves, without
 * running the encoder again.  Asynchronous. */
int bpd_rewind(bpd_session* s);

/* Copy the tokens decoded so far to the host (synchronises).
 * out_ids: host [batch, max_new]; out_len: host [batch] (either may be NULL). */
int bpd_fetch_output(bpd_session* s, int max_new, int32_t* out_ids, int32_t* out_len, bpd_stats* stats);

/* ---- instrumentation ------------------------------------------------------ */

/* Number of CUDA kernels this library has launched in this process so far. */
long long bpd_kernel_launches(void);

/* Per-phase device timing of the decoder pass.  bpd_profile(s, 1) clears the
 * record and makes every following pass bracket four phases with CUDA events on
 * the session's stream; bpd_profile(s, 0) stops.  bpd_profile_read returns how
 * many times `phase` ran and the summed device time.  Phases: 0 = embedding,
 * decoder layers and final norm; 1 = head hidden layer; 2 = head output layers
 * (+ residual); 3 = vocabulary projection with top-1; for bf16 models also the
 * individual kernels inside phase 0: 4 = embedding, 5 = layer norms, 6 = QKV
 * projection, 7 = self-attention, 8 = output projection, 9 = cross-attention
 * query projection, 10 = cross-attention, 11 = cross-attention output
 * projection, 12 / 13 = feed-forward layers 1 / 2, 14 = verify and commit. */
int bpd_profile(bpd_session* s, int enable);
int bpd_profile_read(bpd_session* s, int phase, int64_t* launches, double* total_ms);

/* Self test of the bounded device-side waits: launches one CTA that waits on a
 * barrier nothing ever arrives on, then one that waits for tagged words nobody
 * writes (the two kinds of wait the kernels have), each with a limit of about
 * limit_us microseconds.  The waits give up, the kernels record their error words
 * and return normally, and the call reports BPD_E_TIMEOUT -- the status a real
 * decode call returns if one of its kernels' waits ever expires.  BPD_OK or
 * BPD_E_CUDA would mean that a wait did not expire the way it should.
 * dev_word: device int32 used as the error word.  Synchronises the stream. */
int bpd_debug_wait_timeout(int32_t* dev_word, int limit_us, void* cuda_stream);

/* ---- single operators (used by tests and profiling) ----------------------- */

/* Top-1 of a vocabulary projection without materialising logits (Section 4's
 * "k separate softmaxes per position", of which only the argmax is needed):
 * out_idx[r] = argmin-id argmax_v sum_c x[r][c] * w[v][c].
 * x: device [rows, d]; w: device [vocab, d]; both of `dtype` (0 = float32,
 * 1 = bfloat16), row-major.  scratch: device workspace of at least
 * bpd_op_vocab_argmax_scratch_bytes(rows, d, vocab, dtype) bytes.
 * out_idx: device int32 [rows]; out_val: device float [rows] or NULL. */
size_t bpd_op_vocab_argmax_scratch_bytes(int rows, int d, int vocab, int dtype);
int bpd_op_vocab_argmax(const void* x, const void* w, int rows, int d, int vocab, int dtype,
                        void* scratch, size_t scratch_bytes, int32_t* out_idx, float* out_val,
                        void* cuda_stream);

/* The same top-1 for callers that cannot hand over a workspace and must not
 * trigger a device allocation: code running under a framework that has already
 * claimed the whole GPU for its own pool, a serving loop that cannot afford the
 * device-wide synchronisation an allocation may cause, or a plug-in callback
 * that is only allowed to enqueue work.  (The paper has no counterpart; this is
 * a deployment convenience.)  The cross-CTA reduction workspace is a fixed
 * 512 KiB array inside the library image, resident on every GPU that loads the
 * library until the process exits.  Limits: rows <= 256, vocab <= 65536
 * (beyond them the call returns BPD_E_NOMEM) and d <= 1024, a multiple of 8
 * (BPD_E_SHAPE, as for bpd_op_vocab_argmax); a refused call leaves the outputs
 * untouched.  Arguments as bpd_op_vocab_argmax, minus the scratch.
 * The call performs no cudaMalloc/cudaFree and uses no allocating library.
 * The first call on each device is a set-up call: it looks the array's device
 * address up (with that device current), and, as with any kernel, the CUDA
 * driver loads the kernel's code when a data type is first launched (memory of
 * the driver's own: about 2 MiB in a fresh process) -- make one call per device
 * and data type at start-up, outside any stream capture; from then on the
 * device's free memory stays exactly as it is across calls.  All calls
 * share the one array: the call clears the arrival counters it needs, but two
 * calls whose kernels may overlap on the GPU (different streams, or different
 * host threads) race on it -- keep them on one stream or serialise them. */
int bpd_op_vocab_argmax_noalloc(const void* x, const void* w, int rows, int d, int vocab, int dtype,
                                int32_t* out_idx, float* out_val, void* cuda_stream);

/* y[r][n] = act(sum_c x[r][c] * w[n][c] + bias[n]); the projection used by every
 * layer.  x: device [rows, in_f] `dtype`; w: device [out_f, in_f] `dtype`; bias:
 * device [out_f] `dtype` or NULL; y: device [rows, out_f] float32; relu != 0
 * applies max(0, .).  scratch as above (bpd_op_linear_scratch_bytes). */
size_t bpd_op_linear_scratch_bytes(int rows, int in_f, int out_f, int dtype);
int bpd_op_linear(const void* x, const void* w, const void* bias, int rows, int in_f, int out_f,
                  int dtype, int relu, void* scratch, size_t scratch_bytes, float* y,
                  void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* BPD_H_ */
