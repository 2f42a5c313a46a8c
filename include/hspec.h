/*
 * hspec.h — C ABI of the H-Spec block-parallel draft step on one B200 (sm_100a).
 *
 * One call of hspec_draft_block runs, for B concurrent requests, one forward pass of
 * the hybrid Mamba-attention drafter of the paper (Sec. 3.3, App. B.1):
 *   last-position target hidden state -> Proj_r -> Proj_dS -> S_init   (Sec. 3.3.1, eq. for S_init)
 *   k block rows (last token, then mask tokens; no positional embedding) (Sec. 3.3.1, "Input-dependent selectivity")
 *   per layer: Mamba-2 mixer scanned over the k rows from S_init          (Sec. 3.3.1)
 *              attention whose keys/values are the target model's own paged KV cache, read
 *              in place, plus the block's causal keys/values              (Sec. 3.3.2)
 *              SwiGLU MLP                                                 (App. B.1 "MLP")
 *   final norm, the target's LM head, arg-max -> k draft tokens           (App. B.2 "Pruned drafter vocabulary": LM head is the target's)
 *   optionally (markov_rank > 0) the causal-correction head between the LM head and the arg-max: a rank-r first-order
 *   dependency between adjacent positions, applied position by position  (Sec. 3.3.3; see hspec_op_markov_head)
 * No drafter-side KV cache exists: the library never writes the KV pools (Sec. 3.2).
 *
 * Precision
 *   Weights arrive as bf16.  hspec_load_weights keeps its own device copy of every tensor; matrices that feed
 *   a tensor-core GEMM are widened once to fp16 (bf16 has 8 significant bits, fp16 has 11: the conversion is
 *   exact for 2^-17 <= |w| <= 65504 and loses at most 2^-25 below that).  Activations the library produces
 *   and feeds to a GEMM (norm outputs, the gated SSM output, the attention output, the SwiGLU product, the
 *   fusion vector, S_init) are fp16 as well, because the MMA needs both operands in one 16-bit type and
 *   bf16 activations (8 bits) put the step's rounding noise at ~3e-2 of the output RMS over a full logits
 *   tensor, above the 2e-2 parity bound.  Accumulation is fp32; the residual stream, scan and softmax are
 *   fp32.  The target's KV pools are read in place as bf16, so q, the block's k/v and the softmax weights
 *   enter the attention MMAs as bf16.
 *   Range: fp16 ends at 65504.  |last_hidden| and every GEMM input the library forms must stay below that; a finite
 *   value beyond it is CLAMPED to +-65504 at the store (never turned into inf) and counted, and hspec_get_stats then
 *   returns HSPEC_ERR_F16_RANGE with the count in f16_range_events.  A target whose hidden states carry outlier channels
 *   above 65504 needs them scaled by the caller (Proj_r is linear: scale last_hidden by s and proj_r by 1/s).
 *
 * Conventions
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are
 *     ordinary host memory.  No torch / C++ types cross this boundary.
 *   - All matrices are row-major [out_features, in_features] bf16; vectors are fp32.
 *   - Every function returns HSPEC_OK (0) or a negative hspec_status; nothing throws or aborts.
 *     hspec_last_error() returns a static or per-handle message for the last failure.
 *   - Work is enqueued on the caller's stream; hspec_draft_block performs no host synchronisation.
 *     Asynchronous device faults surface through the CUDA runtime on the caller's next sync;
 *     bounded in-kernel waits that give up set a device status word readable with hspec_get_stats.
 *   - A library built without a usable CUDA device fails loudly (HSPEC_ERR_CUDA): there is no CPU path.
 */
#ifndef HSPEC_H_
#define HSPEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HSPEC_MAX_LAYERS 16
#define HSPEC_MAX_SLOTS 16
#define HSPEC_MAX_K 32            /* block positions per step */

typedef enum {
  HSPEC_OK = 0,
  HSPEC_ERR_INVALID_ARG = -1,        /* NULL pointer, bad handle, B/k out of range */
  HSPEC_ERR_BAD_SHAPE = -2,          /* config or tensor shape the kernels cannot take */
  HSPEC_ERR_NOT_LOADED = -3,         /* a required weight tensor was never loaded */
  HSPEC_ERR_WORKSPACE_TOO_SMALL = -4,
  HSPEC_ERR_PAGE_OUT_OF_RANGE = -5,  /* a page id outside [0, num_pages) or a context length outside [0, max_ctx]: found by the
                                        host-side validation (HSPEC_DEBUG=1, before anything is enqueued) or met by a kernel,
                                        which clamps the length, reads the page as zeros and counts the event */
  HSPEC_ERR_CUDA = -6,               /* a CUDA runtime / driver call failed (message has the text) */
  HSPEC_ERR_TIMEOUT = -7,            /* a bounded in-kernel wait gave up (status word) */
  HSPEC_ERR_F16_RANGE = -8           /* finite values beyond +-65504 reached an fp16 store and were clamped (counted) */
} hspec_status;

typedef enum { HSPEC_BF16 = 0, HSPEC_F32 = 1, HSPEC_I32 = 2, HSPEC_F16 = 3 } hspec_dtype;

/* Shapes of the drafter (App. B.1).  H = Di / P Mamba heads; d_S = H * P * N. */
typedef struct {
  int32_t D;                 /* hidden size of target and drafter */
  int32_t n_fuse;            /* number of target layers whose last-position hidden states are concatenated */
  int32_t r;                 /* fusion rank of Proj_r (the paper sets it to D) */
  int32_t L;                 /* drafter layers, <= HSPEC_MAX_LAYERS */
  int32_t has_attn[HSPEC_MAX_LAYERS]; /* 1: Mamba-attention-MLP layer, 0: Mamba-MLP layer */
  int32_t kv_slot[HSPEC_MAX_LAYERS];  /* which target-layer KV pool layer l's attention reads (layer-wise KV mapping) */
  int32_t n_slots;           /* number of distinct target KV pools passed per step */
  int32_t Di, P, N, G;       /* Mamba-2: inner width, head dim, state dim, B/C groups */
  int32_t d_conv;            /* depthwise conv width (<= 4) */
  int32_t dt_rank;           /* 0: dt projected directly to H; >0: through a rank-dt_rank bottleneck */
  int32_t Hq, Hkv, dh;       /* attention heads (= the target's), head dim (64 or 128) */
  float rope_theta;          /* the target's RoPE base */
  int32_t window;            /* sliding window in tokens, 0 = full context */
  int32_t qk_norm;           /* 1: per-head RMSNorm on q and the block's k before RoPE */
  int32_t F;                 /* SwiGLU width */
  int32_t V;                 /* target vocabulary (rows of `embed`; of `lm_head` too unless V_draft > 0) */
  int32_t V_draft;           /* 0, or the size of a pruned drafter vocabulary (App. B.2 "Pruned drafter vocabulary"): the LM
                                head then has V_draft rows and `vocab_map` translates a row index into a target token id */
  int32_t mask_id;           /* token id whose embedding fills block rows 1..k-1 */
  float rms_eps;
  int32_t page_size;         /* tokens per KV page (16) */
  int32_t max_batch;         /* largest B a step may carry */
  int32_t max_k;             /* largest k a step may carry, <= HSPEC_MAX_K */
  int32_t max_pages_per_req; /* largest page-table row length (bounds the context) */
  int32_t markov_rank;       /* 0, or the rank of the causal-correction head applied after the LM head (Sec. 3.3.3; 256 in
                                App. B.1): tensors `markov_in` [V, rank] and `markov_out` [V or V_draft, rank] are then
                                required and the draft ids follow hspec_op_markov_head's rule */
  int32_t act_bf16;          /* 0 (default): fp16 tensor-core operands, see "Precision".  1: bf16 operands - the GEMM
                                matrices are used where the caller put them (no library copy, except w_gate_up, whose rows
                                the fused SwiGLU epilogue needs interleaved), activations are stored as bf16; no fp16
                                range limit, but 8 instead of 11 significant bits on every GEMM input (measured on the
                                mid-size test step: 2.0e-2 of the hidden state's RMS and 2.3e-2 of the logits' RMS at the
                                maximum, against 4.6e-3 and 5.0e-3 with fp16 operands) */
} hspec_config;

/* A named tensor in DEVICE memory.  hspec_load_weights copies it (converting GEMM matrices to fp16), so
 * the caller may free or reuse it afterwards - except with act_bf16 = 1, where the bf16 GEMM matrices are BORROWED:
 * they must stay valid and unchanged until hspec_destroy.  Names (l = layer index):
 *   embed [V,D]  proj_r [r, n_fuse*D]  proj_ds [H*P*N, r]  final_norm [D]  lm_head [V,D] (or [V_draft,D])
 *   vocab_map [V_draft] int32 (only if V_draft > 0: target token id of each LM-head row, ascending)
 *   markov_in [V, markov_rank]  markov_out [V or V_draft, markov_rank]  (only if markov_rank > 0)
 *   layers.l.mamba.{norm [D], in_proj [Di + (Di+2GN) + (dt_rank or H), D] (rows z | xBC | dt),
 *                   dt_up [H, dt_rank] (only if dt_rank>0), conv_w [Di+2GN, d_conv], conv_b [Di+2GN],
 *                   dt_bias [H], A_log [H], Dskip [H], gnorm [Di], out_proj [D, Di]}
 *   layers.l.attn.{norm [D], wqkv [(Hq+2Hkv)*dh, D] (rows q | k | v), q_norm [dh], k_norm [dh], wo [D, Hq*dh]}
 *   layers.l.mlp.{norm [D], w_gate_up [2F, D] (rows gate | up), w_down [D, F]}
 * Matrices must be HSPEC_BF16 with a 16-byte aligned base; vectors HSPEC_F32. */
typedef struct {
  const char* name;      /* host, NUL-terminated */
  const void* data;      /* device */
  int32_t dtype;         /* hspec_dtype */
  int32_t ndim;          /* 1 or 2 */
  int64_t shape[2];
} hspec_tensor;

/* Inputs of one step (the paper's drafter inputs: last-position hidden states, the target's KV
 * cache in place, the last sampled token; Sec. 3.2 / 3.3). */
typedef struct {
  int32_t B;                     /* requests, 1..max_batch */
  int32_t k;                     /* block positions = draft tokens emitted, 1..max_k */
  const int32_t* page_table;     /* device int32 [B, page_table_stride]: logical page j of request b -> physical page.
                                    Entries at or past ceil(ctx/page_size) are never read. */
  int32_t page_table_stride;     /* row pitch in elements, <= max_pages_per_req */
  const int32_t* ctx_lens;       /* device int32 [B]: tokens of request b already in the target cache (>= 0) */
  int32_t max_ctx;               /* host: an upper bound on every ctx_lens[b]; 0 = page_table_stride*page_size.
                                    Only used to size the split of long contexts; a loose bound costs idle CTAs. */
  const void* last_hidden;       /* device bf16 [B, n_fuse*D]: target hidden state(s) at the last input position */
  const int32_t* last_token;     /* device int32 [B]: last accepted token id (block row 0) */
  const void* const* k_pools;    /* HOST array of n_slots device pointers, each bf16 [num_pages, page_size, Hkv, dh];
                                    keys are stored already rotated by the target.  Never written. */
  const void* const* v_pools;    /* same for values */
  int64_t num_pages;             /* pages in each pool */
  void* stream;                  /* cudaStream_t (0 = default stream) */
  void* workspace;               /* device scratch, >= hspec_workspace_bytes(cfg), 1024-byte aligned; owned by the caller,
                                    contents undefined between calls */
  size_t workspace_bytes;
} hspec_step;

/* Outputs of one step, device memory owned by the caller. */
typedef struct {
  int32_t* draft_ids;   /* int32 [B, k], required: arg-max of the logits, lowest row index on ties; target token ids
                           (mapped through vocab_map when the drafter vocabulary is pruned) */
  float* logits;        /* fp32 [B, k, V] ([B, k, V_draft] when pruned) or NULL (then the logits are never materialised,
                           except in the workspace when markov_rank > 0); with the causal-correction head these are the
                           corrected logits */
  float* hidden;        /* fp32 [B, k, D] or NULL: the residual stream before the final norm */
} hspec_out;

typedef struct hspec_handle hspec_handle;

typedef struct {
  uint64_t kernel_launches;   /* kernels this handle enqueued since it was created */
  uint32_t device_status;     /* 0, or a code written by a bounded in-kernel wait that gave up
                                 (reading it synchronises the handle's last stream) */
  uint32_t launches_last_step;
  uint32_t attn_rescales;     /* informational: (warp, key tile) events in which the attention kernel moved a row's reference
                                 maximum and rescaled its accumulator (peaked score rows; never an error) */
  uint32_t f16_range_events;  /* finite values that left the fp16 range in a store and were clamped to +-65504 */
  uint32_t bad_inputs;        /* out-of-range context lengths / page ids met by a kernel (clamped / read as zeros) */
} hspec_stats;

/* One kernel launch of the last step, as recorded when profiling is on. */
typedef struct {
  char name[40];     /* kernel label, e.g. "gemm:proj_ds", "attn_partial", "mamba_scan" */
  float ms;          /* device time between CUDA events recorded around the launch on the step's stream */
  double flops;      /* algorithmic flops of the launch (GEMMs: 2*M*N*K), 0 if not a contraction */
  double bytes;      /* algorithmic bytes where the library knows them without the context lengths (GEMMs: the
                        weight matrix; scan: S_init), else 0 */
  double io_bytes;   /* GEMMs: activation bytes read and result bytes written besides the weights, else 0 */
} hspec_prof_entry;

/* Validates the config, creates the handle (host memory only; no weights yet).  Sec. 3.3 / App. B.1. */
int hspec_init(const hspec_config* cfg, hspec_handle** out);
/* Device scratch bytes a step of up to (max_batch, max_k, max_pages_per_req) needs. */
size_t hspec_workspace_bytes(const hspec_config* cfg);
/* Copies n named device tensors into library-owned device memory (may be called several times; synchronises the
 * device).  Shapes are checked against the config. */
int hspec_load_weights(hspec_handle* h, const hspec_tensor* tensors, int32_t n);
/* Enqueues one block-parallel draft step (Sec. 3.3) on in->stream.  Needs every tensor loaded.  The first call on a
 * device builds a small RoPE table (one allocation, one copy) and sets kernel attributes; every later call only
 * launches kernels on the stream, so a warmed-up step may be captured in a CUDA graph and replayed: the replay reads
 * the current contents of the same input buffers.  The workspace must hold hspec_workspace_bytes(cfg) bytes, which
 * covers every (B, k) up to (max_batch, max_k). */
int hspec_draft_block(hspec_handle* h, const hspec_step* in, const hspec_out* out);
/* Frees the handle and its weight copies.  Pools and the workspace stay the caller's. */
int hspec_destroy(hspec_handle* h);
/* Message of the last failure on this handle (or of the last failed hspec_init if h is NULL). */
const char* hspec_last_error(const hspec_handle* h);
/* Reads the handle's counters and device status block (synchronises the handle's last stream).  Returns HSPEC_OK, or
 * the most severe condition recorded since the last hspec_clear_status: HSPEC_ERR_TIMEOUT (device_status != 0),
 * HSPEC_ERR_PAGE_OUT_OF_RANGE (bad_inputs != 0), HSPEC_ERR_F16_RANGE (f16_range_events != 0); `out` is filled either way. */
int hspec_get_stats(hspec_handle* h, hspec_stats* out);
/* Failure-path self-test: enqueues a one-thread kernel that waits, for at most limit_ms (1..2000), on a barrier nothing
 * completes; it then gives up, writes a code to the handle's device status word and returns normally (no trap: the
 * context stays usable).  hspec_get_stats afterwards reports HSPEC_ERR_TIMEOUT with device_status != 0, which is how
 * a bounded in-kernel wait that gave up inside a real step surfaces.  hspec_clear_status resets the word. */
int hspec_debug_wait_selftest(hspec_handle* h, int32_t limit_ms, void* stream);
int hspec_clear_status(hspec_handle* h);
/* Measurement aid: when on, every kernel launch of a step is bracketed by CUDA events on the step's stream. */
int hspec_set_profiling(hspec_handle* h, int32_t on);
/* Per-launch times of the LAST step (synchronises its stream).  Returns the number of entries written (<= max_entries)
 * or a negative hspec_status. */
int hspec_get_profile(hspec_handle* h, hspec_prof_entry* out, int32_t max_entries);

/* ------------------------------------------------------------------------------------------------
 * Single-operation entry points: the same kernels the step uses, exposed one at a time so that each
 * can be checked against its definition.  All pointers are DEVICE pointers unless stated; all calls
 * enqueue on `stream` and do not synchronise.
 * ---------------------------------------------------------------------------------------------- */

/* y[M, n_out] = x[M, K] W[n_out, K]^T, x and W both bf16 or both fp16 (in_dtype), fp32 accumulation (every linear
 * map of Sec. 3.3).  out_dtype HSPEC_F32, HSPEC_BF16 or HSPEC_F16; ldy = row pitch of y in elements.  accumulate != 0 (fp32 only):
 * y += result (the residual form).  splits <= 0 lets the library choose how many K-slices to use;
 * `workspace` (>= hspec_gemm_workspace_bytes) is needed when more than one slice is used.
 * Needs K % 8 == 0, 16-byte aligned x and W. */
int hspec_op_gemm(const void* x, const void* W, int32_t in_dtype, void* y, int32_t M, int32_t n_out, int32_t K, int64_t ldy,
                  int32_t out_dtype, int32_t accumulate, int32_t splits, void* workspace, size_t workspace_bytes,
                  void* stream);
size_t hspec_gemm_workspace_bytes(int32_t M, int32_t n_out, int32_t K);
/* LM head fused with arg-max (App. B.2): ids[m] = lowest index of max_v x[m,:] . W[v,:]; logits fp32 [M, V] or NULL.
 * x and W are both bf16 or both fp16 (in_dtype). */
int hspec_op_lm_head_argmax(const void* x, const void* W, int32_t in_dtype, int32_t* ids, float* logits, int32_t M, int32_t V,
                            int32_t K, void* workspace, size_t workspace_bytes, void* stream);
/* The same LM head + arg-max for callers that cannot allocate device memory at the point where they draft: an engine
 * whose KV-cache pool already owns every free byte of HBM (a later cudaMalloc fails), a decode loop that cannot take the
 * device synchronisation and driver lock of an allocation, a plug-in that is handed pointers but no allocator.  (The
 * paper has no counterpart; this is a deployment aid.)  The per-tile (max, index) partials and the status word live in
 * a fixed array inside the library's device image: 8 MiB + 256 B on every GPU that loads the library, held until the
 * process exits.  Limits: M <= 512 rows, V <= 262144; larger sizes are rejected with HSPEC_ERR_BAD_SHAPE.
 * The call allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).  Its FIRST call on a device
 * resolves the array's device address (cudaGetSymbolAddress, with that device current) and, with CUDA's lazy module
 * loading, is also the moment the driver places the array and the kernels' code in device memory: make that first
 * call at start-up - before the host hands the remaining HBM to its pool, and before any stream capture begins; from
 * the second call on, free device memory does not move (the test checks it).  All calls share the array: calls that
 * overlap on the GPU (e.g. on two streams) race.  A bounded wait that gives up inside the call shows in
 * hspec_op_device_status (the ids of such a call are 0x7fffffff).
 * Inputs and outputs are the caller's, as in hspec_op_lm_head_argmax; results are identical to it. */
int hspec_op_lm_head_argmax_noalloc(const void* x, const void* W, int32_t in_dtype, int32_t* ids, float* logits, int32_t M,
                                    int32_t V, int32_t K, void* stream);
/* Status of the hspec_op_* entry points, which take no handle: synchronises the current device, then reads the status
 * block those calls share on this device and the one inside the allocation-free entry point's built-in array.
 * words4 (host, may be NULL) receives {give-up code of a bounded wait or 0, attention rescale events, fp16 range events,
 * out-of-range inputs}; clear != 0 zeroes the blocks afterwards.  Returns like hspec_get_stats.  A handle-less call
 * whose bounded wait gave up has already returned HSPEC_OK when it was enqueued: this is the only place where that
 * shows (arg-max ids of such a call are 0x7fffffff). */
int hspec_op_device_status(uint32_t* words4, int32_t clear);
/* Acceptance rule of speculative decoding (App. A): draft i of request b is accepted if every earlier draft of b
 * was and min(1, P_T / P_D) >= alpha.  p_target, p_draft, alpha: device fp32 [B, k] (probabilities of the drafted
 * tokens under the target and under the drafter, and the caller's uniform draws); n_accept: device int32 [B], the
 * number of leading accepted drafts (the iteration then emits n_accept + 1 tokens).  Ratio, minimum and comparison
 * are fp32 with IEEE division; 0 / 0 rejects, P_D = 0 with P_T > 0 accepts. */
int hspec_op_accept(const float* p_target, const float* p_draft, const float* alpha, int32_t* n_accept, int32_t B, int32_t k,
                    void* stream);
/* Draft probability P_D of App. A: p[m] = softmax(logits[m, 0..V))[ids[m]] for device fp32 logits with row pitch ld
 * elements; ids index the logits' own vocabulary (the drafter's row index when its vocabulary is pruned). */
int hspec_op_token_probs(const float* logits, int64_t ld, const int32_t* ids, float* p, int32_t M, int32_t V, void* stream);
/* Causal correction after the backbone (Sec. 3.3.3; rank 256 in App. B.1): a first-order dependency between adjacent
 * draft positions applied to the logits.  The paper prints no formula; the reading implemented is a low-rank bigram
 * table, logits'[b, i, :] = logits[b, i, :] + W_out . W_in[prev(b, i), :], prev(b, 0) = last_token[b], prev(b, i) =
 * the token chosen at position i - 1 from the adjusted logits (lowest index on ties), positions strictly in order.
 *   logits   device fp32 [B*k, ld] (row b*k + i), adjusted in place when write_logits != 0, else left as they are
 *   W_in     device [V, r]  fp16 or bf16 (w_dtype), one row per possible previous TOKEN id
 *   W_out    device [Vd, r] same type, one row per drafter-vocabulary index; r % 8 == 0, both 16-byte aligned
 *   id_map   device int32 [Vd] drafter-vocabulary index -> token id, or NULL (identity)
 *   ids      device int32 [B*k] out: chosen token ids
 *   workspace >= hspec_markov_workspace_bytes(B, Vd, r), 256-byte aligned.
 * Runs 2k + 1 launches on `stream` (one rank-r product with arg-max per position). */
int hspec_op_markov_head(float* logits, int64_t ld, const void* W_in, const void* W_out, int32_t w_dtype, const int32_t* last_token,
                         const int32_t* id_map, int32_t* ids, int32_t B, int32_t k, int32_t Vd, int32_t r, int32_t write_logits,
                         void* workspace, size_t workspace_bytes, void* stream);
size_t hspec_markov_workspace_bytes(int32_t B, int32_t Vd, int32_t r);
/* The cache write of the KV-injecting block drafters the paper compares with (Sec. 2.2 "KV injection in block
 * drafting"), kept as a measured counter-example to the drafter-side KV bytes the draft step avoids; the draft step
 * itself never calls it.  For T new positions: key rows get the per-head RMSNorm (if k_norm) and rotate-half RoPE at
 * their position, value rows are converted as they are, and both are stored as bf16 in a drafter-side paged cache.
 *   kv fp32 device [T, 2, Hkv, dh] (projected keys | values, e.g. from hspec_op_gemm); k_norm_w fp32 [dh] or NULL
 *   req, pos int32 device [T]: request (page-table row) and absolute position of each row
 *   page_table int32 device [*, page_table_stride]; k_pool, v_pool bf16 device [num_pages, page_size, Hkv, dh], written
 *   in place at (page_table[req, pos / page_size], pos % page_size); all other entries keep their bits.
 * Two rows with the same (req, pos) race. */
int hspec_op_kv_inject_write(const float* kv, const float* k_norm_w, const int32_t* req, const int32_t* pos,
                             const int32_t* page_table, int32_t page_table_stride, void* k_pool, void* v_pool, int32_t T,
                             int32_t Hkv, int32_t dh, int32_t page_size, float theta, float eps, int32_t k_norm, void* stream);
/* RMSNorm over the last axis: y fp16 [M, n] = x fp32 [M, n] / sqrt(mean(x^2) + eps) * w. */
int hspec_op_rmsnorm(const float* x, const float* w, void* y_f16, int32_t M, int32_t n, float eps, void* stream);
/* Mamba-2 mixer core for B requests x k rows (Sec. 3.3.1): causal depthwise conv + SiLU on xBC (zero left
 * context), dt = softplus(dt_raw + dt_bias), decay exp(dt * -exp(A_log)), the selective recurrence over the
 * k rows started from s_init, the D skip, and the SiLU(z) gate.
 *   zxbcdt fp32 [B*k, ld_in]: columns z [Di] | xBC [Di + 2GN] (| dt [H] when dt_raw is NULL)
 *   dt_raw fp32 [B*k, H] or NULL;  s_init fp16 [B, H, P, N] or NULL (zero state)
 *   y_gated fp32 [B*k, Di] = (scan output) * SiLU(z).
 *   workspace: optional device scratch of hspec_scan_workspace_bytes(...) bytes (256-byte aligned); with it the serving
 *   shapes (P = 64, N = 128) run as three kernels (conv, C.B table, state stream), without it as one fused kernel. */
int hspec_op_mamba_scan(const float* zxbcdt, int64_t ld_in, const float* dt_raw, const void* s_init,
                        const float* conv_w, const float* conv_b, const float* dt_bias, const float* A_log,
                        const float* Dskip, float* y_gated, int32_t B, int32_t k, int32_t Di, int32_t P,
                        int32_t N, int32_t G, int32_t d_conv, void* workspace, size_t workspace_bytes, void* stream);
size_t hspec_scan_workspace_bytes(int32_t B, int32_t k, int32_t Di, int32_t N, int32_t G);
/* Per-head RMSNorm (optional) + rotate-half RoPE at positions ctx_lens[b] + i (Sec. 3.3.2, positional alignment).
 * qkv fp32 [B*k, (Hq+2Hkv)*dh] (q | k | v) -> q bf16 [B*k, Hq, dh], kb bf16 [B*k, Hkv, dh], vb bf16 [B*k, Hkv, dh]. */
int hspec_op_qk_norm_rope(const float* qkv, const float* q_norm_w, const float* k_norm_w, const int32_t* ctx_lens,
                          void* q, void* kb, void* vb, int32_t B, int32_t k, int32_t Hq, int32_t Hkv, int32_t dh,
                          float theta, float eps, int32_t qk_norm, void* stream);
/* Block-query GQA attention over the target's paged KV (read in place) plus the block's causal keys (Sec. 3.3.2).
 * q/kb/vb as produced by hspec_op_qk_norm_rope; k_pool/v_pool bf16 [num_pages, page_size, Hkv, dh];
 * o fp16 [B*k, Hq*dh].  window 0 = full.  max_ctx: host upper bound on ctx_lens (0 = stride*page_size).
 * chunk_tokens <= 0 lets the library pick the context split (otherwise rounded up to a multiple of 128).
 * num_pages = pages in each pool. */
int hspec_op_attention(const void* q, const void* kb, const void* vb, const void* k_pool, const void* v_pool,
                       int64_t num_pages, const int32_t* page_table, int32_t page_table_stride, const int32_t* ctx_lens,
                       int32_t max_ctx, void* o, int32_t B, int32_t k, int32_t Hq, int32_t Hkv, int32_t dh,
                       int32_t page_size, int32_t window, int32_t chunk_tokens, void* workspace,
                       size_t workspace_bytes, void* stream);
size_t hspec_attention_workspace_bytes(int32_t B, int32_t k, int32_t Hq, int32_t Hkv, int32_t dh, int32_t max_ctx,
                                       int32_t window, int32_t chunk_tokens);
/* Contiguous copy of one request's prefix out of a paged pool: dst bf16 [ctx_len, Hkv, dh] (pure data movement,
 * bit-exact; used to check the page-table addressing of the attention kernel, Sec. 3.3.2). */
int hspec_debug_gather_kv(const void* pool, const int32_t* page_table_row, int32_t ctx_len, int32_t page_size,
                          int32_t Hkv, int32_t dh, void* dst, void* stream);
/* h fp16 [M, F] = SiLU(gu[:, :F]) * gu[:, F:], gu fp32 [M, 2F] (App. B.1 "MLP"). */
int hspec_op_swiglu(const float* gu, void* h_f16, int32_t M, int32_t F, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HSPEC_H_ */
