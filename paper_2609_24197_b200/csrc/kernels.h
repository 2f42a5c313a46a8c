// Internal interfaces between the kernel files and the C ABI layer (not exported).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdlib>
#include <mutex>
#include <string>
#include <vector>

namespace hspec {

constexpr int GEMM_MAX_STAGES = 8;

// Records the message hspec_last_error(NULL) returns (calling thread).
void set_last_error(const std::string& msg);

// State that CUDA keeps per device (function attributes, small device-side tables, the status block of the
// handle-less entry points) is cached per device index, so one process may drive several GPUs.
constexpr int MAX_DEVICES = 64;
std::mutex& device_setup_mutex();
inline int current_device() {
  int d = -1;
  return (cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < MAX_DEVICES) ? d : -1;
}
// Runs `fn` (returning cudaError_t) once per device, for the current device; a failure is returned and retried on the
// next call.
template <class F>
inline cudaError_t once_per_device(bool (&done)[MAX_DEVICES], F fn) {
  const int d = current_device();
  if (d < 0) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(device_setup_mutex());
  if (done[d]) return cudaSuccess;
  const cudaError_t e = fn(d);
  if (e == cudaSuccess) done[d] = true;
  return e;
}
// Status block (STATUS_WORDS x uint32, zeroed) of the current device for entry points that take no handle.
uint32_t* global_status();
// Status block inside the allocation-free entry point's built-in array, once a call on the current device has
// resolved its address (else null).
uint32_t* noalloc_status_if_resolved();

// Counts kernel launches and, when profiling is on, brackets each launch with a pair of CUDA events
// recorded on the launching stream (read back with elapsed() after the stream is synchronised).
struct Tracker {
  struct Entry {
    char name[40];
    cudaEvent_t a = nullptr, b = nullptr;
    double flops = 0, bytes = 0, io_bytes = 0;
  };
  uint64_t launches = 0;
  bool profiling = false;
  cudaStream_t stream = nullptr;
  std::vector<Entry> entries;
  size_t used = 0;
  void begin_step(cudaStream_t st) { used = 0; stream = st; }
  void begin(const char* name, double flops = 0, double bytes = 0, double io_bytes = 0);   // call right before a launch
  void end();                                                         // call right after it
  void destroy();
};
inline void trk_begin(Tracker* t, const char* name, double flops = 0, double bytes = 0, double io_bytes = 0) {
  if (t) t->begin(name, flops, bytes, io_bytes);
}
// Activation bytes a GEMM launch reads and writes besides its weights: x [M, K] 16-bit in, y [M, n_out] out (a
// residual epilogue reads y as well; the LM-head arg-max epilogue writes logits only when asked).
inline double gemm_io_bytes(int M, int n_out, int K, int mode, bool logits) {
  double out = 0;
  switch (mode) {
    case 0: case 3: out = 4.0 * M * n_out; break;            // fp32 store / K-slice partial
    case 1: case 5: out = 2.0 * M * n_out; break;            // bf16 / fp16 store
    case 2: out = 8.0 * M * n_out; break;                    // fp32 read-modify-write
    case 6: case 7: out = 1.0 * M * n_out; break;            // SwiGLU: 16-bit [M, n_out / 2]
    default: out = logits ? 4.0 * M * n_out : 0; break;      // arg-max
  }
  return 2.0 * M * K + out;
}
inline void trk_end(Tracker* t) { if (t) t->end(); }

// Launch with programmatic stream serialisation: the kernel MUST call pdl_wait() before it touches global data.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
  static const bool off = [] { const char* e = getenv("HSPEC_NO_PDL"); return e && e[0] == '1'; }();
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = off ? 0 : 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

enum GemmEpilogue : int {
  EPI_STORE_F32 = 0,    // y fp32 = acc
  EPI_STORE_BF16 = 1,   // y bf16 = acc
  EPI_ACCUM_F32 = 2,    // y fp32 += acc   (residual)
  EPI_PARTIAL_F32 = 3,  // K-slice partial (internal)
  EPI_ARGMAX = 4,
  EPI_STORE_F16 = 5,    // y fp16 = acc
  EPI_SWIGLU_F16 = 6,   // weight rows interleaved in blocks of 16 (gate | up): h fp16 [M, n_out/2] = SiLU(gate) * up
  EPI_SWIGLU_BF16 = 7,  // the same with h stored as bf16
  EPI_ARGMAX_T = 8,     // arg-max over the ACTIVATION side: the "weights" are a few rows (the requests' factor rows), the
                        // "activations" the vocabulary matrix; every accumulator lane (request) reduces its own columns
};
inline bool epi_is_swiglu(int mode) { return mode == EPI_SWIGLU_F16 || mode == EPI_SWIGLU_BF16; }

struct GemmArgs {       // kernel argument block
  int M, N_out, K;
  int BN;               // activation rows per CTA = UMMA N (multiple of 16, <= 256)
  int WT;               // 128-row weight tiles per CTA (1 or 2): with 2, one activation tile fill feeds two MMAs
  int k_tiles_total, k_tiles_per_split;
  int stages;
  uint32_t tmem_cols;
  int f16;              // both operands fp16 (else both bf16)
  int mode;
  void* out;
  long long ldo;
  float* logits;
  const float* addend;  // EPI_ARGMAX only (one-CTA kernel): value = acc + addend[m * ld_add + n] (may be null)
  long long ld_add;
  int keep_w;           // weights loaded evict-last instead of evict-first
  float* part_val;
  int* part_idx;
  uint32_t* status;
};

struct GemmCall {       // host-side description of one y = x W^T
  const CUtensorMap* tmW;   // weights [n_out, K], box 128 x 64
  const void* x;            // [M, K] in the same 16-bit type as the weights, row pitch ldx elements
  long long ldx;
  bool f16;                 // operands are fp16 (else bf16)
  int M, n_out, K;
  int mode;                 // EPI_STORE_F32 / EPI_STORE_BF16 / EPI_ACCUM_F32 / EPI_ARGMAX
  void* out;
  long long ldo;
  int splits;
  void* splitk_ws;
  size_t splitk_ws_bytes;
  float* logits;            // EPI_ARGMAX only (may be null)
  const float* addend;      // EPI_ARGMAX, one-CTA kernel only: fp32 [M, ld_add] added before the arg-max (may be null)
  long long ld_add;
  bool keep_weights_in_l2;  // one-CTA kernel: the same W is used again by the next launch (keep it in L2 if it fits)
  float* part_val;
  int* part_idx;
  uint32_t* status;
  const char* label;        // profile name (may be null)
  int bn;                   // one-CTA kernel: activation rows per CTA (0 = by the row count)
};

bool make_tmap_16bit_2d(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t ld_elems,
                       int box_rows, bool f16, std::string* err);
int gemm_pick_bn(int M);
int gemm_pick_splits(int M, int n_out, int K, int num_sms, int mode = EPI_STORE_F32);
size_t gemm_splitk_bytes(int M, int n_out, int splits);
cudaError_t gemm_launch(const GemmCall& c, cudaStream_t stream, Tracker* trk, std::string* err);
bool gemm2_preferred(int M, int n_out);        // many rows and at least one full round of cluster tiles
size_t gemm2_tail_bytes();                     // scratch the 2-SM kernel's K-sliced tail wave may use
void gemm2_pick(int M, int n_out, int K, int mode, int* bnt, int* splits);   // tile width and K-slices of the 2-SM kernel
cudaError_t splitk_reduce_launch(const float* part, int splits, int M, int N, void* out, long long ldo, int mode,
                                 cudaStream_t stream, Tracker* trk, uint32_t* status);
cudaError_t gemm2_launch(const GemmCall& c, cudaStream_t stream, Tracker* trk, std::string* err);
cudaError_t argmax_reduce_launch(const float* pv, const int* pi, int n_tiles, int M, int* ids, cudaStream_t stream,
                                 Tracker* trk, const int* id_map = nullptr);

// ---- steps next to the draft block (next_ops.cu)
struct MarkovCall {
  float* logits;                    // fp32 [B*k, ld]: the block's logits (adjusted in place when write_logits)
  long long ld;
  const void *W_in;                 // [V, r] 16-bit: factor row of every possible previous token
  const CUtensorMap* tmW_out;       // [Vd, r] 16-bit, box 128 x 64
  const void* W_out;                // the same matrix by address
  bool f16;
  const int* last_token;            // [B]
  const int* id_map;                // [Vd] draft-vocabulary index -> token id, or null
  int* ids;                         // [B*k] token ids out
  int B, k, Vd, r, write_logits;
  void* ws;                         // markov_workspace_bytes(B, Vd, r)
  uint32_t* status;
};
cudaError_t kv_inject_write_launch(const float* kv, const float* kw, const int32_t* req, const int32_t* pos,
                                   const int32_t* page_table, int page_table_stride, void* k_pool, void* v_pool, int T,
                                   int Hkv, int dh, int page_size, float theta, float eps, int k_norm, cudaStream_t stream);
cudaError_t accept_launch(const float* pt, const float* pd, const float* alpha, int* n_accept, int B, int k, cudaStream_t stream);
cudaError_t token_probs_launch(const float* logits, long long ld, const int* ids, float* p, int M, int V, cudaStream_t stream);
size_t markov_workspace_bytes(int B, int Vd, int r);
cudaError_t markov_launch(const MarkovCall& c, cudaStream_t stream, Tracker* trk, std::string* err);

// ---- attention (attention.cu)
struct AttnCall {
  const void *q, *kb, *vb;          // bf16 [B*k, Hq, dh], [B*k, Hkv, dh] x2
  const void *k_pool, *v_pool;      // bf16 [num_pages, page, Hkv, dh]
  long long num_pages;
  uint32_t* status;                 // device status word for bounded waits
  const int32_t* page_table;
  int page_table_stride;
  const int32_t* ctx_lens;
  int max_ctx;                      // host bound on ctx_lens
  void* o;                          // fp16 (or bf16 when o_bf16) [B*k, Hq*dh]
  bool o_bf16;
  int B, k, Hq, Hkv, dh, page_size, window;
  int chunk_tokens;                 // <= 0: choose
  void* ws;
  size_t ws_bytes;
};
int attn_pick_chunk(int B, int Hkv, int max_ctx, int window, int num_sms);
size_t attn_workspace_bytes(int B, int k, int Hq, int Hkv, int dh, int max_ctx, int window, int chunk_tokens);
cudaError_t attention_launch(const AttnCall& c, cudaStream_t stream, Tracker* trk, std::string* err);
bool attention_tc_supported(const AttnCall& c);
cudaError_t attention_tc_launch(const AttnCall& c, int max_chunks, cudaStream_t stream, Tracker* trk, std::string* err);
cudaError_t gather_kv_launch(const void* pool, const int32_t* row, int ctx_len, int page_size, int Hkv, int dh,
                             void* dst, cudaStream_t stream);

// ---- scan (scan.cu)
struct ScanCall {
  const float* zxbcdt; long long ld_in;
  const float* dt_raw;              // [B*k, H] or null (then the dt columns of zxbcdt)
  const void* s_init;               // fp16 [B, H, P, N] or null
  const float *conv_w, *conv_b, *dt_bias, *A_log, *Dskip;
  float* y_gated;                   // [B*k, Di]
  int B, k, Di, P, N, G, d_conv;
  void* ws;                         // optional scratch (scan_workspace_bytes): enables the three-kernel fast path
  size_t ws_bytes;
};
size_t scan_workspace_bytes(int B, int k, int Di, int N, int G);
cudaError_t scan_launch(const ScanCall& c, cudaStream_t stream, Tracker* trk, std::string* err);

// ---- element-wise kernels (elementwise.cu)
cudaError_t embed_rows_launch(const void* embed_bf16, const int32_t* last_token, int mask_id, float* X, int B, int k,
                              int D, cudaStream_t stream);
cudaError_t rmsnorm_launch(const float* x, const float* w, void* y_16, int M, int n, float eps, cudaStream_t stream,
                           uint32_t* status, bool bf16_out = false);
cudaError_t qk_norm_rope_launch(const float* qkv, const float* qw, const float* kw, const int32_t* ctx_lens, void* q,
                                void* kb, void* vb, int B, int k, int Hq, int Hkv, int dh, float theta, float eps,
                                int qk_norm, cudaStream_t stream);
cudaError_t swiglu_launch(const float* gu, void* h_16, int M, int F, cudaStream_t stream, uint32_t* status, bool bf16_out = false);
cudaError_t copy_f32_launch(const float* src, float* dst, size_t n, cudaStream_t stream);

}  // namespace hspec
