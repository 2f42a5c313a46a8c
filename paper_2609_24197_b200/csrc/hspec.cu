// C ABI of the H-Spec draft step: handle, weight registry, workspace plan and the kernel sequence.
#include "../../include/hspec.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>
#include <unordered_map>
#include <vector>

#include "common.cuh"
#include "kernels.h"

using namespace hspec;

namespace {

constexpr int kNumSMs = 148;   // B200; only used to size grids and K-slices
thread_local std::string g_err;

struct Weight {
  void* data = nullptr;      // library-owned device copy (GEMM matrices as fp16, everything else as given); with bf16
                             // activations the GEMM matrices are the caller's own (owned = false)
  bool owned = true;
  int dtype = 0;
  int64_t rows = 0, cols = 0;
  bool has_tm = false;
  CUtensorMap tm;
};

struct Dims {
  int H, d_S, d_xBC, d_dt, d_in_proj, d_qkv;
  int Vd;   // rows of the LM head: the target vocabulary, or the pruned drafter vocabulary
};

Dims dims_of(const hspec_config& c) {
  Dims d;
  d.H = c.Di / c.P;
  d.d_S = d.H * c.P * c.N;
  d.d_xBC = c.Di + 2 * c.G * c.N;
  d.d_dt = c.dt_rank > 0 ? c.dt_rank : d.H;
  d.d_in_proj = c.Di + d.d_xBC + d.d_dt;
  d.d_qkv = (c.Hq + 2 * c.Hkv) * c.dh;
  d.Vd = c.V_draft > 0 ? c.V_draft : c.V;
  return d;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
int imax(int a, int b) { return a > b ? a : b; }

// Offsets of the step's scratch buffers inside the caller's workspace.
struct Plan {
  size_t X, U, U2, BIG, LH, Fv, SINIT, SCAN, scan_bytes, DTL, DT, YG, Q, KB, VB, ATT, SPLITK, AMAXV, AMAXI, LOGITS, MARKOV, total;
  size_t att_bytes, splitk_bytes;
  int attn_chunk, max_ctx;
};

size_t splitk_need(int M, int n_out, int K) {
  if (gemm2_preferred(M, n_out)) return gemm2_tail_bytes();
  return gemm_splitk_bytes(M, n_out, gemm_pick_splits(M, n_out, K, kNumSMs));
}

Plan make_plan(const hspec_config& c, int B, int k, int max_ctx) {
  const Dims d = dims_of(c);
  const size_t M = size_t(B) * k;
  Plan p{};
  size_t at = 0;
  auto take = [&](size_t bytes) { size_t o = at; at = align_up(at + bytes, 1024); return o; };
  p.X = take(M * c.D * 4);
  p.U = take(M * size_t(imax(imax(c.D, c.Di), c.Hq * c.dh)) * 2);
  p.U2 = take(M * size_t(c.F) * 2);
  p.BIG = take(M * size_t(imax(imax(d.d_in_proj, d.d_qkv), 2 * c.F)) * 4);
  p.LH = take(size_t(B) * c.n_fuse * c.D * 2);
  p.Fv = take(size_t(B) * c.r * 2);
  p.SINIT = take(size_t(B) * d.d_S * 2);
  p.DTL = take(M * size_t(imax(c.dt_rank, 8)) * 2);
  p.DT = take(M * size_t(d.H) * 4);
  p.YG = take(M * size_t(c.Di) * 4);
  p.scan_bytes = scan_workspace_bytes(B, k, c.Di, c.N, c.G);
  p.SCAN = take(p.scan_bytes);
  p.Q = take(M * size_t(c.Hq) * c.dh * 2);
  p.KB = take(M * size_t(c.Hkv) * c.dh * 2);
  p.VB = take(M * size_t(c.Hkv) * c.dh * 2);
  p.max_ctx = max_ctx;
  p.attn_chunk = attn_pick_chunk(B, c.Hkv, max_ctx, c.window, kNumSMs);
  p.att_bytes = attn_workspace_bytes(B, k, c.Hq, c.Hkv, c.dh, max_ctx, c.window, p.attn_chunk);
  p.ATT = take(p.att_bytes);
  size_t sk = 0;
  auto upd = [&](size_t v) { if (v > sk) sk = v; };
  upd(splitk_need(B, c.r, c.n_fuse * c.D));
  upd(splitk_need(B, d.d_S, c.r));
  upd(splitk_need(int(M), d.d_in_proj, c.D));
  if (c.dt_rank > 0) upd(splitk_need(int(M), d.H, c.dt_rank));
  upd(splitk_need(int(M), c.D, c.Di));
  upd(splitk_need(int(M), d.d_qkv, c.D));
  upd(splitk_need(int(M), c.D, c.Hq * c.dh));
  upd(splitk_need(int(M), 2 * c.F, c.D));
  upd(splitk_need(int(M), c.D, c.F));
  p.splitk_bytes = sk;
  p.SPLITK = take(sk);
  const size_t vt = 2 * ((size_t(d.Vd) + 255) / 256);   // 128-row tiles, in pairs (the 2-SM kernel's indexing)
  p.AMAXV = take(vt * M * 4);
  p.AMAXI = take(vt * M * 4);
  if (c.markov_rank > 0) {
    // the causal-correction head works on materialised fp32 logits of the whole block
    p.LOGITS = take(M * size_t(d.Vd) * 4);
    p.MARKOV = take(markov_workspace_bytes(B, d.Vd, c.markov_rank));
  }
  p.total = at;
  return p;
}

const char* check_config(const hspec_config& c) {
  if (c.D < 8 || c.D % 8) return "D must be a positive multiple of 8";
  if (c.n_fuse < 1 || c.r < 8 || c.r % 8) return "n_fuse >= 1 and r a multiple of 8 are required";
  if (c.L < 1 || c.L > HSPEC_MAX_LAYERS) return "L out of range";
  if (c.P < 1 || c.Di < c.P || c.Di % c.P || c.Di % 8) return "Di must be a multiple of P and of 8";
  if (c.N < 1 || c.N > 256 || c.P > 128) return "Mamba state dim N <= 256 and head dim P <= 128 are supported";
  if (c.G < 1 || (c.Di / c.P) % c.G) return "Mamba heads must divide into G groups";
  if (c.d_conv < 1 || c.d_conv > 4) return "d_conv must be 1..4";
  if (c.dt_rank < 0 || c.dt_rank % 8) return "dt_rank must be 0 or a multiple of 8";
  if (c.dh != 64 && c.dh != 128) return "attention head dim must be 64 or 128";
  if (c.Hkv < 1 || c.Hq < c.Hkv || c.Hq % c.Hkv) return "Hq must be a multiple of Hkv";
  if (c.F < 8 || c.F % 8) return "F must be a multiple of 8";
  if (c.V < 2 || c.mask_id < 0 || c.mask_id >= c.V) return "V / mask_id out of range";
  if (c.V_draft < 0 || c.V_draft > c.V) return "V_draft must be 0 or at most V";
  if (c.page_size < 1 || c.max_batch < 1 || c.max_pages_per_req < 1) return "page_size, max_batch, max_pages_per_req must be positive";
  if (c.max_k < 1 || c.max_k > HSPEC_MAX_K) return "max_k out of range";
  if (c.max_k * (c.Hq / c.Hkv) > 1024) return "k * Hq/Hkv too large";
  if (c.n_slots < 0 || c.n_slots > HSPEC_MAX_SLOTS) return "n_slots out of range";
  if (c.window < 0) return "window must be >= 0";
  if (c.markov_rank < 0 || c.markov_rank % 8) return "markov_rank must be 0 or a multiple of 8";
  for (int l = 0; l < c.L; ++l)
    if (c.has_attn[l] && (c.kv_slot[l] < 0 || c.kv_slot[l] >= c.n_slots)) return "kv_slot out of range";
  return nullptr;
}

uint32_t* g_status[MAX_DEVICES] = {};   // status blocks of the handle-less single-op entry points, one per device

int fail(hspec_handle* h, int code, const std::string& msg);

}  // namespace

namespace hspec {

void set_last_error(const std::string& msg) { g_err = msg; }

std::mutex& device_setup_mutex() {
  static std::mutex m;
  return m;
}

uint32_t* global_status() {
  const int d = current_device();
  if (d < 0) return nullptr;
  std::lock_guard<std::mutex> lock(device_setup_mutex());
  if (!g_status[d]) {
    uint32_t* p = nullptr;
    if (cudaMalloc(&p, STATUS_WORDS * 4) != cudaSuccess) return nullptr;
    if (cudaMemset(p, 0, STATUS_WORDS * 4) != cudaSuccess) { cudaFree(p); return nullptr; }
    g_status[d] = p;
  }
  return g_status[d];
}

// HSPEC_NVTX=1: every launch of a step sits inside an NVTX range named like its profile entry, so a timeline tool
// shows "gemm:proj_ds", "attn_partial", ... (header-only NVTX: a no-op unless a tool is attached).
static bool nvtx_on() {
  static const bool on = [] { const char* e = getenv("HSPEC_NVTX"); return e && e[0] == '1'; }();
  return on;
}

void Tracker::begin(const char* name, double flops, double bytes, double io_bytes) {
  ++launches;
  if (nvtx_on()) nvtxRangePushA(name);
  if (!profiling) return;
  if (used == entries.size()) {
    Entry e;
    cudaEventCreate(&e.a);
    cudaEventCreate(&e.b);
    entries.push_back(e);
  }
  Entry& e = entries[used];
  memset(e.name, 0, sizeof(e.name));
  strncpy(e.name, name, sizeof(e.name) - 1);
  e.flops = flops; e.bytes = bytes; e.io_bytes = io_bytes;
  cudaEventRecord(e.a, stream);
}

void Tracker::end() {
  if (nvtx_on()) nvtxRangePop();
  if (!profiling) return;
  cudaEventRecord(entries[used].b, stream);
  ++used;
}

void Tracker::destroy() {
  for (Entry& e : entries) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
  entries.clear();
  used = 0;
}

}  // namespace hspec

struct hspec_handle {
  hspec_config cfg;
  Dims d;
  std::unordered_map<std::string, Weight> w;
  std::string err;
  Tracker trk;
  uint32_t launches_last_step = 0;
  uint32_t* d_status = nullptr;
  cudaStream_t last_stream = nullptr;
  bool debug = false;
};

namespace {

int fail(hspec_handle* h, int code, const std::string& msg) {
  if (h) h->err = msg;
  g_err = msg;
  return code;
}

#define CUDA_TRY(h, expr)                                                                         \
  do {                                                                                            \
    cudaError_t e__ = (expr);                                                                     \
    if (e__ != cudaSuccess)                                                                       \
      return fail(h, HSPEC_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__) +        \
                                         (errtxt.empty() ? "" : " (" + errtxt + ")"));          \
  } while (0)

// expected (rows, cols, dtype, is_gemm_weight) of a tensor name; rows = -1 if the name is unknown
bool expected_shape(const hspec_config& c, const Dims& d, const std::string& name, int64_t* rows, int64_t* cols,
                    int* dtype, bool* gemm) {
  *gemm = false; *dtype = HSPEC_F32; *cols = 0;
  auto mat = [&](int64_t r, int64_t cc, bool g) { *rows = r; *cols = cc; *dtype = HSPEC_BF16; *gemm = g; return true; };
  auto vec = [&](int64_t r) { *rows = r; *cols = 0; *dtype = HSPEC_F32; return true; };
  if (name == "embed") return mat(c.V, c.D, false);
  if (name == "proj_r") return mat(c.r, int64_t(c.n_fuse) * c.D, true);
  if (name == "proj_ds") return mat(d.d_S, c.r, true);
  if (name == "final_norm") return vec(c.D);
  if (name == "lm_head") return mat(d.Vd, c.D, true);
  if (name == "markov_in") return c.markov_rank > 0 ? mat(c.V, c.markov_rank, true) : false;
  if (name == "markov_out") return c.markov_rank > 0 ? mat(d.Vd, c.markov_rank, true) : false;
  if (name == "vocab_map") { if (c.V_draft <= 0) return false; *rows = c.V_draft; *cols = 0; *dtype = HSPEC_I32; return true; }
  if (name.rfind("layers.", 0) != 0) return false;
  const size_t dot = name.find('.', 7);
  if (dot == std::string::npos) return false;
  const int l = atoi(name.substr(7, dot - 7).c_str());
  if (l < 0 || l >= c.L) return false;
  const std::string s = name.substr(dot + 1);
  if (s == "mamba.norm") return vec(c.D);
  if (s == "mamba.in_proj") return mat(d.d_in_proj, c.D, true);
  if (s == "mamba.dt_up") return c.dt_rank > 0 ? mat(d.H, c.dt_rank, true) : false;
  if (s == "mamba.conv_w") { *rows = d.d_xBC; *cols = c.d_conv; *dtype = HSPEC_F32; return true; }
  if (s == "mamba.conv_b") return vec(d.d_xBC);
  if (s == "mamba.dt_bias" || s == "mamba.A_log" || s == "mamba.Dskip") return vec(d.H);
  if (s == "mamba.gnorm") return vec(c.Di);
  if (s == "mamba.out_proj") return mat(c.D, c.Di, true);
  if (s == "attn.norm") return vec(c.D);
  if (s == "attn.wqkv") return mat(d.d_qkv, c.D, true);
  if (s == "attn.q_norm" || s == "attn.k_norm") return vec(c.dh);
  if (s == "attn.wo") return mat(c.D, int64_t(c.Hq) * c.dh, true);
  if (s == "mlp.norm") return vec(c.D);
  if (s == "mlp.w_gate_up") return mat(2 * int64_t(c.F), c.D, true);
  if (s == "mlp.w_down") return mat(c.D, c.F, true);
  return false;
}

std::vector<std::string> required_names(const hspec_config& c) {
  std::vector<std::string> n = {"embed", "proj_r", "proj_ds", "final_norm", "lm_head"};
  if (c.V_draft > 0) n.push_back("vocab_map");
  if (c.markov_rank > 0) { n.push_back("markov_in"); n.push_back("markov_out"); }
  for (int l = 0; l < c.L; ++l) {
    const std::string p = "layers." + std::to_string(l) + ".";
    for (const char* s : {"mamba.norm", "mamba.in_proj", "mamba.conv_w", "mamba.conv_b", "mamba.dt_bias", "mamba.A_log",
                          "mamba.Dskip", "mamba.gnorm", "mamba.out_proj", "mlp.norm", "mlp.w_gate_up", "mlp.w_down"})
      n.push_back(p + s);
    if (c.dt_rank > 0) n.push_back(p + "mamba.dt_up");
    if (c.has_attn[l])
      for (const char* s : {"attn.norm", "attn.wqkv", "attn.q_norm", "attn.k_norm", "attn.wo"}) n.push_back(p + s);
  }
  return n;
}

__global__ void bf16_to_f16_kernel(const __nv_bfloat16* __restrict__ src, __half* __restrict__ dst, size_t n,
                                   uint32_t* status) {
  pdl_wait();
  pdl_trigger();
  for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < n; i += size_t(gridDim.x) * blockDim.x)
    dst[i] = f16_sat(__bfloat162float(src[i]), status);
}

// w_gate_up [2F, K] bf16 (rows gate | up) -> fp16 with rows interleaved in blocks of 16:
// dst rows [32j, 32j+16) = gate rows [16j, 16j+16), dst rows [32j+16, 32j+32) = up rows [16j, 16j+16).
__global__ void interleave_gate_up_kernel(const __nv_bfloat16* __restrict__ src, void* __restrict__ dst, int F, int K,
                                          uint32_t* status, int keep_bf16) {
  const size_t total = size_t(2) * F * K;
  for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < total; i += size_t(gridDim.x) * blockDim.x) {
    const size_t r = i / K, c = i % K;
    const size_t blk = r >> 5, w = r & 31;
    const size_t src_row = (w < 16) ? blk * 16 + w : size_t(F) + blk * 16 + (w - 16);
    if (keep_bf16) reinterpret_cast<__nv_bfloat16*>(dst)[i] = src[src_row * K + c];
    else reinterpret_cast<__half*>(dst)[i] = f16_sat(__bfloat162float(src[src_row * K + c]), status);
  }
}

// Self-test of the bounded-wait path: waits on a barrier that nothing will ever complete, for a short limit, then
// records the give-up in the status word and returns normally (no trap, the context stays usable).
__global__ void wait_selftest_kernel(uint32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    fence_mbar_init();
    if (!mbar_wait(smem_u32(&bar), 0, limit_ns)) atomicExch(status, STATUS_TIMEOUT_SELFTEST);
  }
}

__global__ void cvt_cols_f16_kernel(const float* __restrict__ src, long long ld, int col0, int ncols, int M,
                                    void* __restrict__ dst, uint32_t* status, int bf16_out) {
  pdl_wait();
  pdl_trigger();
  const int total = M * ncols;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x)
    store_act16(dst, size_t(i), src[size_t(i / ncols) * ld + col0 + i % ncols], bf16_out != 0, status);
}

}  // namespace

extern "C" {

const char* hspec_last_error(const hspec_handle* h) { return h ? h->err.c_str() : g_err.c_str(); }

int hspec_init(const hspec_config* cfg, hspec_handle** out) {
  if (!cfg || !out) return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_init: NULL argument");
  *out = nullptr;
  if (const char* why = check_config(*cfg)) return fail(nullptr, HSPEC_ERR_BAD_SHAPE, std::string("hspec_init: ") + why);
  hspec_handle* h = new (std::nothrow) hspec_handle();
  if (!h) return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_init: out of host memory");
  h->cfg = *cfg;
  h->d = dims_of(*cfg);
  const char* dbg = getenv("HSPEC_DEBUG");
  h->debug = dbg && dbg[0] && dbg[0] != '0';
  *out = h;
  return HSPEC_OK;
}

size_t hspec_workspace_bytes(const hspec_config* cfg) {
  if (!cfg || check_config(*cfg)) return 0;
  // The layout of a step depends on its own (B, k): how the contexts are cut into chunks and how many K-slices a GEMM
  // uses change at thresholds, so a smaller step can need MORE of some scratch buffer than the largest one.  The
  // size handed out covers every (B, k) the handle accepts.
  const int max_ctx = cfg->max_pages_per_req * cfg->page_size;
  size_t total = 0;
  for (int B = 1; B <= cfg->max_batch; ++B)
    for (int k = 1; k <= cfg->max_k; ++k) {
      const size_t t = make_plan(*cfg, B, k, max_ctx).total;
      if (t > total) total = t;
    }
  return total;
}

int hspec_load_weights(hspec_handle* h, const hspec_tensor* t, int32_t n) {
  if (!h || (!t && n > 0) || n < 0) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_load_weights: bad argument");
  std::string errtxt;
  int dev_count = 0;
  if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count < 1)
    return fail(h, HSPEC_ERR_CUDA, "hspec_load_weights: no CUDA device; this library has no CPU path");
  if (!h->d_status) {
    CUDA_TRY(h, cudaMalloc(&h->d_status, STATUS_WORDS * 4));
    CUDA_TRY(h, cudaMemset(h->d_status, 0, STATUS_WORDS * 4));
  }
  for (int i = 0; i < n; ++i) {
    if (!t[i].name || !t[i].data) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_load_weights: tensor without name or data");
    const std::string name = t[i].name;
    int64_t rows, cols; int dtype; bool gemm;
    if (!expected_shape(h->cfg, h->d, name, &rows, &cols, &dtype, &gemm))
      return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_load_weights: unknown tensor name '" + name + "'");
    const int64_t got_r = t[i].shape[0], got_c = t[i].ndim > 1 ? t[i].shape[1] : 0;
    if (t[i].dtype != dtype || got_r != rows || got_c != cols || t[i].ndim != (cols ? 2 : 1))
      return fail(h, HSPEC_ERR_BAD_SHAPE, "hspec_load_weights: '" + name + "' has the wrong shape or dtype (expected [" +
                                              std::to_string(rows) + (cols ? "," + std::to_string(cols) : "") + "])");
    auto old = h->w.find(name);
    if (old != h->w.end()) { if (old->second.owned) cudaFree(old->second.data); h->w.erase(old); }
    Weight w;
    w.dtype = dtype; w.rows = rows; w.cols = cols;
    const size_t count = size_t(rows) * size_t(cols ? cols : 1);
    const size_t bytes = count * ((dtype == HSPEC_F32 || dtype == HSPEC_I32) ? 4 : 2);
    const bool bf16_mode = h->cfg.act_bf16 != 0;
    const bool is_gate_up = name.size() >= 13 && name.compare(name.size() - 13, 13, "mlp.w_gate_up") == 0 && h->cfg.F % 16 == 0;
    if (gemm && bf16_mode && !is_gate_up) {
      // bf16 operands: the matrix is used where it lies (borrowed until hspec_destroy)
      w.data = const_cast<void*>(t[i].data);
      w.owned = false;
      if (!make_tmap_16bit_2d(&w.tm, w.data, rows, cols, cols, 128, false, &errtxt))
        return fail(h, HSPEC_ERR_BAD_SHAPE, "hspec_load_weights: '" + name + "': " + errtxt);
      w.has_tm = true;
      h->w[name] = w;
      continue;
    }
    CUDA_TRY(h, cudaMalloc(&w.data, bytes));
    if (gemm) {
      // bf16 -> fp16: exact for every value with |w| in [2^-17, 65504]; smaller ones lose at most 2^-25
      const int blocks = int(std::min<size_t>((count + 255) / 256, 148 * 32));
      if (is_gate_up)
        interleave_gate_up_kernel<<<blocks, 256>>>(reinterpret_cast<const __nv_bfloat16*>(t[i].data), w.data, h->cfg.F,
                                                   int(cols), h->d_status, bf16_mode ? 1 : 0);
      else
        bf16_to_f16_kernel<<<blocks, 256>>>(reinterpret_cast<const __nv_bfloat16*>(t[i].data),
                                            reinterpret_cast<__half*>(w.data), count, h->d_status);
      CUDA_TRY(h, cudaGetLastError());
      if (!make_tmap_16bit_2d(&w.tm, w.data, rows, cols, cols, 128, !bf16_mode, &errtxt)) {
        cudaFree(w.data);
        return fail(h, HSPEC_ERR_BAD_SHAPE, "hspec_load_weights: '" + name + "': " + errtxt);
      }
      w.has_tm = true;
    } else {
      CUDA_TRY(h, cudaMemcpy(w.data, t[i].data, bytes, cudaMemcpyDeviceToDevice));
    }
    h->w[name] = w;
  }
  CUDA_TRY(h, cudaDeviceSynchronize());
  return HSPEC_OK;
}

int hspec_destroy(hspec_handle* h) {
  if (!h) return HSPEC_ERR_INVALID_ARG;
  if (h->d_status) cudaFree(h->d_status);
  for (auto& kv : h->w) if (kv.second.owned) cudaFree(kv.second.data);
  h->trk.destroy();
  delete h;
  return HSPEC_OK;
}

int hspec_get_stats(hspec_handle* h, hspec_stats* out) {
  if (!h || !out) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_get_stats: NULL argument");
  out->kernel_launches = h->trk.launches;
  out->launches_last_step = h->launches_last_step;
  out->device_status = 0;
  out->attn_rescales = out->f16_range_events = out->bad_inputs = 0;
  if (h->d_status) {
    std::string errtxt;
    uint32_t words[4] = {0, 0, 0, 0};
    CUDA_TRY(h, cudaStreamSynchronize(h->last_stream));
    CUDA_TRY(h, cudaMemcpy(words, h->d_status, sizeof(words), cudaMemcpyDeviceToHost));
    out->device_status = words[STATUS_WORD_CODE];
    out->attn_rescales = words[STATUS_WORD_RESCALES];
    out->f16_range_events = words[STATUS_WORD_F16_RANGE];
    out->bad_inputs = words[STATUS_WORD_BAD_INPUT];
  }
  if (out->device_status) return fail(h, HSPEC_ERR_TIMEOUT, "a bounded in-kernel wait gave up (device status word is set)");
  if (out->bad_inputs)
    return fail(h, HSPEC_ERR_PAGE_OUT_OF_RANGE, "a kernel met a context length or page id out of range (clamped / read as zeros)");
  if (out->f16_range_events)
    return fail(h, HSPEC_ERR_F16_RANGE, "finite values left the fp16 range and were clamped to +-65504");
  return HSPEC_OK;
}

int hspec_draft_block(hspec_handle* h, const hspec_step* in, const hspec_out* out) {
  if (!h || !in || !out) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_draft_block: NULL argument");
  const hspec_config& c = h->cfg;
  const Dims& d = h->d;
  if (in->B < 1 || in->B > c.max_batch || in->k < 1 || in->k > c.max_k)
    return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_draft_block: B or k out of range");
  if (!in->ctx_lens || !in->last_hidden || !in->last_token || !out->draft_ids || !in->workspace)
    return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_draft_block: NULL input or output pointer");
  bool any_attn = false;
  for (int l = 0; l < c.L; ++l) any_attn |= c.has_attn[l] != 0;
  if (any_attn) {
    if (!in->page_table || !in->k_pools || !in->v_pools || in->page_table_stride < 1 ||
        in->page_table_stride > c.max_pages_per_req)
      return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_draft_block: page table / pools missing or stride out of range");
    for (int s = 0; s < c.n_slots; ++s)
      if (!in->k_pools[s] || !in->v_pools[s]) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_draft_block: NULL KV pool");
  }
  if (reinterpret_cast<uintptr_t>(in->workspace) & 1023)
    return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_draft_block: workspace must be 1024-byte aligned");
  for (const std::string& nm : required_names(c))
    if (h->w.find(nm) == h->w.end()) return fail(h, HSPEC_ERR_NOT_LOADED, "hspec_draft_block: tensor '" + nm + "' was never loaded");

  const int B = in->B, k = in->k, M = B * k;
  int max_ctx = in->max_ctx > 0 ? in->max_ctx : in->page_table_stride * c.page_size;
  if (max_ctx > c.max_pages_per_req * c.page_size) max_ctx = c.max_pages_per_req * c.page_size;
  const Plan p = make_plan(c, B, k, max_ctx);
  if (in->workspace_bytes < p.total)
    return fail(h, HSPEC_ERR_WORKSPACE_TOO_SMALL, "hspec_draft_block: workspace needs " + std::to_string(p.total) + " bytes");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(in->stream);
  h->last_stream = st;
  std::string errtxt;

  if (h->debug && any_attn) {   // host-side validation of the page table (synchronises; debug only)
    std::vector<int32_t> ctx(B), pt(size_t(B) * in->page_table_stride);
    CUDA_TRY(h, cudaStreamSynchronize(st));
    CUDA_TRY(h, cudaMemcpy(ctx.data(), in->ctx_lens, sizeof(int32_t) * B, cudaMemcpyDeviceToHost));
    CUDA_TRY(h, cudaMemcpy(pt.data(), in->page_table, sizeof(int32_t) * pt.size(), cudaMemcpyDeviceToHost));
    for (int b = 0; b < B; ++b) {
      if (ctx[b] < 0 || ctx[b] > max_ctx) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_draft_block: ctx_lens out of range");
      const int np = (ctx[b] + c.page_size - 1) / c.page_size;
      for (int j = 0; j < np; ++j) {
        const int32_t pg = pt[size_t(b) * in->page_table_stride + j];
        if (pg < 0 || pg >= in->num_pages) return fail(h, HSPEC_ERR_PAGE_OUT_OF_RANGE, "hspec_draft_block: page id out of range");
      }
    }
  }

  uint8_t* ws = reinterpret_cast<uint8_t*>(in->workspace);
  float* X = reinterpret_cast<float*>(ws + p.X);
  void* U = ws + p.U;
  void* U2 = ws + p.U2;
  float* BIG = reinterpret_cast<float*>(ws + p.BIG);
  void* LH = ws + p.LH;
  void* Fv = ws + p.Fv;
  void* SINIT = ws + p.SINIT;
  void* DTL = ws + p.DTL;
  float* DT = reinterpret_cast<float*>(ws + p.DT);
  float* YG = reinterpret_cast<float*>(ws + p.YG);
  void *Q = ws + p.Q, *KB = ws + p.KB, *VB = ws + p.VB;
  Tracker* trk = &h->trk;
  trk->begin_step(st);
  const uint64_t launches0 = trk->launches;
  const double Md = double(M);

  const bool bf = c.act_bf16 != 0;                 // bf16 tensor-core operands instead of fp16
  auto W = [&](const std::string& nm) -> const Weight& { return h->w.at(nm); };
  auto fptr = [&](const std::string& nm) { return reinterpret_cast<const float*>(h->w.at(nm).data); };
  auto gemm = [&](const std::string& wname, const char* label, const void* x, int rows, int mode, void* o,
                  long long ldo) -> cudaError_t {
    const Weight& w = W(wname);
    GemmCall g{};
    g.tmW = &w.tm; g.x = x; g.f16 = !bf; g.ldx = w.cols; g.M = rows; g.n_out = int(w.rows); g.K = int(w.cols);
    g.mode = mode; g.out = o; g.ldo = ldo;
    g.splits = gemm_pick_splits(rows, g.n_out, g.K, kNumSMs, mode);
    g.splitk_ws = ws + p.SPLITK; g.splitk_ws_bytes = p.splitk_bytes;
    g.status = h->d_status; g.label = label;
    return gemm_launch(g, st, trk, &errtxt);
  };
  // element-wise launches: bracket with the tracker (name, algorithmic bytes)
#define EW(name, bytes, call) do { trk->begin(name, 0, bytes); cudaError_t e_ = (call); trk->end(); CUDA_TRY(h, e_); } while (0)

  EW("embed_rows", Md * c.D * 6, embed_rows_launch(W("embed").data, in->last_token, c.mask_id, X, B, k, c.D, st));
  // S_init = Proj_dS(Proj_r(concat h)): once per step, shared by all layers
  const void* lh_in = LH;
  if (bf && (reinterpret_cast<uintptr_t>(in->last_hidden) & 15) == 0) {
    lh_in = in->last_hidden;                       // already the operand type: read in place
  } else {
    const size_t n_lh = size_t(B) * c.n_fuse * c.D;
    trk->begin("cvt_last_hidden", 0, double(n_lh) * 4);
    if (bf) CUDA_TRY(h, cudaMemcpyAsync(LH, in->last_hidden, n_lh * 2, cudaMemcpyDeviceToDevice, st));
    else bf16_to_f16_kernel<<<int(std::min<size_t>((n_lh + 255) / 256, 148 * 8)), 256, 0, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(in->last_hidden), reinterpret_cast<__half*>(LH), n_lh, h->d_status);
    trk->end();
    CUDA_TRY(h, cudaGetLastError());
  }
  CUDA_TRY(h, gemm("proj_r", "gemm:proj_r", lh_in, B, bf ? EPI_STORE_BF16 : EPI_STORE_F16, Fv, c.r));
  // (S_init is an output the scan consumes, not a GEMM operand: it stays fp16 in both modes)
  CUDA_TRY(h, gemm("proj_ds", "gemm:proj_ds", Fv, B, EPI_STORE_F16, SINIT, d.d_S));

  for (int l = 0; l < c.L; ++l) {
    const std::string pre = "layers." + std::to_string(l) + ".";
    // ---- Mamba-2 mixer from the injected state
    EW("rmsnorm", Md * c.D * 6, rmsnorm_launch(X, fptr(pre + "mamba.norm"), U, M, c.D, c.rms_eps, st, h->d_status, bf));
    CUDA_TRY(h, gemm(pre + "mamba.in_proj", "gemm:in_proj", U, M, EPI_STORE_F32, BIG, d.d_in_proj));
    const float* dt_raw = nullptr;
    if (c.dt_rank > 0) {
      trk->begin("cvt_dt_cols", 0, Md * c.dt_rank * 6);
      cvt_cols_f16_kernel<<<(M * c.dt_rank + 255) / 256, 256, 0, st>>>(BIG, d.d_in_proj, c.Di + d.d_xBC, c.dt_rank, M,
                                                                     DTL, h->d_status, bf ? 1 : 0);
      trk->end();
      CUDA_TRY(h, cudaGetLastError());
      CUDA_TRY(h, gemm(pre + "mamba.dt_up", "gemm:dt_up", DTL, M, EPI_STORE_F32, DT, d.H));
      dt_raw = DT;
    }
    ScanCall sc{};
    sc.zxbcdt = BIG; sc.ld_in = d.d_in_proj; sc.dt_raw = dt_raw; sc.s_init = SINIT;
    sc.conv_w = fptr(pre + "mamba.conv_w"); sc.conv_b = fptr(pre + "mamba.conv_b");
    sc.dt_bias = fptr(pre + "mamba.dt_bias"); sc.A_log = fptr(pre + "mamba.A_log"); sc.Dskip = fptr(pre + "mamba.Dskip");
    sc.y_gated = YG; sc.B = B; sc.k = k; sc.Di = c.Di; sc.P = c.P; sc.N = c.N; sc.G = c.G; sc.d_conv = c.d_conv;
    sc.ws = ws + p.SCAN; sc.ws_bytes = p.scan_bytes;
    CUDA_TRY(h, scan_launch(sc, st, trk, &errtxt));
    EW("rmsnorm_gated", Md * c.Di * 6, rmsnorm_launch(YG, fptr(pre + "mamba.gnorm"), U, M, c.Di, c.rms_eps, st, h->d_status, bf));
    CUDA_TRY(h, gemm(pre + "mamba.out_proj", "gemm:out_proj", U, M, EPI_ACCUM_F32, X, c.D));
    // ---- attention over the target's KV (in place) + the block
    if (c.has_attn[l]) {
      EW("rmsnorm", Md * c.D * 6, rmsnorm_launch(X, fptr(pre + "attn.norm"), U, M, c.D, c.rms_eps, st, h->d_status, bf));
      CUDA_TRY(h, gemm(pre + "attn.wqkv", "gemm:wqkv", U, M, EPI_STORE_F32, BIG, d.d_qkv));
      EW("qk_norm_rope", Md * d.d_qkv * 6,
         qk_norm_rope_launch(BIG, fptr(pre + "attn.q_norm"), fptr(pre + "attn.k_norm"), in->ctx_lens, Q, KB, VB, B, k, c.Hq,
                             c.Hkv, c.dh, c.rope_theta, c.rms_eps, c.qk_norm, st));
      AttnCall a{};
      a.q = Q; a.kb = KB; a.vb = VB;
      a.k_pool = in->k_pools[c.kv_slot[l]]; a.v_pool = in->v_pools[c.kv_slot[l]];
      a.num_pages = in->num_pages; a.status = h->d_status;
      a.page_table = in->page_table; a.page_table_stride = in->page_table_stride; a.ctx_lens = in->ctx_lens;
      a.max_ctx = max_ctx; a.o = U; a.o_bf16 = bf; a.B = B; a.k = k; a.Hq = c.Hq; a.Hkv = c.Hkv; a.dh = c.dh;
      a.page_size = c.page_size; a.window = c.window; a.chunk_tokens = p.attn_chunk;
      a.ws = ws + p.ATT; a.ws_bytes = p.att_bytes;
      CUDA_TRY(h, attention_launch(a, st, trk, &errtxt));
      CUDA_TRY(h, gemm(pre + "attn.wo", "gemm:wo", U, M, EPI_ACCUM_F32, X, c.D));
    }
    // ---- SwiGLU MLP
    EW("rmsnorm", Md * c.D * 6, rmsnorm_launch(X, fptr(pre + "mlp.norm"), U, M, c.D, c.rms_eps, st, h->d_status, bf));
    if (c.F % 16 == 0) {
      // gate/up rows were interleaved at load: the GEMM epilogue applies SiLU(gate) * up and writes h directly.
      // U is both the GEMM's input (D columns) and h's home (F columns), so h goes to a second fp16 buffer.
      CUDA_TRY(h, gemm(pre + "mlp.w_gate_up", "gemm:gate_up", U, M, bf ? EPI_SWIGLU_BF16 : EPI_SWIGLU_F16, U2, c.F));
    } else {
      CUDA_TRY(h, gemm(pre + "mlp.w_gate_up", "gemm:gate_up", U, M, EPI_STORE_F32, BIG, 2 * c.F));
      EW("swiglu", Md * c.F * 10, swiglu_launch(BIG, U2, M, c.F, st, h->d_status, bf));
    }
    CUDA_TRY(h, gemm(pre + "mlp.w_down", "gemm:down", U2, M, EPI_ACCUM_F32, X, c.D));
  }
  if (out->hidden) EW("copy_hidden", Md * c.D * 8, copy_f32_launch(X, out->hidden, size_t(M) * c.D, st));
  // ---- final norm, LM head fused with the per-row arg-max
  EW("rmsnorm", Md * c.D * 6, rmsnorm_launch(X, fptr("final_norm"), U, M, c.D, c.rms_eps, st, h->d_status, bf));
  const int* id_map = c.V_draft > 0 ? reinterpret_cast<const int*>(W("vocab_map").data) : nullptr;
  if (c.markov_rank > 0) {
    // ---- LM head to fp32 logits, then the causal correction position by position (Sec. 3.3.3)
    float* logits = out->logits ? out->logits : reinterpret_cast<float*>(ws + p.LOGITS);
    const Weight& w = W("lm_head");
    GemmCall g{};
    g.tmW = &w.tm; g.x = U; g.f16 = !bf; g.ldx = c.D; g.M = M; g.n_out = d.Vd; g.K = c.D; g.mode = EPI_STORE_F32; g.splits = 1;
    g.out = logits; g.ldo = d.Vd; g.status = h->d_status; g.label = "gemm:lm_head";
    CUDA_TRY(h, gemm_launch(g, st, trk, &errtxt));
    MarkovCall mc{};
    mc.logits = logits; mc.ld = d.Vd; mc.W_in = W("markov_in").data; mc.tmW_out = &W("markov_out").tm; mc.W_out = W("markov_out").data; mc.f16 = !bf;
    mc.last_token = in->last_token; mc.id_map = id_map; mc.ids = out->draft_ids; mc.B = B; mc.k = k; mc.Vd = d.Vd;
    mc.r = c.markov_rank; mc.write_logits = out->logits != nullptr; mc.ws = ws + p.MARKOV; mc.status = h->d_status;
    CUDA_TRY(h, markov_launch(mc, st, trk, &errtxt));
  } else {
    const Weight& w = W("lm_head");
    GemmCall g{};
    g.tmW = &w.tm; g.x = U; g.f16 = !bf; g.ldx = c.D; g.M = M; g.n_out = d.Vd; g.K = c.D; g.mode = EPI_ARGMAX; g.splits = 1;
    g.logits = out->logits; g.ldo = d.Vd;
    g.part_val = reinterpret_cast<float*>(ws + p.AMAXV); g.part_idx = reinterpret_cast<int*>(ws + p.AMAXI);
    g.status = h->d_status; g.label = "gemm:lm_head_argmax";
    CUDA_TRY(h, gemm_launch(g, st, trk, &errtxt));
    CUDA_TRY(h, argmax_reduce_launch(g.part_val, g.part_idx, (d.Vd + 127) / 128, M, out->draft_ids, st, trk, id_map));
  }
#undef EW
  h->launches_last_step = uint32_t(trk->launches - launches0);
  return HSPEC_OK;
}

int hspec_debug_wait_selftest(hspec_handle* h, int32_t limit_ms, void* stream) {
  if (!h || limit_ms < 1 || limit_ms > 2000) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_debug_wait_selftest: bad argument");
  std::string errtxt;
  if (!h->d_status) {
    CUDA_TRY(h, cudaMalloc(&h->d_status, STATUS_WORDS * 4));
    CUDA_TRY(h, cudaMemset(h->d_status, 0, STATUS_WORDS * 4));
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  h->last_stream = st;
  wait_selftest_kernel<<<1, 32, 0, st>>>(h->d_status, (unsigned long long)limit_ms * 1000000ull);
  CUDA_TRY(h, cudaGetLastError());
  return HSPEC_OK;
}

int hspec_clear_status(hspec_handle* h) {
  if (!h) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_clear_status: NULL handle");
  std::string errtxt;
  if (h->d_status) {
    CUDA_TRY(h, cudaStreamSynchronize(h->last_stream));
    CUDA_TRY(h, cudaMemset(h->d_status, 0, STATUS_WORDS * 4));
  }
  return HSPEC_OK;
}

int hspec_set_profiling(hspec_handle* h, int32_t on) {
  if (!h) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_set_profiling: NULL handle");
  h->trk.profiling = on != 0;
  return HSPEC_OK;
}

int hspec_get_profile(hspec_handle* h, hspec_prof_entry* out, int32_t max_entries) {
  if (!h || (!out && max_entries > 0)) return fail(h, HSPEC_ERR_INVALID_ARG, "hspec_get_profile: NULL argument");
  std::string errtxt;
  if (!h->trk.profiling) return 0;
  CUDA_TRY(h, cudaStreamSynchronize(h->trk.stream));
  int n = 0;
  for (size_t i = 0; i < h->trk.used && n < max_entries; ++i, ++n) {
    const Tracker::Entry& e = h->trk.entries[i];
    float ms = 0.f;
    CUDA_TRY(h, cudaEventElapsedTime(&ms, e.a, e.b));
    memset(out[n].name, 0, sizeof(out[n].name));
    strncpy(out[n].name, e.name, sizeof(out[n].name) - 1);
    out[n].ms = ms; out[n].flops = e.flops; out[n].bytes = e.bytes; out[n].io_bytes = e.io_bytes;
  }
  return n;
}

// ------------------------------------------------------------------ single-op entry points
#define OP_TRY(expr)                                                                                         \
  do {                                                                                                       \
    cudaError_t e__ = (expr);                                                                                \
    if (e__ != cudaSuccess)                                                                                  \
      return fail(nullptr, HSPEC_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__) +             \
                                               (errtxt.empty() ? "" : " (" + errtxt + ")"));               \
  } while (0)

size_t hspec_gemm_workspace_bytes(int32_t M, int32_t n_out, int32_t K) {
  return gemm_splitk_bytes(M, n_out, 16) + gemm2_tail_bytes() + size_t((n_out + 127) / 128) * M * 8 + 2048;
}

int hspec_op_gemm(const void* x, const void* Wt, int32_t in_dtype, void* y, int32_t M, int32_t n_out, int32_t K, int64_t ldy,
                  int32_t out_dtype, int32_t accumulate, int32_t splits, void* workspace, size_t workspace_bytes,
                  void* stream) {
  if (!x || !Wt || !y || M < 1 || n_out < 1 || K < 8 || K % 8) return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_gemm: bad argument");
  if (accumulate && out_dtype != HSPEC_F32) return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_gemm: accumulate needs fp32 output");
  std::string errtxt;
  CUtensorMap tm;
  if (in_dtype != HSPEC_BF16 && in_dtype != HSPEC_F16) return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_gemm: x and W must both be bf16 or both fp16");
  if (!make_tmap_16bit_2d(&tm, Wt, n_out, K, K, 128, in_dtype == HSPEC_F16, &errtxt)) return fail(nullptr, HSPEC_ERR_BAD_SHAPE, "hspec_op_gemm: " + errtxt);
  GemmCall g{};
  g.tmW = &tm; g.x = x; g.f16 = (in_dtype == HSPEC_F16); g.ldx = K; g.M = M; g.n_out = n_out; g.K = K;
  g.mode = accumulate ? EPI_ACCUM_F32 : (out_dtype == HSPEC_BF16 ? EPI_STORE_BF16 : out_dtype == HSPEC_F16 ? EPI_STORE_F16 : EPI_STORE_F32);
  g.out = y; g.ldo = ldy;
  g.splits = splits > 0 ? splits : gemm_pick_splits(M, n_out, K, kNumSMs);
  g.splitk_ws = workspace; g.splitk_ws_bytes = workspace_bytes;
  g.status = global_status();
  if (!g.status) return fail(nullptr, HSPEC_ERR_CUDA, "hspec_op_gemm: cannot allocate the status word");
  OP_TRY(gemm_launch(g, reinterpret_cast<cudaStream_t>(stream), nullptr, &errtxt));
  return HSPEC_OK;
}

int hspec_op_lm_head_argmax(const void* x, const void* Wt, int32_t in_dtype, int32_t* ids, float* logits, int32_t M, int32_t V, int32_t K,
                            void* workspace, size_t workspace_bytes, void* stream) {
  if (!x || !Wt || !ids || !workspace || M < 1 || V < 1 || K < 8 || K % 8)
    return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_lm_head_argmax: bad argument");
  const size_t vt = (size_t(V) + 127) / 128;
  if (workspace_bytes < vt * M * 8 + 1024) return fail(nullptr, HSPEC_ERR_WORKSPACE_TOO_SMALL, "hspec_op_lm_head_argmax: workspace too small");
  std::string errtxt;
  CUtensorMap tm;
  if (!make_tmap_16bit_2d(&tm, Wt, V, K, K, 128, in_dtype == HSPEC_F16, &errtxt)) return fail(nullptr, HSPEC_ERR_BAD_SHAPE, "hspec_op_lm_head_argmax: " + errtxt);
  GemmCall g{};
  g.tmW = &tm; g.x = x; g.f16 = (in_dtype == HSPEC_F16); g.ldx = K; g.M = M; g.n_out = V; g.K = K; g.mode = EPI_ARGMAX; g.splits = 1;
  g.logits = logits; g.ldo = V;
  g.part_val = reinterpret_cast<float*>(workspace);
  g.part_idx = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(workspace) + align_up(vt * M * 4, 256));
  g.status = global_status();
  if (!g.status) return fail(nullptr, HSPEC_ERR_CUDA, "hspec_op_lm_head_argmax: cannot allocate the status word");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  OP_TRY(gemm_launch(g, st, nullptr, &errtxt));
  OP_TRY(argmax_reduce_launch(g.part_val, g.part_idx, int(vt), M, ids, st, nullptr));
  return HSPEC_OK;
}

int hspec_op_accept(const float* p_target, const float* p_draft, const float* alpha, int32_t* n_accept, int32_t B, int32_t k,
                    void* stream) {
  if (!p_target || !p_draft || !alpha || !n_accept || B < 1 || k < 1)
    return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_accept: bad argument");
  std::string errtxt;
  OP_TRY(accept_launch(p_target, p_draft, alpha, n_accept, B, k, reinterpret_cast<cudaStream_t>(stream)));
  return HSPEC_OK;
}

int hspec_op_token_probs(const float* logits, int64_t ld, const int32_t* ids, float* p, int32_t M, int32_t V, void* stream) {
  if (!logits || !ids || !p || M < 1 || V < 1 || ld < V) return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_token_probs: bad argument");
  std::string errtxt;
  OP_TRY(token_probs_launch(logits, ld, ids, p, M, V, reinterpret_cast<cudaStream_t>(stream)));
  return HSPEC_OK;
}

int hspec_op_kv_inject_write(const float* kv, const float* k_norm_w, const int32_t* req, const int32_t* pos,
                             const int32_t* page_table, int32_t page_table_stride, void* k_pool, void* v_pool, int32_t T,
                             int32_t Hkv, int32_t dh, int32_t page_size, float theta, float eps, int32_t k_norm, void* stream) {
  if (!kv || !req || !pos || !page_table || !k_pool || !v_pool || (k_norm && !k_norm_w) || T < 1 || Hkv < 1 || dh < 2 ||
      page_size < 1 || page_table_stride < 1)
    return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_kv_inject_write: bad argument");
  std::string errtxt;
  OP_TRY(kv_inject_write_launch(kv, k_norm_w, req, pos, page_table, page_table_stride, k_pool, v_pool, T, Hkv, dh, page_size,
                                theta, eps, k_norm, reinterpret_cast<cudaStream_t>(stream)));
  return HSPEC_OK;
}

int hspec_op_device_status(uint32_t* words4, int32_t clear) {
  std::string errtxt;
  uint32_t total[4] = {0, 0, 0, 0};
  OP_TRY(cudaDeviceSynchronize());
  uint32_t* blocks[2] = {nullptr, noalloc_status_if_resolved()};
  {
    const int d = current_device();
    if (d < 0) return fail(nullptr, HSPEC_ERR_CUDA, "hspec_op_device_status: no current CUDA device");
    std::lock_guard<std::mutex> lock(device_setup_mutex());
    blocks[0] = g_status[d];
  }
  for (uint32_t* blk : blocks) {
    if (!blk) continue;
    uint32_t w[4];
    OP_TRY(cudaMemcpy(w, blk, sizeof(w), cudaMemcpyDeviceToHost));
    if (total[0] == 0) total[0] = w[0];
    for (int i = 1; i < 4; ++i) total[i] += w[i];
    if (clear) OP_TRY(cudaMemset(blk, 0, STATUS_WORDS * 4));
  }
  if (words4) memcpy(words4, total, sizeof(total));
  if (total[STATUS_WORD_CODE]) return fail(nullptr, HSPEC_ERR_TIMEOUT, "a bounded in-kernel wait gave up (device status word is set)");
  if (total[STATUS_WORD_BAD_INPUT]) return fail(nullptr, HSPEC_ERR_PAGE_OUT_OF_RANGE, "a kernel met a context length or page id out of range");
  if (total[STATUS_WORD_F16_RANGE]) return fail(nullptr, HSPEC_ERR_F16_RANGE, "finite values left the fp16 range and were clamped");
  return HSPEC_OK;
}

size_t hspec_markov_workspace_bytes(int32_t B, int32_t Vd, int32_t r) {
  if (B < 1 || Vd < 1 || r < 1) return 0;
  return markov_workspace_bytes(B, Vd, r);
}

int hspec_op_markov_head(float* logits, int64_t ld, const void* W_in, const void* W_out, int32_t w_dtype, const int32_t* last_token,
                         const int32_t* id_map, int32_t* ids, int32_t B, int32_t k, int32_t Vd, int32_t r, int32_t write_logits,
                         void* workspace, size_t workspace_bytes, void* stream) {
  if (!logits || !W_in || !W_out || !last_token || !ids || !workspace || B < 1 || k < 1 || Vd < 1 || r < 8 || r % 8 || ld < Vd ||
      (w_dtype != HSPEC_F16 && w_dtype != HSPEC_BF16))
    return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_markov_head: bad argument");
  if (workspace_bytes < markov_workspace_bytes(B, Vd, r) || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return fail(nullptr, HSPEC_ERR_WORKSPACE_TOO_SMALL, "hspec_op_markov_head: workspace too small or not 256-byte aligned");
  std::string errtxt;
  CUtensorMap tm;
  if (!make_tmap_16bit_2d(&tm, W_out, Vd, r, r, 128, w_dtype == HSPEC_F16, &errtxt))
    return fail(nullptr, HSPEC_ERR_BAD_SHAPE, "hspec_op_markov_head: " + errtxt);
  MarkovCall mc{};
  mc.logits = logits; mc.ld = ld; mc.W_in = W_in; mc.tmW_out = &tm; mc.W_out = W_out; mc.f16 = (w_dtype == HSPEC_F16);
  mc.last_token = last_token; mc.id_map = id_map; mc.ids = ids; mc.B = B; mc.k = k; mc.Vd = Vd; mc.r = r;
  mc.write_logits = write_logits; mc.ws = workspace;
  mc.status = global_status();
  if (!mc.status) return fail(nullptr, HSPEC_ERR_CUDA, "hspec_op_markov_head: cannot allocate the status word");
  OP_TRY(markov_launch(mc, reinterpret_cast<cudaStream_t>(stream), nullptr, &errtxt));
  return HSPEC_OK;
}

int hspec_op_rmsnorm(const float* x, const float* w, void* y, int32_t M, int32_t n, float eps, void* stream) {
  if (!x || !w || !y || M < 1 || n < 1) return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_rmsnorm: bad argument");
  std::string errtxt;
  OP_TRY(rmsnorm_launch(x, w, y, M, n, eps, reinterpret_cast<cudaStream_t>(stream), global_status()));
  return HSPEC_OK;
}

int hspec_op_mamba_scan(const float* zxbcdt, int64_t ld_in, const float* dt_raw, const void* s_init, const float* conv_w,
                        const float* conv_b, const float* dt_bias, const float* A_log, const float* Dskip, float* y_gated,
                        int32_t B, int32_t k, int32_t Di, int32_t P, int32_t N, int32_t G, int32_t d_conv, void* workspace,
                        size_t workspace_bytes, void* stream) {
  if (!zxbcdt || !conv_w || !conv_b || !dt_bias || !A_log || !Dskip || !y_gated || B < 1 || P < 1 || P > 128 || N < 1 ||
      N > 256 || d_conv < 1 || d_conv > 4)
    return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_mamba_scan: bad argument");
  std::string errtxt;
  ScanCall sc{};
  sc.zxbcdt = zxbcdt; sc.ld_in = ld_in; sc.dt_raw = dt_raw; sc.s_init = s_init; sc.conv_w = conv_w; sc.conv_b = conv_b;
  sc.dt_bias = dt_bias; sc.A_log = A_log; sc.Dskip = Dskip; sc.y_gated = y_gated;
  sc.B = B; sc.k = k; sc.Di = Di; sc.P = P; sc.N = N; sc.G = G; sc.d_conv = d_conv;
  sc.ws = workspace; sc.ws_bytes = workspace_bytes;
  OP_TRY(scan_launch(sc, reinterpret_cast<cudaStream_t>(stream), nullptr, &errtxt));
  return HSPEC_OK;
}

size_t hspec_scan_workspace_bytes(int32_t B, int32_t k, int32_t Di, int32_t N, int32_t G) {
  return scan_workspace_bytes(B, k, Di, N, G);
}

int hspec_op_qk_norm_rope(const float* qkv, const float* qw, const float* kw, const int32_t* ctx_lens, void* q, void* kb,
                          void* vb, int32_t B, int32_t k, int32_t Hq, int32_t Hkv, int32_t dh, float theta, float eps,
                          int32_t qk_norm, void* stream) {
  if (!qkv || !ctx_lens || !q || !kb || !vb || (qk_norm && (!qw || !kw)))
    return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_qk_norm_rope: bad argument");
  std::string errtxt;
  OP_TRY(qk_norm_rope_launch(qkv, qw, kw, ctx_lens, q, kb, vb, B, k, Hq, Hkv, dh, theta, eps, qk_norm,
                             reinterpret_cast<cudaStream_t>(stream)));
  return HSPEC_OK;
}

static int resolve_chunk(int B, int Hkv, int max_ctx, int window, int chunk_tokens) {
  if (chunk_tokens > 0) return ((chunk_tokens + 127) / 128) * 128;
  return attn_pick_chunk(B, Hkv, max_ctx, window, kNumSMs);
}

size_t hspec_attention_workspace_bytes(int32_t B, int32_t k, int32_t Hq, int32_t Hkv, int32_t dh, int32_t max_ctx,
                                       int32_t window, int32_t chunk_tokens) {
  return attn_workspace_bytes(B, k, Hq, Hkv, dh, max_ctx, window, resolve_chunk(B, Hkv, max_ctx, window, chunk_tokens));
}

int hspec_op_attention(const void* q, const void* kb, const void* vb, const void* k_pool, const void* v_pool,
                       int64_t num_pages, const int32_t* page_table, int32_t page_table_stride, const int32_t* ctx_lens, int32_t max_ctx,
                       void* o, int32_t B, int32_t k, int32_t Hq, int32_t Hkv, int32_t dh, int32_t page_size, int32_t window,
                       int32_t chunk_tokens, void* workspace, size_t workspace_bytes, void* stream) {
  if (!q || !kb || !vb || !k_pool || !v_pool || !page_table || !ctx_lens || !o || !workspace || B < 1 || k < 1 ||
      k > HSPEC_MAX_K || page_size < 1)
    return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_attention: bad argument");
  std::string errtxt;
  AttnCall a{};
  a.q = q; a.kb = kb; a.vb = vb; a.k_pool = k_pool; a.v_pool = v_pool; a.page_table = page_table;
  a.num_pages = num_pages; a.status = global_status();
  if (!a.status) return fail(nullptr, HSPEC_ERR_CUDA, "hspec_op_attention: cannot allocate the status word");
  a.page_table_stride = page_table_stride; a.ctx_lens = ctx_lens;
  a.max_ctx = max_ctx > 0 ? max_ctx : page_table_stride * page_size;
  a.o = o; a.B = B; a.k = k; a.Hq = Hq; a.Hkv = Hkv; a.dh = dh; a.page_size = page_size; a.window = window;
  a.chunk_tokens = resolve_chunk(B, Hkv, a.max_ctx, window, chunk_tokens);
  a.ws = workspace; a.ws_bytes = workspace_bytes;
  OP_TRY(attention_launch(a, reinterpret_cast<cudaStream_t>(stream), nullptr, &errtxt));
  return HSPEC_OK;
}

int hspec_debug_gather_kv(const void* pool, const int32_t* page_table_row, int32_t ctx_len, int32_t page_size, int32_t Hkv,
                          int32_t dh, void* dst, void* stream) {
  if (!pool || !page_table_row || !dst || ctx_len < 0 || (Hkv * dh * 2) % 16)
    return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_debug_gather_kv: bad argument");
  std::string errtxt;
  OP_TRY(gather_kv_launch(pool, page_table_row, ctx_len, page_size, Hkv, dh, dst, reinterpret_cast<cudaStream_t>(stream)));
  return HSPEC_OK;
}

int hspec_op_swiglu(const float* gu, void* h_f16, int32_t M, int32_t F, void* stream) {
  if (!gu || !h_f16 || M < 1 || F < 1) return fail(nullptr, HSPEC_ERR_INVALID_ARG, "hspec_op_swiglu: bad argument");
  std::string errtxt;
  OP_TRY(swiglu_launch(gu, h_f16, M, F, reinterpret_cast<cudaStream_t>(stream), global_status()));
  return HSPEC_OK;
}

}  // extern "C"
