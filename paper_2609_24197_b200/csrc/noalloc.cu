// LM head + arg-max for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they draft: a serving engine that has
// already handed every free byte of HBM to its KV-cache pool (a later allocation simply fails), a latency-critical
// decode loop that cannot afford the implicit device synchronisation and driver lock an allocation takes, or a
// plug-in that is given device pointers but no allocator.  For them the per-tile (max, index) partials of the fused
// arg-max — the scratch that hspec_op_lm_head_argmax takes from a caller-allocated workspace — live in a fixed
// array inside the library's own device image, together with the status word for bounded waits.
//
// The array is part of every process image that loads the library: each GPU that loads it holds these bytes until
// the process exits.  All calls share it, so two calls that overlap on the GPU (different streams) race on the
// partials; the contents left by one call are garbage to the next, which overwrites every slot it reads.
#include "../../include/hspec.h"

#include <mutex>
#include <string>

#include "kernels.h"

namespace {

constexpr int NA_MAX_ROWS = 512;        // activation rows per call
constexpr int NA_MAX_TILES = 2048;      // 128-row vocabulary tiles: V <= 262144
constexpr int NA_MAX_DEVICES = 64;

struct NoAllocScratch {
  uint32_t status[64];                                   // word 0: bounded-wait status (must start at zero: it does,
                                                         // and only a give-up ever writes it)
  float part_val[size_t(NA_MAX_TILES) * NA_MAX_ROWS];
  int part_idx[size_t(NA_MAX_TILES) * NA_MAX_ROWS];
};

// 8 MiB + 256 B per GPU.  In HOST code this name is only a handle for cudaGetSymbolAddress, not a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

std::mutex g_setup_mutex;
void* g_scratch_ptr[NA_MAX_DEVICES] = {};

// Once per device, with that device current: resolve the array's device address.
int scratch_for_current_device(NoAllocScratch** out, std::string* why) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { *why = std::string("cudaGetDevice: ") + cudaGetErrorString(e); return HSPEC_ERR_CUDA; }
  if (dev < 0 || dev >= NA_MAX_DEVICES) { *why = "device index out of range"; return HSPEC_ERR_INVALID_ARG; }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || p == nullptr) {
      *why = std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e);
      return HSPEC_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
  }
  *out = reinterpret_cast<NoAllocScratch*>(g_scratch_ptr[dev]);
  return HSPEC_OK;
}

}  // namespace

namespace hspec {
uint32_t* noalloc_status_if_resolved() {
  const int dev = current_device();
  if (dev < 0 || dev >= NA_MAX_DEVICES) return nullptr;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  return g_scratch_ptr[dev] ? reinterpret_cast<NoAllocScratch*>(g_scratch_ptr[dev])->status : nullptr;
}
}  // namespace hspec

namespace {

int na_fail(int code, const std::string& msg) {
  hspec::set_last_error("hspec_op_lm_head_argmax_noalloc: " + msg);
  return code;
}

}  // namespace

extern "C" int hspec_op_lm_head_argmax_noalloc(const void* x, const void* W, int32_t in_dtype, int32_t* ids, float* logits,
                                               int32_t M, int32_t V, int32_t K, void* stream) {
  using namespace hspec;
  if (!x || !W || !ids || M < 1 || V < 1 || K < 8 || K % 8) return na_fail(HSPEC_ERR_INVALID_ARG, "bad argument");
  if (in_dtype != HSPEC_BF16 && in_dtype != HSPEC_F16) return na_fail(HSPEC_ERR_INVALID_ARG, "x and W must both be bf16 or both fp16");
  const int tiles = 2 * ((V + 255) / 256);               // 128-row tiles, counted in pairs as the 2-SM kernel indexes them
  if (M > NA_MAX_ROWS || tiles > NA_MAX_TILES)
    return na_fail(HSPEC_ERR_BAD_SHAPE, "the built-in scratch holds at most " + std::to_string(NA_MAX_ROWS) + " rows and a vocabulary of " +
                                            std::to_string(NA_MAX_TILES * 128) + " (got M=" + std::to_string(M) + ", V=" + std::to_string(V) +
                                            "); use hspec_op_lm_head_argmax with a workspace instead");
  std::string why;
  NoAllocScratch* s = nullptr;
  if (int rc = scratch_for_current_device(&s, &why)) return na_fail(rc, why);
  CUtensorMap tm;
  if (!make_tmap_16bit_2d(&tm, W, V, K, K, 128, in_dtype == HSPEC_F16, &why)) return na_fail(HSPEC_ERR_BAD_SHAPE, why);
  GemmCall g{};
  g.tmW = &tm; g.x = x; g.f16 = (in_dtype == HSPEC_F16); g.ldx = K; g.M = M; g.n_out = V; g.K = K; g.mode = EPI_ARGMAX; g.splits = 1;
  g.logits = logits; g.ldo = V;
  g.part_val = s->part_val; g.part_idx = s->part_idx;     // device addresses obtained above, never the symbol itself
  g.status = s->status;
  g.label = "gemm:lm_head_argmax";
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t e = gemm_launch(g, st, nullptr, &why);
  if (e != cudaSuccess) return na_fail(HSPEC_ERR_CUDA, std::string(cudaGetErrorString(e)) + (why.empty() ? "" : " (" + why + ")"));
  e = argmax_reduce_launch(g.part_val, g.part_idx, (V + 127) / 128, M, ids, st, nullptr);
  if (e != cudaSuccess) return na_fail(HSPEC_ERR_CUDA, cudaGetErrorString(e));
  return HSPEC_OK;
}
