// Row-wise and element-wise kernels of the draft step (all fp32 math; bf16 only where a tensor-core
// operand is produced).
#include "common.cuh"
#include "kernels.h"

#include <cstdlib>

namespace hspec {

namespace {

// Block rows: row 0 of each request is the embedding of its last token, rows 1..k-1 the mask-token
// embedding; no positional embedding is added (paper Sec. 3.3.1).
__global__ void embed_rows_kernel(const __nv_bfloat16* __restrict__ embed, const int32_t* __restrict__ last_token,
                                  int mask_id, float* __restrict__ X, int k, int D) {
  pdl_wait();
  pdl_trigger();
  const int m = blockIdx.x;
  const int b = m / k, i = m % k;
  const int tok = (i == 0) ? last_token[b] : mask_id;
  const __nv_bfloat16* src = embed + size_t(tok) * D;
  float* dst = X + size_t(m) * D;
  if ((D & 3) == 0 && ((reinterpret_cast<uintptr_t>(embed) | reinterpret_cast<uintptr_t>(X)) & 15) == 0) {
    // four elements per thread and step: 8-byte loads, 16-byte stores
    for (int d4 = threadIdx.x; d4 < D / 4; d4 += blockDim.x) {
      const uint2 t = __ldg(reinterpret_cast<const uint2*>(src) + d4);
      reinterpret_cast<float4*>(dst)[d4] = make_float4(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u),
                                                       __uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u));
    }
    return;
  }
  for (int d = threadIdx.x; d < D; d += blockDim.x) dst[d] = __bfloat162float(src[d]);
}

__device__ __forceinline__ float block_sum(float v, float* red) {
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  const int warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if ((threadIdx.x & 31) == 0) red[warp] = v;
  __syncthreads();
  float t = (threadIdx.x < nw) ? red[threadIdx.x] : 0.f;
  if (warp == 0) {
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    if (threadIdx.x == 0) red[0] = t;
  }
  __syncthreads();
  const float r = red[0];
  __syncthreads();
  return r;
}

// y = x / sqrt(mean(x^2) + eps) * w, one CTA per row, fp16 (or bf16) out.  VPT = 16-byte vectors a thread keeps in
// registers between the two passes.
template <int VPT>
__global__ void rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ w, void* __restrict__ y,
                               int n, float eps, uint32_t* status, int bf16_out) {
  pdl_wait();
  pdl_trigger();
  __shared__ float red[32];
  const float* xr = x + size_t(blockIdx.x) * n;
  uint16_t* yr = reinterpret_cast<uint16_t*>(y) + size_t(blockIdx.x) * n;      // a row of 16-bit values, either type
  if ((n & 3) == 0 && n <= 4 * VPT * int(blockDim.x)) {
    // 16-byte loads, the row stays in registers between the two passes
    float4 v[VPT];
    const int nv = n >> 2;
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int d4 = threadIdx.x + i * blockDim.x;
      v[i] = d4 < nv ? reinterpret_cast<const float4*>(xr)[d4] : make_float4(0.f, 0.f, 0.f, 0.f);
      ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
    const float inv = rsqrtf(block_sum(ss, red) / float(n) + eps);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int d4 = threadIdx.x + i * blockDim.x;
      if (d4 < nv) {
        // (fetching the gains together with the row, before the block-wide sum, measured slower: 27 against 23 us)
        const float4 g = reinterpret_cast<const float4*>(w)[d4];
        // (a normalised value is at most sqrt(n) |w|; the saturating convert still guards a huge gain or a NaN-free
        // overflow of x * inv)
        uint2 out;
        if (bf16_out) {
          out.x = pack_bf16(v[i].x * inv * g.x, v[i].y * inv * g.y);
          out.y = pack_bf16(v[i].z * inv * g.z, v[i].w * inv * g.w);
        } else {
          const __half2 lo = __halves2half2(f16_sat(v[i].x * inv * g.x, status), f16_sat(v[i].y * inv * g.y, status));
          const __half2 hi = __halves2half2(f16_sat(v[i].z * inv * g.z, status), f16_sat(v[i].w * inv * g.w, status));
          out.x = *reinterpret_cast<const uint32_t*>(&lo);
          out.y = *reinterpret_cast<const uint32_t*>(&hi);
        }
        reinterpret_cast<uint2*>(yr)[d4] = out;
      }
    }
    return;
  }
  float ss = 0.f;
  for (int d = threadIdx.x; d < n; d += blockDim.x) { const float v = xr[d]; ss += v * v; }
  const float tot = block_sum(ss, red);
  const float inv = rsqrtf(tot / float(n) + eps);
  for (int d = threadIdx.x; d < n; d += blockDim.x) store_act16(yr, d, xr[d] * inv * w[d], bf16_out != 0, status);
}

// Per (row, head): optional RMSNorm over dh, then rotate-half RoPE at position ctx_len + i.
// The angle is one fp32 product pos * inv_freq[j]; sin/cos are the accurate library versions.
// One warp per (row, head), eight warps per block; heads run over q heads, then k heads, then v heads (v is only
// converted).
__global__ void qk_norm_rope_kernel(const float* __restrict__ qkv, const float* __restrict__ qw,
                                    const float* __restrict__ kw, const float* __restrict__ inv_freq,
                                    const int32_t* __restrict__ ctx_lens, __nv_bfloat16* __restrict__ q,
                                    __nv_bfloat16* __restrict__ kb, __nv_bfloat16* __restrict__ vb, int k, int Hq,
                                    int Hkv, int dh, float eps, int qk_norm, int n_pairs) {
  pdl_wait();
  pdl_trigger();
  const int pair = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (pair >= n_pairs) return;
  const int heads = Hq + 2 * Hkv;
  const int m = pair / heads, hh = pair % heads;
  const int lane = threadIdx.x & 31;
  const float* src = qkv + size_t(m) * (Hq + 2 * Hkv) * dh + size_t(hh) * dh;
  const int half = dh / 2;
  if (hh >= Hq + Hkv) {                               // values: plain conversion
    __nv_bfloat16* dst = vb + (size_t(m) * Hkv + (hh - Hq - Hkv)) * dh;
    for (int d = lane; d < dh; d += 32) dst[d] = __float2bfloat16_rn(src[d]);
    return;
  }
  const bool is_q = hh < Hq;
  const float* w = is_q ? qw : kw;
  float inv = 1.f;
  if (qk_norm) {
    float ss = 0.f;
    for (int d = lane; d < dh; d += 32) { const float v = src[d]; ss += v * v; }
    for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    inv = rsqrtf(ss / float(dh) + eps);
  }
  const float pos = float(ctx_lens[m / k] + m % k);
  __nv_bfloat16* dst = is_q ? q + (size_t(m) * Hq + hh) * dh : kb + (size_t(m) * Hkv + (hh - Hq)) * dh;
  for (int j = lane; j < half; j += 32) {
    float v1 = src[j] * inv, v2 = src[j + half] * inv;
    if (qk_norm) { v1 *= w[j]; v2 *= w[j + half]; }
    float sn, cs;
    sincosf(pos * inv_freq[j], &sn, &cs);
    dst[j] = __float2bfloat16_rn(v1 * cs - v2 * sn);
    dst[j + half] = __float2bfloat16_rn(v2 * cs + v1 * sn);
  }
}

// Same operation, one CTA per row (dh a multiple of 4): the row's dh/2 sines and cosines are computed once into shared
// memory and serve all Hq + Hkv heads (a warp per head recomputed them 72 times per row at the 32B-class shapes), a
// warp takes every eighth head with 8-byte loads, the loads of ROPE_HB heads in flight together.  The arithmetic per
// element is that of the kernel above.
constexpr int ROPE_HB = 5;
__global__ void __launch_bounds__(256)
qk_norm_rope_row_kernel(const float* __restrict__ qkv, const float* __restrict__ qw, const float* __restrict__ kw,
                        const float* __restrict__ inv_freq, const int32_t* __restrict__ ctx_lens,
                        __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ kb, __nv_bfloat16* __restrict__ vb,
                        int k, int Hq, int Hkv, int dh, float eps, int qk_norm) {
  pdl_wait();
  pdl_trigger();
  __shared__ __align__(8) float cs_s[64], sn_s[64];
  const int m = blockIdx.x, half = dh / 2, heads = Hq + 2 * Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float pos = float(ctx_lens[m / k] + m % k);
  for (int j = threadIdx.x; j < half; j += blockDim.x) sincosf(pos * inv_freq[j], &sn_s[j], &cs_s[j]);
  __syncthreads();
  const float* row = qkv + size_t(m) * heads * dh;
  // dh <= 128: a lane's share of a head is one pair of rotation pairs, j = 2 lane and 2 lane + 1 (lanes past dh / 4
  // hold zeros and store nothing, but take part in the warp reduction)
  const int j2 = lane;
  const bool act = j2 < half / 2;
  for (int h0 = warp; h0 < heads; h0 += 8 * ROPE_HB) {
    float2 a[ROPE_HB], b[ROPE_HB];
#pragma unroll
    for (int u = 0; u < ROPE_HB; ++u) {
      const int hh = h0 + u * 8;
      if (hh < heads && act) {
        a[u] = *reinterpret_cast<const float2*>(row + size_t(hh) * dh + 2 * j2);
        b[u] = *reinterpret_cast<const float2*>(row + size_t(hh) * dh + half + 2 * j2);
      } else {
        a[u] = b[u] = make_float2(0.f, 0.f);
      }
    }
#pragma unroll
    for (int u = 0; u < ROPE_HB; ++u) {
      const int hh = h0 + u * 8;
      if (hh >= heads) continue;                            // warp-uniform
      if (hh >= Hq + Hkv) {                                 // values: plain conversion
        if (act) {
          __nv_bfloat16* dst = vb + (size_t(m) * Hkv + (hh - Hq - Hkv)) * dh;
          *reinterpret_cast<__nv_bfloat162*>(dst + 2 * j2) = __floats2bfloat162_rn(a[u].x, a[u].y);
          *reinterpret_cast<__nv_bfloat162*>(dst + half + 2 * j2) = __floats2bfloat162_rn(b[u].x, b[u].y);
        }
        continue;
      }
      const bool is_q = hh < Hq;
      float inv = 1.f;
      if (qk_norm) {
        float ss = a[u].x * a[u].x + a[u].y * a[u].y + b[u].x * b[u].x + b[u].y * b[u].y;
        for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        inv = rsqrtf(ss / float(dh) + eps);
      }
      if (!act) continue;
      float v1x = a[u].x * inv, v1y = a[u].y * inv, v2x = b[u].x * inv, v2y = b[u].y * inv;
      if (qk_norm) {
        const float* w = is_q ? qw : kw;
        const float2 wa = *reinterpret_cast<const float2*>(w + 2 * j2), wb = *reinterpret_cast<const float2*>(w + half + 2 * j2);
        v1x *= wa.x; v1y *= wa.y; v2x *= wb.x; v2y *= wb.y;
      }
      const float2 cs = *reinterpret_cast<const float2*>(cs_s + 2 * j2), sn = *reinterpret_cast<const float2*>(sn_s + 2 * j2);
      __nv_bfloat16* dst = is_q ? q + (size_t(m) * Hq + hh) * dh : kb + (size_t(m) * Hkv + (hh - Hq)) * dh;
      *reinterpret_cast<__nv_bfloat162*>(dst + 2 * j2) = __floats2bfloat162_rn(v1x * cs.x - v2x * sn.x, v1y * cs.y - v2y * sn.y);
      *reinterpret_cast<__nv_bfloat162*>(dst + half + 2 * j2) = __floats2bfloat162_rn(v2x * cs.x + v1x * sn.x, v2y * cs.y + v1y * sn.y);
    }
  }
}

// The comparison drafters' cache write (Sec. 2.2 "KV injection in block drafting"): one warp per (new position, head).
// Key heads: optional RMSNorm over dh, rotate-half RoPE at the position, bf16, into the paged key pool; value heads:
// bf16 into the paged value pool.  Row t belongs to request req[t] and sits at absolute position pos[t].
__global__ void kv_inject_write_kernel(const float* __restrict__ kv, const float* __restrict__ kw,
                                       const float* __restrict__ inv_freq, const int32_t* __restrict__ req,
                                       const int32_t* __restrict__ pos, const int32_t* __restrict__ page_table,
                                       int page_table_stride, __nv_bfloat16* __restrict__ k_pool,
                                       __nv_bfloat16* __restrict__ v_pool, int Hkv, int dh, int page_size, float eps,
                                       int k_norm, int n_pairs) {
  pdl_wait();
  pdl_trigger();
  const int pair = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (pair >= n_pairs) return;
  const int t = pair / (2 * Hkv), hh = pair % (2 * Hkv);
  const int lane = threadIdx.x & 31;
  const float* src = kv + (size_t(t) * 2 * Hkv + hh) * dh;
  const int p = pos[t];
  const int page = page_table[size_t(req[t]) * page_table_stride + p / page_size];
  const size_t slot = (size_t(page) * page_size + p % page_size) * Hkv;
  if (hh >= Hkv) {                                    // values: plain conversion
    __nv_bfloat16* dst = v_pool + (slot + (hh - Hkv)) * dh;
    for (int d = lane; d < dh; d += 32) dst[d] = __float2bfloat16_rn(src[d]);
    return;
  }
  const int half = dh / 2;
  float inv = 1.f;
  if (k_norm) {
    float ss = 0.f;
    for (int d = lane; d < dh; d += 32) { const float v = src[d]; ss += v * v; }
    for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    inv = rsqrtf(ss / float(dh) + eps);
  }
  const float fp = float(p);
  __nv_bfloat16* dst = k_pool + (slot + hh) * dh;
  for (int j = lane; j < half; j += 32) {
    float v1 = src[j] * inv, v2 = src[j + half] * inv;
    if (k_norm) { v1 *= kw[j]; v2 *= kw[j + half]; }
    float sn, cs;
    sincosf(fp * inv_freq[j], &sn, &cs);
    dst[j] = __float2bfloat16_rn(v1 * cs - v2 * sn);
    dst[j + half] = __float2bfloat16_rn(v2 * cs + v1 * sn);
  }
}

__global__ void swiglu_kernel(const float* __restrict__ gu, void* __restrict__ h, int M, int F, uint32_t* status, int bf16_out) {
  pdl_wait();
  pdl_trigger();
  const long long total = (long long)M * F;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int m = int(idx / F), f = int(idx % F);
    const float gte = gu[size_t(m) * 2 * F + f], up = gu[size_t(m) * 2 * F + F + f];
    store_act16(h, size_t(idx), silu_f(gte) * up, bf16_out != 0, status);
  }
}

__global__ void copy_f32_kernel(const float* __restrict__ src, float* __restrict__ dst, size_t n) {
  pdl_wait();
  pdl_trigger();
  for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < n; i += size_t(gridDim.x) * blockDim.x)
    dst[i] = src[i];
}

// inv_freq table per (device, theta, dh): theta^(-2j/dh) evaluated in double, rounded to fp32, kept on that device.
struct RopeTable { int device; float theta; int dh; float* dev; };
constexpr int MAX_ROPE_TABLES = 64;
RopeTable g_rope[MAX_ROPE_TABLES];
int g_n_rope = 0;

const float* rope_table(float theta, int dh) {
  const int device = current_device();
  if (device < 0) return nullptr;
  std::lock_guard<std::mutex> lock(device_setup_mutex());
  for (int i = 0; i < g_n_rope; ++i)
    if (g_rope[i].device == device && g_rope[i].theta == theta && g_rope[i].dh == dh) return g_rope[i].dev;
  if (g_n_rope == MAX_ROPE_TABLES) return nullptr;
  float host[128];
  const int half = dh / 2;
  for (int j = 0; j < half; ++j) host[j] = float(pow(double(theta), -2.0 * double(j) / double(dh)));
  float* dev = nullptr;
  if (cudaMalloc(&dev, sizeof(float) * half) != cudaSuccess) return nullptr;
  if (cudaMemcpy(dev, host, sizeof(float) * half, cudaMemcpyHostToDevice) != cudaSuccess) { cudaFree(dev); return nullptr; }
  g_rope[g_n_rope++] = RopeTable{device, theta, dh, dev};
  return dev;
}

int grid_for(long long total, int threads) {
  long long b = (total + threads - 1) / threads;
  return int(b > 148 * 16 ? 148 * 16 : (b < 1 ? 1 : b));
}

}  // namespace

cudaError_t embed_rows_launch(const void* embed_bf16, const int32_t* last_token, int mask_id, float* X, int B, int k,
                              int D, cudaStream_t stream) {
  cudaError_t e = launch_pdl(embed_rows_kernel, dim3(B * k), dim3(256), 0, stream, (const __nv_bfloat16*)embed_bf16, last_token, mask_id, X, k, D);
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t rmsnorm_launch(const float* x, const float* w, void* y_16, int M, int n, float eps, cudaStream_t stream,
                           uint32_t* status, bool bf16_out) {
  // 256 threads with up to six vectors each as long as the row fits (n <= 6144), else 512: at n = 5120 the profiler
  // timed 16.5-17.1 us with 256 threads, 18.1-19.5 with 512, 19.6-21.0 with 128 (twelve vectors each)
  const int threads = n <= 4 * 6 * 256 ? 256 : 512;
  cudaError_t e = launch_pdl(rmsnorm_kernel<6>, dim3(M), dim3(threads), 0, stream, x, w, y_16, n, eps, status, bf16_out ? 1 : 0);
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t qk_norm_rope_launch(const float* qkv, const float* qw, const float* kw, const int32_t* ctx_lens, void* q,
                                void* kb, void* vb, int B, int k, int Hq, int Hkv, int dh, float theta, float eps,
                                int qk_norm, cudaStream_t stream) {
  if (dh > 256 || (dh & 1)) return cudaErrorInvalidValue;
  const float* tab = rope_table(theta, dh);
  if (!tab) return cudaErrorMemoryAllocation;
  if ((dh & 3) == 0 && dh <= 128) {
    cudaError_t e = launch_pdl(qk_norm_rope_row_kernel, dim3(B * k), dim3(256), 0, stream, qkv, qw, kw, tab, ctx_lens,
                               (__nv_bfloat16*)q, (__nv_bfloat16*)kb, (__nv_bfloat16*)vb, k, Hq, Hkv, dh, eps, qk_norm);
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  const int n_pairs = B * k * (Hq + 2 * Hkv);
  cudaError_t e = launch_pdl(qk_norm_rope_kernel, dim3((n_pairs + 7) / 8), dim3(256), 0, stream, qkv, qw, kw, tab, ctx_lens,
                             (__nv_bfloat16*)q, (__nv_bfloat16*)kb, (__nv_bfloat16*)vb, k, Hq, Hkv, dh, eps, qk_norm, n_pairs);
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t kv_inject_write_launch(const float* kv, const float* kw, const int32_t* req, const int32_t* pos,
                                   const int32_t* page_table, int page_table_stride, void* k_pool, void* v_pool, int T,
                                   int Hkv, int dh, int page_size, float theta, float eps, int k_norm, cudaStream_t stream) {
  if (dh > 256 || (dh & 1)) return cudaErrorInvalidValue;
  const float* tab = rope_table(theta, dh);
  if (!tab) return cudaErrorMemoryAllocation;
  const int n_pairs = T * 2 * Hkv;
  kv_inject_write_kernel<<<(n_pairs + 7) / 8, 256, 0, stream>>>(kv, kw, tab, req, pos, page_table, page_table_stride,
                                                                (__nv_bfloat16*)k_pool, (__nv_bfloat16*)v_pool, Hkv, dh,
                                                                page_size, eps, k_norm, n_pairs);
  return cudaGetLastError();
}

cudaError_t swiglu_launch(const float* gu, void* h_16, int M, int F, cudaStream_t stream, uint32_t* status, bool bf16_out) {
  cudaError_t e = launch_pdl(swiglu_kernel, dim3(grid_for((long long)M * F, 256)), dim3(256), 0, stream, gu, h_16, M, F,
                             status, bf16_out ? 1 : 0);
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t copy_f32_launch(const float* src, float* dst, size_t n, cudaStream_t stream) {
  cudaError_t e = launch_pdl(copy_f32_kernel, dim3(grid_for((long long)n, 256)), dim3(256), 0, stream, src, dst, n);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace hspec
