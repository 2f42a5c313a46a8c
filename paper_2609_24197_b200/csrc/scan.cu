// Mamba-2 mixer core over the k block rows, started from the injected state (paper Sec. 3.3.1).
//
// One CTA per (request, head).  Because the recurrence S_i = a_i S_{i-1} + dt_i x_i B_i^T is linear,
// all k positions are evaluated in one pass without carrying the state:
//   y_t = exp(c_t) * (S_init C_t)  +  sum_{s<=t} exp(c_t - c_s) dt_s (C_t . B_s) x_s  +  D x_t,
//   c_t = sum_{r<=t} dt_r A   (inclusive prefix sum over the block positions, one warp shuffle scan).
// S_init (fp16 [P, N] per head) is read from HBM exactly once with 16-byte loads; it is the only
// large operand, so the kernel is bound by that read.  The causal depthwise conv + SiLU of x, B, C
// (zero left context), softplus(dt), the D skip and the SiLU(z) gate are fused around it.
#include "common.cuh"
#include "kernels.h"

namespace hspec {

namespace {

constexpr int SCAN_THREADS = 128;
constexpr int KMAX = 32;

struct ScanArgs {
  const float* zxbcdt; long long ld_in;
  const float* dt_raw;
  const __half* s_init;
  const float *conv_w, *conv_b, *dt_bias, *A_log, *Dskip;
  float* y;
  int B, k, Di, P, N, G, H, d_conv, d_xBC;
  int NP;          // padded N (row pitch of the staged state in floats)
};

__device__ __forceinline__ float softplus_f(float v) { return v > 20.f ? v : log1pf(expf(v)); }

__global__ void __launch_bounds__(SCAN_THREADS)
mamba_scan_kernel(ScanArgs a) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ __align__(16) float sm[];
  const int tid = threadIdx.x;
  const int h = blockIdx.x, b = blockIdx.y;
  const int g = h / (a.H / a.G);
  const int k = a.k, P = a.P, N = a.N;
  float* xs = sm;                    // [k][P]
  float* Bs = xs + KMAX * P;         // [k][N]
  float* Cs = Bs + KMAX * N;         // [k][N]
  float* Wm = Cs + KMAX * N;         // [k][k]  exp(c_t - c_s) dt_s (C_t . B_s), s <= t
  float* dec = Wm + KMAX * KMAX;     // [k]     exp(c_t)
  float* dts = dec + KMAX;           // [k]
  float* cum = dts + KMAX;           // [k]
  float* Ss = cum + KMAX;            // [P][NP] staged S_init (fp32)
  const size_t row0 = size_t(b) * k;

  // ---- conv + SiLU for this head's x channels and its group's B, C channels
  const int n_ch = P + 2 * N;
  for (int idx = tid; idx < k * n_ch; idx += SCAN_THREADS) {
    const int i = idx / n_ch, cc = idx % n_ch;
    int ch;                          // channel inside xBC
    if (cc < P) ch = h * P + cc;
    else if (cc < P + N) ch = a.Di + g * N + (cc - P);
    else ch = a.Di + a.G * N + g * N + (cc - P - N);
    float acc = a.conv_b[ch];
    for (int j = 0; j < a.d_conv; ++j) {
      const int src = i - (a.d_conv - 1) + j;
      if (src >= 0) acc += a.conv_w[ch * a.d_conv + j] * a.zxbcdt[(row0 + src) * a.ld_in + a.Di + ch];
    }
    const float v = silu_f(acc);
    if (cc < P) xs[i * P + cc] = v;
    else if (cc < P + N) Bs[i * N + (cc - P)] = v;
    else Cs[i * N + (cc - P - N)] = v;
  }
  // ---- dt, cumulative log-decay (warp 0: inclusive shuffle scan over the k <= 32 positions)
  if (tid < 32) {
    float dt = 0.f, dA = 0.f;
    if (tid < k) {
      const float raw = a.dt_raw ? a.dt_raw[(row0 + tid) * a.H + h]
                                 : a.zxbcdt[(row0 + tid) * a.ld_in + a.Di + a.d_xBC + h];
      dt = softplus_f(raw + a.dt_bias[h]);
      dA = dt * (-expf(a.A_log[h]));
    }
    float c = dA;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const float up = __shfl_up_sync(0xffffffffu, c, off);
      if (tid >= off) c += up;
    }
    if (tid < k) { dts[tid] = dt; cum[tid] = c; dec[tid] = expf(c); }
  }
  // ---- stage S_init[b, h] (fp16 -> fp32), 16-byte loads
  if (a.s_init != nullptr) {
    const __half* src = a.s_init + (size_t(b) * a.H + h) * P * N;
    if ((N & 7) == 0) {
      const int vec = P * N / 8;
      for (int idx = tid; idx < vec; idx += SCAN_THREADS) {
        const uint4 raw = reinterpret_cast<const uint4*>(src)[idx];
        const int p = (idx * 8) / N, n = (idx * 8) % N;
        float* d = Ss + p * a.NP + n;
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[e]));
          d[2 * e] = f.x;
          d[2 * e + 1] = f.y;
        }
      }
    } else {
      for (int idx = tid; idx < P * N; idx += SCAN_THREADS)
        Ss[(idx / N) * a.NP + idx % N] = __half2float(src[idx]);
    }
  }
  __syncthreads();
  // ---- W[t][s] = exp(c_t - c_s) dt_s (C_t . B_s) for s <= t
  for (int idx = tid; idx < k * k; idx += SCAN_THREADS) {
    const int t = idx / k, s = idx % k;
    float w = 0.f;
    if (s <= t) {
      float dot = 0.f;
      for (int n = 0; n < N; ++n) dot += Cs[t * N + n] * Bs[s * N + n];
      w = expf(cum[t] - cum[s]) * dts[s] * dot;
    }
    Wm[t * KMAX + s] = w;
  }
  __syncthreads();
  // ---- outputs: thread owns head channel p for all k positions
  const float Dh = a.Dskip[h];
  for (int p = tid; p < P; p += SCAN_THREADS) {
    float acc[KMAX];
#pragma unroll
    for (int t = 0; t < KMAX; ++t) acc[t] = 0.f;
    if (a.s_init != nullptr) {
      const float* srow = Ss + p * a.NP;
      for (int n = 0; n < N; ++n) {
        const float sv = srow[n];
#pragma unroll
        for (int t = 0; t < KMAX; ++t)
          if (t < k) acc[t] += Cs[t * N + n] * sv;
      }
    }
#pragma unroll
    for (int t = 0; t < KMAX; ++t) {
      if (t < k) {
        float y = dec[t] * acc[t] + Dh * xs[t * P + p];
        for (int s = 0; s <= t; ++s) y += Wm[t * KMAX + s] * xs[s * P + p];
        const size_t row = row0 + t;
        const float z = a.zxbcdt[row * a.ld_in + h * P + p];
        a.y[row * a.Di + h * P + p] = y * silu_f(z);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// Fast path for the serving shapes (P = 64, N = 128 here; any N % 32 == 0, P % 8 == 0 instantiation):
// one warp per head, HPC heads of one B/C group per CTA.  The state term  Y[t, p] = sum_n C[t, n] S[p, n]
// is a [k x N] x [N x P] contraction per head and runs on mma.sync m16n8k16 (fp16 in, fp32 out):
//   * S_init goes from HBM straight into the B fragments: each lane loads 16 contiguous bytes
//     S[p = 8j + lane/4][32 kp + 8 (lane%4) .. +7], which feed TWO k-steps; the contraction index is
//     permuted accordingly (a sum does not care), and the A fragments of C use the same permutation;
//   * no shared-memory staging of the state, every byte of S_init is read exactly once.
// The conv + SiLU of the group's B and C is computed once per CTA and shared by its heads; the k x k
// intra-block term, the decay prefix sums (warp shuffle scan), the D skip and the SiLU(z) gate stay fp32.
template <int P, int N, int MT>
__global__ void __launch_bounds__(128)
mamba_scan_mma_kernel(ScanArgs a) {
  pdl_wait();
  pdl_trigger();
  constexpr int HPC = 4;                 // heads (= warps) per CTA
  constexpr int NT = P / 8;              // n-tiles of the MMA (head channels)
  constexpr int KP = N / 32;             // k-step pairs
  constexpr int ROWS = MT * 16;          // padded block positions
  extern __shared__ __align__(16) float sm[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h0 = blockIdx.x * HPC, b = blockIdx.y;
  const int hpg = a.H / a.G;
  const int g = h0 / hpg;
  const int k = a.k;
  float* Bs = sm;                                    // [ROWS][N+1]
  float* Cs = Bs + ROWS * (N + 1);                   // [ROWS][N+1]
  float* CB = Cs + ROWS * (N + 1);                   // [ROWS][ROWS+1]   C_t . B_s
  float* xs = CB + ROWS * (ROWS + 1);                // [ROWS][HPC*P]
  float* Wm = xs + ROWS * HPC * P;                   // [HPC][ROWS][ROWS+1]
  float* dts = Wm + HPC * ROWS * (ROWS + 1);         // [HPC][ROWS]
  float* cum = dts + HPC * ROWS;                     // [HPC][ROWS]
  __half* C16 = reinterpret_cast<__half*>(cum + HPC * ROWS);   // [ROWS][N] fp16 head of C (rows >= k are zero)
  __half* C16lo = C16 + ROWS * N;                              // [ROWS][N] fp16 of the remainder C - head
  const size_t row0 = size_t(b) * k;

  // ---- phase 1: causal conv + SiLU for x of the CTA's heads and B, C of their group
  constexpr int NCH = HPC * P + 2 * N;
  for (int idx = tid; idx < ROWS * NCH; idx += 128) {
    const int i = idx / NCH, cc = idx % NCH;
    float v = 0.f;
    if (i < k) {
      int ch;
      if (cc < HPC * P) ch = h0 * P + cc;
      else if (cc < HPC * P + N) ch = a.Di + g * N + (cc - HPC * P);
      else ch = a.Di + a.G * N + g * N + (cc - HPC * P - N);
      float acc = a.conv_b[ch];
      for (int j = 0; j < a.d_conv; ++j) {
        const int src = i - (a.d_conv - 1) + j;
        if (src >= 0) acc += a.conv_w[ch * a.d_conv + j] * a.zxbcdt[(row0 + src) * a.ld_in + a.Di + ch];
      }
      v = silu_f(acc);
    }
    if (cc < HPC * P) xs[i * HPC * P + cc] = v;
    else if (cc < HPC * P + N) Bs[i * (N + 1) + (cc - HPC * P)] = v;
    else {
      // C = hi + lo with both parts fp16: the tensor-core contraction then carries ~22 bits of C
      const __half hi = __float2half_rn(v);
      Cs[i * (N + 1) + (cc - HPC * P - N)] = v;
      C16[i * N + (cc - HPC * P - N)] = hi;
      C16lo[i * N + (cc - HPC * P - N)] = __float2half_rn(v - __half2float(hi));
    }
  }
  // ---- per head (warp): dt, inclusive prefix sum of dt * A over the block positions
  const int h = h0 + warp;
  {
    float dt = 0.f, dA = 0.f;
    if (lane < k) {
      const float raw = a.dt_raw ? a.dt_raw[(row0 + lane) * a.H + h]
                                 : a.zxbcdt[(row0 + lane) * a.ld_in + a.Di + a.d_xBC + h];
      dt = softplus_f(raw + a.dt_bias[h]);
      dA = dt * (-expf(a.A_log[h]));
    }
    float c = dA;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const float up = __shfl_up_sync(0xffffffffu, c, off);
      if (lane >= off) c += up;
    }
    if (lane < ROWS) { dts[warp * ROWS + lane] = dt; cum[warp * ROWS + lane] = c; }
  }
  __syncthreads();
  // ---- phase 2: CB[t][s] = C_t . B_s (shared by the CTA's heads), s <= t
  for (int idx = tid; idx < ROWS * ROWS; idx += 128) {
    const int t = idx / ROWS, s2 = idx % ROWS;
    float dot = 0.f;
    if (s2 <= t && t < k) {
      const float* cr = Cs + t * (N + 1);
      const float* br = Bs + s2 * (N + 1);
#pragma unroll 8
      for (int n = 0; n < N; ++n) dot += cr[n] * br[n];
    }
    CB[t * (ROWS + 1) + s2] = dot;
  }
  __syncthreads();
  // ---- per head: W[t][s] = exp(c_t - c_s) dt_s CB[t][s]
  float* Wh = Wm + warp * ROWS * (ROWS + 1);
  for (int idx = lane; idx < ROWS * ROWS; idx += 32) {
    const int t = idx / ROWS, s2 = idx % ROWS;
    float w = 0.f;
    if (s2 <= t && t < k) w = expf(cum[warp * ROWS + t] - cum[warp * ROWS + s2]) * dts[warp * ROWS + s2] * CB[t * (ROWS + 1) + s2];
    Wh[t * (ROWS + 1) + s2] = w;
  }
  __syncwarp();

  // ---- phase 3: state term on the tensor cores, S_init read once from global into the B fragments
  const int gq = lane >> 2, tq = lane & 3;
  float acc[MT][NT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int j = 0; j < NT; ++j) { acc[mt][j][0] = acc[mt][j][1] = acc[mt][j][2] = acc[mt][j][3] = 0.f; }
  if (a.s_init != nullptr) {
    const __half* S = a.s_init + (size_t(b) * a.H + h) * P * N;
#pragma unroll
    for (int kp = 0; kp < KP; ++kp) {
      uint4 sv[NT];
#pragma unroll
      for (int j = 0; j < NT; ++j)
        sv[j] = __ldg(reinterpret_cast<const uint4*>(S + size_t(j * 8 + gq) * N + kp * 32 + tq * 8));
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const uint4 c_lo = *reinterpret_cast<const uint4*>(C16 + (mt * 16 + gq) * N + kp * 32 + tq * 8);
        const uint4 c_hi = *reinterpret_cast<const uint4*>(C16 + (mt * 16 + gq + 8) * N + kp * 32 + tq * 8);
        const uint4 r_lo = *reinterpret_cast<const uint4*>(C16lo + (mt * 16 + gq) * N + kp * 32 + tq * 8);
        const uint4 r_hi = *reinterpret_cast<const uint4*>(C16lo + (mt * 16 + gq + 8) * N + kp * 32 + tq * 8);
        const uint32_t a0[4] = {c_lo.x, c_hi.x, c_lo.y, c_hi.y};     // first virtual k-step
        const uint32_t a1[4] = {c_lo.z, c_hi.z, c_lo.w, c_hi.w};     // second virtual k-step
        const uint32_t e0[4] = {r_lo.x, r_hi.x, r_lo.y, r_hi.y};     // the same two k-steps of the remainder
        const uint32_t e1[4] = {r_lo.z, r_hi.z, r_lo.w, r_hi.w};
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          mma_f16_16816(acc[mt][j], a0, sv[j].x, sv[j].y);
          mma_f16_16816(acc[mt][j], a1, sv[j].z, sv[j].w);
          mma_f16_16816(acc[mt][j], e0, sv[j].x, sv[j].y);
          mma_f16_16816(acc[mt][j], e1, sv[j].z, sv[j].w);
        }
      }
    }
  }
  // ---- epilogue: decay, intra-block term, D skip, gate
  const float Dh = a.Dskip[h];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int t = mt * 16 + gq + half * 8;
      if (t >= k) continue;
      const float dec = expf(cum[warp * ROWS + t]);
      float y[NT][2];
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const float2 xv = *reinterpret_cast<const float2*>(xs + t * HPC * P + warp * P + j * 8 + tq * 2);
        y[j][0] = dec * acc[mt][j][half * 2] + Dh * xv.x;
        y[j][1] = dec * acc[mt][j][half * 2 + 1] + Dh * xv.y;
      }
      for (int s2 = 0; s2 <= t; ++s2) {
        const float w = Wh[t * (ROWS + 1) + s2];
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          const float2 xv = *reinterpret_cast<const float2*>(xs + s2 * HPC * P + warp * P + j * 8 + tq * 2);
          y[j][0] += w * xv.x;
          y[j][1] += w * xv.y;
        }
      }
      const size_t row = row0 + t;
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const int col = h * P + j * 8 + tq * 2;
        const float2 z = *reinterpret_cast<const float2*>(a.zxbcdt + row * a.ld_in + col);
        *reinterpret_cast<float2*>(a.y + row * a.Di + col) = make_float2(y[j][0] * silu_f(z.x), y[j][1] * silu_f(z.y));
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// Three-kernel form of the fast path (used when the caller provides scratch): the small per-position
// operands are prepared once per request and group, so the kernel that streams S_init has no
// block-wide phases in front of its loads.
//   scan_conv_kernel   causal depthwise conv + SiLU of every xBC channel (thread = 4 channels x 4 positions);
//                      C is also written as fp16 head + fp16 remainder for the tensor-core contraction
//   scan_cb_kernel     CB[b, g, t, s] = C_t . B_s for s <= t
//   mamba_scan_stream_kernel  one warp per head: everything it needs is fetched up front (cp.async for the
//                      shared operands, 16-byte loads of S_init straight into the MMA fragments)
constexpr int CONV_ROWS = 4;                                 // block positions per thread
// thread = (VEC adjacent channels, group of four block positions): the filter reads raw inputs only, so the groups are
// independent; a thread's seven (vector) loads are in flight together and it needs few registers.  VEC = 4 (16-byte
// loads and stores) when every channel offset and row stride is a multiple of four, else 1.  (One thread per channel
// walking all k rows held 72 registers, three blocks per SM, and reached 25 % of the DRAM peak with its warps waiting
// on loads; one channel and four rows per thread was bound by the instruction issue, 85 %, most of it set-up.)
template <int VEC>
__global__ void __launch_bounds__(256)
scan_conv_kernel(ScanArgs a, float* __restrict__ xact, __half* __restrict__ c16) {
  pdl_wait();
  pdl_trigger();
  const int ch = (blockIdx.x * blockDim.x + threadIdx.x) * VEC;
  const int n_grp = (a.k + CONV_ROWS - 1) / CONV_ROWS;
  const int b = blockIdx.y / n_grp, i0 = (blockIdx.y % n_grp) * CONV_ROWS;
  if (ch >= a.d_xBC) return;
  float w[VEC][4], bias[VEC];
#pragma unroll
  for (int v = 0; v < VEC; ++v) {
    if (VEC == 4 && a.d_conv == 4) {                         // a channel's four taps in one 16-byte load
      const float4 t = __ldg(reinterpret_cast<const float4*>(a.conv_w) + ch + v);
      w[v][0] = t.x; w[v][1] = t.y; w[v][2] = t.z; w[v][3] = t.w;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) w[v][j] = (j >= 4 - a.d_conv) ? a.conv_w[(ch + v) * a.d_conv + j - (4 - a.d_conv)] : 0.f;   // right-aligned taps
    }
  }
  if (VEC == 4) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(a.conv_b + ch));
    bias[0] = t.x; bias[VEC > 1 ? 1 : 0] = t.y; bias[VEC > 1 ? 2 : 0] = t.z; bias[VEC > 1 ? 3 : 0] = t.w;
  } else {
    bias[0] = a.conv_b[ch];
  }
  const size_t row0 = size_t(b) * a.k;
  const int GN = a.G * a.N;
  const int c_col = ch - a.Di - GN;                          // >= 0 for C channels
  float in[CONV_ROWS + 3][VEC];                              // rows i0 - 3 .. i0 + 3 (zero left context before the block)
#pragma unroll
  for (int j = 0; j < CONV_ROWS + 3; ++j) {
    const int i = i0 - 3 + j;
    const bool ok = i >= 0 && i < a.k;
    const float* src = a.zxbcdt + (row0 + (ok ? i : 0)) * a.ld_in + a.Di + ch;
    if (VEC == 4) {
      const float4 t = ok ? __ldg(reinterpret_cast<const float4*>(src)) : make_float4(0.f, 0.f, 0.f, 0.f);
      in[j][0] = t.x; in[j][VEC > 1 ? 1 : 0] = t.y; in[j][VEC > 1 ? 2 : 0] = t.z; in[j][VEC > 1 ? 3 : 0] = t.w;
    } else {
      in[j][0] = ok ? __ldg(src) : 0.f;
    }
  }
#pragma unroll
  for (int r = 0; r < CONV_ROWS; ++r) {
    const int i = i0 + r;
    if (i >= a.k) break;
    float o[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v)
      o[v] = silu_f(bias[v] + w[v][0] * in[r][v] + w[v][1] * in[r + 1][v] + w[v][2] * in[r + 2][v] + w[v][3] * in[r + 3][v]);
    float* dst = xact + (row0 + i) * a.d_xBC + ch;
    if (VEC == 4) *reinterpret_cast<float4*>(dst) = make_float4(o[0], o[VEC > 1 ? 1 : 0], o[VEC > 1 ? 2 : 0], o[VEC > 1 ? 3 : 0]);
    else dst[0] = o[0];
    if (c_col >= 0) {
      __half hi[VEC], lo[VEC];
#pragma unroll
      for (int v = 0; v < VEC; ++v) { hi[v] = __float2half_rn(o[v]); lo[v] = __float2half_rn(o[v] - __half2float(hi[v])); }
      __half* d_hi = c16 + ((row0 + i) * 2 + 0) * GN + c_col;
      __half* d_lo = c16 + ((row0 + i) * 2 + 1) * GN + c_col;
      if (VEC == 4) {
        *reinterpret_cast<uint2*>(d_hi) = *reinterpret_cast<const uint2*>(hi);
        *reinterpret_cast<uint2*>(d_lo) = *reinterpret_cast<const uint2*>(lo);
      } else {
        d_hi[0] = hi[0];
        d_lo[0] = lo[0];
      }
    }
  }
}

// CB[b, g, t, s] = C_t . B_s for s <= t.  One block per (request, group): the block's B and C rows are staged in shared
// memory (rows padded by four floats so that the 16-byte reads of a warp's threads spread over the banks), each thread
// takes (t, s) pairs with float4 dot products in the order n = 0 .. N - 1 of the scalar loop it replaces (that loop read
// both rows from global memory one float at a time and ran at the L1's limit).
__global__ void __launch_bounds__(256)
scan_cb_kernel(ScanArgs a, const float* __restrict__ xact, float* __restrict__ cb) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ __align__(16) float cb_sm[];
  const int g = blockIdx.x, b = blockIdx.y;
  const int k = a.k, N = a.N, ldr = N + 4;
  const size_t row0 = size_t(b) * k;
  const int GN = a.G * N;
  float* Bs = cb_sm;                 // [k][N + 4]
  float* Cs = cb_sm + k * ldr;       // [k][N + 4]
  for (int idx = threadIdx.x; idx < 2 * k * (N / 4); idx += blockDim.x) {
    const int which = idx / (k * (N / 4)), rem = idx % (k * (N / 4)), r = rem / (N / 4), c4 = rem % (N / 4);
    const float4 v = *reinterpret_cast<const float4*>(xact + (row0 + r) * a.d_xBC + a.Di + which * GN + g * N + c4 * 4);
    *reinterpret_cast<float4*>((which ? Cs : Bs) + r * ldr + c4 * 4) = v;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < k * k; idx += blockDim.x) {
    const int t = idx / k, s2 = idx % k;
    float dot = 0.f;
    if (s2 <= t) {
      const float4* cr = reinterpret_cast<const float4*>(Cs + t * ldr);
      const float4* br = reinterpret_cast<const float4*>(Bs + s2 * ldr);
      for (int n4 = 0; n4 < N / 4; ++n4) {
        const float4 c = cr[n4], bb = br[n4];
        dot += c.x * bb.x; dot += c.y * bb.y; dot += c.z * bb.z; dot += c.w * bb.w;
      }
    }
    cb[((size_t(b) * a.G + g) * KMAX + t) * KMAX + s2] = dot;
  }
}

template <int P, int N, int MT>
__global__ void __launch_bounds__(128, MT == 1 ? 4 : 3)
mamba_scan_stream_kernel(ScanArgs a, const float* __restrict__ xact, const __half* __restrict__ c16,
                         const float* __restrict__ cb) {
  pdl_wait();
  pdl_trigger();
  constexpr int HPC = 4, NT = P / 8, ROWS = MT * 16;
  constexpr int XS = P + 8;                                    // floats per x row in shared memory (padded: the fragment reads
                                                               // of rows tq and columns gq then fall on 32 different banks)
  constexpr int CS = 2 * N + 8;                                // halves per C row (hi | lo | 16 bytes of padding: the 16-byte
                                                               // fragment reads, 32 bytes apart along a row, of rows gq and gq + 1
                                                               // then fall on different banks)
  extern __shared__ __align__(16) float sm[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h0 = blockIdx.x * HPC, b = blockIdx.y;
  const int hpg = a.H / a.G, g = h0 / hpg, k = a.k, GN = a.G * N;
  const int h = h0 + warp;
  const size_t row0 = size_t(b) * k;
  __half* C16 = reinterpret_cast<__half*>(sm);                 // [ROWS][CS]  (hi, lo), rows >= k zero
  float* CB = sm + ROWS * CS / 2;                                   // [ROWS][ROWS]
  float* xs = CB + ROWS * ROWS + warp * (ROWS * XS);           // per warp [ROWS][XS]
  float* Wh = CB + ROWS * ROWS + HPC * ROWS * XS + warp * ROWS * (ROWS + 1);   // per warp [ROWS][ROWS+1]

  // ---- state fragments of the first two k-step pairs: issued before anything else
  const int gq = lane >> 2, tq = lane & 3;
  const __half* S = a.s_init ? a.s_init + (size_t(b) * a.H + h) * P * N : nullptr;
  // (32-byte loads: the four lanes of a row then cover a whole 128-byte line per instruction; with 16-byte loads every
  // line was touched twice, and the state's loads were a quarter of the L1's work)
  uint4 sv0[NT][2];
  if (S != nullptr) {
#pragma unroll
    for (int j = 0; j < NT; ++j) ldg_nc_32B(S + size_t(j * 8 + gq) * N + tq * 16, sv0[j][0], sv0[j][1]);
  }
  // ---- shared operands (C halves, CB) and this head's x rows: cp.async, zero fill for the padding rows
  for (int idx = tid; idx < ROWS * 2 * N / 8; idx += 128) {
    const int r = idx / (2 * N / 8), rest = idx % (2 * N / 8), half = rest / (N / 8), c8 = rest % (N / 8);
    cp_async16(smem_u32(C16 + r * CS + half * N + c8 * 8), c16 + ((row0 + min(r, k - 1)) * 2 + half) * GN + g * N + c8 * 8, r < k);
  }
  for (int idx = tid; idx < ROWS * ROWS / 4; idx += 128) {
    const int r = idx / (ROWS / 4), c4 = idx % (ROWS / 4);
    cp_async16(smem_u32(CB + r * ROWS + c4 * 4), cb + ((size_t(b) * a.G + g) * KMAX + r) * KMAX + c4 * 4, true);
  }
  for (int idx = lane; idx < ROWS * P / 4; idx += 32) {
    const int r = idx / (P / 4), c4 = idx % (P / 4);
    cp_async16(smem_u32(xs + r * XS + c4 * 4), xact + (row0 + min(r, k - 1)) * a.d_xBC + h * P + c4 * 4, r < k);
  }
  cp_async_commit();
  // ---- dt, inclusive prefix sum of dt * A over the block positions (one warp shuffle scan per head)
  float dt = 0.f, dA = 0.f;
  if (lane < k) {
    const float raw = a.dt_raw ? a.dt_raw[(row0 + lane) * a.H + h] : a.zxbcdt[(row0 + lane) * a.ld_in + a.Di + a.d_xBC + h];
    dt = softplus_f(raw + a.dt_bias[h]);
    dA = dt * (-expf(a.A_log[h]));
  }
  float cum = dA;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const float up = __shfl_up_sync(0xffffffffu, cum, off);
    if (lane >= off) cum += up;
  }
  cp_async_wait<0>();
  __syncthreads();
  // ---- W[t][s] = exp(c_t - c_s) dt_s CB[t][s] for s <= t, plus the skip weight D on the diagonal: lane s owns
  // column s; the rows past k are zero
  const float Dh = a.Dskip[h];
  for (int t = 0; t < ROWS; ++t) {
    const float ct = __shfl_sync(0xffffffffu, cum, t & 31);
    float w = 0.f;
    if (t < k && lane <= t) w = __expf(ct - cum) * dt * CB[t * ROWS + lane];
    if (t < k && lane == t) w += Dh;
    if (lane < ROWS) Wh[t * (ROWS + 1) + lane] = w;
  }
  __syncwarp();
  // ---- state term on the tensor cores
  float acc[MT][NT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int j = 0; j < NT; ++j) { acc[mt][j][0] = acc[mt][j][1] = acc[mt][j][2] = acc[mt][j][3] = 0.f; }
  if (S != nullptr) {
#pragma unroll
    // the contraction index is permuted (the same way for C and for the state): within a chunk of 64, lane tq's 16
    // consecutive elements serve four k-steps, four elements each
    for (int kq = 0; kq < N / 64; ++kq) {
      uint4 sv[NT][2];
      if (kq >= 1) {
#pragma unroll
        for (int j = 0; j < NT; ++j) ldg_nc_32B(S + size_t(j * 8 + gq) * N + kq * 64 + tq * 16, sv[j][0], sv[j][1]);
      } else {
#pragma unroll
        for (int j = 0; j < NT; ++j) { sv[j][0] = sv0[j][0]; sv[j][1] = sv0[j][1]; }
      }
#pragma unroll
      for (int piece = 0; piece < 2; ++piece) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const __half* c0 = C16 + (mt * 16 + gq) * CS + kq * 64 + tq * 16 + piece * 8;
          const __half* c1 = C16 + (mt * 16 + gq + 8) * CS + kq * 64 + tq * 16 + piece * 8;
          const uint4 c_lo = *reinterpret_cast<const uint4*>(c0), c_hi = *reinterpret_cast<const uint4*>(c1);
          const uint4 r_lo = *reinterpret_cast<const uint4*>(c0 + N), r_hi = *reinterpret_cast<const uint4*>(c1 + N);
          const uint32_t a0[4] = {c_lo.x, c_hi.x, c_lo.y, c_hi.y}, a1[4] = {c_lo.z, c_hi.z, c_lo.w, c_hi.w};
          const uint32_t e0[4] = {r_lo.x, r_hi.x, r_lo.y, r_hi.y}, e1[4] = {r_lo.z, r_hi.z, r_lo.w, r_hi.w};
#pragma unroll
          for (int j = 0; j < NT; ++j) {
            mma_f16_16816(acc[mt][j], a0, sv[j][piece].x, sv[j][piece].y);
            mma_f16_16816(acc[mt][j], a1, sv[j][piece].z, sv[j][piece].w);
            mma_f16_16816(acc[mt][j], e0, sv[j][piece].x, sv[j][piece].y);
            mma_f16_16816(acc[mt][j], e1, sv[j][piece].z, sv[j][piece].w);
          }
        }
      }
    }
  }
  // ---- decay of the state term: row t of the accumulator times exp(c_t)
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const float d_lo = __expf(__shfl_sync(0xffffffffu, cum, (mt * 16 + gq) & 31));
    const float d_hi = __expf(__shfl_sync(0xffffffffu, cum, (mt * 16 + gq + 8) & 31));
#pragma unroll
    for (int j = 0; j < NT; ++j) { acc[mt][j][0] *= d_lo; acc[mt][j][1] *= d_lo; acc[mt][j][2] *= d_hi; acc[mt][j][3] *= d_hi; }
  }
  // ---- intra-block term and D skip, y_t += sum_{s <= t} W[t][s] x_s, as a [ROWS x ROWS] x [ROWS x P] product on the
  // tensor cores: tf32 operands keep fp32's range (W is a product of exponentials, dt and a 128-term dot product), and
  // each operand is split in two tf32 parts, three products per k-step, for ~21 bits.  (The scalar form read x from
  // shared memory once per (t, s) pair and thread, and the kernel ran at the L1's limit.)
#pragma unroll
  for (int ks = 0; ks < ROWS / 8; ++ks) {
    uint32_t ah[MT][4], al[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const float* wr = Wh + (mt * 16 + gq) * (ROWS + 1) + ks * 8 + tq;
      split_tf32(wr[0], ah[mt][0], al[mt][0]);
      split_tf32(wr[8 * (ROWS + 1)], ah[mt][1], al[mt][1]);
      split_tf32(wr[4], ah[mt][2], al[mt][2]);
      split_tf32(wr[8 * (ROWS + 1) + 4], ah[mt][3], al[mt][3]);
    }
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      uint32_t bh[2], bl[2];
      split_tf32(xs[(ks * 8 + tq) * XS + j * 8 + gq], bh[0], bl[0]);
      split_tf32(xs[(ks * 8 + tq + 4) * XS + j * 8 + gq], bh[1], bl[1]);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        if (ks * 8 > mt * 16 + 15) continue;                   // W is lower triangular: nothing in this k-step for these rows
        mma_tf32_1688(acc[mt][j], al[mt], bh[0], bh[1]);
        mma_tf32_1688(acc[mt][j], ah[mt], bl[0], bl[1]);
        mma_tf32_1688(acc[mt][j], ah[mt], bh[0], bh[1]);
      }
    }
  }
  // ---- gate and store
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int t = mt * 16 + gq + half * 8;
      if (t >= k) continue;
      const size_t row = row0 + t;
      float2 z[NT];
#pragma unroll
      for (int j = 0; j < NT; ++j) z[j] = *reinterpret_cast<const float2*>(a.zxbcdt + row * a.ld_in + h * P + j * 8 + tq * 2);
#pragma unroll
      for (int j = 0; j < NT; ++j)
        *reinterpret_cast<float2*>(a.y + row * a.Di + h * P + j * 8 + tq * 2) =
            make_float2(acc[mt][j][half * 2] * silu_f(z[j].x), acc[mt][j][half * 2 + 1] * silu_f(z[j].y));
    }
  }
}

template <int MT>
size_t scan_stream_smem() {
  constexpr int P = 64, N = 128, HPC = 4, ROWS = MT * 16;
  return sizeof(__half) * ROWS * (2 * N + 8) + sizeof(float) * (ROWS * ROWS + HPC * ROWS * (P + 8) + HPC * ROWS * (ROWS + 1));
}

template <int MT>
size_t scan_mma_smem() {
  constexpr int P = 64, N = 128, HPC = 4, ROWS = MT * 16;
  return sizeof(float) * (2 * ROWS * (N + 1) + ROWS * (ROWS + 1) + ROWS * HPC * P + HPC * ROWS * (ROWS + 1) + 2 * HPC * ROWS) +
         sizeof(__half) * 2 * ROWS * N;
}

}  // namespace

size_t scan_workspace_bytes(int B, int k, int Di, int N, int G) {
  const size_t M = size_t(B) * k, d_xBC = size_t(Di) + 2 * size_t(G) * N;
  return M * d_xBC * 4 + size_t(B) * G * KMAX * KMAX * 4 + M * 2 * size_t(G) * N * 2 + 256;
}

cudaError_t scan_launch(const ScanCall& c, cudaStream_t stream, Tracker* trk, std::string* err) {
  if (c.k < 1 || c.k > KMAX) { if (err) *err = "scan: k out of range"; return cudaErrorInvalidValue; }
  if (c.Di % c.P) { if (err) *err = "scan: Di must be a multiple of P"; return cudaErrorInvalidValue; }
  ScanArgs a{};
  a.zxbcdt = c.zxbcdt; a.ld_in = c.ld_in; a.dt_raw = c.dt_raw; a.s_init = (const __half*)c.s_init;
  a.conv_w = c.conv_w; a.conv_b = c.conv_b; a.dt_bias = c.dt_bias; a.A_log = c.A_log; a.Dskip = c.Dskip;
  a.y = c.y_gated; a.B = c.B; a.k = c.k; a.Di = c.Di; a.P = c.P; a.N = c.N; a.G = c.G; a.H = c.Di / c.P;
  a.d_conv = c.d_conv; a.d_xBC = c.Di + 2 * c.G * c.N;
  a.NP = c.N + 1;                                    // odd pitch: threads of a warp own consecutive p
  if (a.H % c.G) { if (err) *err = "scan: heads must divide into groups"; return cudaErrorInvalidValue; }
  // serving shapes: tensor-core path (needs 8-byte aligned rows for the float2 accesses)
  if (c.P == 64 && c.N == 128 && (a.H / c.G) % 4 == 0 && c.ld_in % 2 == 0 && c.Di % 4 == 0 && c.ws != nullptr &&
      (reinterpret_cast<uintptr_t>(c.s_init) & 31) == 0 &&     // its 32-byte loads of the state
      c.ws_bytes >= scan_workspace_bytes(c.B, c.k, c.Di, c.N, c.G)) {
    const bool two = c.k > 16;
    const size_t M = size_t(c.B) * c.k;
    float* xact = reinterpret_cast<float*>(c.ws);
    float* cbw = xact + M * a.d_xBC;
    __half* c16 = reinterpret_cast<__half*>(cbw + size_t(c.B) * c.G * KMAX * KMAX);
    trk_begin(trk, "scan_conv", 0, double(M) * a.d_xBC * 8);
    const bool vec4 = a.Di % 4 == 0 && (c.G * c.N) % 4 == 0 && a.ld_in % 4 == 0 &&
                      ((reinterpret_cast<uintptr_t>(a.zxbcdt) | reinterpret_cast<uintptr_t>(c.ws) | reinterpret_cast<uintptr_t>(a.conv_w) |
                        reinterpret_cast<uintptr_t>(a.conv_b)) & 15) == 0;
    const dim3 grid_c((a.d_xBC / (vec4 ? 4 : 1) + 255) / 256, c.B * ((c.k + CONV_ROWS - 1) / CONV_ROWS));
    if (vec4) launch_pdl(scan_conv_kernel<4>, grid_c, dim3(256), 0, stream, a, xact, c16);
    else launch_pdl(scan_conv_kernel<1>, grid_c, dim3(256), 0, stream, a, xact, c16);
    trk_end(trk);
    trk_begin(trk, "scan_cb", 0, 0);
    launch_pdl(scan_cb_kernel, dim3(c.G, c.B), dim3(256), size_t(2) * c.k * (c.N + 4) * sizeof(float), stream, a, xact, (float*)cbw);
    trk_end(trk);
    const size_t smem_s = two ? scan_stream_smem<2>() : scan_stream_smem<1>();
    static bool sset[2][MAX_DEVICES] = {};
    {
      const cudaError_t e = once_per_device(sset[two ? 1 : 0], [two, smem_s](int) {
        return two ? cudaFuncSetAttribute(mamba_scan_stream_kernel<64, 128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_s))
                   : cudaFuncSetAttribute(mamba_scan_stream_kernel<64, 128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_s));
      });
      if (e != cudaSuccess) return e;
    }
    dim3 grid_s(a.H / 4, c.B);
    trk_begin(trk, "mamba_scan", 2.0 * c.B * c.k * a.H * c.P * c.N, double(c.B) * a.H * c.P * c.N * 2);
    if (two) launch_pdl(mamba_scan_stream_kernel<64, 128, 2>, grid_s, dim3(128), smem_s, stream, a, (const float*)xact, (const __half*)c16, (const float*)cbw);
    else launch_pdl(mamba_scan_stream_kernel<64, 128, 1>, grid_s, dim3(128), smem_s, stream, a, (const float*)xact, (const __half*)c16, (const float*)cbw);
    trk_end(trk);
    return cudaGetLastError();
  }
  if (c.P == 64 && c.N == 128 && (a.H / c.G) % 4 == 0 && c.ld_in % 2 == 0 && c.Di % 2 == 0) {
    const bool two = c.k > 16;
    const size_t smem_f = two ? scan_mma_smem<2>() : scan_mma_smem<1>();
    static bool fset[2][MAX_DEVICES] = {};
    {
      const cudaError_t e = once_per_device(fset[two ? 1 : 0], [two, smem_f](int) {
        return two ? cudaFuncSetAttribute(mamba_scan_mma_kernel<64, 128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_f))
                   : cudaFuncSetAttribute(mamba_scan_mma_kernel<64, 128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_f));
      });
      if (e != cudaSuccess) return e;
    }
    dim3 grid_f(a.H / 4, c.B);
    trk_begin(trk, "mamba_scan", 2.0 * c.B * c.k * a.H * c.P * c.N, double(c.B) * a.H * c.P * c.N * 2);
    if (two) mamba_scan_mma_kernel<64, 128, 2><<<grid_f, 128, smem_f, stream>>>(a);
    else mamba_scan_mma_kernel<64, 128, 1><<<grid_f, 128, smem_f, stream>>>(a);
    trk_end(trk);
    return cudaGetLastError();
  }
  const size_t smem = sizeof(float) * (size_t(KMAX) * c.P + 2 * size_t(KMAX) * c.N + KMAX * KMAX + 3 * KMAX +
                                       size_t(c.P) * a.NP);
  if (smem > 48 * 1024) {
    // the largest size asked for so far, per device (the attribute is a per-device property of the function)
    static size_t smem_set[MAX_DEVICES] = {};
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(device_setup_mutex());
    if (smem > smem_set[dev]) {
      cudaError_t e = cudaFuncSetAttribute(mamba_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
      if (e != cudaSuccess) { if (err) *err = "scan: state tile does not fit in shared memory"; return e; }
      smem_set[dev] = smem;
    }
  }
  dim3 grid(a.H, c.B);
  trk_begin(trk, "mamba_scan", 0, double(c.B) * a.H * c.P * c.N * 2);
  mamba_scan_kernel<<<grid, SCAN_THREADS, smem, stream>>>(a);
  trk_end(trk);
  return cudaGetLastError();
}

}  // namespace hspec
