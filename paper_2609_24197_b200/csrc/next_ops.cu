// Steps next to the draft block: the acceptance rule of App. A, the draft probability it divides by, and the
// causal correction of Sec. 3.3.3 (a first-order dependency between adjacent draft positions applied to the logits).
#include "common.cuh"
#include "kernels.h"

#include <cstdlib>

namespace hspec {

namespace {

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ------------------------------------------------------------------ acceptance rule (App. A)
// One warp per request: n[b] = number of leading positions with min(1, P_T / P_D) >= alpha, all in fp32 with IEEE
// division.  0 / 0 (NaN) rejects; P_D = 0 with P_T > 0 (+inf) accepts.
__global__ void accept_kernel(const float* __restrict__ pt, const float* __restrict__ pd, const float* __restrict__ alpha,
                              int* __restrict__ n_accept, int B, int k) {
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  int n = k;
  for (int base = 0; base < k; base += 32) {
    const int i = base + lane;
    bool ok = true;
    if (i < k) {
      const float r = __fdiv_rn(pt[size_t(b) * k + i], pd[size_t(b) * k + i]);
      ok = !(r != r) && fminf(1.0f, r) >= alpha[size_t(b) * k + i];
    }
    const unsigned bad = __ballot_sync(0xffffffffu, !ok);
    if (bad != 0u) { n = base + __ffs(bad) - 1; break; }
  }
  if (lane == 0) n_accept[b] = n;
}

// ------------------------------------------------------------------ softmax probability of one token per row
// One block per row, one pass over the fp32 logits: every thread keeps a running (max, sum of exp) over its
// elements, the block merges them; p = exp(z[id] - max) / sum.
__global__ void token_probs_kernel(const float* __restrict__ logits, long long ld, const int* __restrict__ ids,
                                   float* __restrict__ p, int V) {
  const int m = blockIdx.x;
  const float* z = logits + size_t(m) * ld;
  float mx = -INFINITY, sum = 0.f;
  auto add = [&](float v) {                       // (-inf entries contribute nothing, also while the maximum is still -inf)
    if (v > mx) { sum = sum * __expf(mx - v) + 1.f; mx = v; }
    else if (v > -INFINITY) sum += __expf(v - mx);
  };
  const bool vec = ((reinterpret_cast<uintptr_t>(z) & 15) == 0);
  const int V4 = vec ? (V >> 2) : 0;
  for (int i = threadIdx.x; i < V4; i += blockDim.x) {
    const float4 v = __ldcs(reinterpret_cast<const float4*>(z) + i);
    // local maximum first: one rescale per four elements
    const float m4 = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
    if (m4 > mx) { sum *= __expf(mx - m4); mx = m4; }
    if (mx > -INFINITY) sum += __expf(v.x - mx) + __expf(v.y - mx) + __expf(v.z - mx) + __expf(v.w - mx);
  }
  for (int i = V4 * 4 + threadIdx.x; i < V; i += blockDim.x) add(z[i]);
  auto merge = [&](float omx, float osum) {
    const float nm = fmaxf(mx, omx);
    if (nm == -INFINITY) return;
    sum = (mx > -INFINITY ? sum * __expf(mx - nm) : 0.f) + (omx > -INFINITY ? osum * __expf(omx - nm) : 0.f);
    mx = nm;
  };
  for (int off = 16; off > 0; off >>= 1) {
    const float omx = __shfl_xor_sync(0xffffffffu, mx, off);
    const float osum = __shfl_xor_sync(0xffffffffu, sum, off);
    merge(omx, osum);
  }
  __shared__ float smx[32], ssum[32];
  if ((threadIdx.x & 31) == 0) { smx[threadIdx.x >> 5] = mx; ssum[threadIdx.x >> 5] = sum; }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int nw = blockDim.x >> 5;
    mx = threadIdx.x < nw ? smx[threadIdx.x] : -INFINITY;
    sum = threadIdx.x < nw ? ssum[threadIdx.x] : 0.f;
    for (int off = 16; off > 0; off >>= 1) {
      const float omx = __shfl_xor_sync(0xffffffffu, mx, off);
      const float osum = __shfl_xor_sync(0xffffffffu, sum, off);
      merge(omx, osum);
    }
    if (threadIdx.x == 0) p[m] = expf(z[ids[m]] - mx) / sum;
  }
}

// ------------------------------------------------------------------ Markov head (Sec. 3.3.3)
// x[b, :] = W_in[prev[b], :] (16-bit rows copied as they are): the predecessor's factor row, the activation of the
// position's rank-r product with W_out.
__global__ void markov_gather_kernel(const uint16_t* __restrict__ W_in, const int* __restrict__ prev, long long prev_stride,
                                     uint16_t* __restrict__ x, int r) {
  pdl_wait();
  pdl_trigger();
  const int b = blockIdx.x;
  const uint16_t* src = W_in + size_t(prev[size_t(b) * prev_stride]) * r;
  for (int i = threadIdx.x; i < (r >> 3); i += blockDim.x)
    reinterpret_cast<uint4*>(x + size_t(b) * r)[i] = reinterpret_cast<const uint4*>(src)[i];
}

// Position i of every request: lowest index among the per-tile maxima -> ids[b * k + i] (mapped to a token id when the
// drafter's vocabulary is pruned), and the factor row of that token -> x[b, :] for position i + 1.
// The partials are [tile][request]: a block takes eight consecutive requests, thread (tid % 8, tid / 8) walks every
// 128th tile of its request, so that eight neighbouring threads read one 32-byte sector (1024 threads: there are only
// B / 8 blocks, and the kernel sits between two dependent GEMMs, so its latency counts).
__global__ void __launch_bounds__(1024)
markov_reduce_gather_kernel(const float* __restrict__ pv, const int* __restrict__ pi, int n_tiles, int B,
                            int* __restrict__ ids, int k, int i, const int* __restrict__ id_map,
                            const uint16_t* __restrict__ W_in, uint16_t* __restrict__ x, int r, int gather) {
  pdl_wait();
  pdl_trigger();
  const int rr = threadIdx.x & 7, b = blockIdx.x * 8 + rr;
  float v = -INFINITY;
  int idx = 0x7fffffff;
  auto take = [&](float ov, int oi) { if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; } };
  if (b < B) {
    for (int t = threadIdx.x >> 3; t < n_tiles; t += 256) {          // two tiles' loads in flight per step
      const int t2 = t + 128;
      const float v1 = pv[size_t(t) * B + b], v2 = t2 < n_tiles ? pv[size_t(t2) * B + b] : -INFINITY;
      const int i1 = pi[size_t(t) * B + b], i2 = t2 < n_tiles ? pi[size_t(t2) * B + b] : 0x7fffffff;
      take(v1, i1);
      take(v2, i2);
    }
  }
  for (int off = 8; off < 32; off <<= 1) take(__shfl_xor_sync(0xffffffffu, v, off), __shfl_xor_sync(0xffffffffu, idx, off));
  __shared__ float sv[32][8];
  __shared__ int si[32][8];
  __shared__ int token[8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane < 8) { sv[warp][lane] = v; si[warp][lane] = idx; }
  __syncthreads();
  if (threadIdx.x < 8) {
    int tok = 0;
    if (b < B) {
      v = sv[0][rr]; idx = si[0][rr];
      for (int w = 1; w < 32; ++w) take(sv[w][rr], si[w][rr]);
      tok = id_map ? id_map[idx] : idx;
      ids[size_t(b) * k + i] = tok;
    }
    token[rr] = tok;
  }
  __syncthreads();
  if (gather) {
    // warp w copies the factor row of request blockIdx.x * 8 + w (16 bytes per lane and step)
    const int bw = blockIdx.x * 8 + warp;
    if (warp < 8 && bw < B) {
      const uint16_t* src = W_in + size_t(token[warp]) * r;
      for (int j = lane; j < (r >> 3); j += 32)
        reinterpret_cast<uint4*>(x + size_t(bw) * r)[j] = reinterpret_cast<const uint4*>(src)[j];
    }
  }
}

}  // namespace

cudaError_t accept_launch(const float* pt, const float* pd, const float* alpha, int* n_accept, int B, int k, cudaStream_t stream) {
  accept_kernel<<<(B + 7) / 8, 256, 0, stream>>>(pt, pd, alpha, n_accept, B, k);
  return cudaGetLastError();
}

cudaError_t token_probs_launch(const float* logits, long long ld, const int* ids, float* p, int M, int V, cudaStream_t stream) {
  token_probs_kernel<<<M, 512, 0, stream>>>(logits, ld, ids, p, V);
  return cudaGetLastError();
}

// From 65 to 128 requests the head's GEMM runs with the operands' roles exchanged: the requests' factor rows x [B, r]
// sit on the MMA's M side (one 128-row tile), the vocabulary matrix W_out on the N side in tiles of 128 rows, so that an
// accumulator lane is a request and its arg-max over the tile's vocabulary rows runs inside one thread, its addends
// 512 contiguous bytes fetched four groups ahead.  (With the vocabulary on the lanes every group of 16 columns goes
// through a 32-shuffle reduction network and 16 separate addend loads: 23 000 of a CTA's 29 000 clocks at 128
// requests.  Measured per step of 16 positions at 128 requests, V = 152 064, r = 256: 1.68 ms -> 1.42 ms; with 32
// requests only a quarter of the lanes would work and the vocabulary-on-lanes form is as fast, 0.34 against 0.36 ms
// for 8 positions.)
constexpr int MARKOV_T_MIN_B = 65, MARKOV_T_MAX_B = 128, MARKOV_T_TILE = 128;

size_t markov_workspace_bytes(int B, int Vd, int r) {
  const size_t vt = (size_t(Vd) + 127) / 128;
  return round_up(size_t(B) * r * 2, 256) + 2 * round_up(vt * B * 4, 256) + 256;
}

cudaError_t markov_launch(const MarkovCall& c, cudaStream_t stream, Tracker* trk, std::string* err) {
  const size_t vt = (size_t(c.Vd) + 127) / 128;
  uint8_t* ws = reinterpret_cast<uint8_t*>(c.ws);
  uint16_t* x = reinterpret_cast<uint16_t*>(ws);
  float* part_val = reinterpret_cast<float*>(ws + round_up(size_t(c.B) * c.r * 2, 256));
  int* part_idx = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(part_val) + round_up(vt * c.B * 4, 256));
  trk_begin(trk, "markov_gather");
  markov_gather_kernel<<<c.B, 32, 0, stream>>>(reinterpret_cast<const uint16_t*>(c.W_in), c.last_token, 1, x, c.r);
  trk_end(trk);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const bool transposed = c.B >= MARKOV_T_MIN_B && c.B <= MARKOV_T_MAX_B && c.W_out != nullptr;
  CUtensorMap tm_x;
  if (transposed && !make_tmap_16bit_2d(&tm_x, x, c.B, c.r, c.r, 128, c.f16, err)) return cudaErrorInvalidValue;
  const size_t n_part = transposed ? (size_t(c.Vd) + MARKOV_T_TILE - 1) / MARKOV_T_TILE : vt;
  for (int i = 0; i < c.k; ++i) {
    GemmCall g{};
    if (transposed) {
      g.tmW = &tm_x; g.x = c.W_out; g.ldx = c.r; g.M = c.Vd; g.n_out = c.B; g.mode = EPI_ARGMAX_T; g.bn = MARKOV_T_TILE;
    } else {
      g.tmW = c.tmW_out; g.x = x; g.ldx = c.r; g.M = c.B; g.n_out = c.Vd; g.mode = EPI_ARGMAX;
    }
    g.f16 = c.f16; g.K = c.r; g.splits = 1;
    g.addend = c.logits + size_t(i) * c.ld;                 // row b of this GEMM is row b * k + i of the block's logits
    g.ld_add = (long long)c.k * c.ld;
    g.logits = c.write_logits ? c.logits + size_t(i) * c.ld : nullptr;
    g.ldo = (long long)c.k * c.ld;
    g.part_val = part_val; g.part_idx = part_idx; g.status = c.status;
    g.keep_weights_in_l2 = true;                            // W_out (78 MB at V = 152 064, r = 256) serves every position
    g.label = "markov";
    e = gemm_launch(g, stream, trk, err);
    if (e != cudaSuccess) return e;
    trk_begin(trk, "markov_reduce");
    launch_pdl(markov_reduce_gather_kernel, dim3((c.B + 7) / 8), dim3(1024), 0, stream, (const float*)part_val, (const int*)part_idx,
               int(n_part), c.B, c.ids, c.k, i, c.id_map, reinterpret_cast<const uint16_t*>(c.W_in), x, c.r, int(i + 1 < c.k));
    trk_end(trk);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace hspec
