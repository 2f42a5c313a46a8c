// bf16 GEMM y = x W^T on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), sm_100a.
//
// Every dense map of the draft step is "few activation rows times a tall weight matrix".  The
// weight rows therefore sit on the MMA's M side (128 output features per CTA = 128 TMEM lanes) and
// the activation rows on its N side (BN = 16..256 rows = BN TMEM columns), so a step with one
// request and a step with 256 requests run the same kernel: the accumulator tile is y^T.
//
//   warp 0 : TMA producer  (weights [128 x 64] and activations [BN x 64] per stage, 128-byte swizzle)
//   warp 1 : allocates TMEM, issues tcgen05.mma (one elected thread), commits stages back
//   warps 2..5 : epilogue, one TMEM lane quarter each: tcgen05.ld -> registers -> global
//
// Epilogues: fp32 / bf16 store, fp32 accumulate-into (residual), fp32 K-slice partial, and the
// LM-head form that reduces each activation row's (max, index) over the CTA's 128 vocabulary rows.
//
// A CTA can also own TWO weight tiles (WT = 2, two accumulators in TMEM) so that one activation fill per k-step feeds
// two MMAs: 1.5 bytes of shared-memory fill per weight byte instead of 2 at 128 activation rows.  Measured on the
// state projection at 128 rows it changes nothing (5.55 TB/s either way: the profiler shows L2-to-SM traffic down
// from 2.0x to 1.5x the weight bytes, DRAM at 73 % and the tensor pipe at 43 % - neither the fill nor a pipe is the
// limit there), so it stays off unless HSPEC_GEMM_WT=2 asks for it.
#include "common.cuh"
#include "kernels.h"

#include <cuda.h>

#include <cstdio>
#include <cstdlib>

namespace hspec {

namespace {

constexpr int TILE_W = 128;       // weight rows per CTA (UMMA M)
constexpr int TILE_K = 64;        // bf16 elements per stage along K = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr uint32_t A_STAGE_BYTES = TILE_W * TILE_K * 2;   // 16 KiB

struct __align__(8) GemmSmemTail {
  uint64_t full[GEMM_MAX_STAGES];
  uint64_t empty[GEMM_MAX_STAGES];
  uint64_t tmem_full;
  uint32_t tmem_base;
  uint32_t abort_flag;
  float red_val[4][256];   // LM-head epilogue: per lane-quarter (max, index) of each activation row
  int red_idx[4][256];
};

__global__ void __launch_bounds__(192, 2)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmArgs g) {
#ifdef HSPEC_GEMM_CLOCK
  const long long clk_start = clock64();     // measurement build: one CTA prints where its clocks went
#endif
  extern __shared__ uint8_t smem_raw[];
  // 128-byte swizzle needs 1024-byte aligned tiles
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t b_stage_bytes = g.BN * TILE_K * 2;
  const uint32_t a_stage_bytes = uint32_t(g.WT) * A_STAGE_BYTES;
  const uint32_t stage_bytes = a_stage_bytes + b_stage_bytes;
  GemmSmemTail* tail = reinterpret_cast<GemmSmemTail*>(smem + size_t(g.stages) * stage_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_m = blockIdx.x;            // activation-row tile (fastest: CTAs sharing a weight tile run together)
  const int tile_n = blockIdx.y;            // weight-row tile (WT consecutive 128-row tiles)
  const int split = blockIdx.z;
  const int kt_begin = split * g.k_tiles_per_split;
  const int kt_end = min(g.k_tiles_total, kt_begin + g.k_tiles_per_split);
  const int n_kt = kt_end - kt_begin;       // >= 1 by construction of the grid
  const uint32_t tmem_cols = g.tmem_cols;

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int s = 0; s < g.stages; ++s) {
      mbar_init(smem_u32(&tail->full[s]), 1);
      mbar_init(smem_u32(&tail->empty[s]), 1);
    }
    mbar_init(smem_u32(&tail->tmem_full), 1);
    tail->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tail->tmem_base), tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = tail->tmem_base;
  pdl_wait();                                   // set-up done: now the previous kernel's results may be read
  pdl_trigger();
#ifdef HSPEC_GEMM_CLOCK
  const long long clk_setup = clock64();
#endif

  if (warp == 0) {
    if (lane == 0) {
      // weights are streamed once per step, unless the caller runs the same matrix again right away
      const uint64_t pol_w = g.keep_w ? policy_evict_last() : policy_evict_first();
      const uint64_t pol_x = policy_evict_last();    // activations are re-read by every weight tile
      for (int i = 0; i < n_kt; ++i) {
        const int s = i % g.stages;
        const uint32_t round = i / g.stages;
        if (round > 0 && !mbar_wait(smem_u32(&tail->empty[s]), (round - 1) & 1)) {
          atomicExch(g.status, STATUS_TIMEOUT_PRODUCER);
          atomicExch(&tail->abort_flag, 1u);
          break;
        }
        const uint32_t full = smem_u32(&tail->full[s]);
        mbar_expect_tx(full, stage_bytes);
        uint8_t* sa = smem + size_t(s) * stage_bytes;
        for (int w = 0; w < g.WT; ++w)       // (a tile wholly past the last weight row is zero-filled by the copy)
          tma_load_2d(smem_u32(sa + w * A_STAGE_BYTES), &tmA, (kt_begin + i) * TILE_K, (tile_n * g.WT + w) * TILE_W, full, pol_w);
        tma_load_2d(smem_u32(sa + a_stage_bytes), &tmB, (kt_begin + i) * TILE_K, tile_m * g.BN, full, pol_x);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_m128(g.BN, g.f16 != 0);
      bool ok = true;
      for (int i = 0; i < n_kt && ok; ++i) {
        const int s = i % g.stages;
        const uint32_t round = i / g.stages;
        if (!mbar_wait(smem_u32(&tail->full[s]), round & 1)) {
          atomicExch(g.status, STATUS_TIMEOUT_MMA);
          atomicExch(&tail->abort_flag, 1u);
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + size_t(s) * stage_bytes);
        const uint64_t db = umma_desc_kmajor_sw128(sa + a_stage_bytes);
        for (int w = 0; w < g.WT; ++w) {
          const uint64_t da = umma_desc_kmajor_sw128(sa + w * A_STAGE_BYTES);
#pragma unroll
          for (int kk = 0; kk < TILE_K / UMMA_K; ++kk) {
            // advancing K inside the swizzle row: +32 bytes = +2 in the descriptor's 16-byte units
            umma_bf16(tmem_acc + uint32_t(w * g.BN), da + uint64_t(kk * 2), db + uint64_t(kk * 2), idesc, (i > 0 || kk > 0) ? 1u : 0u);
          }
        }
        umma_commit(smem_u32(&tail->empty[s]));   // stage reusable once these MMAs have read it
      }
      // accumulator complete (or aborted: release the epilogue either way)
      if (ok) umma_commit(smem_u32(&tail->tmem_full));
      else mbar_arrive(smem_u32(&tail->tmem_full));
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;                         // TMEM lane quarter this warp may read
    if (g.addend != nullptr && g.mode == EPI_ARGMAX) {
      // the addend rows of this tile do not depend on the accumulator: pull this warp's 128-byte piece of every
      // row into L2 while the main loop runs (one line per lane and pass)
      const int n_w = tile_n * TILE_W + q * 32;
      if (n_w < g.N_out)
        for (int c = lane; c < g.BN; c += 32) {
          const int m = tile_m * g.BN + c;
          if (m < g.M) asm volatile("prefetch.global.L2 [%0];" ::"l"(g.addend + size_t(m) * g.ld_add + n_w));
        }
    }
    // EPI_ARGMAX_T: lane = request, its addends for the tile's columns are BN contiguous floats.  They do not depend on
    // the accumulator: the first 64 are requested before the wait for it, and every group of 16 is re-filled as soon as
    // it is used (64 loads per thread in flight; one dependent round trip per group made a CTA's epilogue 30 us).
    float aq[4][16];
    const int n_t = tile_n * TILE_W + q * 32 + lane;
    const bool t_on = g.mode == EPI_ARGMAX_T && g.addend != nullptr && n_t < g.N_out;
    auto load_aq = [&](float (&dst)[16], int c_first) {
      const int mf = tile_m * g.BN + c_first;
      const float* arow = g.addend + size_t(n_t) * g.ld_add + mf;
      if (t_on && c_first < g.BN && mf + 16 <= g.M && (reinterpret_cast<uintptr_t>(arow) & 15) == 0) {
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4) {
          const float4 t = __ldg(reinterpret_cast<const float4*>(arow) + j4);
          dst[4 * j4] = t.x; dst[4 * j4 + 1] = t.y; dst[4 * j4 + 2] = t.z; dst[4 * j4 + 3] = t.w;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) dst[j] = (t_on && c_first < g.BN && mf + j < g.M) ? __ldg(arow + j) : 0.f;
      }
    };
    if (g.mode == EPI_ARGMAX_T) {
#pragma unroll
      for (int u = 0; u < 4; ++u) load_aq(aq[u], u * 16);
    }
    bool ok = mbar_wait(smem_u32(&tail->tmem_full), 0);
#ifdef HSPEC_GEMM_CLOCK
    const long long clk_acc = clock64();
#endif
    if (!ok) atomicExch(g.status, STATUS_TIMEOUT_EPILOGUE);
    tc_fence_after();
    if (*reinterpret_cast<volatile uint32_t*>(&tail->abort_flag)) ok = false;
    const int m0 = tile_m * g.BN;
    // EPI_ARGMAX_T: this lane's running (max, lowest column) over the tile's columns
    float t_best = -INFINITY;
    int t_idx = 0x7fffffff;
    if (g.mode == EPI_ARGMAX_T) {
      // value = acc + addend[request][vocabulary row]; the arg-max over the tile's vocabulary rows runs inside the
      // thread (ascending columns, strict comparison: the lowest index wins ties), no shuffles
      const bool n_ok_t = n_t < g.N_out;
      for (int c00 = 0; c00 < g.BN && ok; c00 += 64) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int c0 = c00 + u * 16;
          if (c0 >= g.BN) break;                    // warp-uniform
          uint32_t r[16];
          tmem_ld16(tmem_acc + (uint32_t(q * 32) << 16) + uint32_t(c0), r);
          tmem_ld_wait();
          float add[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) add[j] = aq[u][j];
          load_aq(aq[u], c0 + 64);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            const float val = __uint_as_float(r[j]) + add[j];
            if (n_ok_t && m < g.M) {
              if (g.logits != nullptr) g.logits[size_t(n_t) * g.ldo + m] = val;
              if (val > t_best) { t_best = val; t_idx = m; }
            }
          }
        }
      }
    }
    for (int w = 0; w < g.WT && g.mode != EPI_ARGMAX_T; ++w) {   // (WT = 2 is never combined with the arg-max epilogues)
    const int tile_w = tile_n * g.WT + w;           // 128-row weight tile of this pass
    const int n = tile_w * TILE_W + q * 32 + lane;  // output feature (weight row) of this thread
    const bool n_ok = n < g.N_out;
    // Addend of the arg-max epilogue (the causal-correction head): the loads of the next 16 columns are issued before
    // this batch is reduced.  Measured on that head's CTAs (-DHSPEC_GEMM_CLOCK; K = 256, 128 requests): the epilogue
    // takes 23 000 of a CTA's 29 000 clocks - 10 000 with neither addend nor reduction, +6 000 for the reduction network,
    // +7 500 for the addend - and a queue of 64 loads per thread instead of 16 changes nothing: with two CTAs of four
    // epilogue warps per SM it is the warps' instruction latency, not memory, that sets the pace.
    float add_next[16];
    auto load_addend = [&](int c_first) {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int m = m0 + c_first + j;
#ifdef HSPEC_GEMM_NOADDEND                   // measurement build
        add_next[j] = float(m);
#else
        add_next[j] = (n_ok && c_first < g.BN && m < g.M) ? __ldcs(g.addend + size_t(m) * g.ld_add + n) : 0.f;
#endif
      }
    };
    const bool with_addend = g.mode == EPI_ARGMAX && g.addend != nullptr;
    if (with_addend && ok) load_addend(0);

    for (int c0 = 0; c0 < g.BN && ok; c0 += 16) {
      uint32_t r[16];
      tmem_ld16(tmem_acc + (uint32_t(q * 32) << 16) + uint32_t(w * g.BN + c0), r);
      tmem_ld_wait();
      if (g.mode == EPI_STORE_F32 || g.mode == EPI_PARTIAL_F32) {
        float* out = reinterpret_cast<float*>(g.out) + (g.mode == EPI_PARTIAL_F32 ? size_t(split) * g.M * g.ldo : 0);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = m0 + c0 + j;
          if (n_ok && m < g.M) out[size_t(m) * g.ldo + n] = __uint_as_float(r[j]);
        }
      } else if (g.mode == EPI_ACCUM_F32) {
        // read-modify-write of the residual stream: issue the 16 loads together, then add and store
        float* out = reinterpret_cast<float*>(g.out);
        float old[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = m0 + c0 + j;
          old[j] = (n_ok && m < g.M) ? __ldcg(out + size_t(m) * g.ldo + n) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = m0 + c0 + j;
          if (n_ok && m < g.M) out[size_t(m) * g.ldo + n] = old[j] + __uint_as_float(r[j]);
        }
      } else if (g.mode == EPI_STORE_BF16) {
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(g.out);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = m0 + c0 + j;
          if (n_ok && m < g.M) out[size_t(m) * g.ldo + n] = __float2bfloat16_rn(__uint_as_float(r[j]));
        }
      } else if (g.mode == EPI_SWIGLU_F16 || g.mode == EPI_SWIGLU_BF16) {
        const int f = tile_w * 64 + q * 16 + (lane & 15);
        swiglu_store16(r, g.out, g.mode == EPI_SWIGLU_BF16, g.ldo, m0 + c0, g.M, f, 2 * f < g.N_out, lane, g.status);
      } else if (g.mode == EPI_STORE_F16) {
        __half* out = reinterpret_cast<__half*>(g.out);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = m0 + c0 + j;
          if (n_ok && m < g.M) out[size_t(m) * g.ldo + n] = f16_sat(__uint_as_float(r[j]), g.status);
        }
      } else {  // EPI_ARGMAX: logits optional, (max, lowest index) over this warp's 32 vocabulary rows
        float add[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) add[j] = with_addend ? add_next[j] : 0.f;
        if (with_addend) load_addend(c0 + 16);
        float v[16];
        int vi[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = m0 + c0 + j;
          v[j] = n_ok ? __uint_as_float(r[j]) + add[j] : -INFINITY;
          vi[j] = n;
          if (g.logits != nullptr && n_ok && m < g.M) g.logits[size_t(m) * g.ldo + n] = v[j];
        }
        int row = 0;
#ifndef HSPEC_GEMM_NOARGMAX                   // measurement build
        warp_argmax16(v, vi, lane, row);
#endif
        if ((lane & 1) == 0) { tail->red_val[q][c0 + row] = v[0]; tail->red_idx[q][c0 + row] = vi[0]; }
      }
    }
    }
    if (g.mode == EPI_ARGMAX_T) {
      // per (column tile, request): [tile_m][N_out]
      const int n = tile_n * TILE_W + q * 32 + lane;
      if (n < g.N_out) {
        g.part_val[size_t(tile_m) * g.N_out + n] = ok ? t_best : -INFINITY;
        g.part_idx[size_t(tile_m) * g.N_out + n] = ok ? t_idx : 0x7fffffff;
      }
    }
    if (g.mode == EPI_ARGMAX) {
      asm volatile("bar.sync 1, 128;" ::: "memory");      // the four epilogue warps only
      const int t = threadIdx.x - 64;                     // 0..127
      for (int c = t; c < g.BN; c += 128) {
        const int m = m0 + c;
        if (m >= g.M) continue;
        float v = tail->red_val[0][c];
        int idx = tail->red_idx[0][c];
#pragma unroll
        for (int qq = 1; qq < 4; ++qq) {
          const float ov = tail->red_val[qq][c];
          const int oi = tail->red_idx[qq][c];
          if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
        }
        if (!ok) { v = -INFINITY; idx = 0x7fffffff; }
        g.part_val[size_t(tile_n) * g.M + m] = v;
        g.part_idx[size_t(tile_n) * g.M + m] = idx;
      }
    }
#ifdef HSPEC_GEMM_CLOCK
    if (blockIdx.y == gridDim.y / 2 && blockIdx.x == 0 && blockIdx.z == 0 && threadIdx.x == 64)
      printf("gemm cta %d: set-up %lld clocks, until the accumulator is complete %lld, epilogue %lld\n", int(blockIdx.y),
             clk_setup - clk_start, clk_acc - clk_setup, clock64() - clk_acc);
#endif
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_acc, tmem_cols);
  }
}

// Sum the K-slice partials in slice order (deterministic) and apply the final store.
__global__ void splitk_reduce_kernel(const float* __restrict__ part, int splits, int M, int N, void* out,
                                     long long ldo, int mode, uint32_t* status) {
  pdl_wait();
  pdl_trigger();
  const long long total = (long long)M * N;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int m = int(i / N), n = int(i % N);
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) acc += part[(size_t(s) * M + m) * N + n];
    if (mode == EPI_STORE_F32) reinterpret_cast<float*>(out)[size_t(m) * ldo + n] = acc;
    else if (mode == EPI_ACCUM_F32) reinterpret_cast<float*>(out)[size_t(m) * ldo + n] += acc;
    else if (mode == EPI_STORE_F16) reinterpret_cast<__half*>(out)[size_t(m) * ldo + n] = f16_sat(acc, status);
    else if (mode == EPI_SWIGLU_F16 || mode == EPI_SWIGLU_BF16) {
      // n runs over interleaved rows; lower half of each 32-row block = gate, upper half = up of the same 16 features
      if ((n & 31) < 16) {
        float up = 0.f;
        for (int s = 0; s < splits; ++s) up += part[(size_t(s) * M + m) * N + n + 16];
        const int f = (n >> 5) * 16 + (n & 15);
        store_act16(out, size_t(m) * ldo + f, silu_f(acc) * up, mode == EPI_SWIGLU_BF16, status);
      }
    }
    else reinterpret_cast<__nv_bfloat16*>(out)[size_t(m) * ldo + n] = __float2bfloat16_rn(acc);
  }
}

// The same for fp32 outputs whose row length and pitch are multiples of four: 16-byte loads and stores, one row
// per blockIdx.y, every slice's load issued before the first add.
template <int SPLITS>
__global__ void splitk_reduce_f32x4_kernel(const float* __restrict__ part, int M, int N, float* __restrict__ out,
                                           long long ldo, int accumulate) {
  pdl_wait();
  pdl_trigger();
  const int m = blockIdx.y;
  const size_t slice = size_t(M) * N;
  for (int n4 = blockIdx.x * blockDim.x + threadIdx.x; n4 < (N >> 2); n4 += gridDim.x * blockDim.x) {
    float4 v[SPLITS];
#pragma unroll
    for (int s = 0; s < SPLITS; ++s) v[s] = __ldcs(reinterpret_cast<const float4*>(part + s * slice + size_t(m) * N) + n4);
    float4* dst = reinterpret_cast<float4*>(out + size_t(m) * ldo) + n4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 old = accumulate ? *dst : acc;
#pragma unroll
    for (int s = 0; s < SPLITS; ++s) { acc.x += v[s].x; acc.y += v[s].y; acc.z += v[s].z; acc.w += v[s].w; }
    if (accumulate) { acc.x = old.x + acc.x; acc.y = old.y + acc.y; acc.z = old.z + acc.z; acc.w = old.w + acc.w; }
    *dst = acc;
  }
}

// ids[m] = lowest index among the per-tile maxima (tiles are in ascending vocabulary order).
// The partials are [tile][row]: a block takes eight consecutive rows, thread (r = tid % 8, tid / 8) walks every 32nd
// tile of row r, so that eight neighbouring threads read one 32-byte sector (a block per row read 4 bytes of every
// sector it touched: 33 us for 19 MB at M = 2048, V = 152 064).
__device__ __forceinline__ void argmax_take(float& v, int& idx, float ov, int oi) {
  if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
}
__global__ void __launch_bounds__(256)
argmax_reduce_kernel(const float* __restrict__ pv, const int* __restrict__ pi, int n_tiles, int M,
                     int* __restrict__ ids, const int* __restrict__ id_map) {
  pdl_wait();
  pdl_trigger();
  const int r = threadIdx.x & 7, m = blockIdx.x * 8 + r;
  float v = -INFINITY;
  int idx = 0x7fffffff;
  if (m < M) {
    for (int t = threadIdx.x >> 3; t < n_tiles; t += 32) argmax_take(v, idx, pv[size_t(t) * M + m], pi[size_t(t) * M + m]);
  }
  // lanes r, r + 8, r + 16, r + 24 of a warp hold the same row
  for (int off = 8; off < 32; off <<= 1)
    argmax_take(v, idx, __shfl_xor_sync(0xffffffffu, v, off), __shfl_xor_sync(0xffffffffu, idx, off));
  __shared__ float sv[8][8];
  __shared__ int si[8][8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane < 8) { sv[warp][lane] = v; si[warp][lane] = idx; }
  __syncthreads();
  if (threadIdx.x < 8 && m < M) {
    v = sv[0][r]; idx = si[0][r];
    for (int w = 1; w < 8; ++w) argmax_take(v, idx, sv[w][r], si[w][r]);
    ids[m] = id_map ? id_map[idx] : idx;                    // pruned drafter vocabulary: row index -> token id
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool g_attr_done[MAX_DEVICES] = {};
int g_smem_optin[MAX_DEVICES] = {};

}  // namespace

// 2-D bf16/fp16 row-major [rows, cols] tensor, box [box_rows x 64 columns], 128-byte swizzle, zero fill.
bool make_tmap_16bit_2d(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t ld_elems,
                        int box_rows, bool f16, std::string* err) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { if (err) *err = "cuTensorMapEncodeTiled is not available from the CUDA driver"; return false; }
  if ((reinterpret_cast<uintptr_t>(base) & 15) || ((ld_elems * 2) & 15)) {
    if (err) *err = "TMA operand needs a 16-byte aligned base and row pitch";
    return false;
  }
  cuuint64_t dims[2] = {cuuint64_t(cols), cuuint64_t(rows)};
  cuuint64_t strides[1] = {cuuint64_t(ld_elems) * 2};
  cuuint32_t box[2] = {cuuint32_t(TILE_K), cuuint32_t(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(tm, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    if (err) *err = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string(int(r));
    return false;
  }
  return true;
}

int gemm_pick_bn(int M) {
  if (M >= 256) return 256;
  return ((M + 15) / 16) * 16;
}

int gemm_pick_splits(int M, int n_out, int K, int num_sms, int mode) {
  if (gemm2_preferred(M, n_out)) {
    int bnt = 256, s = 1;
    gemm2_pick(M, n_out, K, mode, &bnt, &s);
    return s;
  }
  // Weight streaming (few rows): keep every SM fed.  Many rows: one slice (tensor-bound, no reduction pass).
  const int k_tiles = (K + TILE_K - 1) / TILE_K;
  const int tiles = ((n_out + TILE_W - 1) / TILE_W) * ((M + 255) / 256);
  if (tiles >= num_sms || k_tiles < 8) return 1;
  int want = (2 * num_sms + tiles - 1) / tiles;
  int max_by_k = k_tiles / 4;               // at least 4 K-tiles per slice
  int s = want < max_by_k ? want : max_by_k;
  if (s > 16) s = 16;
  return s < 1 ? 1 : s;
}

size_t gemm_splitk_bytes(int M, int n_out, int splits) {
  return splits > 1 ? size_t(splits) * M * n_out * sizeof(float) : 0;
}

// Launches y = x W^T.  tmW must describe W with box rows 128; x is described here (box rows BN).
cudaError_t gemm_launch(const GemmCall& c, cudaStream_t stream, Tracker* trk, std::string* err) {
  if (c.addend == nullptr && gemm2_preferred(c.M, c.n_out)) return gemm2_launch(c, stream, trk, err);
  {
    // the opt-in shared-memory limit is a per-device function attribute
    const cudaError_t e = once_per_device(g_attr_done, [](int dev) {
      cudaError_t e2 = cudaDeviceGetAttribute(&g_smem_optin[dev], cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
      if (e2 != cudaSuccess) return e2;
      return cudaFuncSetAttribute(gemm_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, g_smem_optin[dev]);
    });
    if (e != cudaSuccess) return e;
  }
  const int smem_optin = g_smem_optin[current_device()];
  GemmArgs g{};
  g.M = c.M; g.N_out = c.n_out; g.K = c.K;
  g.BN = c.bn > 0 ? c.bn : gemm_pick_bn(c.M);
  g.k_tiles_total = (c.K + TILE_K - 1) / TILE_K;
  int splits = c.splits < 1 ? 1 : c.splits;
  if (splits > g.k_tiles_total) splits = g.k_tiles_total;
  g.k_tiles_per_split = (g.k_tiles_total + splits - 1) / splits;
  splits = (g.k_tiles_total + g.k_tiles_per_split - 1) / g.k_tiles_per_split;   // no empty slice
  // Two weight tiles per CTA: only on request (HSPEC_GEMM_WT=2, measurements), see the note at the top of the file.
  static const int wt_env = [] { const char* e = getenv("HSPEC_GEMM_WT"); return e ? atoi(e) : 0; }();
  const int n_tiles_w = (c.n_out + TILE_W - 1) / TILE_W;
  g.WT = (wt_env == 2 && g.BN <= 128 && c.mode != EPI_ARGMAX && c.addend == nullptr) ? 2 : 1;
  uint32_t cols = 32;
  while (cols < uint32_t(g.WT * g.BN)) cols <<= 1;
  g.tmem_cols = cols;
  const size_t stage_bytes = size_t(g.WT) * A_STAGE_BYTES + size_t(g.BN) * TILE_K * 2;
  const size_t fixed = sizeof(GemmSmemTail) + 1024;
  // Weight streaming (narrow activation tile): size the ring so that TWO CTAs fit on an SM; one CTA's prologue and
  // epilogue then overlap the other's stream.  Wide tiles take the whole SM.
  const size_t budget = (g.BN <= 128) ? size_t(smem_optin) / 2 - 1024 : size_t(smem_optin);
  int stages = int((budget - fixed) / stage_bytes);
  if (stages > GEMM_MAX_STAGES) stages = GEMM_MAX_STAGES;
  if (stages > g.k_tiles_per_split) stages = g.k_tiles_per_split < 2 ? 2 : g.k_tiles_per_split;
  if (stages < 2) { if (err) *err = "shared memory too small for the GEMM pipeline"; return cudaErrorInvalidValue; }
  g.stages = stages;
  g.status = c.status;
  g.f16 = c.f16 ? 1 : 0;
  g.logits = c.logits; g.addend = c.addend; g.ld_add = c.ld_add; g.part_val = c.part_val; g.part_idx = c.part_idx;
  g.keep_w = c.keep_weights_in_l2 ? 1 : 0;
  g.ldo = c.ldo;
  if (splits > 1) {
    if (c.mode == EPI_ARGMAX) { if (err) *err = "LM-head epilogue cannot be K-sliced"; return cudaErrorInvalidValue; }
    if (c.splitk_ws == nullptr || c.splitk_ws_bytes < gemm_splitk_bytes(c.M, c.n_out, splits)) {
      if (err) *err = "K-slice workspace too small";
      return cudaErrorInvalidValue;
    }
    g.mode = EPI_PARTIAL_F32; g.out = c.splitk_ws; g.ldo = c.n_out;
  } else {
    g.mode = c.mode; g.out = c.out;
  }
  CUtensorMap tmB;
  if (!make_tmap_16bit_2d(&tmB, c.x, c.M, c.K, c.ldx, g.BN, c.f16, err)) return cudaErrorInvalidValue;
  dim3 grid((c.M + g.BN - 1) / g.BN, (n_tiles_w + g.WT - 1) / g.WT, splits);
  const size_t smem = size_t(stages) * stage_bytes + fixed;
  trk_begin(trk, c.label ? c.label : "gemm", 2.0 * c.M * c.n_out * c.K, 2.0 * c.n_out * c.K,
            gemm_io_bytes(c.M, c.n_out, c.K, c.mode, c.logits != nullptr));
  cudaError_t e = launch_pdl(gemm_tcgen05_kernel, grid, dim3(192), smem, stream, *c.tmW, tmB, g);
  trk_end(trk);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (splits > 1)
    e = splitk_reduce_launch(reinterpret_cast<const float*>(c.splitk_ws), splits, c.M, c.n_out, c.out, c.ldo, c.mode, stream, trk,
                             c.status);
  return e;
}

cudaError_t splitk_reduce_launch(const float* part, int splits, int M, int N, void* out, long long ldo, int mode,
                                 cudaStream_t stream, Tracker* trk, uint32_t* status) {
  const long long total = (long long)M * N;
  trk_begin(trk, "splitk_reduce", 0, double(splits + 1) * M * N * 4);
  const bool f32 = mode == EPI_STORE_F32 || mode == EPI_ACCUM_F32;
  if (f32 && (N & 3) == 0 && (ldo & 3) == 0 && (reinterpret_cast<uintptr_t>(out) & 15) == 0 && splits >= 2 && splits <= 4) {
    // (the sum order s = 0, 1, ... and "old + sum" match the generic kernel bit for bit)
    dim3 grid((N / 4 + 255) / 256, M);
    float* o = reinterpret_cast<float*>(out);
    const int acc = mode == EPI_ACCUM_F32;
    if (splits == 2) launch_pdl(splitk_reduce_f32x4_kernel<2>, grid, dim3(256), 0, stream, part, M, N, o, ldo, acc);
    else if (splits == 3) launch_pdl(splitk_reduce_f32x4_kernel<3>, grid, dim3(256), 0, stream, part, M, N, o, ldo, acc);
    else launch_pdl(splitk_reduce_f32x4_kernel<4>, grid, dim3(256), 0, stream, part, M, N, o, ldo, acc);
  } else {
    int blocks = int((total + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    launch_pdl(splitk_reduce_kernel, dim3(blocks), dim3(256), 0, stream, part, splits, M, N, out, ldo, mode, status);
  }
  trk_end(trk);
  return cudaGetLastError();
}

cudaError_t argmax_reduce_launch(const float* pv, const int* pi, int n_tiles, int M, int* ids, cudaStream_t stream,
                                 Tracker* trk, const int* id_map) {
  trk_begin(trk, "argmax_reduce", 0, double(n_tiles) * M * 8);
  launch_pdl(argmax_reduce_kernel, dim3((M + 7) / 8), dim3(256), 0, stream, pv, pi, n_tiles, M, ids, id_map);
  trk_end(trk);
  return cudaGetLastError();
}

}  // namespace hspec
