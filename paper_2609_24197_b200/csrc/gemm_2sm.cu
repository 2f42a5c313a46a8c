// y = x W^T for many activation rows (M >= 256): the tensor-bound regime of the draft step.
//
// Two CTAs on two SMs form one MMA unit (tcgen05 cta_group::2): the pair owns a [256 weight rows x BNT
// activation rows] tile of y^T.  Each CTA loads its own 128 weight rows and only HALF of the activation tile per
// k-step (the MMA reads the B operand from both CTAs' shared memory), which halves the shared-memory fill per
// flop compared with the one-CTA kernel; the accumulator lives in both CTAs' TMEM (128 lanes each).
// The kernel is persistent: one cluster per SM pair walks a static list of tiles; two TMEM accumulators
// alternate so the epilogue of one tile (tcgen05.ld -> global stores) overlaps the main loop of the next.
//
//   warp 0   TMA producer (both CTAs; both signal the LEADER CTA's "full" barrier)
//   warp 1   TMEM allocation (both CTAs), MMA issue + commits (leader CTA only, one thread)
//   warps 2..5  epilogue (both CTAs, their own 128 accumulator lanes)
// No TMA load is multicast; the only cluster-wide signal is tcgen05.commit to both CTAs' barriers.
//
// A pipeline stage holds TWO 64-column k-steps (64 KB per CTA at 256-wide tiles, three stages): every barrier round of
// the MMA thread (wait for "full", commit to "empty") costs the tensor pipe about 150 clocks whatever the order of the
// operations, so it is paid once per eight MMAs instead of once per four.  (Three k-steps per stage leave room for two
// stages only: 1 291 against 1 331 TFLOP/s on M = 2048, n_out = 25600, K = 5120.)
//
// Measurement builds (HSPEC_NVCC_FLAGS): -DHSPEC_GEMM2_NOLOAD (no operand is fetched), -DHSPEC_GEMM2_NOMMA (no MMA is
// issued, stages are released unread), -DHSPEC_GEMM2_NOEPI (accumulators are not read out), -DHSPEC_GEMM2_NOSTORE (read out, not stored), -DHSPEC_GEMM2_NOARGMAX (LM-head epilogue without its reduction network), -DHSPEC_GEMM2_CLOCK (CTA 0 prints its SM clock count and the wall time); HSPEC_GEMM2_KSUB=1 in the
// environment goes back to one k-step per stage.  On M = 2048, n_out = 25600, K = 5120, SM clocks per 256 x 256 x 16
// instruction (the arithmetic needs 128): MMA issue alone, no barrier at all 128; one k-step per stage 167 alone and
// 182 with loads and read-out; two k-steps per stage 146 and 160.
#include "common.cuh"
#include "kernels.h"

#include <cstdio>
#include <cstdlib>
#include <cstring>

namespace hspec {

namespace {

constexpr int TILE_K = 64;
constexpr uint32_t A_BYTES = 128 * TILE_K * 2;     // 16 KiB: this CTA's 128 weight rows

struct Gemm2Args {
  int M, N_out, K;
  int BNT;                 // activation rows per cluster tile (128 or 256); each CTA stages BNT/2
  int k_tiles, stages;
  int ksub;                // 64-column k-steps per pipeline stage (1 or 2): one barrier round per stage
  int n_tiles_w, n_tiles_m;
  // Work units: the first n_full_tiles tiles run whole (full waves of the SM pairs); each of the remaining "tail" tiles
  // is cut into tail_splits K-slices so that the last, partly filled wave keeps every pair busy.  A slice stores an
  // fp32 partial tile to `part` ([tail tile][slice][activation row][256 weight rows]); a second kernel sums them.
  int n_full_tiles, tail_splits, k_tiles_per_split;
  float* part;
  int f16, mode;
  void* out;
  long long ldo;
  float* logits;
  float* part_val;
  int* part_idx;
  uint32_t* status;
};

struct __align__(8) Tail2 {
  uint64_t full[GEMM_MAX_STAGES];
  uint64_t empty[GEMM_MAX_STAGES];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  uint32_t abort_flag;
  float red_val[4][256];
  int red_idx[4][256];
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc_2sm(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_2sm() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_2sm(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// TMA load issued by either CTA of the pair; the byte count is credited to the barrier at the same offset in
// the leader CTA (rank bit of the shared::cluster address cleared).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const void* tmap, int c0, int c1, uint32_t bar_local,
                                                 uint64_t policy) {
  const uint32_t bar_leader = bar_local & 0xFEFFFFFFu;
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(bar_leader), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void umma_2sm(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives (once every MMA issued so far has finished) on the barrier at this offset in BOTH CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}
__device__ __forceinline__ uint32_t idesc_m256(uint32_t n, bool f16) {
  const uint32_t fmt = f16 ? 0u : 1u;
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((n >> 3) << 17) | ((256u >> 4) << 24);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(192, 1)
gemm_2sm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, Gemm2Args g) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t b_bytes = uint32_t(g.BNT / 2) * TILE_K * 2;
  const uint32_t sub_bytes = A_BYTES + b_bytes;                    // one k-step: this CTA's weight rows + its half of the activations
  const uint32_t stage_bytes = uint32_t(g.ksub) * sub_bytes;
  Tail2* tail = reinterpret_cast<Tail2*>(smem + size_t(g.stages) * stage_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  const int total_tiles = g.n_tiles_w * g.n_tiles_m;
  const int total_units = g.n_full_tiles + (total_tiles - g.n_full_tiles) * g.tail_splits;
  // unit u < n_full_tiles: tile u, all of K; else tail tile n_full_tiles + v / tail_splits, K-slice v % tail_splits
  auto decode = [&](int u, int& tile, int& sp, int& kt_begin, int& kt_end) {
    if (u < g.n_full_tiles) { tile = u; sp = -1; kt_begin = 0; kt_end = g.k_tiles; return; }
    const int v = u - g.n_full_tiles;
    tile = g.n_full_tiles + v / g.tail_splits;
    sp = g.tail_splits > 1 ? v % g.tail_splits : -1;          // -1: the unit is a whole tile with the real epilogue
    kt_begin = (v % g.tail_splits) * g.k_tiles_per_split;
    kt_end = min(g.k_tiles, kt_begin + g.k_tiles_per_split);
  };
  const uint32_t tmem_cols = 2u * uint32_t(g.BNT);           // two accumulators (256 or 512 columns)

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int s = 0; s < g.stages; ++s) {
      mbar_init(smem_u32(&tail->full[s]), 1);
      mbar_init(smem_u32(&tail->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&tail->tmem_full[a]), 1);
      mbar_init(smem_u32(&tail->tmem_empty[a]), 256);        // 128 epilogue threads of each CTA (leader's copy is used)
    }
    tail->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_2sm(smem_u32(&tail->tmem_base), tmem_cols);
    tmem_relinquish_2sm();
  }
  tc_fence_before();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = tail->tmem_base;
  volatile uint32_t* abort_flag = &tail->abort_flag;
  pdl_wait();                                   // set-up done: now the previous kernel's results may be read
  pdl_trigger();
#ifdef HSPEC_GEMM2_CLOCK
  const long long clk0 = clock64();
  const uint64_t ns0 = global_timer_ns();
#endif

  if (warp == 0) {
    if (lane == 0) {
      // Weights at normal L2 priority, activations evict-last.  Evict-first weights ran a few percent faster in
      // short isolated runs, but ncu showed 2.4x the algorithmic DRAM reads (the clusters that share a weight tile
      // drift apart and fetch it again), and in a long power-capped step the extra DRAM traffic costs clock:
      // 13.5 vs 13.75 ms per step at conc128_32b.
      // (With a single activation tile nobody shares a weight tile: the weights stream through once, evict-first.)
      const uint64_t pol_w = g.n_tiles_m == 1 ? policy_evict_first() : policy_evict_normal(), pol_x = policy_evict_last();
      uint32_t it = 0;
      bool ok = true;
      for (int unit = cluster_id; unit < total_units && ok; unit += n_clusters) {
        int tile, sp, kt_begin, kt_end;
        decode(unit, tile, sp, kt_begin, kt_end);
        const int tn = tile / g.n_tiles_m, tm = tile % g.n_tiles_m;
        for (int kt = kt_begin; kt < kt_end; kt += g.ksub, ++it) {
          const int s = it % g.stages;
          const uint32_t lap = it / g.stages;
          if (lap > 0 && !mbar_wait(smem_u32(&tail->empty[s]), (lap - 1) & 1)) {
            atomicExch(g.status, STATUS_TIMEOUT_PRODUCER);
            *abort_flag = 1;
            ok = false;
            break;
          }
          const int n_sub = min(g.ksub, kt_end - kt);
          const uint32_t full = smem_u32(&tail->full[s]);
#ifdef HSPEC_GEMM2_NOLOAD
          // measurement build: no operand is fetched, the MMAs run on whatever the stage holds (results are garbage);
          // shows the rate of the MMA issue + epilogue alone
          if (rank == 0) mbar_arrive(full);
          (void)pol_w; (void)pol_x; (void)tn; (void)tm; (void)n_sub;
#else
          if (rank == 0) mbar_expect_tx(full, 2 * uint32_t(n_sub) * sub_bytes);   // both CTAs' bytes land on the leader's barrier
          for (int sub = 0; sub < n_sub; ++sub) {
            uint8_t* sa = smem + size_t(s) * stage_bytes + size_t(sub) * sub_bytes;
            tma_load_2d_pair(smem_u32(sa), &tmA, (kt + sub) * TILE_K, tn * 256 + int(rank) * 128, full, pol_w);
            tma_load_2d_pair(smem_u32(sa + A_BYTES), &tmB, (kt + sub) * TILE_K, tm * g.BNT + int(rank) * (g.BNT / 2), full, pol_x);
          }
#endif
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = idesc_m256(uint32_t(g.BNT), g.f16 != 0);
      uint32_t it = 0, tile_count = 0;
      bool ok = true;
      for (int unit = cluster_id; unit < total_units && ok; unit += n_clusters, ++tile_count) {
        int tile, sp, kt_begin, kt_end;
        decode(unit, tile, sp, kt_begin, kt_end);
        const uint32_t acc = tile_count & 1, use = tile_count >> 1;
        if (use > 0 && !mbar_wait(smem_u32(&tail->tmem_empty[acc]), (use - 1) & 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + acc * uint32_t(g.BNT);
        for (int kt = kt_begin; kt < kt_end; kt += g.ksub, ++it) {
          const int s = it % g.stages;
          const uint32_t lap = it / g.stages;
          // (every barrier round in this thread costs the tensor pipe ~150 clocks: with two k-steps per stage it is
          // paid once per eight MMAs instead of once per four)
          if (!mbar_wait(smem_u32(&tail->full[s]), lap & 1)) { ok = false; break; }
          tc_fence_after();
          const int n_sub = min(g.ksub, kt_end - kt);
          for (int sub = 0; sub < n_sub; ++sub) {
            const uint32_t sa = smem_u32(smem + size_t(s) * stage_bytes + size_t(sub) * sub_bytes);
            const uint64_t da = umma_desc_kmajor_sw128(sa), db = umma_desc_kmajor_sw128(sa + A_BYTES);
#ifndef HSPEC_GEMM2_NOMMA                   // measurement build: stages are released unread (shows the load path's own rate)
#pragma unroll
            for (int kk = 0; kk < TILE_K / 16; ++kk)
              umma_2sm(tmem_acc, da + uint64_t(kk * 2), db + uint64_t(kk * 2), idesc, (kt > kt_begin || sub > 0 || kk > 0) ? 1u : 0u);
#else
            (void)da; (void)db; (void)idesc;
#endif
          }
          umma_commit_pair(smem_u32(&tail->empty[s]));
        }
        if (ok) umma_commit_pair(smem_u32(&tail->tmem_full[acc]));
      }
      if (!ok) { atomicExch(g.status, STATUS_TIMEOUT_MMA); *abort_flag = 1; }
    }
  } else {
    // ---------------------------------------------------------------- epilogue (both CTAs)
    const int q = warp & 3;
    uint32_t tile_count = 0;
    bool ok = true;
    const uint32_t empty_leader0 = mapa_rank(smem_u32(&tail->tmem_empty[0]), 0);
    const uint32_t empty_leader1 = mapa_rank(smem_u32(&tail->tmem_empty[1]), 0);
    for (int unit = cluster_id; unit < total_units && ok; unit += n_clusters, ++tile_count) {
      int tile, sp, kt_begin, kt_end;
      decode(unit, tile, sp, kt_begin, kt_end);
      const int tn = tile / g.n_tiles_m, tm = tile % g.n_tiles_m;
      const int mode = sp >= 0 ? EPI_PARTIAL_F32 : g.mode;
      const uint32_t acc = tile_count & 1, use = tile_count >> 1;
      if (!mbar_wait(smem_u32(&tail->tmem_full[acc]), use & 1)) {
        atomicExch(g.status, STATUS_TIMEOUT_EPILOGUE);
        ok = false;
        break;
      }
      tc_fence_after();
      const int tile_n128 = tn * 2 + int(rank);               // 128-row weight tile of this CTA
      const int n = tile_n128 * 128 + q * 32 + lane;
      const bool n_ok = n < g.N_out;
      const int m0 = tm * g.BNT;
      const uint32_t tmem_acc = tmem_base + acc * uint32_t(g.BNT) + (uint32_t(q * 32) << 16);
#ifdef HSPEC_GEMM2_NOEPI
      const int c_first = g.BNT;                            // measurement build: the accumulator is handed back unread
#else
      const int c_first = 0;
#endif
      for (int c0 = c_first; c0 < g.BNT; c0 += 16) {
        if (m0 + c0 >= g.M && mode != EPI_ARGMAX) break;    // rows past M: nothing to store (warp-uniform)
        uint32_t r[16];
        tmem_ld16(tmem_acc + uint32_t(c0), r);
        tmem_ld_wait();
#ifdef HSPEC_GEMM2_NOSTORE                   // measurement build: the accumulator is read but nothing is written
        if (r[0] == 0x7fc12345u && g.M < 0) g.status[0] = r[1];
        continue;
#endif
        if (mode == EPI_PARTIAL_F32) {
          // slice of a tail tile: [tail tile][slice][activation row of the tile][256 weight rows of the pair]
          float* out = g.part + (size_t(tile - g.n_full_tiles) * g.tail_splits + sp) * size_t(g.BNT) * 256 +
                       int(rank) * 128 + q * 32 + lane;
#pragma unroll
          for (int j = 0; j < 16; ++j) out[size_t(c0 + j) * 256] = __uint_as_float(r[j]);
        } else if (mode == EPI_STORE_F32) {
          float* out = reinterpret_cast<float*>(g.out);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            if (n_ok && m < g.M) out[size_t(m) * g.ldo + n] = __uint_as_float(r[j]);
          }
        } else if (mode == EPI_ACCUM_F32) {
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
        } else if (mode == EPI_SWIGLU_F16 || mode == EPI_SWIGLU_BF16) {
          const int f = tile_n128 * 64 + q * 16 + (lane & 15);
          swiglu_store16(r, g.out, mode == EPI_SWIGLU_BF16, g.ldo, m0 + c0, g.M, f, 2 * f < g.N_out, lane, g.status);
        } else if (mode == EPI_STORE_F16) {
          __half* out = reinterpret_cast<__half*>(g.out);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            if (n_ok && m < g.M) out[size_t(m) * g.ldo + n] = f16_sat(__uint_as_float(r[j]), g.status);
          }
        } else if (mode == EPI_STORE_BF16) {
          __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(g.out);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            if (n_ok && m < g.M) out[size_t(m) * g.ldo + n] = __float2bfloat16_rn(__uint_as_float(r[j]));
          }
        } else {  // EPI_ARGMAX
          float v[16];
          int vi[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            v[j] = n_ok ? __uint_as_float(r[j]) : -INFINITY;
            vi[j] = n;
            if (g.logits != nullptr && n_ok && m < g.M) g.logits[size_t(m) * g.ldo + n] = v[j];
          }
          // (The network costs the LM head 4 % - 2.34 -> 2.24 ms per step without it - mostly as clock under the power cap.
          // One redux.sync maximum + ballot per column instead of the shuffle rounds: 2.56 ms.)
          int row = 0;
#ifndef HSPEC_GEMM2_NOARGMAX                 // measurement build: no reduction network (ids are wrong)
          warp_argmax16(v, vi, lane, row);
#endif
          if ((lane & 1) == 0) { tail->red_val[q][c0 + row] = v[0]; tail->red_idx[q][c0 + row] = vi[0]; }
        }
      }
      // accumulator drained: hand it back to the MMA issuer in the leader CTA
      tc_fence_before();
      mbar_arrive_cluster(acc ? empty_leader1 : empty_leader0);
      if (mode == EPI_ARGMAX) {
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int t = threadIdx.x - 64;
        for (int c = t; c < g.BNT; c += 128) {
          const int m = m0 + c;
          if (m >= g.M || tile_n128 * 128 >= g.N_out) continue;   // the pair's second half may lie wholly past V
          float v = tail->red_val[0][c];
          int idx = tail->red_idx[0][c];
#pragma unroll
          for (int qq = 1; qq < 4; ++qq) {
            const float ov = tail->red_val[qq][c];
            const int oi = tail->red_idx[qq][c];
            if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
          }
          g.part_val[size_t(tile_n128) * g.M + m] = v;
          g.part_idx[size_t(tile_n128) * g.M + m] = idx;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");        // red_* is reused by the next tile
      }
    }
  }
#ifdef HSPEC_GEMM2_CLOCK
  if (blockIdx.x == 0 && threadIdx.x == 64) {
    const long long dc = clock64() - clk0;
    const uint64_t dn = global_timer_ns() - ns0;
    printf("gemm_2sm cta 0: %lld SM clocks in %llu ns = %.0f MHz\n", dc, (unsigned long long)dn, double(dc) * 1e3 / double(dn));
  }
#endif
  tc_fence_before();
  cluster_sync_all();           // neither CTA may leave while its pair still reads its shared memory or TMEM
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_2sm(tmem_base, tmem_cols);
  }
}

// Sums the K-slices of the tail tiles in slice order (deterministic) and applies the real epilogue.
// Block = (tail tile, group of 4 activation rows); thread = one of the pair's 256 weight rows; all slices' loads are
// issued before the first add.
constexpr int TAIL_MAX_SPLITS = 8, TAIL_ROWS = 4;
__global__ void __launch_bounds__(256)
gemm2_tail_reduce_kernel(Gemm2Args g) {
  pdl_wait();
  pdl_trigger();
  const int tail = blockIdx.x, tile = g.n_full_tiles + tail;
  const int tn = tile / g.n_tiles_m, tm = tile % g.n_tiles_m;
  const int n = tn * 256 + threadIdx.x;
  const int m_base = tm * g.BNT + blockIdx.y * TAIL_ROWS;
  if (m_base >= g.M) return;
  const float* src = g.part + size_t(tail) * g.tail_splits * g.BNT * 256 + size_t(blockIdx.y) * TAIL_ROWS * 256 + threadIdx.x;
  float v[TAIL_MAX_SPLITS][TAIL_ROWS];
#pragma unroll
  for (int sp = 0; sp < TAIL_MAX_SPLITS; ++sp)
#pragma unroll
    for (int j = 0; j < TAIL_ROWS; ++j)
      v[sp][j] = (sp < g.tail_splits && m_base + j < g.M) ? __ldcs(src + (size_t(sp) * g.BNT + j) * 256) : 0.f;
  const int lane = threadIdx.x & 31;
  // SwiGLU epilogue: weight rows are interleaved in blocks of 16 (gate | up), so lanes l and l ^ 16 of a warp hold the
  // gate and the up projection of feature f
  const int f = (tn * 2 + (threadIdx.x >> 7)) * 64 + ((threadIdx.x >> 5) & 3) * 16 + (lane & 15);
#pragma unroll
  for (int j = 0; j < TAIL_ROWS; ++j) {
    const int m = m_base + j;
    if (m >= g.M) break;                                    // uniform over the block
    float acc = 0.f;
#pragma unroll
    for (int sp = 0; sp < TAIL_MAX_SPLITS; ++sp)
      if (sp < g.tail_splits) acc += v[sp][j];
    if (g.mode == EPI_SWIGLU_F16 || g.mode == EPI_SWIGLU_BF16) {
      const float up = __shfl_xor_sync(0xffffffffu, acc, 16);
      if (lane < 16 && 2 * f < g.N_out) store_act16(g.out, size_t(m) * g.ldo + f, silu_f(acc) * up, g.mode == EPI_SWIGLU_BF16, g.status);
      continue;
    }
    if (n >= g.N_out) continue;
    const size_t o = size_t(m) * g.ldo + n;
    if (g.mode == EPI_STORE_F32) reinterpret_cast<float*>(g.out)[o] = acc;
    else if (g.mode == EPI_ACCUM_F32) reinterpret_cast<float*>(g.out)[o] += acc;
    else if (g.mode == EPI_STORE_F16) reinterpret_cast<__half*>(g.out)[o] = f16_sat(acc, g.status);
    else reinterpret_cast<__nv_bfloat16*>(g.out)[o] = __float2bfloat16_rn(acc);
  }
}

bool g_attr_done2[MAX_DEVICES] = {};
int g_smem_optin2[MAX_DEVICES] = {};

}  // namespace

bool gemm2_preferred(int M, int n_out) {
  static const bool off = [] { const char* e = getenv("HSPEC_GEMM_1SM"); return e && e[0] == '1'; }();
  static const int min_m = [] { const char* e = getenv("HSPEC_GEMM2_MIN_M"); return e ? atoi(e) : 0; }();   // measurements only
  if (off) return false;
  if (min_m > 0) return M >= min_m;
  // From 256 rows on the contractions are tensor-bound; even a partly filled wave of pair tiles beats the one-CTA
  // kernel with K-slices and its reduction pass.  At 128..255 rows only a matrix of 2^18 weight rows or more (the
  // state projection) goes this way: streaming it, the pair kernel measured 5.65 against 5.51 TB/s at 128 rows (at 64
  // rows the one-CTA kernel wins, 6.24 against 6.01), and the step's small matrices keep the kernel they are tuned for.
  return M >= 256 || (M >= 128 && n_out >= (1 << 18));
}

// Tile width (activation rows per pair tile) and the number of K-slices for the tiles of the last, partly filled wave,
// by a simple model: full waves of the 74 SM pairs x k-steps x cost of a k-step, plus the tail wave (k-steps / slices),
// a fixed cost per wave (pipeline fill, the last epilogue) and, with slices, the pass that sums the partial tiles.
// One cost unit ~ 2.2 ns (a k-step of a 256-wide pair tile = 256 units ~ 0.56 us).
void gemm2_pick(int M, int n_out, int K, int mode, int* bnt_out, int* splits_out) {
  const int tw = (n_out + 255) / 256;
  const int k_tiles = (K + TILE_K - 1) / TILE_K;
  const bool may_split = mode != EPI_ARGMAX;            // every other epilogue can be applied after the slices are summed
  double best_cost = 1e30;
  int best_bnt = 256, best_s = 1;
  for (int bnt : {256, 128}) {
    const int tiles = tw * ((M + bnt - 1) / bnt);
    const int full_waves = tiles / 74, tail = tiles % 74;
    // a 128-wide tile needs 96 B/clk of shared-memory fill per SM at full MMA rate, a 256-wide one 64 B/clk:
    // measured, the narrow tile runs ~1.5x slower per flop
    const double kstep = bnt * (bnt == 128 ? 1.5 : 1.0);
    for (int s = 1; s <= 8; ++s) {
      if (s > 1 && (!may_split || tail == 0 || tail * s > 74 || k_tiles / s < 8)) continue;
      const int kps = (k_tiles + s - 1) / s;
      if (s > 1 && kps * (s - 1) >= k_tiles) continue;         // an empty last slice
      double cost = double(full_waves) * (k_tiles * kstep + 1500.0);
      if (tail > 0) cost += kps * kstep + 1500.0;
      // (the pass that sums the slices: its bytes at 4 TB/s plus 2 us; with 4, 8, 12 or 20 us fewer launches are sliced and
      // the 256-row steps get slower, 1.93 -> 1.95 / 2.02 / 2.07 / 2.10 ms at paper_8b; no difference at 2048 rows)
      if (s > 1) cost += (double(s + 2) * tail * bnt * 256 * 4.0 / 4.0e6 + 2.0) * 455.0;
      if (cost < best_cost) { best_cost = cost; best_bnt = bnt; best_s = s; }
    }
  }
  static const int bnt_env = [] { const char* e = getenv("HSPEC_GEMM2_BNT"); return e ? atoi(e) : 0; }();   // measurements only
  if (bnt_env == 128 || bnt_env == 256) { best_bnt = bnt_env; best_s = 1; }
  *bnt_out = best_bnt;
  *splits_out = best_s;
}

// Scratch for the tail tiles' partials: at most one wave of pair tiles, each up to 256 x 256 fp32, times the slices.
size_t gemm2_tail_bytes() { return size_t(74) * 256 * 256 * 4; }

cudaError_t gemm2_launch(const GemmCall& c, cudaStream_t stream, Tracker* trk, std::string* err) {
  {
    const cudaError_t e = once_per_device(g_attr_done2, [](int dev) {
      cudaError_t e2 = cudaDeviceGetAttribute(&g_smem_optin2[dev], cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
      if (e2 != cudaSuccess) return e2;
      return cudaFuncSetAttribute(gemm_2sm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, g_smem_optin2[dev]);
    });
    if (e != cudaSuccess) return e;
  }
  const int smem_optin2 = g_smem_optin2[current_device()];
  Gemm2Args g{};
  g.M = c.M; g.N_out = c.n_out; g.K = c.K;
  int splits = 1;
  gemm2_pick(c.M, c.n_out, c.K, c.mode, &g.BNT, &splits);
  g.k_tiles = (c.K + TILE_K - 1) / TILE_K;
  g.n_tiles_w = (c.n_out + 255) / 256;
  g.n_tiles_m = (c.M + g.BNT - 1) / g.BNT;
  const int tiles = g.n_tiles_w * g.n_tiles_m;
  const int tail = tiles % 74;
  if (c.splits > 0) splits = c.splits;                    // the caller fixed the number of K-slices (of the tail tiles)
  if (c.mode == EPI_ARGMAX || tail == 0) splits = 1;
  if (splits > g.k_tiles) splits = g.k_tiles;
  if (splits > TAIL_MAX_SPLITS) splits = TAIL_MAX_SPLITS;
  while (splits > 1 && size_t(tail) * splits * g.BNT * 256 * 4 > c.splitk_ws_bytes) --splits;   // never more than the scratch holds
  if (c.splitk_ws == nullptr) splits = 1;
  g.k_tiles_per_split = (g.k_tiles + splits - 1) / splits;
  splits = (g.k_tiles + g.k_tiles_per_split - 1) / g.k_tiles_per_split;   // no empty slice
  g.tail_splits = splits;
  g.n_full_tiles = splits > 1 ? tiles - tail : tiles;
  g.part = reinterpret_cast<float*>(c.splitk_ws);
  g.f16 = c.f16 ? 1 : 0; g.mode = c.mode; g.out = c.out; g.ldo = c.ldo;
  if (c.addend != nullptr) { if (err) *err = "the 2-SM kernel has no addend epilogue"; return cudaErrorInvalidValue; }
  g.logits = c.logits; g.part_val = c.part_val; g.part_idx = c.part_idx; g.status = c.status;
  static const int ksub_env = [] { const char* e = getenv("HSPEC_GEMM2_KSUB"); return e ? atoi(e) : 0; }();   // measurements only
  g.ksub = (ksub_env == 1 || ksub_env == 2) ? ksub_env : 2;
  const size_t stage_bytes = size_t(g.ksub) * (A_BYTES + size_t(g.BNT / 2) * TILE_K * 2);
  const size_t fixed = sizeof(Tail2) + 1024;
  int stages = int((size_t(smem_optin2) - fixed) / stage_bytes);
  if (stages > GEMM_MAX_STAGES) stages = GEMM_MAX_STAGES;
  if (stages < 2) { if (err) *err = "shared memory too small for the 2-SM GEMM pipeline"; return cudaErrorInvalidValue; }
  g.stages = stages;
  CUtensorMap tmB;
  if (!make_tmap_16bit_2d(&tmB, c.x, c.M, c.K, c.ldx, g.BNT / 2, c.f16, err)) return cudaErrorInvalidValue;
  const int total = g.n_full_tiles + (tiles - g.n_full_tiles) * splits;
  const int clusters = total < 74 ? total : 74;
  const size_t smem = size_t(stages) * stage_bytes + fixed;
  // profile name "gemm2:<what>" tells this kernel's launches from the one-CTA kernel's "gemm:<what>"
  std::string label = "gemm2:";
  if (c.label) { const char* colon = strchr(c.label, ':'); label += colon ? colon + 1 : c.label; }
  trk_begin(trk, label.c_str(), 2.0 * c.M * c.n_out * c.K, 2.0 * c.n_out * c.K,
            gemm_io_bytes(c.M, c.n_out, c.K, c.mode, c.logits != nullptr));
  cudaError_t e = launch_pdl(gemm_2sm_kernel, dim3(2 * clusters), dim3(192), smem, stream, *c.tmW, tmB, g);
  trk_end(trk);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e == cudaSuccess && splits > 1) {
    trk_begin(trk, "gemm2_tail_reduce", 0, double(splits + 1) * tail * g.BNT * 256 * 4);
    launch_pdl(gemm2_tail_reduce_kernel, dim3(tail, g.BNT / TAIL_ROWS), dim3(256), 0, stream, g);
    trk_end(trk);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace hspec
