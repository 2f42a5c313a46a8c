// Block-query GQA attention over the target's paged KV, tcgen05 version (dh = 128, 16-token pages).
//
// Same decomposition as attention.cu — CTA = (request, KV head, context chunk[, 128-row tile]), partials
// (m, l, O) per chunk merged afterwards — but both contractions run on the 5th-generation tensor cores:
//
//   warp 8      producer: K/V pages -> shared memory.  Full 128-key tiles are 32 TMA boxes (one
//               [16 tokens x 64 dh] box per page and head-dim half, 128-byte swizzle: each box is the page's rows
//               of this KV head exactly as the target stored them).  The ragged end of the context and the block's
//               own keys/values go through plain 16-byte loads with zero fill, so no garbage row is ever multiplied.
//   warp 9      issues S = Q K^T (A = Q, B = K tile, both K-major) into one of two TMEM S buffers, then
//               O += P V (A = P read from TMEM, B = V tile as an MN-major operand) into the TMEM O buffer.
//   warps 0..7  softmax: two threads per query row (= TMEM lane), 64 key columns each; they exchange their half-row
//               maxima through shared memory.  Each reads its S half-row, masks by selection, keeps a
//               reference maximum that only moves when the row maximum outgrows it by 2^8 (then, rarely, rescales
//               its O row in TMEM), writes P (bf16, two keys per 32-bit column) into one of two TMEM P buffers.
//
// The MMA warp issues S_{t+1} before it waits for P_t, so the tensor core works on the next tile's scores while
// the softmax warps are busy, and the producer runs NS tiles ahead.  Every wait is bounded.
#include "common.cuh"
#include "kernels.h"

#include <cstdio>

namespace hspec {

namespace {

constexpr int KT = 128;            // keys per tile
constexpr int DH = 128;
constexpr int NS = 3;              // K/V stages in shared memory
constexpr int HALF_BYTES = 128 * 128;            // [128 rows x 64 bf16] = 16 KiB
constexpr int TILE_BYTES = 2 * HALF_BYTES;       // one operand tile [128 x 128] bf16
constexpr float NEG = -1.0e30f;
constexpr float LAZY = 8.0f;       // rescale only when the row maximum exceeds the reference by 2^8

struct AttnTcArgs {
  const __nv_bfloat16 *q, *kb, *vb, *k_pool, *v_pool;
  const int32_t* page_table;
  const int32_t* ctx_lens;
  float* ws_o;
  float* ws_ml;
  uint32_t* status;
  int page_table_stride;
  int B, k, Hq, Hkv, rep, R, n_row_tiles;
  int chunk, max_chunks, window;
  float scale_log2;
};

struct __align__(8) AttnTcBars {
  uint64_t q_ready, o_done;
  uint64_t k_full[NS], v_full[NS], kv_empty[NS];
  uint64_t s_ready[2], p_ready[2], pv_done[2];
  uint32_t tmem_base;
  uint32_t abort_flag;
  __half xmax[2][2][128];  // [tile parity][column half][row]: half-row maxima exchanged between the two threads of a row
                           // (1 KiB; reused as float [2][128] for the final row-sum exchange)
};

// byte offset of (row, 16-byte chunk 0..15) inside a [128 x 128] bf16 operand tile stored as two K-major halves
// with the 128-byte swizzle (the layout TMA writes and the UMMA descriptors read)
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return uint32_t((chunk >> 3) * HALF_BYTES + (row >> 3) * 1024 + (row & 7) * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// adds to the barrier's expected byte count without arriving on it
__device__ __forceinline__ void mbar_expect_tx_only(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* tmap, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

// MN-major B operand (V tile: rows = keys, 128 bytes = 64 head-dim elements per row and half), 128-byte swizzle:
// LBO = distance between the two 64-element head-dim halves, SBO = distance between 8-key groups.
__device__ __forceinline__ uint64_t umma_desc_mnmajor_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= uint64_t((smem_addr & 0x3FFFF) >> 4);
  d |= uint64_t(HALF_BYTES >> 4) << 16;
  d |= uint64_t(1024 >> 4) << 32;
  d |= uint64_t(1) << 46;
  d |= uint64_t(2) << 61;
  return d;
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
// 2^x by the special-function unit alone (flush-to-zero form: no range fix-up code around it)
__device__ __forceinline__ float ex2_ftz(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[tmem] * B[smem desc]: the A operand (128 rows x 16 bf16 = 8 columns) is read from tensor memory
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}

// instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = 128, A K-major, B K-major or MN-major
__device__ __forceinline__ uint32_t idesc_bf16_128x128(bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// Geometry of one CTA's key range, computed identically by every role.
struct Range {
  int base;        // first position of the visible prefix, rounded down to a page boundary
  int n_chunks;
  int p_begin;     // first position of this chunk
  int n_full;      // 128-key tiles fetched by TMA
  int rem;         // valid prefix keys after the full tiles (only in the last chunk)
  int n_manual;    // 0, 1 or 2 hand-loaded tiles (ragged end and/or the block's own keys)
  int T;           // tiles in total
  bool last;
};

__device__ __forceinline__ Range make_range(int ctx, int window, int chunk, int c, int k) {
  Range g;
  const int lo0 = (window > 0) ? max(0, ctx - window + 1) : 0;
  g.base = lo0 & ~15;
  const int len = ctx - g.base;
  g.n_chunks = max(1, (len + chunk - 1) / chunk);
  g.last = (c == g.n_chunks - 1);
  g.p_begin = g.base + c * chunk;
  const int p_end = min(ctx, g.p_begin + chunk);
  const int span = max(0, p_end - g.p_begin);
  g.n_full = span / KT;
  g.rem = span - g.n_full * KT;
  g.n_manual = g.last ? ((g.rem + k <= KT) ? 1 : 2) : 0;
  g.T = g.n_full + g.n_manual;
  return g;
}

// For manual tile index mi (0 or 1): how many prefix keys and block keys it holds, and where the prefix keys start.
__device__ __forceinline__ void manual_tile(const Range& g, int mi, int k, int& n_prefix, int& prefix_start, int& n_block) {
  prefix_start = g.p_begin + g.n_full * KT;
  if (g.n_manual == 1) { n_prefix = g.rem; n_block = k; }
  else if (mi == 0) { n_prefix = g.rem; n_block = 0; }
  else { n_prefix = 0; n_block = k; }
}

__global__ void __launch_bounds__(320, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, AttnTcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                               // 32 KiB
  uint8_t* sKV = sQ + TILE_BYTES;                   // NS x (K 32 KiB + V 32 KiB)
  AttnTcBars* bars = reinterpret_cast<AttnTcBars*>(sKV + NS * 2 * TILE_BYTES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.z, kvh = blockIdx.y;
  const int c = blockIdx.x / a.n_row_tiles, rt = blockIdx.x % a.n_row_tiles;
  const int ctx = a.ctx_lens[b];
  const Range g = make_range(ctx, a.window, a.chunk, c, a.k);
  if (c >= g.n_chunks) return;                      // uniform for the whole CTA

  if (tid == 0) {
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
    mbar_init(smem_u32(&bars->q_ready), 8);            // one arrival per softmax warp
    mbar_init(smem_u32(&bars->o_done), 1);
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&bars->k_full[s]), 1);
      mbar_init(smem_u32(&bars->v_full[s]), 1);
      mbar_init(smem_u32(&bars->kv_empty[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bars->s_ready[i]), 1);
      mbar_init(smem_u32(&bars->p_ready[i]), 8);
      mbar_init(smem_u32(&bars->pv_done[i]), 1);
    }
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  const uint32_t tmem_o = tmem;                     // columns [0, 128)
  const uint32_t tmem_s0 = tmem + 128;              // S buffers: columns [128, 256) and [256, 384)
  const uint32_t tmem_p0 = tmem + 384;              // P buffers (bf16 pairs): columns [384, 448) and [448, 512)
  volatile uint32_t* abort_flag = &bars->abort_flag;
  const int row0 = rt * 128;

  if (warp == 8) {
    // ================================================================= producer
    const int32_t* ptab = a.page_table + size_t(b) * a.page_table_stride;
    // page ids are fetched one tile ahead (lanes 0..7, one page each): no dependent global load on the issue path
    int page_next = (lane < 8 && g.n_full > 0) ? ptab[(g.p_begin >> 4) + lane] : 0;
    for (int t = 0; t < g.T; ++t) {
      const int page_cur = page_next;
      if (lane < 8 && t + 1 < g.n_full) page_next = ptab[(g.p_begin >> 4) + (t + 1) * 8 + lane];
      const int s = t % NS;
      if (t >= NS && !mbar_wait(smem_u32(&bars->kv_empty[s]), ((t / NS) - 1) & 1)) {
        if (lane == 0) { atomicExch(a.status, STATUS_TIMEOUT_PRODUCER); *abort_flag = 1; }
        break;
      }
      if (*abort_flag) break;
      uint8_t* dK = sKV + s * 2 * TILE_BYTES;
      uint8_t* dV = dK + TILE_BYTES;
      if (t < g.n_full) {
        const uint32_t kf = smem_u32(&bars->k_full[s]), vf = smem_u32(&bars->v_full[s]);
        if (lane == 0) { mbar_expect_tx(kf, TILE_BYTES); mbar_expect_tx(vf, TILE_BYTES); }
        __syncwarp();
        if (lane < 8) {                                   // one lane per page: K first (the score MMA needs it first)
          const int page = page_cur;
          tma_load_4d(smem_u32(dK) + lane * 2048, &tmK, 0, kvh, 0, page, kf);
          tma_load_4d(smem_u32(dK) + HALF_BYTES + lane * 2048, &tmK, 64, kvh, 0, page, kf);
        }
        __syncwarp();
        if (lane < 8) {
          const int page = page_cur;
          tma_load_4d(smem_u32(dV) + lane * 2048, &tmV, 0, kvh, 0, page, vf);
          tma_load_4d(smem_u32(dV) + HALF_BYTES + lane * 2048, &tmV, 64, kvh, 0, page, vf);
        }
      } else {
        // ragged end of the prefix and / or the block's own keys.  Whole pages of the ragged end still come by
        // TMA; the last partial page and the block rows come through cp.async (zero fill for every unused row,
        // so nothing that is not a real key or value is ever multiplied).
        int n_prefix, prefix_start, n_block;
        manual_tile(g, t - g.n_full, a.k, n_prefix, prefix_start, n_block);
        const int full_pages = n_prefix >> 4;
        const int tma_rows = full_pages << 4;
        const uint32_t kf = smem_u32(&bars->k_full[s]), vf = smem_u32(&bars->v_full[s]);
        if (lane == 0 && full_pages > 0) { mbar_expect_tx_only(kf, full_pages * 4096); mbar_expect_tx_only(vf, full_pages * 4096); }
        __syncwarp();
        if (lane < full_pages) {
          const int page = ptab[(prefix_start >> 4) + lane];
          tma_load_4d(smem_u32(dK) + lane * 2048, &tmK, 0, kvh, 0, page, kf);
          tma_load_4d(smem_u32(dK) + HALF_BYTES + lane * 2048, &tmK, 64, kvh, 0, page, kf);
          tma_load_4d(smem_u32(dV) + lane * 2048, &tmV, 0, kvh, 0, page, vf);
          tma_load_4d(smem_u32(dV) + HALF_BYTES + lane * 2048, &tmV, 64, kvh, 0, page, vf);
        }
        for (int idx = lane; idx < (KT - tma_rows) * 16; idx += 32) {
          const int r = tma_rows + (idx >> 4), chunk16 = idx & 15;
          const bool valid = r < n_prefix + n_block;
          size_t off = 0;
          const __nv_bfloat16 *srcK = a.k_pool, *srcV = a.v_pool;
          if (r < n_prefix) {
            const int p = prefix_start + r;
            const int page = ptab[p >> 4];
            off = ((size_t(page) * 16 + (p & 15)) * a.Hkv + kvh) * DH + chunk16 * 8;
          } else if (valid) {
            srcK = a.kb; srcV = a.vb;
            off = ((size_t(b) * a.k + (r - n_prefix)) * a.Hkv + kvh) * DH + chunk16 * 8;
          }
          cp_async16(smem_u32(dK) + tile_off(r, chunk16), srcK + off, valid);
          cp_async16(smem_u32(dV) + tile_off(r, chunk16), srcV + off, valid);
        }
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) { mbar_arrive(smem_u32(&bars->k_full[s])); mbar_arrive(smem_u32(&bars->v_full[s])); }
      }
    }
  } else if (warp == 9) {
    // ================================================================= MMA issuer
    if (lane == 0) {
      const uint32_t id_qk = idesc_bf16_128x128(false), id_pv = idesc_bf16_128x128(true);
      bool ok = mbar_wait(smem_u32(&bars->q_ready), 0);
#ifdef HSPEC_ATTN_TIMING
      long long w_k = 0, w_p = 0, w_v = 0, m0;
#endif
      auto issue_s = [&](int t) -> bool {
        const int s = t % NS;
#ifdef HSPEC_ATTN_TIMING
        m0 = clock64();
#endif
        if (!mbar_wait(smem_u32(&bars->k_full[s]), (t / NS) & 1)) return false;
#ifdef HSPEC_ATTN_TIMING
        w_k += clock64() - m0;
#endif
        tc_fence_after();
        const uint32_t kbase = smem_u32(sKV + s * 2 * TILE_BYTES);
        const uint32_t qbase = smem_u32(sQ);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
          const uint64_t da = umma_desc_kmajor_sw128(qbase + (ks >> 2) * HALF_BYTES) + uint64_t((ks & 3) * 2);
          const uint64_t db = umma_desc_kmajor_sw128(kbase + (ks >> 2) * HALF_BYTES) + uint64_t((ks & 3) * 2);
          umma_bf16(tmem_s0 + (t & 1) * 128, da, db, id_qk, ks > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&bars->s_ready[t & 1]));
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int t = 0; t < g.T && ok; ++t) {
        if (t + 1 < g.T) ok = issue_s(t + 1);
        if (!ok) break;
        const int s = t % NS;
#ifdef HSPEC_ATTN_TIMING
        m0 = clock64();
#endif
        if (!mbar_wait(smem_u32(&bars->p_ready[t & 1]), (t >> 1) & 1)) { ok = false; break; }
#ifdef HSPEC_ATTN_TIMING
        w_p += clock64() - m0; m0 = clock64();
#endif
        if (!mbar_wait(smem_u32(&bars->v_full[s]), (t / NS) & 1)) { ok = false; break; }
#ifdef HSPEC_ATTN_TIMING
        w_v += clock64() - m0;
#endif
        tc_fence_after();
        const uint32_t vbase = smem_u32(sKV + s * 2 * TILE_BYTES + TILE_BYTES);
#pragma unroll
        for (int ks = 0; ks < KT / 16; ++ks) {
          // A = 16 keys of P = 8 TMEM columns of the P buffer; B = the same 16 keys (rows) of V
          const uint64_t db = umma_desc_mnmajor_sw128(vbase + ks * 2048);
          umma_bf16_ts(tmem_o, tmem_p0 + (t & 1) * 64 + ks * 8, db, id_pv, (t > 0 || ks > 0) ? 1u : 0u);
        }
        umma_commit(smem_u32(&bars->kv_empty[s]));
        umma_commit(smem_u32(&bars->pv_done[t & 1]));
      }
#ifdef HSPEC_ATTN_TIMING
      if ((blockIdx.x + blockIdx.y * 7 + blockIdx.z * 13) % 97 == 0)
        printf("  mma (%d,%d,%d): wait_k=%lld wait_p=%lld wait_v=%lld\n", blockIdx.x, blockIdx.y, blockIdx.z, w_k, w_p, w_v);
#endif
      if (ok) umma_commit(smem_u32(&bars->o_done));
      else {
        atomicExch(a.status, STATUS_TIMEOUT_MMA);
        *abort_flag = 1;
        mbar_arrive(smem_u32(&bars->o_done));
      }
    }
  } else {
    // ================================================================= softmax warps: two threads per query row
    // warps 0..3 own key columns [0, 64) of the tile, warps 4..7 columns [64, 128); warp w reads TMEM lane quarter
    // w % 4, so threads tid and tid + 128 share a row and exchange their half-row maxima through shared memory.
    const int r_local = tid & 127;                   // TMEM lane = query row of the tile
    const int hf = tid >> 7;                         // which half of the key columns
    const int rg = row0 + r_local;                   // row among the k * rep rows of this KV head
    const bool row_ok = rg < a.R;
    const int i_blk = rg / a.rep;                    // block position of the row
    {   // Q row -> shared memory (zeros for padding rows): each thread of the pair writes one head-dim half
      const __nv_bfloat16* src = a.q + ((size_t(b) * a.k + (row_ok ? i_blk : 0)) * a.Hq + kvh * a.rep + (row_ok ? rg % a.rep : 0)) * DH;
#pragma unroll
      for (int c8 = 0; c8 < 8; ++c8) {
        const int ch = hf * 8 + c8;
        const uint4 v = row_ok ? *reinterpret_cast<const uint4*>(src + ch * 8) : make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(sQ + tile_off(r_local, ch)) = v;
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->q_ready));
    }
    const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
    float m_ref = NEG, l_sum = 0.f;
    bool ok = true;
#ifdef HSPEC_ATTN_TIMING
    long long t_wait_s = 0, t_wait_pv = 0, t_start = clock64(), t_mark, t_ld = 0, t_bar = 0, t_exp = 0, t_st = 0;
#endif
    for (int t = 0; t < g.T && ok; ++t) {
#ifdef HSPEC_ATTN_TIMING
      t_mark = clock64();
#endif
      if (!mbar_wait(smem_u32(&bars->s_ready[t & 1]), (t >> 1) & 1)) { ok = false; break; }
#ifdef HSPEC_ATTN_TIMING
      t_wait_s += clock64() - t_mark;
#endif
      tc_fence_after();
#ifdef HSPEC_ATTN_TIMING
      t_mark = clock64();
#endif
      float s[64];
      const int col0 = hf * 64;                      // first key column of this thread
#pragma unroll
      for (int j = 0; j < 2; ++j) tmem_ld32(tmem_s0 + (t & 1) * 128 + lane_base + col0 + j * 32, reinterpret_cast<uint32_t*>(s + j * 32));
      tmem_ld_wait();
#ifdef HSPEC_ATTN_TIMING
      t_ld += clock64() - t_mark; t_mark = clock64();
#endif
      // ---- mask by selection (raw scores; the positive scale is folded into the exponent below)
      if (t < g.n_full) {
        const int key0 = g.p_begin + t * KT + col0;
        if (a.window > 0 && key0 < g.base + 16 + a.k) {                   // leading edge of the window
#pragma unroll
          for (int j = 0; j < 64; ++j)
            if ((ctx + i_blk) - (key0 + j) >= a.window) s[j] = -INFINITY;
        }
      } else {
        int n_prefix, prefix_start, n_block;
        manual_tile(g, t - g.n_full, a.k, n_prefix, prefix_start, n_block);
#pragma unroll
        for (int j = 0; j < 64; ++j) {
          const int col = col0 + j;
          bool vis;
          if (col < n_prefix) vis = a.window <= 0 || (ctx + i_blk) - (prefix_start + col) < a.window;
          else {
            const int jb = col - n_prefix;
            vis = jb < n_block && jb <= i_blk && (a.window <= 0 || i_blk - jb < a.window);
          }
          if (!vis) s[j] = -INFINITY;
        }
      }
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};         // four chains instead of one
#pragma unroll
      for (int j = 0; j < 64; j += 4) {
        mx4[0] = fmaxf(mx4[0], s[j]); mx4[1] = fmaxf(mx4[1], s[j + 1]);
        mx4[2] = fmaxf(mx4[2], s[j + 2]); mx4[3] = fmaxf(mx4[3], s[j + 3]);
      }
      // exchanged as fp16 (rounded UP, so the reference never undershoots): both threads of the row then hold the
      // same two values and take the same decision; the reference maximum need not be the exact maximum
      const __half mx_own = __float2half_ru(fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])));
      bars->xmax[t & 1][hf][r_local] = mx_own;
      asm volatile("bar.sync 1, 256;" ::: "memory");                        // the eight softmax warps
      const float mx = fmaxf(__half2float(mx_own), __half2float(bars->xmax[t & 1][hf ^ 1][r_local])) * a.scale_log2;
#ifdef HSPEC_ATTN_TIMING
      t_bar += clock64() - t_mark;
#endif
      // ---- reference maximum moves only when the row maximum outgrows it by 2^LAZY (same decision in both halves)
      float factor = 1.f;
      const bool grow = mx > m_ref + LAZY;
      if (grow) { factor = ex2_ftz(m_ref - mx); m_ref = mx; }
      if (t > 0 && __any_sync(0xffffffffu, grow)) {
        // O of the tiles so far must be complete before it is rescaled; each thread rescales its 64 columns
        if (!mbar_wait(smem_u32(&bars->pv_done[(t - 1) & 1]), ((t - 1) >> 1) & 1)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          uint32_t o[32];
          tmem_ld32(tmem_o + lane_base + col0 + j * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
          tmem_st32(tmem_o + lane_base + col0 + j * 32, o);
        }
        tmem_st_wait();
      }
      l_sum *= factor;
      // ---- P = exp2(s - m_ref) -> bf16 pairs -> this thread's half of the TMEM P buffer
#ifdef HSPEC_ATTN_TIMING
      t_mark = clock64();
#endif
      if (t >= 2 && !mbar_wait(smem_u32(&bars->pv_done[t & 1]), ((t >> 1) - 1) & 1)) { ok = false; break; }
#ifdef HSPEC_ATTN_TIMING
      t_wait_pv += clock64() - t_mark;
#endif
#ifdef HSPEC_ATTN_TIMING
      t_mark = clock64();
#endif
      const float neg_m = -m_ref;
      float ls4[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t w[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const float p0 = ex2_ftz(fmaf(s[2 * e], a.scale_log2, neg_m));
        const float p1 = ex2_ftz(fmaf(s[2 * e + 1], a.scale_log2, neg_m));
        ls4[e & 1] += p0; ls4[2 + (e & 1)] += p1;
        w[e] = pack_bf16(p0, p1);
      }
#ifdef HSPEC_ATTN_TIMING
      t_exp += clock64() - t_mark; t_mark = clock64();
#endif
      tmem_st32(tmem_p0 + (t & 1) * 64 + lane_base + hf * 32, w);
      l_sum += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
      tmem_st_wait();
#ifdef HSPEC_ATTN_TIMING
      t_st += clock64() - t_mark;
#endif
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->p_ready[t & 1]));   // one arrival per warp, after all its lanes' stores
    }
#ifdef HSPEC_ATTN_TIMING
    if (tid == 0 && (blockIdx.x + blockIdx.y * 7 + blockIdx.z * 13) % 97 == 0)
      printf("attn cta (%d,%d,%d): T=%d total=%lld wait_s=%lld wait_pv=%lld ld=%lld max+bar=%lld exp=%lld st=%lld clocks\n", blockIdx.x, blockIdx.y,
             blockIdx.z, g.T, clock64() - t_start, t_wait_s, t_wait_pv, t_ld, t_bar, t_exp, t_st);
#endif
    if (!ok) { atomicExch(a.status, STATUS_TIMEOUT_EPILOGUE); *abort_flag = 1; }
    // ---- partial (m, l, O) of this chunk: the row sum is the sum of the two halves
    float* xl = reinterpret_cast<float*>(&bars->xmax[0][0][0]);            // [2][128] floats
    asm volatile("bar.sync 1, 256;" ::: "memory");                          // everyone is done with the maxima
    xl[hf * 128 + r_local] = l_sum;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const float l_row = l_sum + xl[(hf ^ 1) * 128 + r_local];
    if (ok && mbar_wait(smem_u32(&bars->o_done), 0) && !*abort_flag) {
      tc_fence_after();
      const size_t slab = (size_t(b) * a.Hkv + kvh) * a.max_chunks + c;
      float* dst = a.ws_o + (slab * a.R + (row_ok ? rg : 0)) * DH + hf * 64;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        uint32_t o[32];
        tmem_ld32(tmem_o + lane_base + hf * 64 + j * 32, o);
        tmem_ld_wait();
        if (row_ok) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<uint4*>(dst + j * 32 + e) = make_uint4(o[e], o[e + 1], o[e + 2], o[e + 3]);
        }
      }
      if (row_ok && hf == 0) {
        float* ml = a.ws_ml + (slab * a.R + rg) * 2;
        ml[0] = (m_ref == NEG) ? -INFINITY : m_ref;
        ml[1] = l_row;
      }
    }
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// One block per (row of the block, query head): merge the chunk partials in chunk order (page-aligned chunk geometry).
__global__ void attn_tc_merge_kernel(AttnTcArgs a, __half* __restrict__ o, int n_pairs) {
  // one warp per (row, head): each lane merges four adjacent head-dim columns with 16-byte loads
  const int pair = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (pair >= n_pairs) return;
  const int m = pair / a.Hq, hq = pair % a.Hq;
  const int b = m / a.k, i = m % a.k;
  const int kvh = hq / a.rep, r = i * a.rep + hq % a.rep;
  const Range g = make_range(a.ctx_lens[b], a.window, a.chunk, 0, a.k);
  const size_t slab0 = (size_t(b) * a.Hkv + kvh) * a.max_chunks;
  float m_tot = -INFINITY;
  for (int c = 0; c < g.n_chunks; ++c) m_tot = fmaxf(m_tot, a.ws_ml[((slab0 + c) * a.R + r) * 2]);
  const float ref = (m_tot == -INFINITY) ? 0.f : m_tot;
  const int d4 = threadIdx.x & 31;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float L = 0.f;
  for (int c = 0; c < g.n_chunks; ++c) {
    const float* ml = a.ws_ml + ((slab0 + c) * a.R + r) * 2;
    const float w = exp2f(ml[0] - ref);
    L += ml[1] * w;
    const float4 v = reinterpret_cast<const float4*>(a.ws_o + ((slab0 + c) * a.R + r) * DH)[d4];
    acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
  }
  const float inv = 1.f / L;
  __half2 lo = __floats2half2_rn(acc.x * inv, acc.y * inv), hi = __floats2half2_rn(acc.z * inv, acc.w * inv);
  uint2 out;
  out.x = *reinterpret_cast<uint32_t*>(&lo);
  out.y = *reinterpret_cast<uint32_t*>(&hi);
  reinterpret_cast<uint2*>(o + (size_t(m) * a.Hq + hq) * DH)[d4] = out;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 4-D view of a pool [num_pages, 16, Hkv, dh] bf16; one box = the 16 rows of one page for one KV head and one
// 64-element half of the head dim (16 x 128 bytes).
bool make_pool_tmap(CUtensorMap* tm, const void* pool, int64_t num_pages, int Hkv, std::string* err) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
      if (err) *err = "cuTensorMapEncodeTiled is not available";
      return false;
    }
    enc = reinterpret_cast<EncodeTiledFn>(p);
  }
  if (reinterpret_cast<uintptr_t>(pool) & 15) { if (err) *err = "KV pool must be 16-byte aligned"; return false; }
  cuuint64_t dims[4] = {cuuint64_t(DH), cuuint64_t(Hkv), 16, cuuint64_t(num_pages)};
  cuuint64_t strides[3] = {cuuint64_t(DH) * 2, cuuint64_t(Hkv) * DH * 2, cuuint64_t(16) * Hkv * DH * 2};
  cuuint32_t box[4] = {64, 1, 16, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pool), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { if (err) *err = "cuTensorMapEncodeTiled (KV pool) failed with CUresult " + std::to_string(int(r)); return false; }
  return true;
}

}  // namespace

bool attention_tc_supported(const AttnCall& c) {
  return c.dh == 128 && c.page_size == 16 && c.num_pages > 0 && (c.chunk_tokens % KT) == 0 && c.k <= KT;
}

cudaError_t attention_tc_launch(const AttnCall& c, int max_chunks, cudaStream_t stream, Tracker* trk, std::string* err) {
  AttnTcArgs a{};
  a.q = (const __nv_bfloat16*)c.q; a.kb = (const __nv_bfloat16*)c.kb; a.vb = (const __nv_bfloat16*)c.vb;
  a.k_pool = (const __nv_bfloat16*)c.k_pool; a.v_pool = (const __nv_bfloat16*)c.v_pool;
  a.page_table = c.page_table; a.ctx_lens = c.ctx_lens; a.page_table_stride = c.page_table_stride;
  a.status = c.status;
  a.B = c.B; a.k = c.k; a.Hq = c.Hq; a.Hkv = c.Hkv; a.rep = c.Hq / c.Hkv; a.R = c.k * a.rep;
  a.n_row_tiles = (a.R + 127) / 128;
  a.chunk = c.chunk_tokens; a.max_chunks = max_chunks; a.window = c.window;
  a.scale_log2 = 1.4426950408889634f / sqrtf(float(c.dh));
  const size_t slabs = size_t(c.B) * c.Hkv * max_chunks;
  a.ws_o = reinterpret_cast<float*>(c.ws);
  a.ws_ml = a.ws_o + slabs * a.R * c.dh;
  CUtensorMap tmK, tmV;
  if (!make_pool_tmap(&tmK, c.k_pool, c.num_pages, c.Hkv, err) || !make_pool_tmap(&tmV, c.v_pool, c.num_pages, c.Hkv, err))
    return cudaErrorInvalidValue;
  const size_t smem = size_t(TILE_BYTES) * (1 + 2 * NS) + sizeof(AttnTcBars) + 1024;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid(max_chunks * a.n_row_tiles, c.Hkv, c.B);
  trk_begin(trk, "attn_partial");
  attn_tc_kernel<<<grid, 320, smem, stream>>>(tmK, tmV, a);
  trk_end(trk);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int n_pairs = c.B * c.k * c.Hq;
  trk_begin(trk, "attn_merge");
  attn_tc_merge_kernel<<<(n_pairs + 7) / 8, 256, 0, stream>>>(a, reinterpret_cast<__half*>(c.o), n_pairs);
  trk_end(trk);
  return cudaGetLastError();
}

}  // namespace hspec
