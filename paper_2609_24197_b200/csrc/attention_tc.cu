// Block-query GQA attention over the target's paged KV, tcgen05 version (dh = 128, 16-token pages).
//
// Same decomposition as attention.cu — work item = (request, KV head, context chunk[, 128-row tile]), partials
// (m, l, O) per chunk merged afterwards — but both contractions run on the 5th-generation tensor cores, and the
// kernel is persistent: a small plan kernel writes the work list (longest items first), one CTA per SM walks it.
//
//   warp 8      K producer, warp 10 V producer: pages -> their own rings of 32 KiB slots in shared memory (3 + 3
//               slots).  Full 128-key tiles are 16 TMA boxes per operand (one [16 tokens x 64 dh] box per page and
//               head-dim half, 128-byte swizzle: each box is the page's rows of this KV head exactly as the target
//               stored them).  The ragged end of the context and the block's own keys/values go through plain
//               16-byte loads with zero fill, so no garbage row is ever multiplied.  A K slot is released as soon as
//               the tile's scores are computed, a V slot after the P V product; both producers run on into the next
//               work item, so HBM keeps streaming while an item's result is read out.
//   warp 9      issues S = Q K^T (A = Q from shared memory, B = K tile, both K-major) into one of three TMEM S buffers,
//               then O += P V (A = P read from TMEM, B = V tile as an MN-major operand) into the TMEM O buffer.
//   warps 0..7  softmax: two threads per query row (= TMEM lane), 64 key columns each; they exchange their half-row
//               maxima through shared memory.  Each reads its S half-row, masks by selection, keeps a
//               reference maximum that only moves when the row maximum outgrows it by 2^8 (then, rarely, rescales
//               its O row in TMEM), and writes P (bf16, two keys per 32-bit column) over the first half of the S
//               buffer it came from.  During an item's last tile they copy the next item's Q tile into shared
//               memory (cp.async, no registers); at its end they read O out: as a finished fp16 row when the request
//               has a single chunk, else as an fp32 partial for the merge kernel.
//
// The MMA warp keeps the scores two tiles ahead of the softmax warps (O and three score buffers fill the 512 TMEM
// columns): S_{t+1} and S_{t+2} are issued before it waits for P_t, so the softmax warps always find the next tile's
// scores waiting and the issuing thread's time on a score product is off the P_t -> P V -> S -> softmax chain (-3 %
// against two buffers).  The lookahead crosses item boundaries: the softmax warps copy the next item's Q tile into
// shared memory while they work on the current item's last tile - every product that reads the old Q has finished by
// then - so the next item's first scores are computed during the current item's last P V product and read-out
// (another -3 % at 32B-class shapes, -5..8 % where the items are short).  Every wait is bounded; a timed-out role sets
// a status word and the CTA unwinds.
#include "common.cuh"
#include "kernels.h"

#include <cstdio>

namespace hspec {

namespace {

constexpr int KT = 128;            // keys per tile
constexpr int DH = 128;
constexpr int NSK = 3, NSV = 3;    // slots of the K ring and of the V ring (7 x 32 KiB = all of shared memory)
constexpr int NSB = 3;             // score buffers in tensor memory: the MMA warp runs two tiles of scores ahead of the softmax
constexpr int KV_HALF = KT * 128;                // K or V tile: [128 keys x 64 bf16] = 16 KiB per head-dim half
constexpr int KV_BYTES = 2 * KV_HALF;            // one K or V tile [128 keys x 128 dh] bf16 = 32 KiB
constexpr float NEG = -1.0e30f;
constexpr float LAZY = 8.0f;       // rescale only when the row maximum exceeds the reference by 2^8

struct AttnTcArgs {
  const __nv_bfloat16 *q, *kb, *vb, *k_pool, *v_pool;
  const int32_t* page_table;
  const int32_t* ctx_lens;
  float* ws_o;
  float* ws_ml;
  uint16_t* o_final;     // [B*k, Hq, dh] fp16 (or bf16 when o_bf16): requests whose context is one chunk are finished
                         // here, without partials; the merge kernel writes the others
  int o_bf16;
  uint32_t* status;
  int page_table_stride;
  int B, k, Hq, Hkv, rep, R, n_row_tiles;
  int chunk, max_chunks, window;
  int max_ctx;           // host bound on the context lengths: a length outside [0, max_ctx] is clamped and counted
  int num_pages;         // pages in each pool: a page id outside [0, num_pages) is read as zeros and counted
  float scale_log2;
};

// A request's context length as every kernel of the attention uses it: the device array's value clamped to the bound
// the host sized the work list, the partials and the page-table row for.
__device__ __forceinline__ int clamped_ctx(const AttnTcArgs& a, int b) { return min(max(a.ctx_lens[b], 0), a.max_ctx); }

struct __align__(8) AttnTcBars {
  uint64_t q_ready, o_done, o_free, l_ready;
  uint64_t x_ready[2];
  uint64_t k_full[NSK], k_empty[NSK], v_full[NSV], v_empty[NSV];
  uint64_t s_ready[NSB], p_ready[NSB];
  uint32_t tmem_base;
  uint32_t abort_flag;
  float xmax[2][2][128];   // [tile parity][column half][row]: half-row maxima exchanged between the two threads of a row
                           // (2 KiB; one parity's first 512 bytes are reused as a float per row for the final row-sum exchange)
};

// byte offset of (row, 16-byte chunk 0..15) inside a [128 x 128] bf16 operand tile stored as two K-major halves
// with the 128-byte swizzle (the layout TMA writes and the UMMA descriptors read)
template <int HALF>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return uint32_t((chunk >> 3) * HALF + (row >> 3) * 1024 + (row & 7) * 128 + (((chunk & 7) ^ (row & 7)) << 4));
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
  d |= uint64_t(KV_HALF >> 4) << 16;
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
// Waits for the outstanding tensor-memory loads; the 32 destination registers are operands, so no use of them can be
// scheduled ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld32(uint32_t* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
                 "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                 "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
// two fp32 operations in one instruction (sm_100 packed forms): halves the issue slots of the scale-and-subtract and of
// the row-sum adds around the exponentials
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
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

// Work item = (request, KV head, context chunk, 128-row tile); x = request, y = KV head | row tile << 16, z = chunk,
// w = the request's context length (so that one 16-byte load tells a role everything about the item).
struct Item { int b, kvh, rt, c, ctx; };
__device__ __forceinline__ Item unpack_item(const int4 w) {
  Item it;
  it.b = w.x; it.kvh = w.y & 0xffff; it.rt = w.y >> 16; it.c = w.z; it.ctx = w.w;
  return it;
}

// The n-th item of this CTA.  The list is sorted longest first; handing round n out in ascending CTA order for even n and
// in descending order for odd n evens out the CTAs' shares (plain round-robin gives CTA 0 the longest item of every
// round).  Once an index falls past the end of the list, every later one does too.
__device__ __forceinline__ int item_at(int n) {
  const int G = int(gridDim.x), c = int(blockIdx.x);
  return n * G + ((n & 1) ? G - 1 - c : c);
}

// Work list: one item per (request, KV head, context chunk, 128-row tile), longest first (bucketed by tile count),
// heads of one request and chunk next to each other so the CTAs that run them at the same time read neighbouring
// bytes of the same pages.  The order inside a bucket depends on atomics; every item is computed independently, so
// results do not.
__global__ void attn_tc_plan_kernel(AttnTcArgs a, int* __restrict__ count, int4* __restrict__ items) {
  pdl_wait();
  pdl_trigger();
  __shared__ int bucket[64];
  __shared__ int offset[64];
  const int per_chunk = a.Hkv * a.n_row_tiles;
  const int pairs = a.B * a.max_chunks;            // one thread per (request, chunk slot); slots past n_chunks are skipped
  for (int i = threadIdx.x; i < 64; i += blockDim.x) bucket[i] = 0;
  __syncthreads();
  for (int i = threadIdx.x; i < pairs; i += blockDim.x) {
    const int b = i / a.max_chunks, c = i % a.max_chunks;
    if (c == 0 && a.ctx_lens[b] != clamped_ctx(a, b)) atomicAdd(a.status + STATUS_WORD_BAD_INPUT, 1u);
    const Range g = make_range(clamped_ctx(a, b), a.window, a.chunk, c, a.k);
    if (c < g.n_chunks) atomicAdd(&bucket[min(g.T, 63)], per_chunk);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int off = 0;
    for (int T = 63; T >= 0; --T) { offset[T] = off; off += bucket[T]; }
    *count = off;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < pairs; i += blockDim.x) {
    const int b = i / a.max_chunks, c = i % a.max_chunks;
    const int ctx = clamped_ctx(a, b);
    const Range g = make_range(ctx, a.window, a.chunk, c, a.k);
    if (c >= g.n_chunks) continue;
    int at = atomicAdd(&offset[min(g.T, 63)], per_chunk);
    for (int kvh = 0; kvh < a.Hkv; ++kvh)
      for (int rt = 0; rt < a.n_row_tiles; ++rt) items[at++] = make_int4(b, kvh | (rt << 16), c, ctx);
  }
}

// One operand (K or V) of every tile of this CTA's items -> its own ring of 32 KiB slots.  K and V have separate
// rings and separate producer warps because their slots are released at different times (K once the tile's scores
// are computed, V only after the softmax of the tile and the P V product), and a single in-order producer would
// hold the next K loads back behind a V slot that is still in use.
//   Full 128-key tiles are 16 TMA boxes (one [16 tokens x 64 dh] box per page and head-dim half, 128-byte swizzle).
//   The ragged end of the prefix and the block's own rows: whole pages still by TMA, the rest through 16-byte
//   cp.async with zero fill for every unused row, so nothing that is not a real key or value is ever multiplied.
__device__ __forceinline__ void produce_operand(const AttnTcArgs& a, const CUtensorMap* tm, const __nv_bfloat16* pool,
                                                const __nv_bfloat16* blk, uint8_t* ring, uint64_t* full, uint64_t* empty,
                                                volatile uint32_t* abort_flag, const int4* __restrict__ items, int n_items,
                                                int lane, int ns) {
  uint32_t gt = 0;                                 // tiles issued so far, across items
  int4 w_next = items[item_at(0)];
  for (int n = 0; item_at(n) < n_items; ++n) {
    const Item wi = unpack_item(w_next);
    if (item_at(n + 1) < n_items) w_next = items[item_at(n + 1)];         // consumed one item later
    const int b = wi.b, kvh = wi.kvh;
    const Range g = make_range(wi.ctx, a.window, a.chunk, wi.c, a.k);
    const int32_t* ptab = a.page_table + size_t(b) * a.page_table_stride;
    // page ids are fetched one tile ahead (lanes 0..3, one page each): no dependent global load on the issue path
    int page_next = (lane < KT / 16 && g.n_full > 0) ? ptab[(g.p_begin >> 4) + lane] : 0;
    for (int t = 0; t < g.T; ++t, ++gt) {
      const int page_cur = page_next;
      if (lane < KT / 16 && t + 1 < g.n_full) page_next = ptab[(g.p_begin >> 4) + (t + 1) * (KT / 16) + lane];
      const int s = gt % ns;
      if (gt >= uint32_t(ns) && !mbar_wait(smem_u32(&empty[s]), ((gt / ns) - 1) & 1)) {
        if (lane == 0) { atomicExch(a.status, STATUS_TIMEOUT_PRODUCER); *abort_flag = 1; }
        return;
      }
      if (*abort_flag) return;
      uint8_t* dst = ring + s * KV_BYTES;
      const uint32_t bar = smem_u32(&full[s]);
      if (t < g.n_full) {
        if (lane == 0) mbar_expect_tx(bar, KV_BYTES);
        __syncwarp();
        if (lane < KT / 16) {
          // (a page id outside the pool is outside the tensor map: the copy delivers zeros and touches no memory)
          if (unsigned(page_cur) >= unsigned(a.num_pages)) atomicAdd(a.status + STATUS_WORD_BAD_INPUT, 1u);
          tma_load_4d(smem_u32(dst) + lane * 2048, tm, 0, kvh, 0, page_cur, bar);
          tma_load_4d(smem_u32(dst) + KV_HALF + lane * 2048, tm, 64, kvh, 0, page_cur, bar);
        }
      } else {
        int n_prefix, prefix_start, n_block;
        manual_tile(g, t - g.n_full, a.k, n_prefix, prefix_start, n_block);
        const int full_pages = n_prefix >> 4;
        const int tma_rows = full_pages << 4;
        if (lane == 0 && full_pages > 0) mbar_expect_tx_only(bar, full_pages * 4096);
        __syncwarp();
        if (lane < full_pages) {
          const int page = ptab[(prefix_start >> 4) + lane];
          if (unsigned(page) >= unsigned(a.num_pages)) atomicAdd(a.status + STATUS_WORD_BAD_INPUT, 1u);
          tma_load_4d(smem_u32(dst) + lane * 2048, tm, 0, kvh, 0, page, bar);
          tma_load_4d(smem_u32(dst) + KV_HALF + lane * 2048, tm, 64, kvh, 0, page, bar);
        }
        for (int idx = lane; idx < (KT - tma_rows) * 16; idx += 32) {
          const int r = tma_rows + (idx >> 4), chunk16 = idx & 15;
          bool valid = r < n_prefix + n_block;
          size_t off = 0;
          const __nv_bfloat16* src = pool;
          if (r < n_prefix) {
            const int p = prefix_start + r;
            const int page = ptab[p >> 4];
            if (unsigned(page) >= unsigned(a.num_pages)) {       // never form an address from a bad id: zero row, counted once
              valid = false;
              if (chunk16 == 0 && (p & 15) == 0) atomicAdd(a.status + STATUS_WORD_BAD_INPUT, 1u);
            } else {
              off = ((size_t(page) * 16 + (p & 15)) * a.Hkv + kvh) * DH + chunk16 * 8;
            }
          } else if (valid) {
            src = blk;
            off = ((size_t(b) * a.k + (r - n_prefix)) * a.Hkv + kvh) * DH + chunk16 * 8;
          }
          cp_async16(smem_u32(dst) + tile_off<KV_HALF>(r, chunk16), src + off, valid);
        }
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar);
      }
    }
  }
}

// Persistent: one CTA per SM walks the work list (items item_at(0), item_at(1), ...).  All ring and buffer indices
// count tiles across items (gt): K slot = gt % NSK, V slot = gt % NSV, S / P buffer = gt % NSB.
__global__ void __launch_bounds__(352, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, AttnTcArgs a,
               const int* __restrict__ count, const int4* __restrict__ items) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sQ = smem;                               // Q tile, 32 KiB
  uint8_t* sKV = smem + KV_BYTES;                   // K ring (NSK x 32 KiB), then V ring (NSV x 32 KiB)
  AttnTcBars* bars = reinterpret_cast<AttnTcBars*>(sKV + (NSK + NSV) * KV_BYTES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_items = *count;
  if (item_at(0) >= n_items) return;                // uniform for the whole CTA
  if (smem_u32(smem) & 1023) {                      // the swizzled operand tiles need a 1 KiB-aligned base
    if (tid == 0) atomicExch(a.status, STATUS_BAD_SMEM_BASE);
    return;
  }

  if (tid == 0) {
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
    mbar_init(smem_u32(&bars->q_ready), 8);            // one arrival per softmax warp
    mbar_init(smem_u32(&bars->o_free), 8);
    mbar_init(smem_u32(&bars->l_ready), 8);
    mbar_init(smem_u32(&bars->o_done), 1);
    for (int s = 0; s < NSK; ++s) {
      mbar_init(smem_u32(&bars->k_full[s]), 1);
      mbar_init(smem_u32(&bars->k_empty[s]), 1);
    }
    for (int s = 0; s < NSV; ++s) {
      mbar_init(smem_u32(&bars->v_full[s]), 1);
      mbar_init(smem_u32(&bars->v_empty[s]), 1);
    }
    for (int i = 0; i < NSB; ++i) {
      mbar_init(smem_u32(&bars->s_ready[i]), 1);
      mbar_init(smem_u32(&bars->p_ready[i]), 8);
    }
    for (int i = 0; i < 2; ++i) mbar_init(smem_u32(&bars->x_ready[i]), 8);
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
  // tensor memory: O in columns [0, 128), three S buffers in [128, 256), [256, 384) and [384, 512); P (bf16 pairs, 64
  // columns) overwrites the first half of the S buffer it was computed from
  const uint32_t tmem_o = tmem, tmem_s0 = tmem + 128;
  volatile uint32_t* abort_flag = &bars->abort_flag;

  if (warp == 8 || warp == 10) {
    // ================================================================= producers: warp 8 streams K, warp 10 streams V
    const bool is_v = warp == 10;
    produce_operand(a, is_v ? &tmV : &tmK, is_v ? a.v_pool : a.k_pool, is_v ? a.vb : a.kb, sKV + (is_v ? NSK * KV_BYTES : 0),
                    is_v ? bars->v_full : bars->k_full, is_v ? bars->v_empty : bars->k_empty, abort_flag, items, n_items, lane,
                    is_v ? NSV : NSK);
  } else if (warp == 9) {
    // ================================================================= MMA issuer
    if (lane == 0) {
      // fp32 accumulate, bf16 x bf16, M = 128, N = 128; scores: A = Q, B = K tile, both K-major in shared memory;
      // P V: A = P from tensor memory, B = V tile (MN-major)
      const uint32_t id_qk = idesc_bf16_128x128(false), id_pv = idesc_bf16_128x128(true);
      uint32_t gt = 0, n = 0;                        // tiles and items done so far
      bool ok = true;
#ifdef HSPEC_ATTN_TIMING
      long long mk[8] = {0, 0, 0, 0, 0, 0, 0, 0}, m_last = clock64(), m_start = m_last;
#define MCLK(i) { const long long t_now = clock64(); mk[i] += t_now - m_last; m_last = t_now; }
#else
#define MCLK(i)
#endif
      // Two cursors walk this CTA's tiles in the same order.  The P V cursor (item n, global tile gt) follows the softmax
      // warps.  The score cursor (item n_s, tile t_s of T_s, global tile gts) runs up to two tiles ahead of it, ACROSS
      // item boundaries: the softmax warps put the next item's Q tile in place while they work on this item's last tile
      // (every score product of the item has finished by then), so the next item's first scores are computed while this
      // item's last P V product and its read-out are still under way.
      // S = Q K^T of tile gts into S buffer gts % NSB.  The buffer last held P of tile gts - NSB, whose P V product this
      // thread issued earlier; the tensor pipe runs one thread's MMAs in issue order.
      uint32_t gts = 0, n_s = 0;
      int t_s = 0;
      int4 ws_next = items[item_at(0)];
      bool s_valid = true;
      int T_s;
      {
        const Item w0 = unpack_item(ws_next);
        T_s = make_range(w0.ctx, a.window, a.chunk, w0.c, a.k).T;
        if (item_at(1) < n_items) ws_next = items[item_at(1)];
      }
      // returns 1 = issued, 0 = the item's Q tile is not there yet (only when it may come back later), -1 = timed out
      auto issue_s = [&](bool must) -> int {
        if (t_s == 0) {
          const uint32_t qb = smem_u32(&bars->q_ready);
          MCLK(0)
          if (must) { if (!mbar_wait(qb, n_s & 1)) return -1; }
          else if (!mbar_test(qb, n_s & 1)) return 0;
          MCLK(4)
          tc_fence_after();
        }
        const int s = gts % NSK;
        MCLK(0)
        if (!mbar_wait(smem_u32(&bars->k_full[s]), (gts / NSK) & 1)) return -1;
        MCLK(1)
        tc_fence_after();
        const uint32_t kbase = smem_u32(sKV + s * KV_BYTES);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
          const uint64_t da = umma_desc_kmajor_sw128(smem_u32(sQ) + (ks >> 2) * KV_HALF) + uint64_t((ks & 3) * 2);
          const uint64_t db = umma_desc_kmajor_sw128(kbase + (ks >> 2) * KV_HALF) + uint64_t((ks & 3) * 2);
          umma_bf16(tmem_s0 + (gts % NSB) * 128, da, db, id_qk, ks > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&bars->k_empty[s]));
        umma_commit(smem_u32(&bars->s_ready[gts % NSB]));
        ++gts;
        if (++t_s == T_s) {                            // on to the next item (its descriptor was fetched an item ago)
          t_s = 0;
          ++n_s;
          if (item_at(int(n_s)) < n_items) {
            const Item wn = unpack_item(ws_next);
            T_s = make_range(wn.ctx, a.window, a.chunk, wn.c, a.k).T;
            if (item_at(int(n_s) + 1) < n_items) ws_next = items[item_at(int(n_s) + 1)];
          } else {
            s_valid = false;
          }
        }
        return 1;
      };
      int4 w_next = items[item_at(0)];
      for (; item_at(int(n)) < n_items && ok; ++n) {
        const Item wi = unpack_item(w_next);
        if (item_at(int(n) + 1) < n_items) w_next = items[item_at(int(n) + 1)];
        const Range g = make_range(wi.ctx, a.window, a.chunk, wi.c, a.k);
        for (int t = 0; t < g.T && ok; ++t, ++gt) {
          // the scores of this tile must be under way (the softmax warps wait for them); the next two are issued as soon
          // as their K tile and, at an item's first tile, its Q tile are there
          while (ok && s_valid && gts <= gt + 2) {
            const int r = issue_s(gts <= gt);
            if (r < 0) ok = false;
            if (r <= 0) break;
          }
          if (!ok) break;
          const int s = gt % NSV;
          MCLK(0)
          if (!mbar_wait(smem_u32(&bars->p_ready[gt % NSB]), (gt / NSB) & 1)) { ok = false; break; }
          MCLK(2)
          if (!mbar_wait(smem_u32(&bars->v_full[s]), (gt / NSV) & 1)) { ok = false; break; }
          MCLK(3)
          // the first P V product of an item overwrites O: the previous item's accumulator must have been read out
          if (t == 0 && n > 0 && !mbar_wait(smem_u32(&bars->o_free), (n - 1) & 1)) { ok = false; break; }
          MCLK(5)
          tc_fence_after();
          const uint32_t vbase = smem_u32(sKV + (NSK + s) * KV_BYTES);
#pragma unroll
          for (int ks = 0; ks < KT / 16; ++ks) {
            // A = 16 keys of P = 8 TMEM columns; B = the same 16 keys (rows) of V
            const uint64_t db = umma_desc_mnmajor_sw128(vbase + ks * 2048);
            umma_bf16_ts(tmem_o, tmem_s0 + (gt % NSB) * 128 + ks * 8, db, id_pv, (t > 0 || ks > 0) ? 1u : 0u);
          }
          umma_commit(smem_u32(&bars->v_empty[s]));
        }
        if (ok) umma_commit(smem_u32(&bars->o_done));
      }
#ifdef HSPEC_ATTN_TIMING
      MCLK(0)
      if (blockIdx.x == 0 || blockIdx.x == 147)
        printf("cta %d mma: total %lld | issue %lld wait_k %lld wait_p %lld wait_v %lld wait_q %lld wait_ofree %lld\n",
               blockIdx.x, clock64() - m_start, mk[0], mk[1], mk[2], mk[3], mk[4], mk[5]);
#endif
      if (!ok) {
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
    const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
    const int col0 = hf * 64;                        // first key column of this thread
    uint32_t gt = 0, n = 0;
    bool ok = true;
#ifdef HSPEC_ATTN_TIMING
    long long tk[8] = {0, 0, 0, 0, 0, 0, 0, 0}, t_last = clock64(), t_start = t_last;
#define TCLK(i) { const long long t_now = clock64(); tk[i] += t_now - t_last; t_last = t_now; }
#else
#define TCLK(i)
#endif
    // Each thread of a row pair owns one 64-element half (128 bytes) of the Q row.  The half is pulled into L2 an item
    // ahead and read while the item's last P V product drains.
    auto q_half = [&](const Item& wi, bool& row_ok) -> const __nv_bfloat16* {
      const int rg = wi.rt * 128 + r_local;
      row_ok = rg < a.R;
      return a.q + ((size_t(wi.b) * a.k + (row_ok ? rg / a.rep : 0)) * a.Hq + wi.kvh * a.rep + (row_ok ? rg % a.rep : 0)) * DH + hf * 64;
    };
    auto prefetch_q = [&](const Item& wi) {
      bool row_ok;
      const __nv_bfloat16* src = q_half(wi, row_ok);
      if (row_ok) asm volatile("prefetch.global.L2 [%0];" ::"l"(src));
    };
    // Q tile -> shared memory in the swizzled K-major operand layout (zeros for padding rows), by 16-byte asynchronous
    // copies that need no registers: they are issued once the item's last score product has finished and are waited
    // for after the thread has dealt with that tile.
    auto q_copy_issue = [&](const Item& wi) {
      bool row_ok;
      const __nv_bfloat16* src = q_half(wi, row_ok);
#pragma unroll
      for (int c8 = 0; c8 < 8; ++c8) cp_async16(smem_u32(sQ + tile_off<KV_HALF>(r_local, hf * 8 + c8)), src + c8 * 8, row_ok);
      cp_async_commit();
    };
    auto q_copy_finish = [&]() {
      cp_async_wait<0>();
      fence_proxy_async();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->q_ready));
    };
    int4 w_cur = items[item_at(0)];
    int4 w_next = (item_at(1) < n_items) ? items[item_at(1)] : w_cur;
    q_copy_issue(unpack_item(w_cur));
    q_copy_finish();
    for (; item_at(int(n)) < n_items && ok; ++n) {
      const Item wi = unpack_item(w_cur);
      const int b = wi.b, kvh = wi.kvh, c = wi.c, ctx = wi.ctx;
      const Range g = make_range(ctx, a.window, a.chunk, c, a.k);
      const int rg = wi.rt * 128 + r_local;          // row among the k * rep rows of this KV head
      const bool row_ok = rg < a.R;
      const int i_blk = rg / a.rep;                  // block position of the row
      const bool has_next = item_at(int(n) + 1) < n_items;
      int4 w_next2 = w_next;                         // the descriptor is fetched two items ahead
      if (item_at(int(n) + 2) < n_items) w_next2 = items[item_at(int(n) + 2)];
      if (has_next) prefetch_q(unpack_item(w_next));
      float m_ref = NEG, l_sum = 0.f;
      // a warp all of whose 32 rows are padding (fewer than 128 query rows share the KV head) only keeps the
      // barriers' arrival counts: its rows of S, P and O are never read, and a row of P feeds no other row of O
      const bool warp_live = wi.rt * 128 + (warp & 3) * 32 < a.R;
      TCLK(0)
      for (int t = 0; t < g.T && ok; ++t, ++gt) {
        const uint32_t t_s = tmem_s0 + (gt % NSB) * 128 + lane_base;
        if (!mbar_wait(smem_u32(&bars->s_ready[gt % NSB]), (gt / NSB) & 1)) { ok = false; break; }
        // The scores of the item's last tile are there: every product that reads this item's Q tile has finished, and
        // the next item's Q goes in now, so that the tensor core can start on its scores before this item is done.
        const bool q_now = has_next && t == g.T - 1;
        if (q_now) q_copy_issue(unpack_item(w_next));
        if (!warp_live) {
          // The scores run up to two tiles ahead, and the exchange barrier has two slots: this warp must not arrive for
          // tile t + 2 on the slot the live warps still use for tile t, so it waits for the exchange like they do.
          if (lane == 0) {
            mbar_arrive(smem_u32(&bars->x_ready[gt & 1]));
            mbar_arrive(smem_u32(&bars->p_ready[gt % NSB]));
          }
          if (q_now) q_copy_finish();
          if (!mbar_wait(smem_u32(&bars->x_ready[gt & 1]), (gt >> 1) & 1)) { ok = false; break; }
          continue;
        }
        tc_fence_after();
        TCLK(1)
        float s[64];
#pragma unroll
        for (int j = 0; j < 2; ++j) tmem_ld32(t_s + col0 + j * 32, reinterpret_cast<uint32_t*>(s + j * 32));
        tmem_wait_ld32(reinterpret_cast<uint32_t*>(s));
        tmem_wait_ld32(reinterpret_cast<uint32_t*>(s + 32));
        // ---- mask by selection (raw scores; the positive scale is folded into the exponent below)
        if (t < g.n_full) {
          const int key0 = g.p_begin + t * KT + col0;
          if (a.window > 0 && key0 < g.base + 16 + a.k) {                 // leading edge of the window
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
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};       // four chains instead of one
#pragma unroll
        for (int j = 0; j < 64; j += 4) {
          mx4[0] = fmaxf(mx4[0], s[j]); mx4[1] = fmaxf(mx4[1], s[j + 1]);
          mx4[2] = fmaxf(mx4[2], s[j + 2]); mx4[3] = fmaxf(mx4[3], s[j + 3]);
        }
        // both threads of the row then hold the same two values and take the same decision below
        const float mx_own = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        TCLK(2)
        bars->xmax[gt & 1][hf][r_local] = mx_own;
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->x_ready[gt & 1]));       // bounded exchange between the eight softmax warps
        if (!mbar_wait(smem_u32(&bars->x_ready[gt & 1]), (gt >> 1) & 1)) { ok = false; break; }
        // (past this barrier both threads of the row hold their scores in registers: P may overwrite the S columns)
        const float mx = fmaxf(mx_own, bars->xmax[gt & 1][hf ^ 1][r_local]) * a.scale_log2;
        TCLK(3)
        // ---- reference maximum moves only when the row maximum outgrows it by 2^LAZY (same decision in both halves)
        float factor = 1.f;
        const bool grow = mx > m_ref + LAZY;
        if (grow) { factor = ex2_ftz(m_ref - mx); m_ref = mx; }
        if (t > 0 && __any_sync(0xffffffffu, grow)) {
          // O of the tiles so far must be complete before it is rescaled (the barrier that releases the previous
          // tile's V slot is committed behind its P V product); each thread rescales its 64 columns
          if (!mbar_wait(smem_u32(&bars->v_empty[(gt - 1) % NSV]), ((gt - 1) / NSV) & 1)) { ok = false; break; }
          tc_fence_after();
          if (lane == 0 && hf == 0) atomicAdd(a.status + STATUS_WORD_RESCALES, 1u);   // rare; lets a test see the branch run
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            uint32_t o[32];
            tmem_ld32(tmem_o + lane_base + col0 + j * 32, o);
            tmem_wait_ld32(o);
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
            tmem_st32(tmem_o + lane_base + col0 + j * 32, o);
          }
          tmem_st_wait();
        }
        l_sum *= factor;
        TCLK(4)
        // ---- P = exp2(s * scale - m_ref) -> bf16 pairs -> this thread's 32 of the 64 P columns, which lie over the
        // first half of the S buffer (both threads of the row took their scores into registers before the exchange)
        const uint64_t scale2 = pack_f32x2(a.scale_log2, a.scale_log2), neg_m2 = pack_f32x2(-m_ref, -m_ref);
        uint64_t ls2[2] = {0ull, 0ull};               // two packed accumulators = four row-sum chains
        uint32_t pw[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          float x0, x1;
          unpack_f32x2(fma_f32x2(pack_f32x2(s[2 * e], s[2 * e + 1]), scale2, neg_m2), x0, x1);
          const float p0 = ex2_ftz(x0), p1 = ex2_ftz(x1);
          ls2[e & 1] = add_f32x2(ls2[e & 1], pack_f32x2(p0, p1));
          pw[e] = pack_bf16(p0, p1);
        }
        float ls4[4];
        unpack_f32x2(ls2[0], ls4[0], ls4[1]);
        unpack_f32x2(ls2[1], ls4[2], ls4[3]);
        tmem_st32(t_s + hf * 32, pw);
        l_sum += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->p_ready[gt % NSB]));   // one arrival per warp, after all its lanes' stores
        if (q_now) q_copy_finish();
        TCLK(5)
      }
      if (!ok) break;
      // ---- the row sum is the sum of the two halves: the threads of a row swap theirs through the exchange buffer of
      // parity gt & 1, last used two tiles ago.  The next tile (the next item's first) writes the same slots, so a second
      // round of the barrier keeps every thread from going on before its partner has read.
      bars->xmax[gt & 1][hf][r_local] = l_sum;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->l_ready));
      if (!mbar_wait(smem_u32(&bars->l_ready), 0)) { ok = false; break; }
      const float l_row = l_sum + bars->xmax[gt & 1][hf ^ 1][r_local];
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->l_ready));
      if (!mbar_wait(smem_u32(&bars->l_ready), 1)) { ok = false; break; }
      // every MMA of the item has finished once o_done completes
      if (!mbar_wait(smem_u32(&bars->o_done), n & 1) || *abort_flag) { ok = false; break; }
      tc_fence_after();
      TCLK(6)
      const size_t slab = (size_t(b) * a.Hkv + kvh) * a.max_chunks + c;
      const bool whole = g.n_chunks == 1;            // the request's only chunk: normalise and finish here
      if (!warp_live) {
        // nothing to read out
      } else if (whole) {
        // (the last chunk always holds the row's own block key, so the row sum is positive)
        const float inv = 1.f / l_row;
        uint16_t* dsth = a.o_final + ((size_t(b) * a.k + (row_ok ? i_blk : 0)) * a.Hq + kvh * a.rep + (row_ok ? rg % a.rep : 0)) * DH + hf * 64;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          uint32_t o[32];
          tmem_ld32(tmem_o + lane_base + hf * 64 + j * 32, o);
          tmem_wait_ld32(o);
          if (row_ok) {
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint32_t h[4];
#pragma unroll
              for (int q2 = 0; q2 < 4; ++q2) {
                const float v0 = __uint_as_float(o[e + 2 * q2]) * inv, v1 = __uint_as_float(o[e + 2 * q2 + 1]) * inv;
                if (a.o_bf16) {
                  h[q2] = pack_bf16(v0, v1);
                } else {
                  const __half2 v = __halves2half2(f16_sat(v0, a.status), f16_sat(v1, a.status));
                  h[q2] = *reinterpret_cast<const uint32_t*>(&v);
                }
              }
              *reinterpret_cast<uint4*>(dsth + j * 32 + e) = make_uint4(h[0], h[1], h[2], h[3]);
            }
          }
        }
      } else {
        // partial layout [slab][group of 4 head-dim columns][row][4]: a thread owns a row, so for one column group the
        // 32 lanes of a warp write 32 consecutive rows = 512 contiguous bytes (row-major partials would scatter every
        // 16-byte store of a warp over 32 lines, and the item's read-out took 4 000 clocks of the load/store unit)
        float* dst = a.ws_o + slab * a.R * DH + size_t(row_ok ? rg : 0) * 4;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          uint32_t o[32];
          tmem_ld32(tmem_o + lane_base + hf * 64 + j * 32, o);
          tmem_wait_ld32(o);
          if (row_ok) {
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              *reinterpret_cast<uint4*>(dst + size_t(hf * 16 + j * 8 + e / 4) * a.R * 4) = make_uint4(o[e], o[e + 1], o[e + 2], o[e + 3]);
          }
        }
      }
      // O has been read out: the next item's first P V product may overwrite it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->o_free));
      if (row_ok && hf == 0 && !whole) {
        float* ml = a.ws_ml + (slab * a.R + rg) * 2;
        ml[0] = (m_ref == NEG) ? -INFINITY : m_ref;
        ml[1] = l_row;
      }
      w_cur = w_next;
      w_next = w_next2;
      TCLK(7)
    }
#ifdef HSPEC_ATTN_TIMING
    if ((blockIdx.x == 0 || blockIdx.x == 147) && (tid == 0 || tid == 128))
      printf("cta %d tid %d: items %u tiles %u total %lld | q %lld wait_s %lld max %lld xchg %lld rescale %lld exp %lld wait_o %lld item_end %lld\n",
             blockIdx.x, tid, n, gt, clock64() - t_start, tk[0], tk[1], tk[2], tk[3], tk[4], tk[5], tk[6], tk[7]);
#endif
    if (!ok) { atomicExch(a.status, STATUS_TIMEOUT_EPILOGUE); *abort_flag = 1; }
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// Merges the chunk partials in chunk order (page-aligned chunk geometry).  One block per (request, KV head, group of
// 32 of its k * rep rows): lane = row, warp w = head-dim columns [16 w, 16 w + 16), so the loads follow the partials'
// [column group][row][4] layout (512 contiguous bytes per warp) and the finished rows go through shared memory to leave
// as whole 256-byte rows.
constexpr int MERGE_ROW_BYTES = DH * 2 + 16;         // padded: the 32 lanes' 16-byte writes spread over the banks
__global__ void __launch_bounds__(256)
attn_tc_merge_kernel(AttnTcArgs a, uint16_t* __restrict__ o) {
  pdl_wait();
  pdl_trigger();
  __shared__ __align__(16) uint8_t tile[32 * MERGE_ROW_BYTES];
  const int groups = (a.R + 31) / 32;
  const int b = blockIdx.x / (a.Hkv * groups), kvh = (blockIdx.x / groups) % a.Hkv, r0 = (blockIdx.x % groups) * 32;
  const Range g = make_range(clamped_ctx(a, b), a.window, a.chunk, 0, a.k);
  if (g.n_chunks == 1) return;                     // finished by the attention kernel itself (uniform for the block)
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int r = r0 + lane;
  const bool row_ok = r < a.R;
  const size_t slab0 = (size_t(b) * a.Hkv + kvh) * a.max_chunks;
  if (row_ok) {
    float m_tot = -INFINITY;
    for (int c = 0; c < g.n_chunks; ++c) m_tot = fmaxf(m_tot, a.ws_ml[((slab0 + c) * a.R + r) * 2]);
    const float ref = (m_tot == -INFINITY) ? 0.f : m_tot;
    float4 acc[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
    for (int c = 0; c < g.n_chunks; ++c) {
      const float* ml = a.ws_ml + ((slab0 + c) * a.R + r) * 2;
      const float wgt = exp2f(ml[0] - ref);
      L += ml[1] * wgt;
      const float* src = a.ws_o + (slab0 + c) * a.R * DH + size_t(r) * 4;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 v = *reinterpret_cast<const float4*>(src + size_t(w * 4 + q) * a.R * 4);
        acc[q].x += v.x * wgt; acc[q].y += v.y * wgt; acc[q].z += v.z * wgt; acc[q].w += v.w * wgt;
      }
    }
    const float inv = 1.f / L;
    uint32_t h[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (a.o_bf16) {
        h[2 * q] = pack_bf16(acc[q].x * inv, acc[q].y * inv);
        h[2 * q + 1] = pack_bf16(acc[q].z * inv, acc[q].w * inv);
      } else {
        const __half2 lo = __halves2half2(f16_sat(acc[q].x * inv, a.status), f16_sat(acc[q].y * inv, a.status));
        const __half2 hi = __halves2half2(f16_sat(acc[q].z * inv, a.status), f16_sat(acc[q].w * inv, a.status));
        h[2 * q] = *reinterpret_cast<const uint32_t*>(&lo);
        h[2 * q + 1] = *reinterpret_cast<const uint32_t*>(&hi);
      }
    }
    uint4* dst = reinterpret_cast<uint4*>(tile + lane * MERGE_ROW_BYTES + w * 32);
    dst[0] = make_uint4(h[0], h[1], h[2], h[3]);
    dst[1] = make_uint4(h[4], h[5], h[6], h[7]);
  }
  __syncthreads();
  // 16 lanes write one 256-byte row: row rr of the group is block position rr / rep, query head kvh * rep + rr % rep
#pragma unroll
  for (int p = 0; p < 2; ++p) {
    const int rl = w * 4 + p * 2 + (lane >> 4);
    const int rr = r0 + rl;
    if (rr < a.R) {
      const int i = rr / a.rep, hq = kvh * a.rep + rr % a.rep;
      const uint4 v = *reinterpret_cast<const uint4*>(tile + rl * MERGE_ROW_BYTES + (lane & 15) * 16);
      *reinterpret_cast<uint4*>(o + ((size_t(b) * a.k + i) * a.Hq + hq) * DH + (lane & 15) * 8) = v;
    }
  }
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
  a.max_ctx = c.max_ctx < c.page_table_stride * 16 ? c.max_ctx : c.page_table_stride * 16;
  a.num_pages = int(c.num_pages < 0x7fffffff ? c.num_pages : 0x7fffffff);
  a.scale_log2 = 1.4426950408889634f / sqrtf(float(c.dh));
  const size_t slabs = size_t(c.B) * c.Hkv * max_chunks;
  a.ws_o = reinterpret_cast<float*>(c.ws);
  a.o_final = reinterpret_cast<uint16_t*>(c.o);
  a.o_bf16 = c.o_bf16 ? 1 : 0;
  a.ws_ml = a.ws_o + slabs * a.R * c.dh;
  CUtensorMap tmK, tmV;
  if (!make_pool_tmap(&tmK, c.k_pool, c.num_pages, c.Hkv, err) || !make_pool_tmap(&tmV, c.v_pool, c.num_pages, c.Hkv, err))
    return cudaErrorInvalidValue;
  const size_t smem = size_t(KV_BYTES) * (1 + NSK + NSV) + sizeof(AttnTcBars);
  static bool attr_done[MAX_DEVICES] = {};
  static int sm_count[MAX_DEVICES] = {};
  {
    const cudaError_t e0 = once_per_device(attr_done, [smem](int dev) {
      if (cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count[dev] < 1)
        sm_count[dev] = 148;
      return cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    });
    if (e0 != cudaSuccess) return e0;
  }
  const int n_sms = sm_count[current_device()];
  // work list (count + items) behind the partials in the workspace
  int* count = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(a.ws_ml + slabs * a.R * 2) + 15) & ~uintptr_t(15));
  int4* items = reinterpret_cast<int4*>(count + 4);
  trk_begin(trk, "attn_plan");
  launch_pdl(attn_tc_plan_kernel, dim3(1), dim3(256), 0, stream, a, count, items);
  trk_end(trk);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  trk_begin(trk, "attn_partial");
  launch_pdl(attn_tc_kernel, dim3(n_sms), dim3(352), smem, stream, tmK, tmV, a, (const int*)count, (const int4*)items);
  trk_end(trk);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  trk_begin(trk, "attn_merge");
  launch_pdl(attn_tc_merge_kernel, dim3(c.B * c.Hkv * ((a.R + 31) / 32)), dim3(256), 0, stream, a, reinterpret_cast<uint16_t*>(c.o));
  trk_end(trk);
  return cudaGetLastError();
}

}  // namespace hspec
