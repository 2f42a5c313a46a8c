// Block-query GQA attention over the target model's paged KV cache, read in place, plus the
// block's own causal keys/values (paper Sec. 3.3.2).  Nothing is ever written to the pools.
//
// Work item = (request b, KV head, context chunk[, row tile]).  The k*Hq/Hkv query rows that share
// one KV head form the M side of the MMAs, so each K/V byte fetched from HBM is used by all of
// them.  K/V rows stream through a cp.async ring of 64-key tiles (16-byte loads, each token row of
// one head is dh*2 contiguous bytes inside its page).  Long contexts are split into chunks; every
// chunk writes an un-normalised partial (row max, row sum, O) and a second kernel merges the
// chunks in index order, so the result does not depend on scheduling.
#include "common.cuh"
#include "kernels.h"

#include <cstdlib>

namespace hspec {

namespace {

constexpr int KT = 64;        // keys per tile
constexpr int NSTAGE = 3;     // cp.async ring depth

struct AttnArgs {
  const __nv_bfloat16 *q, *kb, *vb, *k_pool, *v_pool;
  const int32_t* page_table;
  const int32_t* ctx_lens;
  float* ws_o;       // [B, Hkv, max_chunks, R, DH]
  float* ws_ml;      // [B, Hkv, max_chunks, R, 2]
  void* o;           // [B*k, Hq*DH] fp16 (or bf16 when o_bf16)
  int o_bf16;
  uint32_t* status;
  int page_table_stride;
  int B, k, Hq, Hkv, rep, R, RT, n_row_tiles;
  int chunk, max_chunks, page_size, window;
  int max_ctx;       // host bound on the context lengths: a length outside [0, max_ctx] is clamped and counted
  int num_pages;     // a page id outside [0, num_pages) is read as zeros and counted
  float scale_log2;
};

// A request's context length as both kernels use it: clamped to the bound the host sized the grid and the partials for.
__device__ __forceinline__ int clamped_ctx(const AttnArgs& a, int b) { return min(max(a.ctx_lens[b], 0), a.max_ctx); }

// Visible prefix range of a request: [lo0, ctx).  With a window W row i sees positions
// > ctx + i - W, so the union over rows starts at ctx - W + 1 (row 0).
__device__ __forceinline__ void visible_range(int ctx, int window, int chunk, int& lo0, int& n_chunks) {
  lo0 = (window > 0) ? max(0, ctx - window + 1) : 0;
  const int len = ctx - lo0;
  n_chunks = max(1, (len + chunk - 1) / chunk);
}

template <int DH>
__device__ __forceinline__ uint32_t swz(int row, int col) {   // byte offset of element (row, col), 16-byte chunks XOR-swizzled
  return uint32_t(row * DH * 2 + ((((col >> 3) ^ (row & 7))) << 4) + ((col & 7) << 1));
}

template <int DH>
__global__ void __launch_bounds__(256)
attn_partial_kernel(AttnArgs a) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.z, kvh = blockIdx.y;
  const int c = blockIdx.x / a.n_row_tiles, rt = blockIdx.x % a.n_row_tiles;
  const int ctx = clamped_ctx(a, b);
  if (tid == 0 && blockIdx.x == 0 && kvh == 0 && ctx != a.ctx_lens[b]) atomicAdd(a.status + STATUS_WORD_BAD_INPUT, 1u);
  int lo0, n_chunks;
  visible_range(ctx, a.window, a.chunk, lo0, n_chunks);
  if (c >= n_chunks) return;
  const bool last = (c == n_chunks - 1);
  const int p_begin = lo0 + c * a.chunk;
  const int p_end = min(ctx, p_begin + a.chunk);
  const int n_pre = (p_end > p_begin) ? (p_end - p_begin + KT - 1) / KT : 0;
  const int n_tiles = n_pre + (last ? 1 : 0);

  uint8_t* sQ = smem;
  uint8_t* sK = sQ + a.RT * DH * 2;
  uint8_t* sV = sK + NSTAGE * KT * DH * 2;
  constexpr int CPR = DH / 8;                        // 16-byte chunks per row

  // ---- Q rows of this tile -> shared (zero for padding rows)
  const int row0 = rt * a.RT;
  for (int idx = tid; idx < a.RT * CPR; idx += nthr) {
    const int r = idx / CPR, ch = idx % CPR;
    const int rg = row0 + r;
    const bool ok = rg < a.R;
    const int i = ok ? rg / a.rep : 0, gq = ok ? rg % a.rep : 0;
    const __nv_bfloat16* src = a.q + ((size_t(b) * a.k + i) * a.Hq + kvh * a.rep + gq) * DH + ch * 8;
    cp_async16(smem_u32(sQ) + swz<DH>(r, ch * 8), src, ok);
  }
  cp_async_commit();

  const int32_t* ptab = a.page_table + size_t(b) * a.page_table_stride;
  auto load_tile = [&](int t) {
    const int st = t % NSTAGE;
    const uint32_t dK = smem_u32(sK) + st * KT * DH * 2, dV = smem_u32(sV) + st * KT * DH * 2;
    if (t < n_pre) {
      const int base = p_begin + t * KT;
      for (int idx = tid; idx < KT * CPR; idx += nthr) {
        const int r = idx / CPR, ch = idx % CPR;
        const int p = base + r;
        bool ok = p < p_end;
        size_t off = 0;
        if (ok) {
          const int page = ptab[p / a.page_size];
          if (unsigned(page) >= unsigned(a.num_pages)) {     // never form an address from a bad id: zero row, counted once
            ok = false;
            if (ch == 0 && p % a.page_size == 0) atomicAdd(a.status + STATUS_WORD_BAD_INPUT, 1u);
          } else {
            off = ((size_t(page) * a.page_size + (p % a.page_size)) * a.Hkv + kvh) * DH + ch * 8;
          }
        }
        cp_async16(dK + swz<DH>(r, ch * 8), a.k_pool + off, ok);
        cp_async16(dV + swz<DH>(r, ch * 8), a.v_pool + off, ok);
      }
    } else {                                          // the block's own keys / values
      for (int idx = tid; idx < KT * CPR; idx += nthr) {
        const int r = idx / CPR, ch = idx % CPR;
        const bool ok = r < a.k;
        const size_t off = ok ? ((size_t(b) * a.k + r) * a.Hkv + kvh) * DH + ch * 8 : 0;
        cp_async16(dK + swz<DH>(r, ch * 8), a.kb + off, ok);
        cp_async16(dV + swz<DH>(r, ch * 8), a.vb + off, ok);
      }
    }
  };

#pragma unroll
  for (int t = 0; t < NSTAGE - 1; ++t) {
    if (t < n_tiles) load_tile(t);
    cp_async_commit();
  }

  // rows of this thread inside the warp's 16-row slab
  const int g = lane >> 2, tq = lane & 3;
  const int r_lo = row0 + warp * 16 + g, r_hi = r_lo + 8;          // global row indices (may be >= R: padding)
  const int i_lo = r_lo / a.rep, i_hi = r_hi / a.rep;              // block position of the row
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  float o[DH / 8][4];
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  uint32_t qf[DH / 16][4];
  bool q_loaded = false;

  for (int t = 0; t < n_tiles; ++t) {
    cp_async_wait<NSTAGE - 2>();
    __syncthreads();
    if (t + NSTAGE - 1 < n_tiles) load_tile(t + NSTAGE - 1);
    cp_async_commit();
    if (!q_loaded) {                                   // Q landed with the first group
      q_loaded = true;
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks)
        ldmatrix_x4(qf[ks], smem_u32(sQ) + swz<DH>(warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, ks * 16 + (lane >> 4) * 8));
    }
    const int st = t % NSTAGE;
    const uint32_t bK = smem_u32(sK) + st * KT * DH * 2, bV = smem_u32(sV) + st * KT * DH * 2;

    // ---- S = Q K^T for 64 keys
    float s[KT / 8][4];
#pragma unroll
    for (int n = 0; n < KT / 8; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
#pragma unroll
      for (int n2 = 0; n2 < KT / 16; ++n2) {
        uint32_t kf[4];
        ldmatrix_x4(kf, bK + swz<DH>(n2 * 16 + (lane & 7) + (lane >> 4) * 8, ks * 16 + ((lane >> 3) & 1) * 8));
        mma_bf16_16816(s[2 * n2], qf[ks], kf[0], kf[1]);
        mma_bf16_16816(s[2 * n2 + 1], qf[ks], kf[2], kf[3]);
      }
    }

    // ---- scale, mask by selection, online softmax (base 2)
    const bool is_block = (t >= n_pre);
    const int key0 = is_block ? 0 : p_begin + t * KT;           // position (prefix) or block index of key 0
    // prefix tile needs masking only at a ragged end or inside the window's leading edge
    const bool need_mask = is_block || (key0 + KT > p_end) || (a.window > 0 && key0 < lo0 + a.k);
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int n = 0; n < KT / 8; ++n) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = s[n][e] * a.scale_log2;
        if (need_mask) {
          const int kk = n * 8 + tq * 2 + (e & 1);
          const int i = (e < 2) ? i_lo : i_hi;
          bool vis;
          if (is_block) vis = (kk <= i) && (kk < a.k) && (a.window <= 0 || i - kk < a.window);
          else vis = (key0 + kk < p_end) && (a.window <= 0 || (ctx + i) - (key0 + kk) < a.window);
          if (!vis) v = -INFINITY;
        }
        s[n][e] = v;
      }
      mx_lo = fmaxf(mx_lo, fmaxf(s[n][0], s[n][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(s[n][2], s[n][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float ref_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, ref_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
    const float al_lo = exp2f(m_lo - ref_lo), al_hi = exp2f(m_hi - ref_hi);   // m = -inf -> 0
    m_lo = mn_lo; m_hi = mn_hi;
    float sum_lo = 0.f, sum_hi = 0.f;
    uint32_t pf[KT / 16][4];
#pragma unroll
    for (int n = 0; n < KT / 8; ++n) {
      const float p0 = exp2f(s[n][0] - ref_lo), p1 = exp2f(s[n][1] - ref_lo);
      const float p2 = exp2f(s[n][2] - ref_hi), p3 = exp2f(s[n][3] - ref_hi);
      sum_lo += p0 + p1; sum_hi += p2 + p3;
      pf[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    l_lo = l_lo * al_lo + sum_lo; l_hi = l_hi * al_hi + sum_hi;
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) { o[n][0] *= al_lo; o[n][1] *= al_lo; o[n][2] *= al_hi; o[n][3] *= al_hi; }

    // ---- O += P V
#pragma unroll
    for (int kt = 0; kt < KT / 16; ++kt) {
#pragma unroll
      for (int d2 = 0; d2 < DH / 16; ++d2) {
        uint32_t vf[4];
        ldmatrix_x4_trans(vf, bV + swz<DH>(kt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, d2 * 16 + (lane >> 4) * 8));
        mma_bf16_16816(o[2 * d2], pf[kt], vf[0], vf[1]);
        mma_bf16_16816(o[2 * d2 + 1], pf[kt], vf[2], vf[3]);
      }
    }
  }
  cp_async_wait<0>();

  // ---- partial (m, l, O) of this chunk
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  const size_t slab = (size_t(b) * a.Hkv + kvh) * a.max_chunks + c;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int r = half ? r_hi : r_lo;
    if (r >= a.R) continue;
    float* dst = a.ws_o + (slab * a.R + r) * DH;
#pragma unroll
    for (int n = 0; n < DH / 8; ++n)
      *reinterpret_cast<float2*>(dst + n * 8 + tq * 2) = make_float2(o[n][half * 2], o[n][half * 2 + 1]);
    if (tq == 0) {
      float* ml = a.ws_ml + (slab * a.R + r) * 2;
      ml[0] = half ? m_hi : m_lo;
      ml[1] = half ? l_hi : l_lo;
    }
  }
}

// One block per (row of the block, query head): merge the chunk partials in chunk order.
template <int DH>
__global__ void attn_merge_kernel(AttnArgs a) {
  pdl_wait();
  pdl_trigger();
  const int m = blockIdx.x;             // b * k + i
  const int hq = blockIdx.y;
  const int b = m / a.k, i = m % a.k;
  const int kvh = hq / a.rep, r = i * a.rep + hq % a.rep;
  const int ctx = clamped_ctx(a, b);
  int lo0, n_chunks;
  visible_range(ctx, a.window, a.chunk, lo0, n_chunks);
  const size_t slab0 = (size_t(b) * a.Hkv + kvh) * a.max_chunks;
  float m_tot = -INFINITY;
  for (int c = 0; c < n_chunks; ++c) m_tot = fmaxf(m_tot, a.ws_ml[((slab0 + c) * a.R + r) * 2]);
  const float ref = (m_tot == -INFINITY) ? 0.f : m_tot;
  for (int d = threadIdx.x; d < DH; d += blockDim.x) {
    float acc = 0.f, L = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
      const float* ml = a.ws_ml + ((slab0 + c) * a.R + r) * 2;
      const float w = exp2f(ml[0] - ref);
      L += ml[1] * w;
      acc += a.ws_o[((slab0 + c) * a.R + r) * DH + d] * w;
    }
    store_act16(a.o, (size_t(m) * a.Hq + hq) * DH + d, acc / L, a.o_bf16 != 0, a.status);
  }
}

__global__ void gather_kv_kernel(const uint4* __restrict__ pool, const int32_t* __restrict__ row, int ctx_len,
                                 int page_size, int Hkv, int dh, uint4* __restrict__ dst) {
  const int vec_per_tok = Hkv * dh * 2 / 16;
  const long long total = (long long)ctx_len * vec_per_tok;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int p = int(idx / vec_per_tok), v = int(idx % vec_per_tok);
    const int page = row[p / page_size];
    dst[idx] = pool[(size_t(page) * page_size + p % page_size) * vec_per_tok + v];
  }
}

int rows_per_cta(int R) { int rt = ((R + 15) / 16) * 16; return rt > 128 ? 128 : rt; }

}  // namespace

int attn_pick_chunk(int B, int Hkv, int max_ctx, int window, int num_sms) {
  // with a window the visible range starts on a page boundary, up to 15 tokens before the window itself: size the
  // chunks for window + 15 tokens, or a request's last few tokens become a chunk (and a merge) of their own
  int lmax = (window > 0 && window + 15 < max_ctx) ? window + 15 : max_ctx;
  if (lmax < 1) lmax = 1;
  int nsplit = (2 * num_sms + B * Hkv - 1) / (B * Hkv);
  if (nsplit < 1) nsplit = 1;
  if (nsplit > 32) nsplit = 32;
  int chunk = (lmax + nsplit - 1) / nsplit;
  chunk = ((chunk + 127) / 128) * 128;
  if (chunk < 256) chunk = 256;
  // long chunks mean fewer partials to write and merge and fewer item boundaries; past 8192 tokens the work list gets
  // too uneven.  Measured at 8, 16, 32 and 64 requests x 8 KV heads with contexts up to 16k and 32k: a cap of 8192 is
  // 3-11 % faster than 4096 wherever it binds and never slower; 16384 loses 5-9 %.
  static const int cap_env = [] { const char* e = getenv("HSPEC_ATTN_CHUNK_CAP"); return e ? atoi(e) : 0; }();   // measurements only
  const int cap = cap_env >= 256 ? cap_env : 8192;
  if (chunk > cap) chunk = cap;
  return chunk;
}

static int max_chunks_of(int max_ctx, int window, int chunk) {
  // with a window the visible range may start up to 15 tokens earlier (page-aligned chunk grid of the tcgen05 path)
  int lmax = (window > 0 && window + 15 < max_ctx) ? window + 15 : max_ctx;
  int n = (lmax + chunk - 1) / chunk;
  return n < 1 ? 1 : n;
}

size_t attn_workspace_bytes(int B, int k, int Hq, int Hkv, int dh, int max_ctx, int window, int chunk_tokens) {
  const int R = k * (Hq / Hkv);
  const size_t slabs = size_t(B) * Hkv * max_chunks_of(max_ctx, window, chunk_tokens);
  const size_t row_tiles = (size_t(R) + 127) / 128;
  return slabs * R * (dh + 2) * sizeof(float) + 256 + slabs * row_tiles * 16 + 64;   // partials + the tcgen05 path's work list
}

cudaError_t attention_launch(const AttnCall& c, cudaStream_t stream, Tracker* trk, std::string* err) {
  if (c.dh != 64 && c.dh != 128) { if (err) *err = "attention head dim must be 64 or 128"; return cudaErrorInvalidValue; }
  if (c.Hq % c.Hkv) { if (err) *err = "Hq must be a multiple of Hkv"; return cudaErrorInvalidValue; }
  AttnArgs a{};
  a.q = (const __nv_bfloat16*)c.q; a.kb = (const __nv_bfloat16*)c.kb; a.vb = (const __nv_bfloat16*)c.vb;
  a.k_pool = (const __nv_bfloat16*)c.k_pool; a.v_pool = (const __nv_bfloat16*)c.v_pool;
  a.page_table = c.page_table; a.ctx_lens = c.ctx_lens; a.o = c.o; a.o_bf16 = c.o_bf16 ? 1 : 0;
  a.page_table_stride = c.page_table_stride;
  a.B = c.B; a.k = c.k; a.Hq = c.Hq; a.Hkv = c.Hkv; a.rep = c.Hq / c.Hkv;
  a.R = c.k * a.rep; a.RT = rows_per_cta(a.R); a.n_row_tiles = (a.R + a.RT - 1) / a.RT;
  a.chunk = c.chunk_tokens; a.max_chunks = max_chunks_of(c.max_ctx, c.window, c.chunk_tokens);
  a.page_size = c.page_size; a.window = c.window;
  a.status = c.status;
  a.max_ctx = c.max_ctx < c.page_table_stride * c.page_size ? c.max_ctx : c.page_table_stride * c.page_size;
  a.num_pages = int(c.num_pages < 0x7fffffff ? c.num_pages : 0x7fffffff);
  a.scale_log2 = 1.4426950408889634f / sqrtf(float(c.dh));
  if (c.k > KT) { if (err) *err = "block longer than one key tile"; return cudaErrorInvalidValue; }
  const size_t need = attn_workspace_bytes(c.B, c.k, c.Hq, c.Hkv, c.dh, c.max_ctx, c.window, c.chunk_tokens);
  if (c.ws == nullptr || c.ws_bytes < need) { if (err) *err = "attention workspace too small"; return cudaErrorInvalidValue; }
  {
    static const bool legacy = [] { const char* e = getenv("HSPEC_ATTN_MMA_SYNC"); return e && e[0] == '1'; }();
    if (!legacy && attention_tc_supported(c)) return attention_tc_launch(c, a.max_chunks, stream, trk, err);
  }
  const size_t slabs = size_t(c.B) * c.Hkv * a.max_chunks;
  a.ws_o = reinterpret_cast<float*>(c.ws);
  a.ws_ml = a.ws_o + slabs * a.R * c.dh;
  const size_t smem = size_t(a.RT) * c.dh * 2 + size_t(2) * NSTAGE * KT * c.dh * 2;
  dim3 grid(a.max_chunks * a.n_row_tiles, c.Hkv, c.B);
  const int threads = a.RT * 2;
  static bool attr_done[MAX_DEVICES] = {};
  cudaError_t e = once_per_device(attr_done, [](int) {
    cudaError_t e2 = cudaFuncSetAttribute(attn_partial_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e2 != cudaSuccess) return e2;
    return cudaFuncSetAttribute(attn_partial_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  });
  if (e != cudaSuccess) return e;
  trk_begin(trk, "attn_partial");
  if (c.dh == 128) attn_partial_kernel<128><<<grid, threads, smem, stream>>>(a);
  else attn_partial_kernel<64><<<grid, threads, smem, stream>>>(a);
  trk_end(trk);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 mgrid(c.B * c.k, c.Hq);
  trk_begin(trk, "attn_merge");
  if (c.dh == 128) attn_merge_kernel<128><<<mgrid, 128, 0, stream>>>(a);
  else attn_merge_kernel<64><<<mgrid, 64, 0, stream>>>(a);
  trk_end(trk);
  return cudaGetLastError();
}

cudaError_t gather_kv_launch(const void* pool, const int32_t* row, int ctx_len, int page_size, int Hkv, int dh,
                             void* dst, cudaStream_t stream) {
  if (ctx_len <= 0) return cudaSuccess;
  const long long total = (long long)ctx_len * Hkv * dh * 2 / 16;
  int blocks = int((total + 255) / 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  gather_kv_kernel<<<blocks, 256, 0, stream>>>((const uint4*)pool, row, ctx_len, page_size, Hkv, dh, (uint4*)dst);
  return cudaGetLastError();
}

}  // namespace hspec
