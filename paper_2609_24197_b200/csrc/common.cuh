// Shared device helpers for the H-Spec draft-step kernels (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hspec {

// The device status block is 64 words.  Word 0 holds the code of a bounded wait that gave up (codes below); the
// other words are event counters that kernels bump with atomicAdd and the host reads back with the block.
enum : uint32_t {
  STATUS_OK = 0,
  STATUS_TIMEOUT_PRODUCER = 0x101,
  STATUS_TIMEOUT_MMA = 0x102,
  STATUS_TIMEOUT_EPILOGUE = 0x103,
  STATUS_BAD_SMEM_BASE = 0x104,
  STATUS_TIMEOUT_SELFTEST = 0x1ff,
};
enum : int {
  STATUS_WORD_CODE = 0,        // first give-up code (0 = none)
  STATUS_WORD_RESCALES = 1,    // attention: (warp, tile) events in which a row's reference maximum moved and its
                               // accumulator row was rescaled in tensor memory
  STATUS_WORD_F16_RANGE = 2,   // finite fp32 values that left the fp16 range in a store and were clamped to +-65504
  STATUS_WORD_BAD_INPUT = 3,   // context lengths outside [0, max_ctx] and page ids outside [0, num_pages) that a kernel
                               // met: the length was clamped, the page's rows were read as zeros
  STATUS_WORDS = 64,
};

// fp32 -> fp16 with saturation: a finite value beyond +-65504 is clamped (instead of becoming inf and, one GEMM later,
// NaN) and counted in the status block; NaN and inf pass through unchanged.
__device__ __forceinline__ __half f16_sat(float v, uint32_t* status) {
  if (fabsf(v) > 65504.f && fabsf(v) < INFINITY) {
    if (status) atomicAdd(status + STATUS_WORD_F16_RANGE, 1u);
    v = copysignf(65504.f, v);
  }
  return __float2half_rn(v);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
  return __uint_as_float(static_cast<uint32_t>(b) << 16);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// (fast exponential and fast division: ~2 ulp each, far inside every tolerance that follows an fp16 or bf16 rounding)
__device__ __forceinline__ float silu_f(float v) { return __fdividef(v, 1.0f + __expf(-v)); }

// Stores v into a 16-bit activation buffer: fp16 with saturation (counted), or bf16 (fp32's range: nothing to clamp).
__device__ __forceinline__ void store_act16(void* base, size_t idx, float v, bool bf16, uint32_t* status) {
  if (bf16) reinterpret_cast<__nv_bfloat16*>(base)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<__half*>(base)[idx] = f16_sat(v, status);
}

// ------------------------------------------------------------------ programmatic dependent launch
// A kernel launched with launch_pdl() may start while the kernel before it on the stream is still running: its CTAs
// run their set-up and then block in pdl_wait() until that kernel has finished and its writes are visible.  Nothing
// produced by an earlier kernel may be read, and nothing may be written to global memory, before pdl_wait().
// pdl_trigger() lets the NEXT kernel on the stream start launching once every CTA of this one has called it.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking look at a barrier phase: true if the phase with this parity has completed.  (try_wait may suspend the
// thread for a while when it has not; this never does.)
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: polls the barrier and gives up after about two seconds of wall time (checked every
// 1024 polls).  Returns false on give-up; the caller records a status code and unwinds.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint64_t limit_ns = 2000000000ull) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u) {
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) return false;
    }
  }
}

// The same bounded wait as a pure spin on test_wait: try_wait may put the thread to sleep for a while when the phase is
// not complete yet, which is what a thread on a latency-critical hand-off (a TMA producer waiting for a free stage, the
// MMA issuer waiting for a full one) cannot afford.
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity, uint64_t limit_ns = 2000000000ull) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_test(bar, parity)) return true;
    if ((i & 4095u) == 4095u) {
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) return false;
    }
  }
}

// 16 rows x 32 lanes -> one (max, lowest index on ties) per row with 32 shuffles instead of 160: every round a lane
// hands half of its rows to its partner and merges the partner's copy of the half it keeps.  After the rounds with
// offsets 16, 8, 4, 2 and a last pairwise round, v[0] / idx[0] of every EVEN lane hold the result of row `row`.
__device__ __forceinline__ void warp_argmax16(float (&v)[16], int (&idx)[16], int lane, int& row) {
#define HSPEC_ARGMAX_ROUND(OFF, HALF)                                                  \
  {                                                                                    \
    const bool up = (lane & OFF) != 0;                                                 \
    _Pragma("unroll") for (int t = 0; t < HALF; ++t) {                                 \
      const float sv = up ? v[t] : v[t + HALF];                                        \
      const int si = up ? idx[t] : idx[t + HALF];                                      \
      const float ov = __shfl_xor_sync(0xffffffffu, sv, OFF);                          \
      const int oi = __shfl_xor_sync(0xffffffffu, si, OFF);                            \
      float kv = up ? v[t + HALF] : v[t];                                              \
      int ki = up ? idx[t + HALF] : idx[t];                                            \
      if (ov > kv || (ov == kv && oi < ki)) { kv = ov; ki = oi; }                      \
      v[t] = kv; idx[t] = ki;                                                          \
    }                                                                                  \
  }
  HSPEC_ARGMAX_ROUND(16, 8)
  HSPEC_ARGMAX_ROUND(8, 4)
  HSPEC_ARGMAX_ROUND(4, 2)
  HSPEC_ARGMAX_ROUND(2, 1)
#undef HSPEC_ARGMAX_ROUND
  const float ov = __shfl_xor_sync(0xffffffffu, v[0], 1);
  const int oi = __shfl_xor_sync(0xffffffffu, idx[0], 1);
  if (ov > v[0] || (ov == v[0] && oi < idx[0])) { v[0] = ov; idx[0] = oi; }
  row = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
}

// ------------------------------------------------------------------ TMA (no multicast anywhere)
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, int c0, int c1, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_normal() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}

// ------------------------------------------------------------------ tcgen05 / TMEM
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], bf16 inputs, fp32 accumulate, issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the mbarrier once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread t of the warp gets lane (base_lane + t).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major operand tile in shared memory, 128-byte swizzle: rows of 64 bf16 (128 B), groups of 8 rows
// 1024 B apart.  Start address, LBO (ignored for swizzled K-major, encoded 1), SBO = 1024 B,
// descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t umma_desc_kmajor_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// Instruction descriptor: fp32 accumulator, A and B both fp16 or both bf16 (the hardware rejects a mixed
// pair as an illegal instruction), both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc_m128(uint32_t n, bool f16) {
  const uint32_t fmt = f16 ? 0u : 1u;
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// SwiGLU epilogue for 16 accumulator columns (activation rows m0 + c0 .. +15).  Weight rows are interleaved in blocks
// of 16: lanes 0..15 of a warp hold the gate pre-activation of 16 features, lanes 16..31 the up projection of the same
// features.  Columns are handled in pairs: the lower half-warp finishes the even column, the upper half the odd one,
// so all 32 lanes compute and store.  `f` is the feature index of this lane (same for lane and lane ^ 16).
__device__ __forceinline__ void swiglu_store16(const uint32_t (&r)[16], void* out, bool bf16, long long ldo, int m_first, int M, int f,
                                               bool f_ok, int lane, uint32_t* status) {
  const bool upper = lane >= 16;
#pragma unroll
  for (int j = 0; j < 16; j += 2) {
    const float mine_even = __uint_as_float(r[j]), mine_odd = __uint_as_float(r[j + 1]);
    const float send = upper ? mine_even : mine_odd;           // what the partner needs from me
    const float recv = __shfl_xor_sync(0xffffffffu, send, 16);
    const float gate = upper ? recv : mine_even;               // upper half: partner's gate of the odd column
    const float up = upper ? mine_odd : recv;                  // lower half: partner's up of the even column
    const int m = m_first + j + (upper ? 1 : 0);
    if (f_ok && m < M) store_act16(out, size_t(m) * ldo + f, silu_f(gate) * up, bf16, status);
  }
}

// ------------------------------------------------------------------ warp-level mma (attention)
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// one 32-byte read-only load (sm_100: 256-bit global loads); p must be 32-byte aligned
__device__ __forceinline__ void ldg_nc_32B(const void* p, uint4& lo, uint4& hi) {
  asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w)
               : "l"(p));
}
// D += A B with tf32 operands (fp32's exponent range, 10 explicit mantissa bits), fp32 accumulate
__device__ __forceinline__ void mma_tf32_1688(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// v = hi + lo with both parts representable in tf32: three products hi*hi + hi*lo + lo*hi carry ~21 bits
__device__ __forceinline__ void split_tf32(float v, uint32_t& hi, uint32_t& lo) {
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(v));
  const float rest = v - __uint_as_float(hi);
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(lo) : "f"(rest));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  int sz = valid ? 16 : 0;   // src-size 0: the 16 bytes are zero-filled, nothing is read
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

}  // namespace hspec
