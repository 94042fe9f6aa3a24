// Inline-PTX building blocks shared by the tensor-core kernels: mbarriers with bounded waits, TMA
// tile loads, tcgen05 MMA / commit / tensor-memory loads, and the descriptors they take.
#pragma once

#include <cuda.h>
#include <stdint.h>

namespace camera {

constexpr unsigned long long DEFAULT_WAIT_LIMIT_NS = 4000000000ull;   // every mbarrier wait gives up after this long
                                                                      // unless the host set another limit
constexpr int UMMA_BK = 64;                                   // bf16 elements per k-block = one 128-byte swizzle row

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
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
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// The CTA's wait state in shared memory: the abort flag (an int, 8-byte aligned) and, WAIT_LIMIT_SLOT ints behind
// it, the limit of every wait in nanoseconds.  One thread sets both up before the first wait.
constexpr int WAIT_LIMIT_SLOT = 4;
__device__ __forceinline__ void wait_state_init(volatile int* abort_flag, unsigned long long limit_ns) {
  *abort_flag = 0;
  *reinterpret_cast<volatile unsigned long long*>(abort_flag + WAIT_LIMIT_SLOT) = limit_ns;
}
__device__ __forceinline__ unsigned long long wait_limit_ns(volatile int* abort_flag) {
  return *reinterpret_cast<volatile unsigned long long*>(abort_flag + WAIT_LIMIT_SLOT);
}

// Bounded wait.  Returns false when the limit ran out or another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  unsigned spins = 0;
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > wait_limit_ns(abort_flag)) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tmap), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

__device__ __forceinline__ void tensormap_acquire(const void* tmap) {
  asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(tmap) : "memory");
}

// Shared-memory matrix descriptor for a K-major bf16 tile whose rows are 128 bytes, stored as
// 8-row x 128-byte atoms with the 128-byte swizzle (what TMA writes with SWIZZLE_128B).
__device__ __forceinline__ unsigned long long make_smem_desc(uint32_t addr) {
  unsigned long long d = 0;
  d |= (unsigned long long)((addr & 0x3ffffu) >> 4);        // start address
  d |= (unsigned long long)1 << 16;                         // leading byte offset (unused for this layout)
  d |= (unsigned long long)(1024 >> 4) << 32;               // stride between 8-row groups
  d |= (unsigned long long)1 << 46;                         // descriptor version
  d |= (unsigned long long)2 << 61;                         // 128-byte swizzle
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t make_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, unsigned long long a, unsigned long long b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16 consecutive accumulator columns of this thread's TMEM lane.  The registers hold the values only
// after tmem_ld_wait, which names them so that no use can be scheduled ahead of it.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait(uint32_t* a) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                 "+r"(a[8]), "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait(uint32_t* a, uint32_t* b) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                 "+r"(a[8]), "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15]),
                 "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]),
                 "+r"(b[8]), "+r"(b[9]), "+r"(b[10]), "+r"(b[11]), "+r"(b[12]), "+r"(b[13]), "+r"(b[14]), "+r"(b[15])
               :
               : "memory");
}

// 32 bytes in one store (the address is 32-byte aligned).
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t* v) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]),
               "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}

// Epilogue of the scoring orientation (a thread = a micro-expert, 16 tokens per call):
// lambda = a_t * SiLU(g) * u; folds lambda^2 and |lambda| into s and m.
// WRITE_H (layer forward): lambda also goes, as bf16, to h[token][micro-expert].  The 16 x 32 values of the warp are
// turned in shared memory (stg: 1 KB of the warp's own, 16-byte aligned) so that a lane stores 16 bytes = 8 consecutive
// micro-experts of one token: two vector stores per lane instead of sixteen 2-byte ones.  hwarp points at
// h[first of the 16 tokens][first of the warp's 32 micro-experts]; tokens from n_store on are not stored.
constexpr int FOLD_STG_BYTES = 16 * 32 * 2;
template <bool WRITE_H>
__device__ __forceinline__ void fold16(const uint32_t* vg, const uint32_t* vu, const float* wb, float& s, float& m,
                                       __nv_bfloat16* hwarp, int h_ld, int n_store, uint8_t* stg, int lane) {
  float a[16];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 w4 = *reinterpret_cast<const float4*>(wb + 4 * q);
    a[4 * q] = w4.x; a[4 * q + 1] = w4.y; a[4 * q + 2] = w4.z; a[4 * q + 3] = w4.w;
  }
  __nv_bfloat16* const col = reinterpret_cast<__nv_bfloat16*>(stg) + lane;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float g = __uint_as_float(vg[j]), up = __uint_as_float(vu[j]);
    const float sig = __fdividef(1.f, 1.f + __expf(-g));
    const float lam = (a[j] * up) * (g * sig);
    s = fmaf(lam, lam, s);
    m = fmaxf(m, fabsf(lam));
    if (WRITE_H) col[j * 32] = __float2bfloat16_rn(lam);
  }
  if (WRITE_H) {
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int q = lane + 32 * i, row = q >> 2, part = q & 3;      // 64 pieces of 16 bytes: 4 per token row
      const uint4 v = *reinterpret_cast<const uint4*>(stg + 16 * q);
      if (row < n_store) *reinterpret_cast<uint4*>(hwarp + (size_t)row * h_ld + 8 * part) = v;
    }
    __syncwarp();
  }
}

}  // namespace camera
