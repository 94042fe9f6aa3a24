// Tensor-core scoring kernel for bf16 layers (Algorithm 1 lines 6-8):
//   Lambda = A[:,e] * SiLU(W_gate X) * (W_up X) is formed tile by tile in tensor memory and reduced
//   to per-micro-expert sum(Lambda^2) and max|Lambda| in the epilogue; it never reaches HBM.
//
// One persistent CTA per SM, 6 warps:
//   warps 0-3  epilogue: tcgen05.ld both accumulators, SiLU * up * router weight, running sum / max
//   warp  4    producer: TMA loads of the two weight tiles (A operands) and the token tile (B operand)
//   warp  5    tensor-memory allocation and the single thread that issues tcgen05.mma
//
// Operand orientation: the MMA's M dimension (128 TMEM lanes) holds 128 micro-experts, its N
// dimension (up to 256 columns) holds tokens.  Two accumulators share every token tile: columns
// 0-255 take W_gate x, columns 256-511 take W_up x of the same 128 micro-experts, so one pass over
// K pulls 64 KB from L2 for 8.4 Mflop.  Every epilogue thread owns one micro-expert for all tokens of
// the tile: gate and up of a (micro-expert, token) pair arrive in the same thread, and the reduction
// over tokens runs down its own registers.
//
// Every wait on an mbarrier is bounded: when a wait runs out the CTA records
// CAMERA_ERR_DEVICE_TIMEOUT in the status word, lets its copies land, frees its tensor memory and
// returns.
#include <cuda.h>
#include <string.h>

#include "common.cuh"

namespace camera {

namespace {

constexpr int U_THREADS = 192;
constexpr int U_STAGES = 3;
constexpr int U_BK = 64;                         // bf16 elements per k-block = one 128-byte swizzle row
constexpr int U_A_BYTES = CH_TILE * 128;         // 128 weight rows x 128 B (one of gate / up)
constexpr int U_B_BYTES = UMMA_TOK * 128;        // 256 token rows x 128 B
constexpr int U_STAGE_BYTES = 2 * U_A_BYTES + U_B_BYTES;
constexpr int U_TMEM_COLS = 512;
constexpr int U_WBUF_BYTES = 4 * UMMA_TOK * 4;   // router weights of a token tile, one copy per epilogue warp
constexpr int U_SMEM_BYTES = U_STAGES * U_STAGE_BYTES + U_WBUF_BYTES + 256 + 1024;
constexpr unsigned long long U_WAIT_LIMIT_NS = 4000000000ull;
static_assert(CH_TILE == 128, "one micro-expert per TMEM lane");

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

// Bounded wait.  Returns false when the limit ran out or another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  unsigned spins = 0;
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > U_WAIT_LIMIT_NS) {
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
__device__ __forceinline__ void tmem_ld_wait(uint32_t* a, uint32_t* b) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                 "+r"(a[8]), "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15]),
                 "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]),
                 "+r"(b[8]), "+r"(b[9]), "+r"(b[10]), "+r"(b[11]), "+r"(b[12]), "+r"(b[13]), "+r"(b[14]), "+r"(b[15])
               :
               : "memory");
}

// lambda = a_t * SiLU(g) * u for 16 tokens of this thread's micro-expert; folds lambda^2 and |lambda|.
__device__ __forceinline__ void fold16(const uint32_t* vg, const uint32_t* vu, const float* wb, float& s, float& m) {
  float a[16];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 w4 = *reinterpret_cast<const float4*>(wb + 4 * q);
    a[4 * q] = w4.x; a[4 * q + 1] = w4.y; a[4 * q + 2] = w4.z; a[4 * q + 3] = w4.w;
  }
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float g = __uint_as_float(vg[j]), up = __uint_as_float(vu[j]);
    const float sig = __fdividef(1.f, 1.f + __expf(-g));
    const float lam = (a[j] * up) * (g * sig);
    s = fmaf(lam, lam, s);
    m = fmaxf(m, fabsf(lam));
  }
}

__global__ void __launch_bounds__(U_THREADS, 1) k_score_umma(const ScoreCtx c) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
  // [stages: A_gate | A_up | B] [wbuf 4 warps x 256 floats] [barriers] [tmem slot] [abort flag]
  float* const wbuf = reinterpret_cast<float*>(base_ptr + U_STAGES * U_STAGE_BYTES);
  const uint32_t bars = base + U_STAGES * U_STAGE_BYTES + U_WBUF_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (U_STAGES + s); };
  const uint32_t tfull_bar = bars + 8u * (2 * U_STAGES);
  const uint32_t tempty_bar = bars + 8u * (2 * U_STAGES + 1);
  uint8_t* const tail = base_ptr + U_STAGES * U_STAGE_BYTES + U_WBUF_BYTES + 8 * (2 * U_STAGES + 2);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(tail + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_units = c.totals->total_units;
  const int n_kb = c.d_model / U_BK;

  if (tid == 0) {
    for (int s = 0; s < U_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tfull_bar, 1);
    mbar_init(tempty_bar, 128);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(U_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const char* maps = static_cast<const char*>(c.tensor_maps);
      for (int unit = blockIdx.x; ok && unit < total_units; unit += gridDim.x) {
        const UnitInfo u = decode_unit(c, unit);
        const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
        const void* map_g = maps + (size_t)128 * (2 * u.e);
        const void* map_u = maps + (size_t)128 * (2 * u.e + 1);
        const void* map_x = maps + (size_t)128 * (2 * c.n_experts + (u.shared_idx < 0 ? 0 : 1));
        tensormap_acquire(map_g);
        tensormap_acquire(map_u);
        tensormap_acquire(map_x);
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int row = u.row0 + tt * UMMA_TOK;
          for (int kb = 0; kb < n_kb; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = base + stage * U_STAGE_BYTES;
            mbar_expect_tx(full_bar(stage), U_STAGE_BYTES);
            // weight rows past d_ff and token rows past the tensor are filled with zeros
            tma_load_2d(a_dst, map_g, full_bar(stage), kb * U_BK, u.ch0);
            tma_load_2d(a_dst + U_A_BYTES, map_u, full_bar(stage), kb * U_BK, u.ch0);
            tma_load_2d(a_dst + 2 * U_A_BYTES, map_x, full_bar(stage), kb * U_BK, row);
            if (++stage == U_STAGES) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok) {
        // let the copies already issued land before the CTA's shared memory is given up
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0, tile_phase = 0;
      bool ok = true;
      for (int unit = blockIdx.x; ok && unit < total_units; unit += gridDim.x) {
        const UnitInfo u = decode_unit(c, unit);
        const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int nv = (min(UMMA_TOK, u.rows - tt * UMMA_TOK) + 15) & ~15;
          const uint32_t idesc = make_idesc(nv);
          // both accumulators are free again once the epilogue has read the previous tile out
          if (!mbar_wait(tempty_bar, tile_phase ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          for (int kb = 0; kb < n_kb; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = base + stage * U_STAGE_BYTES;
            const unsigned long long g_desc = make_smem_desc(a_addr);
            const unsigned long long u_desc = make_smem_desc(a_addr + U_A_BYTES);
            const unsigned long long b_desc = make_smem_desc(a_addr + 2 * U_A_BYTES);
#pragma unroll
            for (int k = 0; k < U_BK / 16; ++k) {   // 16 bf16 = 32 bytes per MMA along K: +2 in 16-byte units
              const uint32_t acc = (uint32_t)((kb | k) != 0);
              umma_bf16(tmem_base, g_desc + 2 * k, b_desc + 2 * k, idesc, acc);
              umma_bf16(tmem_base + UMMA_TOK, u_desc + 2 * k, b_desc + 2 * k, idesc, acc);
            }
            umma_commit(empty_bar(stage));
            if (++stage == U_STAGES) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          umma_commit(tfull_bar);
          tile_phase ^= 1u;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3)
    uint32_t tile_phase = 0;
    bool ok = true;
    float* const wb = wbuf + warp * UMMA_TOK;
    const uint32_t t_gate = tmem_base + ((uint32_t)(warp * 32) << 16);
    const uint32_t t_up = t_gate + UMMA_TOK;
    for (int unit = blockIdx.x; ok && unit < total_units; unit += gridDim.x) {
      const UnitInfo u = decode_unit(c, unit);
      const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
      const float* wsrc = u.shared_idx < 0 ? c.perm_w + u.row0 : c.shared_w + (size_t)u.shared_idx * c.n_tokens + u.row0;
      float s = 0.f, m = 0.f;
      for (int tt = 0; ok && tt < n_tiles; ++tt) {
        const int valid = min(UMMA_TOK, u.rows - tt * UMMA_TOK);
        const int nv = (valid + 15) & ~15;
        // each warp stages the tile's router weights for itself (while the MMAs of the tile run), so
        // the four warps never wait on one another and a wait that runs out can be left warp by warp
        __syncwarp();
        for (int i = lane; i < UMMA_TOK; i += 32) wb[i] = i < valid ? wsrc[tt * UMMA_TOK + i] : 0.f;
        __syncwarp();
        ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar, tile_phase, abort_flag));
        if (!ok) break;
        tc_fence_after();
        // two register sets alternate: the loads of the next 16 columns fly while these are folded
        uint32_t g0[16], u0[16], g1[16], u1[16];
        tmem_ld16(t_gate, g0);
        tmem_ld16(t_up, u0);
        for (int c0 = 0; c0 < nv; c0 += 32) {
          tmem_ld_wait(g0, u0);
          if (c0 + 16 < nv) { tmem_ld16(t_gate + c0 + 16, g1); tmem_ld16(t_up + c0 + 16, u1); }
          fold16(g0, u0, wb + c0, s, m);
          if (c0 + 16 < nv) {
            tmem_ld_wait(g1, u1);
            if (c0 + 32 < nv) { tmem_ld16(t_gate + c0 + 32, g0); tmem_ld16(t_up + c0 + 32, u0); }
            fold16(g1, u1, wb + c0 + 16, s, m);
          }
        }
        tc_fence_before();
        mbar_arrive(tempty_bar);
        tile_phase ^= 1u;
      }
      const int ch = u.ch0 + warp * 32 + lane;
      if (ok && ch < u.f) {
        const size_t slot = (size_t)u.part_slot + warp * 32 + lane;
        c.part_sum[slot] = s;
        c.part_max[slot] = m;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag && tid == 0) atomicExch(&c.totals->status, (int)CAMERA_ERR_DEVICE_TIMEOUT);
  if (warp == 5) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(U_TMEM_COLS) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 row-major [rows, d] matrix, box = 64 columns (128 bytes) x box_rows rows, 128-byte swizzle.
bool encode_2d(EncodeTiledFn fn, void* out, const void* ptr, uint64_t rows, uint64_t d, uint32_t box_rows) {
  CUtensorMap m;
  const cuuint64_t dims[2] = {d, rows};
  const cuuint64_t strides[1] = {d * 2};
  const cuuint32_t box[2] = {(cuuint32_t)U_BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  memcpy(out, &m, sizeof(m));
  return true;
}

}  // namespace

bool umma_shape_ok(const camera_layer_t* L) {
  if (L->dtype != CAMERA_BF16 || L->d_model % U_BK != 0) return false;
  for (int e = 0; e < L->n_routed + L->n_shared; ++e) {
    if ((reinterpret_cast<uintptr_t>(L->w_gate[e]) & 15) || (reinterpret_cast<uintptr_t>(L->w_up[e]) & 15)) return false;
  }
  return true;
}

int encode_tensor_maps(const camera_layer_t* L, const ScoreCtx& c, void* host_maps) {
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return CAMERA_ERR_CUDA;
  char* out = static_cast<char*>(host_maps);
  const int E = c.n_experts;
  for (int e = 0; e < E; ++e) {
    if (!encode_2d(fn, out + (size_t)128 * (2 * e), L->w_gate[e], (uint64_t)L->d_ff[e], (uint64_t)c.d_model, CH_TILE) ||
        !encode_2d(fn, out + (size_t)128 * (2 * e + 1), L->w_up[e], (uint64_t)L->d_ff[e], (uint64_t)c.d_model, CH_TILE))
      return CAMERA_ERR_CUDA;
  }
  if (!encode_2d(fn, out + (size_t)128 * (2 * E), c.x_perm, (uint64_t)(c.max_rows_perm > 0 ? c.max_rows_perm : 1),
                 (uint64_t)c.d_model, UMMA_TOK))
    return CAMERA_ERR_CUDA;
  if (!encode_2d(fn, out + (size_t)128 * (2 * E + 1), c.n_tokens > 0 ? c.x : c.x_perm,
                 (uint64_t)(c.n_tokens > 0 ? c.n_tokens : 1), (uint64_t)c.d_model, UMMA_TOK))
    return CAMERA_ERR_CUDA;
  return CAMERA_OK;
}

cudaError_t launch_score_umma(const ScoreCtx& c, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaError_t e = cudaFuncSetAttribute(k_score_umma, cudaFuncAttributeMaxDynamicSharedMemorySize, U_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  k_score_umma<<<sms, U_THREADS, U_SMEM_BYTES, st>>>(c);
  return cudaGetLastError();
}

}  // namespace camera
