// Tensor-core scoring kernel for bf16 layers (Algorithm 1: Lambda, ColumnSum, ColumnMax):
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
// Work units (one channel tile x one token tile) are handed out in order from a counter in global memory, so
// that the CTAs running at one time share a few neighbouring token tiles and one expert's weights through L2
// and stay in step; which CTA runs a unit does not change the result (one partial per unit and micro-expert).
//
// Every wait on an mbarrier is bounded: when a wait runs out the CTA records
// CAMERA_ERR_DEVICE_TIMEOUT in the status word, lets its copies land, frees its tensor memory and
// returns.
#include <cuda.h>
#include <string.h>

#include "common.cuh"
#include "umma.cuh"

namespace camera {

namespace {

constexpr int U_THREADS = 192;
constexpr int U_STAGES = 3;
constexpr int U_BK = UMMA_BK;
constexpr int U_A_BYTES = CH_TILE * 128;         // 128 weight rows x 128 B (one of gate / up)
constexpr int U_B_BYTES = UMMA_TOK * 128;        // 256 token rows x 128 B
constexpr int U_STAGE_BYTES = 2 * U_A_BYTES + U_B_BYTES;
constexpr int U_TMEM_COLS = 512;
constexpr int U_SCHED = 2;                       // depth of the ring that passes unit numbers between the warps
constexpr int U_WBUF_BYTES = 4 * UMMA_TOK * 4;   // router weights of a token tile, one copy per epilogue warp
constexpr int U_STG_BYTES = 4 * FOLD_STG_BYTES;   // layer forward: where an epilogue warp turns its 16 x 32 values of h
constexpr int U_SMEM_BYTES = U_STAGES * U_STAGE_BYTES + U_WBUF_BYTES + U_STG_BYTES + 256 + 1024;
static_assert(CH_TILE == 128, "one micro-expert per TMEM lane");

template <bool WRITE_H>
__global__ void __launch_bounds__(U_THREADS, 1) k_score_umma(const ScoreCtx c) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
  // [stages: A_gate | A_up | B] [wbuf 4 warps x 256 floats] [barriers] [tmem slot] [abort flag]
  float* const wbuf = reinterpret_cast<float*>(base_ptr + U_STAGES * U_STAGE_BYTES);
  uint8_t* const stg_all = base_ptr + U_STAGES * U_STAGE_BYTES + U_WBUF_BYTES;
  const uint32_t bars = base + U_STAGES * U_STAGE_BYTES + U_WBUF_BYTES + U_STG_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (U_STAGES + s); };
  const uint32_t tfull_bar = bars + 8u * (2 * U_STAGES);
  const uint32_t tempty_bar = bars + 8u * (2 * U_STAGES + 1);
  // work units are handed out in order from a counter in global memory: the producer thread takes the next one and
  // passes its number to the MMA thread and the epilogue warps through a small ring
  auto sfull_bar = [&](int q) { return bars + 8u * (2 * U_STAGES + 2 + q); };
  auto sempty_bar = [&](int q) { return bars + 8u * (2 * U_STAGES + 2 + U_SCHED + q); };
  uint8_t* const tail = base_ptr + U_STAGES * U_STAGE_BYTES + U_WBUF_BYTES + U_STG_BYTES + 8 * (2 * U_STAGES + 2 + 2 * U_SCHED);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(tail + 8);
  volatile int* const sched_unit = reinterpret_cast<volatile int*>(tail + 16);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_units = c.totals->total_units;
  const int n_kb = c.d_model / U_BK;

  if (tid == 0) {
    for (int s = 0; s < U_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tfull_bar, 1);
    mbar_init(tempty_bar, 128);
    for (int q = 0; q < U_SCHED; ++q) { mbar_init(sfull_bar(q), 1); mbar_init(sempty_bar(q), 5); }
    wait_state_init(abort_flag, c.wait_limit_ns);
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
      int q = 0;
      uint32_t qphase = 0;
      while (ok) {
        if (!mbar_wait(sempty_bar(q), qphase ^ 1u, abort_flag)) { ok = false; break; }
        int unit = atomicAdd(&c.totals->unit_counter, 1);
        if (unit >= total_units) unit = -1;
        sched_unit[q] = unit;
        mbar_arrive(sfull_bar(q));
        if (++q == U_SCHED) { q = 0; qphase ^= 1u; }
        if (unit < 0) break;
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
      int q = 0;
      uint32_t qphase = 0;
      while (ok) {
        if (!mbar_wait(sfull_bar(q), qphase, abort_flag)) { ok = false; break; }
        const int unit = sched_unit[q];
        mbar_arrive(sempty_bar(q));
        if (++q == U_SCHED) { q = 0; qphase ^= 1u; }
        if (unit < 0) break;
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
    uint8_t* const stg = stg_all + warp * FOLD_STG_BYTES;
    const uint32_t t_gate = tmem_base + ((uint32_t)(warp * 32) << 16);
    const uint32_t t_up = t_gate + UMMA_TOK;
    int q = 0;
    uint32_t qphase = 0;
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait(sfull_bar(q), qphase, abort_flag));
      if (!ok) break;
      const int unit = sched_unit[q];
      __syncwarp();
      if (lane == 0) mbar_arrive(sempty_bar(q));
      if (++q == U_SCHED) { q = 0; qphase ^= 1u; }
      if (unit < 0) break;
      const UnitInfo u = decode_unit(c, unit);
      const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
      const float* wsrc = u.shared_idx < 0 ? c.perm_w + u.row0 : c.shared_w + (size_t)u.shared_idx * c.shared_ld + u.row0;
      float s = 0.f, m = 0.f;
      // layer forward: where the warp's 32 micro-experts go in h, and the last row h has
      __nv_bfloat16* hbase = nullptr;
      int h_ld = 0, row_limit = 0;
      if (WRITE_H) {
        const ExpertStatic es = c.est[u.e];
        h_ld = es.h_ld;
        hbase = static_cast<__nv_bfloat16*>(es.h) + (size_t)u.row0 * h_ld + u.ch0 + warp * 32;
        row_limit = (u.shared_idx < 0 ? c.max_rows_perm : c.n_tokens) - u.row0;
      }
      for (int tt = 0; ok && tt < n_tiles; ++tt) {
        const int valid = min(UMMA_TOK, u.rows - tt * UMMA_TOK);
        const int nv = (valid + 15) & ~15;
        __nv_bfloat16* const htile = hbase + (size_t)tt * UMMA_TOK * h_ld;
        const int rows_left = row_limit - tt * UMMA_TOK;
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
          fold16<WRITE_H>(g0, u0, wb + c0, s, m, htile + (size_t)c0 * h_ld, h_ld, rows_left - c0, stg, lane);
          if (c0 + 16 < nv) {
            tmem_ld_wait(g1, u1);
            if (c0 + 32 < nv) { tmem_ld16(t_gate + c0 + 32, g0); tmem_ld16(t_up + c0 + 32, u0); }
            fold16<WRITE_H>(g1, u1, wb + c0 + 16, s, m, htile + (size_t)(c0 + 16) * h_ld, h_ld, rows_left - c0 - 16, stg, lane);
          }
        }
        tc_fence_before();
        mbar_arrive(tempty_bar);
        tile_phase ^= 1u;
      }
      const int ch = u.ch0 + warp * 32 + lane;
      // the partials are the scores' input: always when scoring, with the layer forward when scores were asked for
      if ((!WRITE_H || c.energy != nullptr) && ok && ch < u.f) {
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
bool encode_2d(EncodeTiledFn fn, void* out, const void* ptr, uint64_t rows, uint64_t d, uint32_t box_rows,
               uint64_t pitch = 0) {
  if (ptr == nullptr || rows == 0 || d == 0) { memset(out, 0, 128); return true; }
  CUtensorMap m;
  const cuuint64_t dims[2] = {d, rows};
  const cuuint64_t strides[1] = {(pitch ? pitch : d) * 2};
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

bool encode_bf16_2d(void* out, const void* ptr, uint64_t rows, uint64_t d, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  return fn != nullptr && encode_2d(fn, out, ptr, rows, d, box_rows);
}

bool encode_bf16_2d_pitch(void* out, const void* ptr, uint64_t rows, uint64_t cols, uint64_t pitch, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  return fn != nullptr && encode_2d(fn, out, ptr, rows, cols, box_rows, pitch);
}

bool umma_shape_ok(const camera_layer_t* L) {
  if (L->dtype != CAMERA_BF16 || L->d_model % U_BK != 0) return false;
  for (int e = 0; e < L->n_routed + L->n_shared; ++e) {
    if ((reinterpret_cast<uintptr_t>(L->w_gate[e]) & 15) || (reinterpret_cast<uintptr_t>(L->w_up[e]) & 15)) return false;
  }
  return true;
}

int encode_tensor_maps(const camera_layer_t* L, const ScoreCtx& c, void* host_maps, int which) {
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return CAMERA_ERR_CUDA;
  char* out = static_cast<char*>(host_maps);
  const int E = c.n_experts;
  if (which & MAPS_STATIC) {
    for (int e = 0; e < E; ++e) {
      if (!encode_2d(fn, out + (size_t)128 * (2 * e), L->w_gate[e], (uint64_t)L->d_ff[e], (uint64_t)c.d_model, CH_TILE) ||
          !encode_2d(fn, out + (size_t)128 * (2 * e + 1), L->w_up[e], (uint64_t)L->d_ff[e], (uint64_t)c.d_model, CH_TILE))
        return CAMERA_ERR_CUDA;
    }
  }
  if (!(which & MAPS_TOKENS)) return CAMERA_OK;
  if (!encode_2d(fn, out + (size_t)128 * (2 * E), c.x_perm, (uint64_t)(c.max_rows_perm > 0 ? c.max_rows_perm : 1),
                 (uint64_t)c.d_model, UMMA_TOK))
    return CAMERA_ERR_CUDA;
  if (!encode_2d(fn, out + (size_t)128 * (2 * E + 1), c.n_tokens > 0 ? c.x : c.x_perm,
                 (uint64_t)(c.n_tokens > 0 ? c.n_tokens : 1), (uint64_t)c.d_model, UMMA_TOK))
    return CAMERA_ERR_CUDA;
  // the same two matrices in boxes of 128 rows: each CTA of a pair loads half a token tile
  if (!encode_2d(fn, out + (size_t)128 * (2 * E + 2), c.n_tokens > 0 ? c.x : c.x_perm,
                 (uint64_t)(c.n_tokens > 0 ? c.n_tokens : 1), (uint64_t)c.d_model, UMMA_TOK / 2) ||
      !encode_2d(fn, out + (size_t)128 * (2 * E + 5), c.x_perm, (uint64_t)(c.max_rows_perm > 0 ? c.max_rows_perm : 1),
                 (uint64_t)c.d_model, UMMA_TOK / 2))
    return CAMERA_ERR_CUDA;
  return CAMERA_OK;
}

cudaError_t launch_score_umma(const ScoreCtx& c, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaError_t e = cudaFuncSetAttribute(k_score_umma<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, U_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  k_score_umma<false><<<sms, U_THREADS, U_SMEM_BYTES, st>>>(c);
  return cudaGetLastError();
}

// The same kernel with the epilogue that stores h (layer forward).
cudaError_t launch_score_umma_write_h(const ScoreCtx& c, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaError_t e = cudaFuncSetAttribute(k_score_umma<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, U_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  k_score_umma<true><<<sms, U_THREADS, U_SMEM_BYTES, st>>>(c);
  return cudaGetLastError();
}

}  // namespace camera
