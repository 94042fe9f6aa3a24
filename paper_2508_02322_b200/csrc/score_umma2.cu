// Tensor-core scoring kernel for bf16 layers on CTA pairs (Algorithm 1: Lambda, ColumnSum, ColumnMax).
//
// Same computation and the same epilogue as k_score_umma, but two CTAs on neighbouring SMs share one
// MMA (tcgen05 cta_group::2): the pair handles 256 micro-experts x 256 tokens, each CTA keeps the
// W_gate / W_up rows of its own 128 micro-experts and only half of the token tile in shared memory,
// and the tensor cores of both SMs read both halves.  Per k-block a CTA pulls 48 KB from L2 for
// 8.4 Mflop (64 KB without pairing) and reads a third less operand data from shared memory.
//
// Roles per CTA (6 warps): warps 0-3 epilogue, warp 4 lane 0 TMA producer, warp 5 tensor-memory
// allocation; lane 0 of warp 5 of the pair's first CTA issues the MMAs for both.  Barriers:
//   full[s]   (first CTA)  bytes of both CTAs' loads of stage s have landed
//   empty[s]  (each CTA)   the MMAs that read stage s are done           (tcgen05.commit to both CTAs)
//   tfull     (each CTA)   both accumulators of the tile are complete     (tcgen05.commit to both CTAs)
//   tempty    (first CTA)  the epilogue threads of both CTAs have read the accumulators out
// Every wait is bounded, as in k_score_umma.
#include <string.h>

#include "common.cuh"
#include "umma.cuh"
#include "umma_pair.cuh"

namespace camera {

namespace {

constexpr int P_THREADS = 192;
constexpr int P_STAGES = 4;
constexpr int P_A_BYTES = 128 * 128;             // 128 weight rows x 128 B (one of gate / up)
constexpr int P_B_BYTES = 128 * 128;             // this CTA's half of the token tile
constexpr int P_STAGE_BYTES = 2 * P_A_BYTES + P_B_BYTES;
constexpr int P_TMEM_COLS = 512;
constexpr int P_SCHED = 2;                       // depth of the ring that passes unit numbers around the pair
constexpr int P_WBUF_BYTES = 4 * UMMA_TOK * 4;
constexpr int P_STG_BYTES = 4 * FOLD_STG_BYTES;   // layer forward: where an epilogue warp turns its 16 x 32 values of h
constexpr int P_SMEM_BYTES = P_STAGES * P_STAGE_BYTES + P_WBUF_BYTES + P_STG_BYTES + 256 + 1024;

// The layer-forward epilogue with a token on every accumulator row: h = a * SiLU(g) * u for 16 consecutive
// micro-experts of the thread's token, rounded to bf16 and packed into 32 contiguous bytes (one store).
__device__ __forceinline__ void silu_mul16(const uint32_t* vg, const uint32_t* vu, float a, uint32_t* p) {
#pragma unroll
  for (int j = 0; j < 16; j += 2) {
    const float g0 = __uint_as_float(vg[j]), g1 = __uint_as_float(vg[j + 1]);
    const float l0 = (a * __uint_as_float(vu[j])) * (g0 * __fdividef(1.f, 1.f + __expf(-g0)));
    const float l1 = (a * __uint_as_float(vu[j + 1])) * (g1 * __fdividef(1.f, 1.f + __expf(-g1)));
    const __nv_bfloat162 b = __floats2bfloat162_rn(l0, l1);
    p[j >> 1] = *reinterpret_cast<const uint32_t*>(&b);
  }
}

// MODE 0: scoring (partial sums and maxima per micro-expert).  MODE 1: layer forward, h stored from the scoring
// orientation (micro-experts on the accumulator rows, tokens on the columns).  MODE 2: layer forward with the operands
// exchanged: the token tile is the M operand (128 tokens per CTA), the gate and up weights are the N operands (each CTA
// supplies half of the tile's micro-experts), so a thread of the epilogue owns a token and writes runs of consecutive
// micro-experts.  The shared-memory tiles, the loads and the barriers are the same in all three.
enum { PAIR_SCORE = 0, PAIR_H_COLS = 1, PAIR_H_ROWS = 2 };
constexpr int H_TILE_CH = 2 * CH_TILE;          // micro-experts per work unit

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(P_THREADS, 1) k_score_umma_pair(const ScoreCtx c) {
  constexpr bool WRITE_H = MODE == PAIR_H_COLS;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
  // [stages: A_gate | A_up | B half] [wbuf 4 warps x 256 floats] [barriers] [tmem slot] [abort flag]
  float* const wbuf = reinterpret_cast<float*>(base_ptr + P_STAGES * P_STAGE_BYTES);
  uint8_t* const stg_all = base_ptr + P_STAGES * P_STAGE_BYTES + P_WBUF_BYTES;
  const uint32_t bars = base + P_STAGES * P_STAGE_BYTES + P_WBUF_BYTES + P_STG_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (P_STAGES + s); };
  const uint32_t tfull_bar = bars + 8u * (2 * P_STAGES);
  const uint32_t tempty_bar = bars + 8u * (2 * P_STAGES + 1);
  // work units are handed out in order: the first CTA's producer takes the next one from a counter in global memory and
  // writes its number into the ring of both CTAs; sfull (each CTA) = a number is there, sempty (first CTA) = the
  // ten readers of the pair (MMA thread, second CTA's producer, eight epilogue warps) have taken it
  auto sfull_bar = [&](int q) { return bars + 8u * (2 * P_STAGES + 2 + q); };
  auto sempty_bar = [&](int q) { return bars + 8u * (2 * P_STAGES + 2 + P_SCHED + q); };
  uint8_t* const tail = base_ptr + P_STAGES * P_STAGE_BYTES + P_WBUF_BYTES + P_STG_BYTES + 8 * (2 * P_STAGES + 2 + 2 * P_SCHED);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(tail + 8);
  volatile int* const sched_unit = reinterpret_cast<volatile int*>(tail + 16);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int total_units = c.totals->total_units;
  const int n_kb = c.d_model / UMMA_BK;

  if (tid == 0) {
    for (int s = 0; s < P_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tfull_bar, 1);
    mbar_init(tempty_bar, 256);
    for (int q = 0; q < P_SCHED; ++q) { mbar_init(sfull_bar(q), 1); mbar_init(sempty_bar(q), 10); }
    wait_state_init(abort_flag, c.wait_limit_ns);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) {   // one warp of each CTA of the pair takes part in the allocation; both get the same address
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(P_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();     // the other CTA's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer (each CTA loads its own share)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const char* maps = static_cast<const char*>(c.tensor_maps);
      int q = 0;
      uint32_t qphase = 0;
      while (ok) {
        int unit;
        if (rank == 0) {
          if (!mbar_wait_cluster(sempty_bar(q), qphase ^ 1u, abort_flag)) { ok = false; break; }
          unit = atomicAdd(&c.totals->unit_counter, 1);
          if (unit >= total_units) unit = -1;
          sched_unit[q] = unit;
          st_cluster_u32(map_to_cta(smem_u32((const void*)(sched_unit + q)), 1), (uint32_t)unit);
          mbar_arrive(sfull_bar(q));
          mbar_arrive_cluster(map_to_cta(sfull_bar(q), 1));
        } else {
          if (!mbar_wait_cluster(sfull_bar(q), qphase, abort_flag)) { ok = false; break; }
          unit = sched_unit[q];
          mbar_arrive_cluster(map_to_cta(sempty_bar(q), 0));
        }
        if (++q == P_SCHED) { q = 0; qphase ^= 1u; }
        if (unit < 0) break;
        const UnitInfo u = decode_unit(c, unit);
        const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
        const void* map_g = maps + (size_t)128 * (2 * u.e);
        const void* map_u = maps + (size_t)128 * (2 * u.e + 1);
        const void* map_x = maps + (size_t)128 * (2 * c.n_experts + (u.shared_idx < 0 ? 5 : 2));
        tensormap_acquire(map_g);
        tensormap_acquire(map_u);
        tensormap_acquire(map_x);
        // MODE 2: the tile's micro-experts, in whole k-blocks of the second GEMM (h is read 64 columns at a time)
        const int ncv = min(H_TILE_CH, (u.f - u.ch0 + UMMA_BK - 1) & ~(UMMA_BK - 1));
        // past d_ff for the second CTA of an odd last tile: reads zeros
        const int ch = u.ch0 + (MODE == PAIR_H_ROWS ? (int)rank * (ncv >> 1) : 128 * (int)rank);
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int nv = (min(UMMA_TOK, u.rows - tt * UMMA_TOK) + 15) & ~15;
          // this CTA holds tokens [rank * nv/2, +nv/2) of the N operand, or rows [128 rank, +128) of the M operand
          const int row = u.row0 + tt * UMMA_TOK + (int)rank * (MODE == PAIR_H_ROWS ? 128 : (nv >> 1));
          for (int kb = 0; kb < n_kb; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = base + stage * P_STAGE_BYTES;
            const uint32_t full0 = map_to_cta(full_bar(stage), 0);
            if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * P_STAGE_BYTES);
            tma_load_2d_pair(a_dst, map_g, full0, kb * UMMA_BK, ch);
            tma_load_2d_pair(a_dst + P_A_BYTES, map_u, full0, kb * UMMA_BK, ch);
            tma_load_2d_pair(a_dst + 2 * P_A_BYTES, map_x, full0, kb * UMMA_BK, row);
            if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer (first CTA of the pair only)
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0, tile_phase = 0;
      bool ok = true;
      int q = 0;
      uint32_t qphase = 0;
      while (ok) {
        if (!mbar_wait(sfull_bar(q), qphase, abort_flag)) { ok = false; break; }
        const int unit = sched_unit[q];
        mbar_arrive(sempty_bar(q));
        if (++q == P_SCHED) { q = 0; qphase ^= 1u; }
        if (unit < 0) break;
        const UnitInfo u = decode_unit(c, unit);
        const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int nv = (min(UMMA_TOK, u.rows - tt * UMMA_TOK) + 15) & ~15;
          const int ncv = min(H_TILE_CH, (u.f - u.ch0 + UMMA_BK - 1) & ~(UMMA_BK - 1));
          const uint32_t idesc = make_idesc_pair(MODE == PAIR_H_ROWS ? ncv : nv);
          if (!mbar_wait(tempty_bar, tile_phase ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          for (int kb = 0; kb < n_kb; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = base + stage * P_STAGE_BYTES;
            const unsigned long long g_desc = make_smem_desc(a_addr);
            const unsigned long long u_desc = make_smem_desc(a_addr + P_A_BYTES);
            const unsigned long long b_desc = make_smem_desc(a_addr + 2 * P_A_BYTES);
#pragma unroll
            for (int k = 0; k < UMMA_BK / 16; ++k) {
              const uint32_t acc = (uint32_t)((kb | k) != 0);
              if (MODE == PAIR_H_ROWS) {   // [tokens] x [micro-experts]: gate in columns 0-255, up in 256-511
                umma_bf16_pair(tmem_base, b_desc + 2 * k, g_desc + 2 * k, idesc, acc);
                umma_bf16_pair(tmem_base + H_TILE_CH, b_desc + 2 * k, u_desc + 2 * k, idesc, acc);
              } else {                     // [micro-experts] x [tokens]
                umma_bf16_pair(tmem_base, g_desc + 2 * k, b_desc + 2 * k, idesc, acc);
                umma_bf16_pair(tmem_base + UMMA_TOK, u_desc + 2 * k, b_desc + 2 * k, idesc, acc);
              }
            }
            umma_commit_pair(empty_bar(stage));
            if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          umma_commit_pair(tfull_bar);
          tile_phase ^= 1u;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3 of both CTAs)
    uint32_t tile_phase = 0;
    bool ok = true;
    float* const wb = wbuf + warp * UMMA_TOK;
    uint8_t* const stg = stg_all + warp * FOLD_STG_BYTES;
    const uint32_t t_gate = tmem_base + ((uint32_t)(warp * 32) << 16);
    const uint32_t t_up = t_gate + UMMA_TOK;
    const uint32_t tempty0 = map_to_cta(tempty_bar, 0);
    const uint32_t sempty0[P_SCHED] = {map_to_cta(sempty_bar(0), 0), map_to_cta(sempty_bar(1), 0)};
    int q = 0;
    uint32_t qphase = 0;
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait_cluster(sfull_bar(q), qphase, abort_flag));
      if (!ok) break;
      const int unit = sched_unit[q];
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(sempty0[q]);
      if (++q == P_SCHED) { q = 0; qphase ^= 1u; }
      if (unit < 0) break;
      const UnitInfo u = decode_unit(c, unit);
      const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
      const float* wsrc = u.shared_idx < 0 ? c.perm_w + u.row0 : c.shared_w + (size_t)u.shared_idx * c.shared_ld + u.row0;
      float s = 0.f, m = 0.f;
      __nv_bfloat16* hbase = nullptr;
      int h_ld = 0, row_limit = 0;
      if (WRITE_H) {
        const ExpertStatic es = c.est[u.e];
        h_ld = es.h_ld;
        hbase = static_cast<__nv_bfloat16*>(es.h) + (size_t)u.row0 * h_ld + u.ch0 + 128 * (int)rank + warp * 32;
        row_limit = (u.shared_idx < 0 ? c.max_rows_perm : c.n_tokens) - u.row0;
        // h is padded to 128 columns, a pair covers 256: the second CTA of an expert's last pair may have no column
        if (u.ch0 + 128 * (int)rank + warp * 32 >= h_ld) row_limit = 0;
      }
      if constexpr (MODE == PAIR_H_ROWS) {
        const ExpertStatic es = c.est[u.e];
        const int ncv = min(H_TILE_CH, (u.f - u.ch0 + UMMA_BK - 1) & ~(UMMA_BK - 1));
        const int r = 128 * (int)rank + warp * 32 + lane;            // this thread's token row of the tile
        const int buf_rows = (u.shared_idx < 0 ? c.max_rows_perm : c.n_tokens) - u.row0;
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int valid = min(UMMA_TOK, u.rows - tt * UMMA_TOK);
          const int rt = tt * UMMA_TOK + r;
          // rows up to the next multiple of 16 are written (zeros: the second GEMM reads them), none past the buffer
          const bool store = r < ((valid + 15) & ~15) && rt < buf_rows;
          const float a = r < valid ? wsrc[rt] : 0.f;
          __nv_bfloat16* const hrow = static_cast<__nv_bfloat16*>(es.h) + (size_t)(u.row0 + rt) * es.h_ld + u.ch0;
          ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar, tile_phase, abort_flag));
          if (!ok) break;
          tc_fence_after();
          uint32_t g0[16], u0[16], g1[16], u1[16];
          uint32_t pk[8];
          tmem_ld16(t_gate, g0);
          tmem_ld16(t_gate + H_TILE_CH, u0);
          for (int c0 = 0; c0 < ncv; c0 += 32) {
            tmem_ld_wait(g0, u0);
            if (c0 + 16 < ncv) { tmem_ld16(t_gate + c0 + 16, g1); tmem_ld16(t_gate + H_TILE_CH + c0 + 16, u1); }
            silu_mul16(g0, u0, a, pk);
            if (store) st_global_v8(hrow + c0, pk);
            if (c0 + 16 < ncv) {
              tmem_ld_wait(g1, u1);
              if (c0 + 32 < ncv) { tmem_ld16(t_gate + c0 + 32, g0); tmem_ld16(t_gate + H_TILE_CH + c0 + 32, u0); }
              silu_mul16(g1, u1, a, pk);
              if (store) st_global_v8(hrow + c0 + 16, pk);
            }
          }
          tc_fence_before();
          mbar_arrive_cluster(tempty0);
          tile_phase ^= 1u;
        }
      } else {
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int valid = min(UMMA_TOK, u.rows - tt * UMMA_TOK);
          const int nv = (valid + 15) & ~15;
          __nv_bfloat16* const htile = hbase + (size_t)tt * UMMA_TOK * h_ld;
          const int rows_left = row_limit - tt * UMMA_TOK;
          __syncwarp();
          for (int i = lane; i < UMMA_TOK; i += 32) wb[i] = i < valid ? wsrc[tt * UMMA_TOK + i] : 0.f;
          __syncwarp();
          ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar, tile_phase, abort_flag));
          if (!ok) break;
          tc_fence_after();
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
          mbar_arrive_cluster(tempty0);
          tile_phase ^= 1u;
        }
        const int ch = u.ch0 + 128 * (int)rank + warp * 32 + lane;
        // the partials are the scores' input: always when scoring, with the layer forward when scores were asked for
        if ((MODE == PAIR_SCORE || c.energy != nullptr) && ok && ch < u.f) {
          const size_t slot = (size_t)u.part_slot + 128 * rank + warp * 32 + lane;
          c.part_sum[slot] = s;
          c.part_max[slot] = m;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag && tid == 0) atomicExch(&c.totals->status, (int)CAMERA_ERR_DEVICE_TIMEOUT);
  cluster_sync_all();     // neither CTA leaves while the other may still read its shared or tensor memory
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(P_TMEM_COLS) : "memory");
  }
}

}  // namespace

cudaError_t launch_score_umma_pair(const ScoreCtx& c, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaError_t e = cudaFuncSetAttribute(k_score_umma_pair<PAIR_SCORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  k_score_umma_pair<PAIR_SCORE><<<sms & ~1, P_THREADS, P_SMEM_BYTES, st>>>(c);
  return cudaGetLastError();
}

// The same kernel with an epilogue that stores h (layer forward); token_rows picks the orientation with the token
// tile as the M operand.
cudaError_t launch_score_umma_pair_write_h(const ScoreCtx& c, bool token_rows, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  auto kern = token_rows ? k_score_umma_pair<PAIR_H_ROWS> : k_score_umma_pair<PAIR_H_COLS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  kern<<<sms & ~1, P_THREADS, P_SMEM_BYTES, st>>>(c);
  return cudaGetLastError();
}

}  // namespace camera
