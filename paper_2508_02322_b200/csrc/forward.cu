// The layer's output (Eq. 1-2): y_t = sum_e A_{t,e} W_down_e [ SiLU(W_gate_e x_t) * (W_up_e x_t) ], on the routing and
// token lists of the scoring path.  It exists to evaluate a selection: the output of the sliced layer is
// Y_hat = Phi[:,S] W[S,:] of Eq. 7, and camera_output_error gives ||Y - Y_hat||_F^2 and the cosine similarity.
//
//   k_score_umma<WRITE_H>   h = A * SiLU(W_gate x) * (W_up x) per (token row, micro-expert), bf16      (score_umma.cu)
//   k_down_umma(_pair)      y_part[row, :] = W_down h[row, :] per expert, tcgen05, fp32 out (pairs: long token lists)
//   k_unpermute_sum         y[t, :] = sum over the token's k routed rows and its shared-expert rows, fixed order
#include <math.h>
#include <string.h>

#include <vector>

#include "common.cuh"
#include "umma.cuh"
#include "umma_pair.cuh"

namespace camera {

namespace {

constexpr int D_THREADS = 192;
constexpr int D_STAGES = 4;                       // with a full token tile per stage
constexpr int D_MAX_STAGES = 8;                   // with the short boxes of a decode batch
constexpr int D_TILE = 128;                       // output channels (rows of W_down) per work unit = TMEM lanes
constexpr int D_A_BYTES = D_TILE * 128;
constexpr int D_B_BYTES = UMMA_TOK * 128;
constexpr int D_STAGE_BYTES = D_A_BYTES + D_B_BYTES;
constexpr int D_TMEM_COLS = 512;
constexpr int D_SCHED = 2;                        // ring that passes unit numbers from the producer to the other warps
constexpr int D_SMEM_BYTES = D_STAGES * D_STAGE_BYTES + 256 + 1024;      // the budget every configuration stays within

struct DownUnit {
  int e, rows, row0, c0, n_kb, row_limit;
  float* y;
};

// Work units are numbered (token chunk, output-channel tile) with the tile fastest: the CTAs running at one time
// share a chunk of h through L2 while an expert's W_down stays resident.
__device__ __forceinline__ DownUnit decode_down_unit(const ScoreCtx& c, int unit, int n_dt, int tile = D_TILE) {
  DownUnit u;
  const int chunk = unit / n_dt;
  int lo = 0, hi = c.n_experts;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (c.edyn[mid].chunk_begin <= chunk) lo = mid; else hi = mid;
  }
  u.e = lo;
  const ExpertDyn dy = c.edyn[lo];
  const ExpertStatic es = c.est[lo];
  const int ck = chunk - dy.chunk_begin;
  u.rows = min(c.chunk_tokens, dy.rows - ck * c.chunk_tokens);
  u.row0 = dy.row_base + ck * c.chunk_tokens;
  u.c0 = (unit % n_dt) * tile;
  u.n_kb = (es.d_ff + UMMA_BK - 1) / UMMA_BK;
  u.row_limit = (es.shared_idx < 0 ? c.max_rows_perm : c.n_tokens) - u.row0;
  u.y = es.y_part;
  return u;
}

// b_bytes: size of the box of h rows one load brings (128 bytes per row; the map's box is as many rows as a token list
// can have, at most a tile: with a few tokens per expert a full tile's box would triple the bytes L2 has to deliver).
// n_stages: depth of the operand ring; a stage is the W_down tile plus that box, so a decode batch (a box of 64 rows)
// gets 8 stages of 24 KB where a full token tile gets 4 of 48 KB: the kernel then streams W_down from DRAM, and the
// bytes in flight per SM are what hides the latency.
__global__ void __launch_bounds__(D_THREADS, 1)
k_down_umma(const ScoreCtx c, const void* maps_raw, int n_dt, int b_bytes, int n_stages) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int stage_bytes = D_A_BYTES + b_bytes;                 // a multiple of 1024: the swizzled tiles stay aligned
  const uint32_t bars = base + n_stages * stage_bytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (D_MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * D_MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * D_MAX_STAGES + 2 + a); };
  auto sfull_bar = [&](int q) { return bars + 8u * (2 * D_MAX_STAGES + 4 + q); };
  auto sempty_bar = [&](int q) { return bars + 8u * (2 * D_MAX_STAGES + 4 + D_SCHED + q); };
  uint8_t* const tail = base_ptr + n_stages * stage_bytes + 8 * (2 * D_MAX_STAGES + 4 + 2 * D_SCHED);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(tail + 8);
  volatile int* const sched_unit = reinterpret_cast<volatile int*>(tail + 16);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_units = c.totals->total_chunks * n_dt;

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128); }
    for (int q = 0; q < D_SCHED; ++q) { mbar_init(sfull_bar(q), 1); mbar_init(sempty_bar(q), 5); }
    wait_state_init(abort_flag, c.wait_limit_ns);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(D_TMEM_COLS)
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
      const char* maps = static_cast<const char*>(maps_raw);
      int q = 0;
      uint32_t qphase = 0;
      while (ok) {   // units are taken in order from a counter, as in the scoring kernel
        if (!mbar_wait(sempty_bar(q), qphase ^ 1u, abort_flag)) { ok = false; break; }
        // last expert first: the shared experts come last in the numbering and have the longest K, so their
        // units start early instead of forming the tail (with 64 tokens they are 8 times a routed expert's unit)
        int unit = atomicAdd(&c.totals->down_counter, 1);
        unit = unit >= total_units ? -1 : total_units - 1 - unit;
        sched_unit[q] = unit;
        mbar_arrive(sfull_bar(q));
        if (++q == D_SCHED) { q = 0; qphase ^= 1u; }
        if (unit < 0) break;
        const DownUnit u = decode_down_unit(c, unit, n_dt);
        if (u.n_kb == 0) continue;
        const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
        const void* map_w = maps + (size_t)128 * (2 * u.e);
        const void* map_h = maps + (size_t)128 * (2 * u.e + 1);
        tensormap_acquire(map_w);
        tensormap_acquire(map_h);
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int row = u.row0 + tt * UMMA_TOK;
          for (int kb = 0; kb < u.n_kb; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = base + stage * stage_bytes;
            mbar_expect_tx(full_bar(stage), D_A_BYTES + b_bytes);
            // W_down columns past d_ff and rows past d_model, h rows past the buffer: filled with zeros
            tma_load_2d(a_dst, map_w, full_bar(stage), kb * UMMA_BK, u.c0);
            tma_load_2d(a_dst + D_A_BYTES, map_h, full_bar(stage), kb * UMMA_BK, row);
            if (++stage == n_stages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      int q = 0;
      uint32_t qphase = 0;
      while (ok) {
        if (!mbar_wait(sfull_bar(q), qphase, abort_flag)) { ok = false; break; }
        const int unit = sched_unit[q];
        mbar_arrive(sempty_bar(q));
        if (++q == D_SCHED) { q = 0; qphase ^= 1u; }
        if (unit < 0) break;
        const DownUnit u = decode_down_unit(c, unit, n_dt);
        if (u.n_kb == 0) continue;
        const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int nv = (min(UMMA_TOK, u.rows - tt * UMMA_TOK) + 15) & ~15;
          const uint32_t idesc = make_idesc(nv);
          if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * UMMA_TOK);
          for (int kb = 0; kb < u.n_kb; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = base + stage * stage_bytes;
            const unsigned long long a_desc = make_smem_desc(a_addr);
            const unsigned long long b_desc = make_smem_desc(a_addr + D_A_BYTES);
#pragma unroll
            for (int k = 0; k < UMMA_BK / 16; ++k)
              umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (uint32_t)((kb | k) != 0));
            umma_commit(empty_bar(stage));
            if (++stage == n_stages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          umma_commit(tfull_bar(acc));
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3): lane = output channel
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    int q = 0;
    uint32_t qphase = 0;
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait(sfull_bar(q), qphase, abort_flag));
      if (!ok) break;
      const int unit = sched_unit[q];
      __syncwarp();
      if (lane == 0) mbar_arrive(sempty_bar(q));
      if (++q == D_SCHED) { q = 0; qphase ^= 1u; }
      if (unit < 0) break;
      const DownUnit u = decode_down_unit(c, unit, n_dt);
      const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
      const int ch = u.c0 + warp * 32 + lane;
      float* const ycol = u.y + (size_t)u.row0 * c.d_model + ch;
      for (int tt = 0; ok && tt < n_tiles; ++tt) {
        const int nv = (min(UMMA_TOK, u.rows - tt * UMMA_TOK) + 15) & ~15;
        const int n_store = min(nv, u.row_limit - tt * UMMA_TOK);
        float* const ytile = ycol + (size_t)tt * UMMA_TOK * c.d_model;
        if (u.n_kb == 0) {   // an expert without micro-experts contributes zeros
          if (ch < c.d_model)
            for (int j = 0; j < n_store; ++j) ytile[(size_t)j * c.d_model] = 0.f;
          continue;
        }
        ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag));
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(acc * UMMA_TOK);
        for (int c0 = 0; c0 < nv; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(taddr + c0, v);
          tmem_ld_wait(v);
          if (ch < c.d_model) {
#pragma unroll
            for (int j = 0; j < 16; ++j)     // a warp writes 32 consecutive channels of one token row: 128 bytes
              if (c0 + j < n_store) ytile[(size_t)(c0 + j) * c.d_model] = __uint_as_float(v[j]);
          }
        }
        tc_fence_before();
        mbar_arrive(tempty_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag && tid == 0) atomicExch(&c.totals->status, (int)CAMERA_ERR_DEVICE_TIMEOUT);
  if (warp == 5) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(D_TMEM_COLS) : "memory");
  }
}

// The same GEMM on CTA pairs with the token tile as the M operand: the pair computes 256 tokens x 512 output channels
// as two MMAs of N = 256 that share the token tile, so a CTA pulls 48 KB per k-block from L2 for 16.8 Mflop (k_down_umma:
// 48 KB for 4.2 Mflop, which keeps the tensor pipe waiting for L2).  Each CTA holds its 128 token rows of h and its
// halves of the two W_down tiles; the two accumulators fill the 512 TMEM columns, so the short epilogue (a thread owns
// a token and writes 64 contiguous bytes of its output row per 16 columns) runs between tiles.  Barriers and the
// hand-out of work units are those of k_score_umma_pair; every token tile costs 256 rows, so short token lists stay
// with k_down_umma.
constexpr int DP_STAGES = 4;
constexpr int DP_HALF = 256;                      // output channels per MMA
constexpr int DP_TILE = 2 * DP_HALF;              // output channels per work unit
constexpr int DP_A_BYTES = 128 * 128;             // this CTA's 128 token rows of h x 128 B
constexpr int DP_B_BYTES = 128 * 128;             // this CTA's half of one W_down tile
constexpr int DP_STAGE_BYTES = DP_A_BYTES + 2 * DP_B_BYTES;
constexpr int DP_SMEM_BYTES = DP_STAGES * DP_STAGE_BYTES + 256 + 1024;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(D_THREADS, 1)
    k_down_umma_pair(const ScoreCtx c, const void* maps_raw, int n_dt) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + DP_STAGES * DP_STAGE_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };                                   // first CTA
  auto empty_bar = [&](int s) { return bars + 8u * (DP_STAGES + s); };                    // each CTA
  const uint32_t tfull_bar = bars + 8u * (2 * DP_STAGES);                                 // each CTA
  const uint32_t tempty_bar = bars + 8u * (2 * DP_STAGES + 1);                            // first CTA, 256 readers
  auto sfull_bar = [&](int q) { return bars + 8u * (2 * DP_STAGES + 2 + q); };            // each CTA
  auto sempty_bar = [&](int q) { return bars + 8u * (2 * DP_STAGES + 2 + D_SCHED + q); }; // first CTA, 10 readers
  uint8_t* const tail = base_ptr + DP_STAGES * DP_STAGE_BYTES + 8 * (2 * DP_STAGES + 2 + 2 * D_SCHED);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(tail + 8);
  volatile int* const sched_unit = reinterpret_cast<volatile int*>(tail + 16);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int total_units = c.totals->total_chunks * n_dt;

  if (tid == 0) {
    for (int s = 0; s < DP_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tfull_bar, 1);
    mbar_init(tempty_bar, 256);
    for (int q = 0; q < D_SCHED; ++q) { mbar_init(sfull_bar(q), 1); mbar_init(sempty_bar(q), 10); }
    wait_state_init(abort_flag, c.wait_limit_ns);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(D_TMEM_COLS)
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
      const char* maps = static_cast<const char*>(maps_raw);
      int q = 0;
      uint32_t qphase = 0;
      while (ok) {
        int unit;
        if (rank == 0) {
          if (!mbar_wait_cluster(sempty_bar(q), qphase ^ 1u, abort_flag)) { ok = false; break; }
          unit = atomicAdd(&c.totals->down_counter, 1);
          unit = unit >= total_units ? -1 : total_units - 1 - unit;     // last expert first, as in k_down_umma
          sched_unit[q] = unit;
          st_cluster_u32(map_to_cta(smem_u32((const void*)(sched_unit + q)), 1), (uint32_t)unit);
          mbar_arrive(sfull_bar(q));
          mbar_arrive_cluster(map_to_cta(sfull_bar(q), 1));
        } else {
          if (!mbar_wait_cluster(sfull_bar(q), qphase, abort_flag)) { ok = false; break; }
          unit = sched_unit[q];
          mbar_arrive_cluster(map_to_cta(sempty_bar(q), 0));
        }
        if (++q == D_SCHED) { q = 0; qphase ^= 1u; }
        if (unit < 0) break;
        const DownUnit u = decode_down_unit(c, unit, n_dt, DP_TILE);
        if (u.n_kb == 0) continue;
        const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
        const void* map_w = maps + (size_t)128 * (2 * u.e);
        const void* map_h = maps + (size_t)128 * (2 * u.e + 1);
        tensormap_acquire(map_w);
        tensormap_acquire(map_h);
        // the two N operands (d_model is a multiple of 64); this CTA holds the upper or lower half of each
        const int ncv0 = min(DP_HALF, c.d_model - u.c0), ncv1 = max(0, min(DP_HALF, c.d_model - u.c0 - DP_HALF));
        const int wrow0 = u.c0 + (int)rank * (ncv0 >> 1), wrow1 = u.c0 + DP_HALF + (int)rank * (ncv1 >> 1);
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          const int row = u.row0 + tt * UMMA_TOK + 128 * (int)rank;  // this CTA's rows of the M operand
          for (int kb = 0; kb < u.n_kb; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = base + stage * DP_STAGE_BYTES;
            const uint32_t full0 = map_to_cta(full_bar(stage), 0);
            if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * DP_STAGE_BYTES);
            // h rows past the buffer, W_down columns past d_ff and rows past d_model: filled with zeros
            tma_load_2d_pair(a_dst, map_h, full0, kb * UMMA_BK, row);
            tma_load_2d_pair(a_dst + DP_A_BYTES, map_w, full0, kb * UMMA_BK, wrow0);
            tma_load_2d_pair(a_dst + DP_A_BYTES + DP_B_BYTES, map_w, full0, kb * UMMA_BK, wrow1);
            if (++stage == DP_STAGES) { stage = 0; phase ^= 1u; }
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
        if (++q == D_SCHED) { q = 0; qphase ^= 1u; }
        if (unit < 0) break;
        const DownUnit u = decode_down_unit(c, unit, n_dt, DP_TILE);
        if (u.n_kb == 0) continue;
        const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
        const int ncv0 = min(DP_HALF, c.d_model - u.c0), ncv1 = max(0, min(DP_HALF, c.d_model - u.c0 - DP_HALF));
        const uint32_t idesc0 = make_idesc_pair(ncv0), idesc1 = make_idesc_pair(ncv1);
        for (int tt = 0; ok && tt < n_tiles; ++tt) {
          if (!mbar_wait_cluster(tempty_bar, tile_phase ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          for (int kb = 0; kb < u.n_kb; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = base + stage * DP_STAGE_BYTES;
            const unsigned long long a_desc = make_smem_desc(a_addr);
            const unsigned long long b0_desc = make_smem_desc(a_addr + DP_A_BYTES);
            const unsigned long long b1_desc = make_smem_desc(a_addr + DP_A_BYTES + DP_B_BYTES);
#pragma unroll
            for (int k = 0; k < UMMA_BK / 16; ++k) {
              const uint32_t accum = (uint32_t)((kb | k) != 0);
              umma_bf16_pair(tmem_base, a_desc + 2 * k, b0_desc + 2 * k, idesc0, accum);
              if (ncv1 > 0) umma_bf16_pair(tmem_base + DP_HALF, a_desc + 2 * k, b1_desc + 2 * k, idesc1, accum);
            }
            umma_commit_pair(empty_bar(stage));
            if (++stage == DP_STAGES) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          umma_commit_pair(tfull_bar);
          tile_phase ^= 1u;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3 of both CTAs): lane = token
    uint32_t tile_phase = 0;
    bool ok = true;
    const uint32_t tempty0 = map_to_cta(tempty_bar, 0);
    const uint32_t sempty0[D_SCHED] = {map_to_cta(sempty_bar(0), 0), map_to_cta(sempty_bar(1), 0)};
    const int r = 128 * (int)rank + warp * 32 + lane;               // this thread's token row of the tile
    int q = 0;
    uint32_t qphase = 0;
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait_cluster(sfull_bar(q), qphase, abort_flag));
      if (!ok) break;
      const int unit = sched_unit[q];
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(sempty0[q]);
      if (++q == D_SCHED) { q = 0; qphase ^= 1u; }
      if (unit < 0) break;
      const DownUnit u = decode_down_unit(c, unit, n_dt, DP_TILE);
      const int n_tiles = (u.rows + UMMA_TOK - 1) / UMMA_TOK;
      const int ncv = min(DP_TILE, c.d_model - u.c0);
      for (int tt = 0; ok && tt < n_tiles; ++tt) {
        const int nv = (min(UMMA_TOK, u.rows - tt * UMMA_TOK) + 15) & ~15;
        const int rt = tt * UMMA_TOK + r;
        const bool store = r < nv && rt < u.row_limit;
        float* const yrow = u.y + (size_t)(u.row0 + rt) * c.d_model + u.c0;
        if (u.n_kb == 0) {   // an expert without micro-experts contributes zeros
          if (store)
            for (int j = 0; j < ncv; j += 4) *reinterpret_cast<float4*>(yrow + j) = make_float4(0.f, 0.f, 0.f, 0.f);
          continue;
        }
        ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar, tile_phase, abort_flag));
        if (!ok) break;
        tc_fence_after();
        // the unit's output channels are consecutive accumulator columns (the first MMA fills 256 unless it is the last)
        const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
        uint32_t v0[16], v1[16];
        tmem_ld16(taddr, v0);
        for (int c0 = 0; c0 < ncv; c0 += 32) {
          tmem_ld_wait(v0);
          if (c0 + 16 < ncv) tmem_ld16(taddr + c0 + 16, v1);
          if (store) { st_global_v8(yrow + c0, v0); st_global_v8(yrow + c0 + 8, v0 + 8); }
          if (c0 + 16 < ncv) {
            tmem_ld_wait(v1);
            if (c0 + 32 < ncv) tmem_ld16(taddr + c0 + 32, v0);
            if (store) { st_global_v8(yrow + c0 + 16, v1); st_global_v8(yrow + c0 + 24, v1 + 8); }
          }
        }
        tc_fence_before();
        mbar_arrive_cluster(tempty0);
        tile_phase ^= 1u;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag && tid == 0) atomicExch(&c.totals->status, (int)CAMERA_ERR_DEVICE_TIMEOUT);
  cluster_sync_all();     // neither CTA leaves while the other may still read its shared or tensor memory
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(D_TMEM_COLS) : "memory");
  }
}

// y[t, :] = the token's k routed rows of y_perm (in slot order) plus its row of every shared expert.  A block owns up
// to 1024 consecutive output channels of one token (four per thread), so a 64-token decode batch still fills the GPU
// with independent loads; the rows' positions are worked out once per block.
__global__ void __launch_bounds__(256) k_unpermute_sum(const ScoreCtx c, float* __restrict__ y) {
  __shared__ long long pos_s[MAX_TOPK];
  const int k = c.top_k, d = c.d_model;
  const int t = blockIdx.x;
  if ((int)threadIdx.x < k) {
    const int e = c.topk_idx[(size_t)t * k + threadIdx.x];
    long long pos = -1;     // the routers only leave experts in range; anything else adds nothing
    if (e >= 0 && e < c.n_routed) {
      pos = (long long)c.edyn[e].row_base + c.block_hist[(size_t)(t / ROUTER_TOK) * c.n_routed + e] +
            c.local_rank[(size_t)t * k + threadIdx.x];
      if (pos < 0 || pos >= c.max_rows_perm) pos = -1;
    }
    pos_s[threadIdx.x] = pos;
  }
  __syncthreads();
  const int v = (blockIdx.y * 256 + threadIdx.x) << 2;
  if (v >= d) return;
  const float* routed = c.n_routed > 0 ? c.est[0].y_part : nullptr;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
  for (int s = 0; s < k; ++s) {
    if (pos_s[s] < 0) continue;
    const float4 p = *reinterpret_cast<const float4*>(routed + (size_t)pos_s[s] * d + v);
    acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
  }
  for (int s = 0; s < c.n_shared; ++s) {
    const float4 p = *reinterpret_cast<const float4*>(c.est[c.n_routed + s].y_part + (size_t)t * d + v);
    acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
  }
  *reinterpret_cast<float4*>(y + (size_t)t * d + v) = acc;
}

// Per CTA of 8 tokens: sum (y - y_hat)^2, sum y^2, sum of the tokens' cosine similarities, in double.
__global__ void __launch_bounds__(256) k_error_partials(const float* __restrict__ y, const float* __restrict__ yh,
                                                        long long n_tokens, int d, double* __restrict__ part) {
  __shared__ double red[8][3];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long t = (long long)blockIdx.x * 8 + warp;
  double e2 = 0.0, n2 = 0.0, cs = 0.0;
  if (t < n_tokens) {
    double dot = 0.0, h2 = 0.0;
    for (int v = lane; v < d; v += 32) {
      const double a = y[(size_t)t * d + v], b = yh[(size_t)t * d + v];
      e2 += (a - b) * (a - b); n2 += a * a; h2 += b * b; dot += a * b;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      e2 += __shfl_xor_sync(0xffffffffu, e2, o); n2 += __shfl_xor_sync(0xffffffffu, n2, o);
      h2 += __shfl_xor_sync(0xffffffffu, h2, o); dot += __shfl_xor_sync(0xffffffffu, dot, o);
    }
    cs = (n2 > 0.0 && h2 > 0.0) ? dot / sqrt(n2 * h2) : (n2 == h2 ? 1.0 : 0.0);
  }
  if (lane == 0) { red[warp][0] = e2; red[warp][1] = n2; red[warp][2] = cs; }
  __syncthreads();
  if (threadIdx.x < 3) {
    double s = 0.0;
    for (int w = 0; w < 8; ++w) s += red[w][threadIdx.x];
    part[(size_t)blockIdx.x * 3 + threadIdx.x] = s;
  }
}

// One CTA adds the partials in a fixed order.
__global__ void __launch_bounds__(256) k_error_final(const double* __restrict__ part, long long n_part, long long n_tokens,
                                                     double* __restrict__ out) {
  __shared__ double red[256][3];
  double s[3] = {0.0, 0.0, 0.0};
  for (long long i = threadIdx.x; i < n_part; i += 256)
    for (int j = 0; j < 3; ++j) s[j] += part[i * 3 + j];
  for (int j = 0; j < 3; ++j) red[threadIdx.x][j] = s[j];
  __syncthreads();
  if (threadIdx.x < 3) {
    double t = 0.0;
    for (int i = 0; i < 256; ++i) t += red[i][threadIdx.x];
    out[threadIdx.x] = threadIdx.x == 2 ? (n_tokens > 0 ? t / (double)n_tokens : 1.0) : t;
  }
}

// One warp per token: z = x + y, out = z / sqrt(mean(z^2) + eps) in the dtype of x.  The row stays in registers
// between the two passes for d_model <= 8192; longer rows are read twice.
template <typename T>
__global__ void __launch_bounds__(256) k_residual_norm(const T* __restrict__ x, const float* __restrict__ y, long long n_tokens,
                                                       int d, float eps, T* __restrict__ out) {
  constexpr int VN = Vec16<T>::N;
  const int lane = threadIdx.x & 31;
  const long long t = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= n_tokens) return;
  const T* xr = x + (size_t)t * d;
  const float* yr = y + (size_t)t * d;
  float ss = 0.f;
  for (int v = lane * VN; v < d; v += 32 * VN) {
    float xv[VN];
    Vec16<T>::load(xr + v, xv);
#pragma unroll
    for (int i = 0; i < VN; ++i) { const float z = xv[i] + yr[v + i]; ss = fmaf(z, z, ss); }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float scale = rsqrtf(ss / (float)d + eps);
  T* orow = out + (size_t)t * d;
  for (int v = lane * VN; v < d; v += 32 * VN) {
    float xv[VN];
    Vec16<T>::load(xr + v, xv);
#pragma unroll
    for (int i = 0; i < VN; ++i) {
      const float z = (xv[i] + yr[v + i]) * scale;
      if constexpr (sizeof(T) == 2) orow[v + i] = __float2bfloat16_rn(z); else orow[v + i] = z;
    }
  }
}

size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

struct FwdLayout {
  size_t score, maps, h_routed, y_perm, total, score_bytes;
  std::vector<size_t> h_shared, y_shared;
  int h_ld_routed, max_rows_perm;
  std::vector<int> h_ld;
};

FwdLayout fwd_layout(const camera_layer_t* L, int64_t T) {
  FwdLayout f;
  const int E = L->n_routed + L->n_shared;
  const int k = L->n_routed > 0 ? L->top_k : 0;
  f.score_bytes = score_workspace_bytes_any(L, T, true);
  f.max_rows_perm = (int)(T * k + (long long)ROW_ALIGN * L->n_routed);
  int f_max = 0;
  for (int e = 0; e < L->n_routed; ++e) f_max = L->d_ff[e] > f_max ? L->d_ff[e] : f_max;
  f.h_ld_routed = ((f_max + CH_TILE - 1) / CH_TILE) * CH_TILE;
  if (f.h_ld_routed == 0) f.h_ld_routed = CH_TILE;
  f.h_ld.resize(E);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up256(o + bytes); return at; };
  f.score = take(f.score_bytes);
  f.maps = take((size_t)128 * 2 * E);
  f.h_routed = take(L->n_routed > 0 ? (size_t)2 * f.max_rows_perm * f.h_ld_routed : 0);
  f.y_perm = take(L->n_routed > 0 ? sizeof(float) * (size_t)f.max_rows_perm * L->d_model : 0);
  for (int e = 0; e < E; ++e) {
    if (e < L->n_routed) { f.h_ld[e] = f.h_ld_routed; continue; }
    f.h_ld[e] = ((L->d_ff[e] + CH_TILE - 1) / CH_TILE) * CH_TILE;
    if (f.h_ld[e] == 0) f.h_ld[e] = CH_TILE;
    f.h_shared.push_back(take((size_t)2 * T * f.h_ld[e]));
    f.y_shared.push_back(take(sizeof(float) * (size_t)T * L->d_model));
  }
  f.total = o;
  return f;
}

// Which gate/up kernel the layer forward runs.  With the tokens on the accumulator rows the epilogue is short (a
// thread packs 16 micro-experts of its token into one 32-byte store) but every token tile costs 256 rows, where the
// scoring orientation trims a list's last tile to a multiple of 16 tokens; its stores of single bf16 values cost
// about a tenth of the kernel.  Token lists are taken at their average length: the routing is not known here.
bool forward_token_rows(const camera_layer_t* L, int64_t T, uint32_t flags) {
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (sms % 2 != 0) return false;
  if (flags & CAMERA_FORWARD_TOKEN_ROWS) return true;
  if (flags & (CAMERA_SCORE_CTA_PAIR | CAMERA_SCORE_SINGLE_CTA)) return false;
  const int E = L->n_routed + L->n_shared;
  double rows_tile = 0.0, cols_tile = 0.0;
  for (int e = 0; e < E; ++e) {
    const double rows = e < L->n_routed ? (double)T * L->top_k / L->n_routed : (double)T;
    const double f = (double)L->d_ff[e];
    rows_tile += ceil(rows / UMMA_TOK) * UMMA_TOK * ceil(f / UMMA_BK) * UMMA_BK;
    cols_tile += ceil(rows / ROW_ALIGN) * ROW_ALIGN * ceil(f / CH_TILE) * CH_TILE;
  }
  return rows_tile <= 1.10 * cols_tile;
}

}  // namespace
}  // namespace camera

using namespace camera;

extern "C" size_t camera_forward_workspace_bytes(const camera_layer_t* layer, int64_t n_tokens) {
  if (score_workspace_bytes_any(layer, n_tokens, true) == 0) return 0;
  return fwd_layout(layer, n_tokens).total;
}

namespace camera {
namespace {

// The second GEMM and the sum over a token's experts, on the token lists, tables and h that the workspace holds.
// w_down: per expert (HOST array of DEVICE pointers) the matrix that multiplies h.
int down_and_sum(const camera_layer_t* L, const void* const* w_down, int64_t T, float* y, const ScoreCtx& c,
                 const FwdLayout& fl, void* const* h, char* ws, bool long_lists, cudaStream_t st, Prepared* prep) {
  const int E = L->n_routed + L->n_shared;
  // rows of h per load: the pair kernel's 128 per CTA; else a tile, or less where no list can be longer (an expert
  // sees a token at most once)
  const int h_box = long_lists ? 128 : (T <= 32 ? 32 : T <= 64 ? 64 : T <= 128 ? 128 : UMMA_TOK);
  // tensor maps: per expert W_down [d_model rows, d_ff] and h [rows, h_ld].  A prepared layer keeps them on the device
  // and rebuilds them only when the workspace, the token count or the W_down matrices differ from the previous call's.
  bool cached = false;
  char* maps_dev = prep ? prepared_down_maps(prep, ws, T, h_box, w_down, &cached) : ws + fl.maps;
  if (!cached) {
    std::vector<char> maps((size_t)128 * 2 * E);
    const char* own = prep ? prepared_wdown_maps(prep, w_down) : nullptr;     // the layer's own W_down: encoded once
    for (int e = 0; e < E; ++e) {
      const int ld = L->w_down_ld ? L->w_down_ld[e] : L->d_ff[e];
      const uint64_t rows_h = e < L->n_routed ? (uint64_t)(fl.max_rows_perm > 0 ? fl.max_rows_perm : 1) : (uint64_t)T;
      if (own != nullptr) memcpy(maps.data() + (size_t)128 * (2 * e), own + (size_t)128 * e, 128);
      else if (!encode_bf16_2d_pitch(maps.data() + (size_t)128 * (2 * e), L->d_ff[e] > 0 ? w_down[e] : nullptr,
                                     (uint64_t)L->d_model, (uint64_t)L->d_ff[e], (uint64_t)ld, D_TILE))
        return CAMERA_ERR_CUDA;
      if (!encode_bf16_2d_pitch(maps.data() + (size_t)128 * (2 * e + 1), h[e], rows_h, (uint64_t)fl.h_ld[e],
                                (uint64_t)fl.h_ld[e], h_box))
        return CAMERA_ERR_CUDA;
    }
    if (prep) {
      if (upload_params(maps_dev, maps.data(), maps.size(), st) != cudaSuccess) { cudaGetLastError(); return CAMERA_ERR_CUDA; }
      prepared_down_maps_store(prep, ws, T, h_box, w_down);
    } else if (cudaMemcpyAsync(maps_dev, maps.data(), maps.size(), cudaMemcpyHostToDevice, st) != cudaSuccess) {
      cudaGetLastError();
      return CAMERA_ERR_CUDA;
    }
  }
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (long_lists) {   // whole 256-token tiles cost little: CTA pairs, tokens on the accumulator rows
    if (cudaFuncSetAttribute(k_down_umma_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, DP_SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return CAMERA_ERR_CUDA;
    }
    k_down_umma_pair<<<sms & ~1, D_THREADS, DP_SMEM_BYTES, st>>>(c, maps_dev, (L->d_model + DP_TILE - 1) / DP_TILE);
  } else {
    if (cudaFuncSetAttribute(k_down_umma, cudaFuncAttributeMaxDynamicSharedMemorySize, D_SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return CAMERA_ERR_CUDA;
    }
    const int stage_bytes = D_A_BYTES + h_box * 128;
    int n_stages = (D_STAGES * D_STAGE_BYTES) / stage_bytes;
    if (n_stages > D_MAX_STAGES) n_stages = D_MAX_STAGES;
    k_down_umma<<<sms, D_THREADS, D_SMEM_BYTES, st>>>(c, maps_dev, (L->d_model + D_TILE - 1) / D_TILE, h_box * 128, n_stages);
  }
  k_unpermute_sum<<<dim3((unsigned)T, (unsigned)((L->d_model + 1023) / 1024)), 256, 0, st>>>(c, y);
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}

// Per-expert buffers of the forward workspace and the argument checks the forward entry points share.
struct FwdSetup {
  FwdLayout fl;
  std::vector<void*> h;
  std::vector<float*> yp;
};
int forward_setup(const camera_layer_t* L, const void* x, int64_t T, const float* y, void* workspace,
                  size_t workspace_bytes, FwdSetup* s) {
  if (L == nullptr || (y == nullptr && T > 0) || (reinterpret_cast<uintptr_t>(y) & 15)) return CAMERA_ERR_INVALID_ARG;
  if (score_workspace_bytes_any(L, T, true) == 0) return CAMERA_ERR_INVALID_ARG;
  if (L->dtype != CAMERA_BF16 || L->down_layout != CAMERA_DOWN_HF || L->d_model % UMMA_BK != 0 || !umma_shape_ok(L) ||
      (reinterpret_cast<uintptr_t>(x) & 15))
    return CAMERA_ERR_UNSUPPORTED_SHAPE;
  s->fl = fwd_layout(L, T);
  const FwdLayout& fl = s->fl;
  if (workspace == nullptr || workspace_bytes < fl.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CAMERA_ERR_WORKSPACE;
  char* ws = static_cast<char*>(workspace);
  const int E = L->n_routed + L->n_shared;
  s->h.resize(E);
  s->yp.resize(E);
  for (int e = 0; e < E; ++e) {
    if (e < L->n_routed) {
      s->h[e] = ws + fl.h_routed;
      s->yp[e] = reinterpret_cast<float*>(ws + fl.y_perm);
    } else {
      s->h[e] = ws + fl.h_shared[e - L->n_routed];
      s->yp[e] = reinterpret_cast<float*>(ws + fl.y_shared[e - L->n_routed]);
    }
    if (L->w_down_ld == nullptr && L->d_ff[e] % 8 != 0) return CAMERA_ERR_UNSUPPORTED_SHAPE;   // TMA row pitch: 16 bytes
  }
  return CAMERA_OK;
}

// The layer output, and with `energy` also the scores, from one pass over W_gate and W_up.
int forward_impl(const camera_layer_t* L, const void* x, int64_t T, float alpha, float* energy, float* y,
                 const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  FwdSetup fs;
  int rc = forward_setup(L, x, T, y, workspace, workspace_bytes, &fs);
  if (rc != CAMERA_OK) return rc;
  const FwdLayout& fl = fs.fl;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  const ForwardBuffers fb{fs.h.data(), fl.h_ld.data(), fs.yp.data(), false};
  camera_score_aux_t a2;
  memset(&a2, 0, sizeof(a2));
  if (aux) {
    a2 = *aux;
    a2.flags &= ~(uint32_t)CAMERA_SCORE_FORCE_SIMT;
    if (energy == nullptr) a2.flags &= ~(uint32_t)CAMERA_SCORE_ACCUMULATE;
  }
  // the scores are sums and maxima over a micro-expert's tokens: they need the scoring orientation
  const bool long_lists = forward_token_rows(L, T, a2.flags);
  const bool token_rows = energy == nullptr && long_lists;
  if (token_rows) a2.flags = (a2.flags & ~(uint32_t)CAMERA_SCORE_SINGLE_CTA) | CAMERA_SCORE_CTA_PAIR;
  ScoreFront f;
  rc = score_front(L, x, T, alpha, energy, &a2, ws + fl.score, fl.score_bytes, st, &fb, &f);
  if (rc != CAMERA_OK) return rc;
  if (!f.use_umma) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  const ScoreCtx& c = f.c;
  if (energy != nullptr && !(a2.flags & CAMERA_SCORE_OMEGA_GIVEN) && launch_rownorm(c, f.norm_blocks, st) != cudaSuccess) {
    cudaGetLastError();
    return CAMERA_ERR_CUDA;
  }
  if (T == 0) {   // no tokens: the scores of the batches so far (or zeros), no output rows
    if (energy != nullptr && launch_combine(c, st) != cudaSuccess) { cudaGetLastError(); return CAMERA_ERR_CUDA; }
    return CAMERA_OK;
  }

  if ((f.use_pair ? launch_score_umma_pair_write_h(c, token_rows, st) : launch_score_umma_write_h(c, st)) != cudaSuccess) {
    cudaGetLastError();
    return CAMERA_ERR_CUDA;
  }
  if (energy != nullptr && launch_combine(c, st) != cudaSuccess) { cudaGetLastError(); return CAMERA_ERR_CUDA; }
  return down_and_sum(L, L->w_down, T, y, c, fl, fs.h.data(), ws, long_lists, st, f.prep);
}

}  // namespace
}  // namespace camera

extern "C" int camera_layer_forward(const camera_layer_t* L, const void* x, int64_t T, float* y,
                                    const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream) {
  return forward_impl(L, x, T, 0.f, nullptr, y, aux, workspace, workspace_bytes, cuda_stream);
}

extern "C" int camera_score_forward_layer(const camera_layer_t* L, const void* x, int64_t T, float alpha, float* energy,
                                          float* y, const camera_score_aux_t* aux, void* workspace,
                                          size_t workspace_bytes, void* cuda_stream) {
  if (energy == nullptr) return CAMERA_ERR_INVALID_ARG;
  return forward_impl(L, x, T, alpha, energy, y, aux, workspace, workspace_bytes, cuda_stream);
}

namespace camera {
namespace {

constexpr int MASK_EXPERTS = 64;    // experts per launch of k_mask_down (their pointers travel as kernel arguments)
struct MaskArgs {
  const void* src[MASK_EXPERTS];
  void* dst[MASK_EXPERTS];
  int d_ff[MASK_EXPERTS], ld[MASK_EXPERTS], me_off[MASK_EXPERTS];
};

// dst[r, i] = keep[me_off + i] ? src[r, i] : 0 for the W_down [d_model, d_ff] of the expert blockIdx.y names:
// 8 micro-experts (16 bytes of a row, 8 bytes of the mask) per thread and step.
__global__ void __launch_bounds__(256) k_mask_down(const MaskArgs a, const uint8_t* __restrict__ keep, int d_model) {
  const int e = blockIdx.y;
  const int vecs = a.d_ff[e] >> 3;
  const long long total = (long long)d_model * vecs;
  const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(a.src[e]);
  __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(a.dst[e]);
  const uint8_t* k = keep + a.me_off[e];
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(v / vecs), cv = (int)(v - (long long)r * vecs);
    uint4 w = *reinterpret_cast<const uint4*>(src + (size_t)r * a.ld[e] + 8 * cv);
    const uint2 m = *reinterpret_cast<const uint2*>(k + 8 * cv);
    auto sel = [](uint32_t word, uint32_t lo_keep, uint32_t hi_keep) {
      return (lo_keep ? word & 0x0000ffffu : 0u) | (hi_keep ? word & 0xffff0000u : 0u);
    };
    w.x = sel(w.x, m.x & 0xffu, m.x & 0xff00u);
    w.y = sel(w.y, m.x & 0xff0000u, m.x & 0xff000000u);
    w.z = sel(w.z, m.y & 0xffu, m.y & 0xff00u);
    w.w = sel(w.w, m.y & 0xff0000u, m.y & 0xff000000u);
    *reinterpret_cast<uint4*>(dst + (size_t)r * a.ld[e] + 8 * cv) = w;
  }
}

}  // namespace
}  // namespace camera

extern "C" int camera_mask_down_columns(const camera_layer_t* L, const uint8_t* keep_mask, void* const* w_down_out,
                                        void* cuda_stream) {
  if (L == nullptr || keep_mask == nullptr || w_down_out == nullptr || (reinterpret_cast<uintptr_t>(keep_mask) & 7))
    return CAMERA_ERR_INVALID_ARG;
  if (score_workspace_bytes_any(L, 0, true) == 0) return CAMERA_ERR_INVALID_ARG;
  if (L->dtype != CAMERA_BF16 || L->down_layout != CAMERA_DOWN_HF) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  const int E = L->n_routed + L->n_shared;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int me = 0;
  for (int e0 = 0; e0 < E; e0 += MASK_EXPERTS) {
    MaskArgs a;
    memset(&a, 0, sizeof(a));
    const int n = E - e0 < MASK_EXPERTS ? E - e0 : MASK_EXPERTS;
    long long most = 0;
    for (int i = 0; i < n; ++i) {
      const int e = e0 + i;
      const int ld = L->w_down_ld ? L->w_down_ld[e] : L->d_ff[e];
      if (L->d_ff[e] % 8 != 0 || ld % 8 != 0) return CAMERA_ERR_UNSUPPORTED_SHAPE;        // 16-byte pieces of a row
      if (L->d_ff[e] > 0 && (w_down_out[e] == nullptr || (reinterpret_cast<uintptr_t>(w_down_out[e]) & 15)))
        return CAMERA_ERR_INVALID_ARG;
      a.src[i] = L->w_down[e]; a.dst[i] = w_down_out[e]; a.d_ff[i] = L->d_ff[e]; a.ld[i] = ld; a.me_off[i] = me;
      me += L->d_ff[e];
      const long long v = (long long)L->d_model * (L->d_ff[e] >> 3);
      most = v > most ? v : most;
    }
    if (most == 0) continue;
    const long long blocks = (most + 255) / 256;
    k_mask_down<<<dim3((unsigned)(blocks < 1024 ? blocks : 1024), (unsigned)n), 256, 0, st>>>(a, keep_mask, L->d_model);
  }
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}

extern "C" int camera_pruned_output(const camera_layer_t* L, const void* const* w_down_masked, int64_t T, float* y_hat,
                                    const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream) {
  if (w_down_masked == nullptr) return CAMERA_ERR_INVALID_ARG;
  FwdSetup fs;
  int rc = forward_setup(L, nullptr, T, y_hat, workspace, workspace_bytes, &fs);
  if (rc != CAMERA_OK) return rc;
  for (int e = 0; e < L->n_routed + L->n_shared; ++e)
    if (L->d_ff[e] > 0 && (w_down_masked[e] == nullptr || (reinterpret_cast<uintptr_t>(w_down_masked[e]) & 15)))
      return CAMERA_ERR_INVALID_ARG;
  const FwdLayout& fl = fs.fl;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  const ForwardBuffers fb{fs.h.data(), fl.h_ld.data(), fs.yp.data(), true};
  camera_score_aux_t a2;
  memset(&a2, 0, sizeof(a2));
  if (aux) { a2 = *aux; a2.flags &= ~(uint32_t)(CAMERA_SCORE_FORCE_SIMT | CAMERA_SCORE_ACCUMULATE); }
  ScoreFront f;
  rc = score_front(L, nullptr, T, 0.f, nullptr, &a2, ws + fl.score, fl.score_bytes, st, &fb, &f);
  if (rc != CAMERA_OK) return rc;
  if (!f.use_umma) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  if (T == 0) return CAMERA_OK;
  // the work-unit counter of the second GEMM is the one thing the earlier call left used up
  if (cudaMemsetAsync(&f.c.totals->down_counter, 0, sizeof(int), st) != cudaSuccess) { cudaGetLastError(); return CAMERA_ERR_CUDA; }
  return down_and_sum(L, w_down_masked, T, y_hat, f.c, fl, fs.h.data(), ws, forward_token_rows(L, T, a2.flags), st, f.prep);
}

extern "C" size_t camera_output_error_workspace_bytes(int64_t n_tokens) {
  return n_tokens < 0 ? 0 : up256(sizeof(double) * 3 * (size_t)((n_tokens + 7) / 8 + 1));
}

extern "C" int camera_output_error(const float* y, const float* y_hat, int64_t n_tokens, int32_t d_model, double* out,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (n_tokens < 0 || d_model < 1 || out == nullptr || (n_tokens > 0 && (y == nullptr || y_hat == nullptr)))
    return CAMERA_ERR_INVALID_ARG;
  if (workspace == nullptr || workspace_bytes < camera_output_error_workspace_bytes(n_tokens) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CAMERA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  double* part = static_cast<double*>(workspace);
  const long long n_part = (n_tokens + 7) / 8;
  if (n_part > 0) k_error_partials<<<(unsigned)n_part, 256, 0, st>>>(y, y_hat, n_tokens, d_model, part);
  k_error_final<<<1, 256, 0, st>>>(part, n_part, n_tokens, out);
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}

extern "C" int camera_residual_norm(const void* x, int32_t dtype, const float* y, int64_t n_tokens, int32_t d_model, float eps,
                                    void* out, void* cuda_stream) {
  if (n_tokens < 0 || d_model < 8 || d_model % 8 != 0 || !(eps >= 0.f) || (dtype != CAMERA_BF16 && dtype != CAMERA_F32))
    return CAMERA_ERR_INVALID_ARG;
  if (n_tokens == 0) return CAMERA_OK;
  if (x == nullptr || y == nullptr || out == nullptr ||
      ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(out)) & 15))
    return CAMERA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const unsigned grid = (unsigned)((n_tokens + 7) / 8);
  if (dtype == CAMERA_BF16)
    k_residual_norm<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), y, n_tokens, d_model, eps,
                                                          static_cast<__nv_bfloat16*>(out));
  else
    k_residual_norm<float><<<grid, 256, 0, st>>>(static_cast<const float*>(x), y, n_tokens, d_model, eps, static_cast<float*>(out));
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}
