// Tensor-core router for bf16 layers (Algorithm 1: A <- Top&Norm(R X)).
//
// The logit GEMM z = X W_r^T (plus the gate logits of sigmoid-gated shared experts) runs on
// tcgen05 with tokens on the 128 TMEM lanes and experts on the columns, so X is streamed from HBM
// exactly once and every epilogue thread ends up with all logits of one token: softmax, top-k,
// normalisation and the bookkeeping of the stable counting sort need no exchange between threads.
//
// One persistent CTA per SM, 6 warps:
//   warps 0-3  epilogue: each owns 32 consecutive tokens = one block of the counting sort
//   warp  4    producer: TMA loads of the token tile (A operand) and the router rows (B operand)
//   warp  5    tensor-memory allocation and the single thread that issues tcgen05.mma
// Two accumulators alternate, so the routing of one token tile overlaps the loads of the next.
// Waits are bounded as in the scoring kernel.
#include <string.h>

#include "common.cuh"
#include "umma.cuh"

namespace camera {

namespace {

constexpr int RU_THREADS = 192;
constexpr int RU_TOK = 128;                      // tokens per tile (the MMA's M)
constexpr int RU_MAX_COLS = 128;                 // routed + gated-shared logit columns, each padded to 16
constexpr int RU_MAX_STAGES = 8;
constexpr int RU_A_BYTES = RU_TOK * 128;
constexpr int RU_TMEM_COLS = 2 * RU_MAX_COLS;
constexpr int RU_SMEM_BUDGET = 220 * 1024;
static_assert(RU_TOK == 4 * ROUTER_TOK, "one counting-sort block per epilogue warp");

struct RouterShape {
  int nr_pad, ng_pad, ncol, ldl, stage_bytes, stages, smem_bytes;
};

__host__ __device__ inline RouterShape router_shape(const ScoreCtx& c) {
  RouterShape r;
  const int n_gated = (c.flags & CAMERA_SHARED_GATE_SIGMOID) ? c.n_shared : 0;
  r.nr_pad = (c.n_routed + 15) & ~15;
  r.ng_pad = (n_gated + 15) & ~15;
  r.ncol = r.nr_pad + r.ng_pad;
  r.ldl = r.ncol + 1;
  r.stage_bytes = RU_A_BYTES + r.ncol * 128;
  const int fixed = 4 * ROUTER_TOK * r.ldl * 4 + 256 + 1024;
  int st = (RU_SMEM_BUDGET - fixed) / r.stage_bytes;
  r.stages = st > RU_MAX_STAGES ? RU_MAX_STAGES : st;
  r.smem_bytes = r.stages * r.stage_bytes + fixed;
  return r;
}

__global__ void __launch_bounds__(RU_THREADS, 1)
k_router_umma(const ScoreCtx c, const int32_t* idx_in, const float* w_in, int n_tiles) {
  extern __shared__ uint8_t smem_raw[];
  const RouterShape rs = router_shape(c);
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
  // [stages: X tile | router rows | gate rows] [logits 4 warps x 32 x ldl floats] [barriers] [tmem slot] [abort flag]
  float* const logits_all = reinterpret_cast<float*>(base_ptr + rs.stages * rs.stage_bytes);
  const int logit_bytes = 4 * ROUTER_TOK * rs.ldl * 4;
  const uint32_t bars = (base + rs.stages * rs.stage_bytes + logit_bytes + 7u) & ~7u;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (RU_MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * RU_MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * RU_MAX_STAGES + 2 + a); };
  uint8_t* const tail = base_ptr + (bars - base) + 8 * (2 * RU_MAX_STAGES + 4);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(tail + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_kb = c.d_model / UMMA_BK;

  if (tid == 0) {
    for (int s = 0; s < rs.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128); }
    wait_state_init(abort_flag, c.wait_limit_ns);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(RU_TMEM_COLS)
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
      const void* map_x = maps + (size_t)128 * (2 * c.n_experts + 2);
      const void* map_r = maps + (size_t)128 * (2 * c.n_experts + 3);
      const void* map_g = maps + (size_t)128 * (2 * c.n_experts + 4);
      tensormap_acquire(map_x);
      if (rs.nr_pad) tensormap_acquire(map_r);
      if (rs.ng_pad) tensormap_acquire(map_g);
      for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
        for (int kb = 0; kb < n_kb; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t a_dst = base + stage * rs.stage_bytes;
          mbar_expect_tx(full_bar(stage), rs.stage_bytes);
          // token rows past the tensor and weight rows past n_routed / n_shared are filled with zeros
          tma_load_2d(a_dst, map_x, full_bar(stage), kb * UMMA_BK, tile * RU_TOK);
          if (rs.nr_pad) tma_load_2d(a_dst + RU_A_BYTES, map_r, full_bar(stage), kb * UMMA_BK, 0);
          if (rs.ng_pad) tma_load_2d(a_dst + RU_A_BYTES + rs.nr_pad * 128, map_g, full_bar(stage), kb * UMMA_BK, 0);
          if (++stage == rs.stages) { stage = 0; phase ^= 1u; }
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
      const uint32_t idesc = make_idesc(rs.ncol);
      for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * RU_MAX_COLS);
        for (int kb = 0; kb < n_kb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = base + stage * rs.stage_bytes;
          const unsigned long long a_desc = make_smem_desc(a_addr);
          const unsigned long long b_desc = make_smem_desc(a_addr + RU_A_BYTES);
#pragma unroll
          for (int k = 0; k < UMMA_BK / 16; ++k)
            umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (uint32_t)((kb | k) != 0));
          umma_commit(empty_bar(stage));
          if (++stage == rs.stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3): lane = token
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    float* const row = logits_all + (size_t)(warp * ROUTER_TOK + lane) * rs.ldl;   // this token's logits
    const int k = c.top_k;
    const int n_gated = (c.flags & CAMERA_SHARED_GATE_SIGMOID) ? c.n_shared : 0;
    for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
      ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(acc * RU_MAX_COLS);
      for (int c0 = 0; c0 < rs.ncol; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(taddr + c0, v);
        tmem_ld_wait(v);
#pragma unroll
        for (int j = 0; j < 16; ++j) row[c0 + j] = __uint_as_float(v[j]);
      }
      tc_fence_before();
      mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }

      const int blk = tile * (RU_TOK / ROUTER_TOK) + warp;   // counting-sort block of this warp
      const int t = blk * ROUTER_TOK + lane;
      const bool live = t < c.n_tokens;
      if (blk >= c.n_blocks) continue;

      // coefficients of the shared experts: 1, or sigmoid of their gate logit
      if (live) {
        for (int s = 0; s < c.n_shared; ++s) {
          float a = 1.f;
          if (n_gated) a = 1.f / (1.f + expf(-row[rs.nr_pad + s]));
          c.shared_w[(size_t)s * c.shared_ld + t] = a;
        }
      }
      if (c.n_routed == 0) continue;

      int my_e[MAX_TOPK];
#pragma unroll
      for (int s = 0; s < MAX_TOPK; ++s) my_e[s] = -1;
      if (live) {
        float my_p[MAX_TOPK];
        bool bad = false;     // a routing that cannot be used: see the safe pairs below
        if (idx_in != nullptr) {
#pragma unroll
          for (int s = 0; s < MAX_TOPK; ++s) {
            my_p[s] = 0.f;
            if (s < k) {
              my_e[s] = idx_in[(size_t)t * k + s];
              my_p[s] = w_in[(size_t)t * k + s];
              bad = bad || my_e[s] < 0 || my_e[s] >= c.n_routed;
            }
          }
          // a prescribed routing names k distinct experts per token (the ranks below count a token once per expert)
#pragma unroll
          for (int s = 1; s < MAX_TOPK; ++s)
#pragma unroll
            for (int r = 0; r < s; ++r)
              if (s < k && my_e[s] == my_e[r]) bad = true;
        } else {
          float zmax = -INFINITY;
          for (int j = 0; j < c.n_routed; ++j) {
            const float z = row[j] + (c.router_bias ? c.router_bias[j] : 0.f);
            row[j] = z;
            zmax = fmaxf(zmax, z);
          }
          float den = 0.f;
          for (int j = 0; j < c.n_routed; ++j) den += expf(row[j] - zmax);
          // a NaN or +inf logit (a NaN or inf in x or in the router) leaves no softmax to take
          bad = !(den > 0.f) || !isfinite(den);
          float chosen = 0.f;
#pragma unroll
          for (int s = 0; s < MAX_TOPK; ++s) {
            my_p[s] = 0.f;
            if (s < k) {
              float best = -INFINITY;
              int bi = -1;
              for (int j = 0; j < c.n_routed; ++j) {     // strict >: equal logits go to the lower expert
                const float z = row[j];
                if (z > best) { best = z; bi = j; }
              }
              if (bi < 0) { bad = true; bi = 0; }        // fewer than k logits above -inf
              row[bi] = -INFINITY;
              my_e[s] = bi;
              my_p[s] = expf(best - zmax) / den;
              chosen += my_p[s];
            }
          }
          if (c.flags & CAMERA_ROUTER_NORM_TOPK) {
#pragma unroll
            for (int s = 0; s < MAX_TOPK; ++s) my_p[s] /= chosen;
          }
        }
        if (bad) {
          // unusable routing: record it and give the token k distinct experts with coefficient 0, so that every
          // later index stays in range and every pair gets its rank
          atomicExch(&c.totals->status, (int)CAMERA_ERR_INVALID_ARG);
#pragma unroll
          for (int s = 0; s < MAX_TOPK; ++s) { my_e[s] = s < k ? s : -1; my_p[s] = 0.f; }
        }
#pragma unroll
        for (int s = 0; s < MAX_TOPK; ++s) {
          if (s < k) {
            c.topk_idx[(size_t)t * k + s] = my_e[s];
            c.topk_w[(size_t)t * k + s] = my_p[s];
          }
        }
      }
      // rank of each pair among the pairs of the same expert in this block, in (token, slot) order:
      // a token names an expert at most once, so it is the number of lower tokens that chose it
      for (int e = 0; e < c.n_routed; ++e) {
        int slot = -1;
#pragma unroll
        for (int s = 0; s < MAX_TOPK; ++s)
          if (my_e[s] == e) slot = s;
        const unsigned mask = __ballot_sync(0xffffffffu, slot >= 0);
        if (slot >= 0) c.local_rank[(size_t)t * k + slot] = __popc(mask & ((1u << lane) - 1u));
        if (lane == 0) c.block_hist[(size_t)blk * c.n_routed + e] = __popc(mask);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag && tid == 0) atomicExch(&c.totals->status, (int)CAMERA_ERR_DEVICE_TIMEOUT);
  if (warp == 5) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(RU_TMEM_COLS) : "memory");
  }
}

}  // namespace

bool router_umma_ok(const ScoreCtx& c) {
  if (c.dtype != CAMERA_BF16 || c.d_model % UMMA_BK != 0 || c.n_tokens <= 0) return false;
  const RouterShape rs = router_shape(c);
  return rs.ncol >= 16 && rs.ncol <= RU_MAX_COLS && rs.stages >= 2;
}

// Tensor maps of the router: x in boxes of 128 token rows, the router rows and the shared-gate rows
// in one box each (rows past the tensor read as zero).
int encode_router_maps(const ScoreCtx& c, void* host_maps, int which) {
  const RouterShape rs = router_shape(c);
  char* out = static_cast<char*>(host_maps) + (size_t)128 * (2 * c.n_experts + 2);
  if ((which & MAPS_TOKENS) && !encode_bf16_2d(out, c.x, (uint64_t)c.n_tokens, (uint64_t)c.d_model, RU_TOK)) return CAMERA_ERR_CUDA;
  if (!(which & MAPS_STATIC)) return CAMERA_OK;
  if (!encode_bf16_2d(out + 128, rs.nr_pad ? c.w_router : nullptr, (uint64_t)c.n_routed, (uint64_t)c.d_model, rs.nr_pad))
    return CAMERA_ERR_CUDA;
  if (!encode_bf16_2d(out + 256, rs.ng_pad ? c.w_shared_gate : nullptr, (uint64_t)c.n_shared, (uint64_t)c.d_model, rs.ng_pad))
    return CAMERA_ERR_CUDA;
  return CAMERA_OK;
}

cudaError_t launch_router_umma(const ScoreCtx& c, const int32_t* idx_in, const float* w_in, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const RouterShape rs = router_shape(c);
  const int n_tiles = (c.n_tokens + RU_TOK - 1) / RU_TOK;
  cudaError_t e = cudaFuncSetAttribute(k_router_umma, cudaFuncAttributeMaxDynamicSharedMemorySize, rs.smem_bytes);
  if (e != cudaSuccess) return e;
  k_router_umma<<<n_tiles < sms ? n_tiles : sms, RU_THREADS, rs.smem_bytes, st>>>(c, idx_in, w_in, n_tiles);
  return cudaGetLastError();
}

}  // namespace camera
