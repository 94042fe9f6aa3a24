// Router (Algorithm 1: A <- Top&Norm(R X)), the stable counting sort of (token, expert)
// pairs by expert, and the token permutation that lays every expert's tokens out contiguously.
#include "common.cuh"

namespace camera {

namespace {

constexpr int RT_THREADS = 256;
constexpr int RT_TOK = 64;           // tokens per CTA = RT_TOK / ROUTER_TOK blocks of the counting sort
constexpr int RT_KC = 32;            // k-chunk of the logit GEMM
constexpr int RT_COLS = 64;          // logit columns per pass
constexpr int RT_LD = RT_TOK + 4;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One token's routing, by one warp: softmax over the routed logits and the top_k largest (equal logits: lower expert
// first), or the prescribed routing after its checks.  row: the token's logits [n_routed ...] (shared or global
// memory).  Lane s < top_k returns slot s in (my_e, my_p).  A routing that cannot be used (see the status word's
// description) is recorded and replaced by k distinct experts with coefficient 0, so that every later index stays in
// range.
__device__ __forceinline__ void route_token(const ScoreCtx& c, const int32_t* idx_in, const float* w_in, const float* row,
                                            int t, int lane, int& my_e, float& my_p) {
  const int k = c.top_k;
  my_e = 0;
  my_p = 0.f;
  bool bad = false;
  if (idx_in != nullptr) {
    if (lane < k) {
      my_e = idx_in[(size_t)t * k + lane];
      my_p = w_in[(size_t)t * k + lane];
      bad = my_e < 0 || my_e >= c.n_routed;
    }
    // a prescribed routing names k distinct experts per token
    for (int s = 0; s < k; ++s) {
      const int other = __shfl_sync(0xffffffffu, my_e, s);
      if (lane < k && lane != s && other == my_e) bad = true;
    }
  } else {
    float v[MAX_ROUTED / 32];
#pragma unroll
    for (int i = 0; i < MAX_ROUTED / 32; ++i) {
      const int col = lane + 32 * i;
      v[i] = -INFINITY;
      if (col < c.n_routed) v[i] = row[col] + (c.router_bias ? c.router_bias[col] : 0.f);
    }
    float zmax = -INFINITY;
#pragma unroll
    for (int i = 0; i < MAX_ROUTED / 32; ++i) zmax = fmaxf(zmax, v[i]);
    zmax = warp_max(zmax);
    float den = 0.f;
#pragma unroll
    for (int i = 0; i < MAX_ROUTED / 32; ++i) den += (lane + 32 * i < c.n_routed) ? expf(v[i] - zmax) : 0.f;
    den = warp_sum(den);
    // a NaN or +inf logit (a NaN or inf in x or in the router) leaves no softmax to take
    bad = !(den > 0.f) || !isfinite(den);
    float chosen = 0.f;
    for (int s = 0; s < k; ++s) {
      float best = -INFINITY;
      int bi = 0x7fffffff;
#pragma unroll
      for (int i = 0; i < MAX_ROUTED / 32; ++i)
        if (v[i] > best) { best = v[i]; bi = lane + 32 * i; }
#pragma unroll
      for (int o = 16; o; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
      }
      if (bi >= c.n_routed) bad = true;     // fewer than k logits above -inf
      const float p = expf(best - zmax) / den;
#pragma unroll
      for (int i = 0; i < MAX_ROUTED / 32; ++i)
        if (lane + 32 * i == bi) v[i] = -INFINITY;
      if (lane == s) { my_e = bi; my_p = p; }
      chosen += p;
    }
    if (c.flags & CAMERA_ROUTER_NORM_TOPK) my_p /= chosen;
  }
  if (__any_sync(0xffffffffu, bad)) {
    if (lane == 0) atomicExch(&c.totals->status, (int)CAMERA_ERR_INVALID_ARG);
    my_e = lane < c.n_routed ? lane : 0;
    my_p = 0.f;
  }
}

// One block of the counting sort (ROUTER_TOK tokens), by all warps of a CTA: the rank of each (token, slot) pair among
// the pairs of the same expert in the block, in (token, slot) order, and the block's per-expert histogram.
// sel_b: shared memory [ROUTER_TOK * top_k], the pairs' experts (-1 past the last token).
__device__ __forceinline__ void rank_block(const ScoreCtx& c, const int* sel_b, int blk) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const int npairs = ROUTER_TOK * c.top_k;
  int32_t* rank_b = c.local_rank + (size_t)blk * ROUTER_TOK * c.top_k;
  for (int e = warp; e < c.n_routed; e += n_warps) {
    int run = 0;
    for (int base = 0; base < npairs; base += 32) {
      const int p = base + lane;
      const bool m = (p < npairs) && (sel_b[p] == e);
      const unsigned b = __ballot_sync(0xffffffffu, m);
      if (m) rank_b[p] = run + __popc(b & ((1u << lane) - 1u));
      run += __popc(b);
    }
    if (lane == 0) c.block_hist[(size_t)blk * c.n_routed + e] = run;
  }
}

// What follows the logits of RT_TOK consecutive tokens (group `group` of the call): the shared experts' coefficients,
// the tokens' routing, and the bookkeeping of the counting sort.  logits: shared memory [RT_TOK][ldl]; sel_e: shared
// memory [RT_TOK * top_k].  Called by all RT_THREADS threads of a CTA.
__device__ void router_tail(const ScoreCtx& c, const int32_t* idx_in, const float* w_in, const float* logits, int ldl,
                            int group, int* sel_e) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_gated = (c.flags & CAMERA_SHARED_GATE_SIGMOID) ? c.n_shared : 0;
  const int tok0 = group * RT_TOK;
  // coefficients of the shared experts: 1, or sigmoid of their gate logit
  for (int i = tid; i < RT_TOK * c.n_shared; i += RT_THREADS) {
    const int s = i / RT_TOK, tl = i % RT_TOK, t = tok0 + tl;
    if (t < c.n_tokens) {
      float a = 1.f;
      if (n_gated) a = 1.f / (1.f + expf(-logits[tl * ldl + c.n_routed + s]));
      c.shared_w[(size_t)s * c.shared_ld + t] = a;
    }
  }
  const int k = c.top_k;
  if (c.n_routed > 0) {
    for (int tl = warp; tl < RT_TOK; tl += RT_THREADS / 32) {
      const int t = tok0 + tl;
      if (t >= c.n_tokens) {
        if (lane < k) sel_e[tl * k + lane] = -1;
        continue;
      }
      int my_e;
      float my_p;
      route_token(c, idx_in, w_in, logits + tl * ldl, t, lane, my_e, my_p);
      if (lane < k) {
        c.topk_idx[(size_t)t * k + lane] = my_e;
        c.topk_w[(size_t)t * k + lane] = my_p;
        sel_e[tl * k + lane] = my_e;
      }
    }
    __syncthreads();
    for (int sb = 0; sb < RT_TOK / ROUTER_TOK; ++sb) {
      const int blk = group * (RT_TOK / ROUTER_TOK) + sb;
      if (blk >= c.n_blocks) break;
      rank_block(c, sel_e + sb * ROUTER_TOK * k, blk);
    }
  }
}


// One CTA = RT_TOK consecutive tokens.  Logits z = x . w (+bias) in fp32 FMA over all routed
// experts and the sigmoid-gated shared experts; softmax over the routed ones; the top_k largest
// logits are kept (equal logits: lower expert first); weights are the softmax probabilities,
// divided by their sum under CAMERA_ROUTER_NORM_TOPK.  Also emits, for the counting sort, each
// pair's rank among the same expert's pairs of this block and the block's per-expert histogram.
template <typename T>
__global__ void __launch_bounds__(RT_THREADS) k_router(ScoreCtx c, const int32_t* idx_in, const float* w_in) {
  extern __shared__ float smem[];
  const int n_gated = (c.flags & CAMERA_SHARED_GATE_SIGMOID) ? c.n_shared : 0;
  const int nc = c.n_routed + n_gated;
  const int nc_pad = ((nc + RT_COLS - 1) / RT_COLS) * RT_COLS;
  const int ldl = nc_pad + 1;
  float* Xs = smem;                              // [RT_KC][RT_LD]
  float* Ws = Xs + RT_KC * RT_LD;                // [RT_KC][RT_LD]
  float* logits = Ws + RT_KC * RT_LD;            // [RT_TOK][ldl]
  int* sel_e = reinterpret_cast<int*>(logits + RT_TOK * ldl);  // [RT_TOK * top_k]

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int tok0 = blockIdx.x * RT_TOK;
  const int d = c.d_model;
  const T* X = static_cast<const T*>(c.x);
  constexpr int VN = Vec16<T>::N;
  constexpr int VPR = RT_KC / VN;                // vectors per row of a k-chunk

  for (int col0 = 0; col0 < nc_pad; col0 += RT_COLS) {
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < d; k0 += RT_KC) {
      __syncthreads();
      for (int v = tid; v < RT_TOK * VPR; v += RT_THREADS) {
        const int row = v / VPR, kv = (v % VPR) * VN;
        float f[VN];
#pragma unroll
        for (int i = 0; i < VN; ++i) f[i] = 0.f;
        const int t = tok0 + row;
        if (t < c.n_tokens && k0 + kv < d) Vec16<T>::load(X + (size_t)t * d + k0 + kv, f);
#pragma unroll
        for (int i = 0; i < VN; ++i) Xs[(kv + i) * RT_LD + row] = f[i];
      }
      for (int v = tid; v < RT_COLS * VPR; v += RT_THREADS) {
        const int row = v / VPR, kv = (v % VPR) * VN;
        float f[VN];
#pragma unroll
        for (int i = 0; i < VN; ++i) f[i] = 0.f;
        const int col = col0 + row;
        if (col < nc && k0 + kv < d) {
          const T* wrow = col < c.n_routed
              ? static_cast<const T*>(c.w_router) + (size_t)col * d
              : static_cast<const T*>(c.w_shared_gate) + (size_t)(col - c.n_routed) * d;
          Vec16<T>::load(wrow + k0 + kv, f);
        }
#pragma unroll
        for (int i = 0; i < VN; ++i) Ws[(kv + i) * RT_LD + row] = f[i];
      }
      __syncthreads();
#pragma unroll 8
      for (int k = 0; k < RT_KC; ++k) {
        const float4 a = *reinterpret_cast<const float4*>(Xs + k * RT_LD + ty * 4);
        const float4 b = *reinterpret_cast<const float4*>(Ws + k * RT_LD + tx * 4);
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) logits[(ty * 4 + i) * ldl + col0 + tx * 4 + j] = acc[i][j];
  }
  __syncthreads();

  router_tail(c, idx_in, w_in, logits, ldl, blockIdx.x, sel_e);
}

// One CTA per routed expert: exclusive scan of its per-block counts over the blocks (in place).
__global__ void __launch_bounds__(256) k_block_scan(ScoreCtx c) {
  __shared__ int wsum[8];
  __shared__ int chunk_total;
  const int e = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int run = 0;
  for (int base = 0; base < c.n_blocks; base += 256) {
    const int b = base + tid;
    const int v = b < c.n_blocks ? c.block_hist[(size_t)b * c.n_routed + e] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    int woff = 0;
    for (int w = 0; w < warp; ++w) woff += wsum[w];
    if (tid == 255) chunk_total = woff + incl;
    if (b < c.n_blocks) c.block_hist[(size_t)b * c.n_routed + e] = run + woff + incl - v;
    __syncthreads();
    run += chunk_total;
  }
  if (tid == 0) c.counts[e] = run;
}

// One warp: lays the experts' token lists out back to back (each padded to ROW_ALIGN rows) and numbers the scoring
// work units and partial slots.  A lane takes an expert; the running offsets are warp scans.
__device__ void plan_body(const ScoreCtx& c, int lane) {
  int row = 0, units = 0, chunks = 0;
  long long part = 0;
  for (int base = 0; base < c.n_experts; base += 32) {
    const int e = base + lane;
    const bool valid = e < c.n_experts, routed = e < c.n_routed;
    const int rows = valid ? (routed ? c.counts[e] : c.n_tokens) : 0;
    const int f = valid ? c.est[e].d_ff : 0;
    const int n_chunks = (rows + c.chunk_tokens - 1) / c.chunk_tokens;
    // what this expert adds to the four running offsets, then inclusive scans over the 32 lanes
    int a_row = valid && routed ? (rows + ROW_ALIGN - 1) / ROW_ALIGN * ROW_ALIGN : 0;
    int a_units = n_chunks * ((f + c.ch_tile - 1) / c.ch_tile), a_chunks = n_chunks;
    long long a_part = (long long)n_chunks * f;
    int s_row = a_row, s_units = a_units, s_chunks = a_chunks;
    long long s_part = a_part;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t_row = __shfl_up_sync(0xffffffffu, s_row, o), t_units = __shfl_up_sync(0xffffffffu, s_units, o);
      const int t_chunks = __shfl_up_sync(0xffffffffu, s_chunks, o);
      const long long t_part = __shfl_up_sync(0xffffffffu, s_part, o);
      if (lane >= o) { s_row += t_row; s_units += t_units; s_chunks += t_chunks; s_part += t_part; }
    }
    if (valid) {
      ExpertDyn dy;
      dy.rows = rows;
      dy.row_base = routed ? row + s_row - a_row : 0;
      dy.n_chunks = n_chunks;
      dy.unit_begin = units + s_units - a_units;
      dy.part_begin = part + s_part - a_part;
      dy.chunk_begin = chunks + s_chunks - a_chunks;
      dy.pad = 0;
      c.edyn[e] = dy;
      c.unit_prefix[e] = dy.unit_begin;
      if (!routed) c.counts[e] = c.n_tokens;
    }
    row += __shfl_sync(0xffffffffu, s_row, 31);
    units += __shfl_sync(0xffffffffu, s_units, 31);
    chunks += __shfl_sync(0xffffffffu, s_chunks, 31);
    part += __shfl_sync(0xffffffffu, s_part, 31);
  }
  if (row > c.max_rows_perm || part > c.max_part) {   // cannot happen with a workspace of the size the query gives
    if (lane == 0) atomicExch(&c.totals->status, (int)CAMERA_ERR_WORKSPACE);
    units = 0;
    chunks = 0;
    __syncwarp();
    for (int e = lane; e < c.n_experts; e += 32) {
      c.unit_prefix[e] = 0;
      c.edyn[e].n_chunks = 0; c.edyn[e].rows = 0; c.edyn[e].chunk_begin = 0;
    }
  }
  if (lane == 0) {
    c.unit_prefix[c.n_experts] = units;
    c.totals->total_units = units;
    c.totals->total_rows = row;
    c.totals->total_chunks = chunks;
    c.totals->unit_counter = 0;
    c.totals->down_counter = 0;
  }
}

__global__ void __launch_bounds__(32) k_plan(ScoreCtx c) { plan_body(c, threadIdx.x); }

// ---- small batches (a decode step): the same routing, token lists and plan from three launches that spread the
// logit sums over the GPU, instead of five whose first runs on one SM --------------------------------------------
constexpr int RS_MAX_TOK = 128;      // tokens such a call may have
constexpr int RS_MAX_COLS = 128;     // logit columns (routed experts + gated shared experts)
constexpr int RS_WARPS = 4;          // warps per CTA of the logit kernel: they split d_model between them
constexpr int RS_TOK = 2, RS_COLS = 8;   // a CTA's share: the logits of RS_TOK tokens x RS_COLS columns

// Logits of a small batch: a CTA forms the full-length dot products of RS_TOK tokens with RS_COLS router rows (its
// warps take every RS_WARPS-th piece of d_model, lanes stride a piece; fp32 FMA, a shuffle tree, then the warps' sums
// in order), so the few hundred KB of tokens and router rows are read by every SM at once instead of streaming
// through one.  logits: [n_tokens][nc_ld] fp32.
template <typename T>
__global__ void __launch_bounds__(32 * RS_WARPS) k_router_logits_small(ScoreCtx c, float* __restrict__ logits, int nc, int nc_ld) {
  constexpr int VN = Vec16<T>::N;
  __shared__ float red[RS_WARPS][RS_TOK * RS_COLS];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_cg = (nc + RS_COLS - 1) / RS_COLS;
  const int t0 = ((int)blockIdx.x / n_cg) * RS_TOK, c0 = ((int)blockIdx.x % n_cg) * RS_COLS;
  const int d = c.d_model;
  const T* X = static_cast<const T*>(c.x);
  const T* wrow[RS_COLS];
#pragma unroll
  for (int j = 0; j < RS_COLS; ++j) {
    const int col = min(c0 + j, nc - 1);          // columns past the last repeat it; their sums are not written
    wrow[j] = col < c.n_routed ? static_cast<const T*>(c.w_router) + (size_t)col * d
                               : static_cast<const T*>(c.w_shared_gate) + (size_t)(col - c.n_routed) * d;
  }
  float acc[RS_TOK][RS_COLS];
#pragma unroll
  for (int i = 0; i < RS_TOK; ++i)
#pragma unroll
    for (int j = 0; j < RS_COLS; ++j) acc[i][j] = 0.f;
  for (int k = (warp * 32 + lane) * VN; k < d; k += RS_WARPS * 32 * VN) {
    float xv[RS_TOK][VN];
#pragma unroll
    for (int i = 0; i < RS_TOK; ++i) Vec16<T>::load(X + (size_t)min(t0 + i, c.n_tokens - 1) * d + k, xv[i]);
#pragma unroll
    for (int j = 0; j < RS_COLS; ++j) {
      float wv[VN];
      Vec16<T>::load(wrow[j] + k, wv);
#pragma unroll
      for (int q = 0; q < VN; ++q)
#pragma unroll
        for (int i = 0; i < RS_TOK; ++i) acc[i][j] = fmaf(xv[i][q], wv[q], acc[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < RS_TOK; ++i)
#pragma unroll
    for (int j = 0; j < RS_COLS; ++j) {
      float v = acc[i][j];
#pragma unroll
      for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) red[warp][i * RS_COLS + j] = v;
    }
  __syncthreads();
  if (threadIdx.x < RS_TOK * RS_COLS) {
    const int i = threadIdx.x / RS_COLS, j = threadIdx.x % RS_COLS;
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < RS_WARPS; ++w) v += red[w][threadIdx.x];
    if (t0 + i < c.n_tokens && c0 + j < nc) logits[(size_t)(t0 + i) * nc_ld + c0 + j] = v;
  }
}

// A warp per token: the shared experts' coefficients and the token's routing from its logits (global memory).
__global__ void __launch_bounds__(RT_THREADS)
k_route_tokens_small(ScoreCtx c, const int32_t* idx_in, const float* w_in, const float* __restrict__ lg, int nc_ld) {
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (RT_THREADS / 32) + (threadIdx.x >> 5);
  if (t >= c.n_tokens) return;
  const float* row = lg + (size_t)t * nc_ld;
  const bool gated = (c.flags & CAMERA_SHARED_GATE_SIGMOID) != 0;
  for (int s = lane; s < c.n_shared; s += 32)
    c.shared_w[(size_t)s * c.shared_ld + t] = gated ? 1.f / (1.f + expf(-row[c.n_routed + s])) : 1.f;
  if (c.n_routed == 0) return;
  int my_e;
  float my_p;
  route_token(c, idx_in, w_in, row, t, lane, my_e, my_p);
  if (lane < c.top_k) {
    c.topk_idx[(size_t)t * c.top_k + lane] = my_e;
    c.topk_w[(size_t)t * c.top_k + lane] = my_p;
  }
}

// One CTA: for all tokens what k_router's last part, k_block_scan and k_plan do (there are at most
// RS_MAX_TOK / ROUTER_TOK blocks of the counting sort).  With so few pairs a thread finds its pair's rank by looking
// at the pairs before it in the block.
__global__ void __launch_bounds__(RT_THREADS) k_rank_plan_small(ScoreCtx c) {
  __shared__ int sel_e[RS_MAX_TOK * MAX_TOPK];
  __shared__ int hist[(RS_MAX_TOK / ROUTER_TOK) * MAX_ROUTED];
  const int tid = threadIdx.x, k = c.top_k;
  if (c.n_routed > 0) {
    const int n_pairs = c.n_tokens * k, per_block = ROUTER_TOK * k;
    for (int i = tid; i < n_pairs; i += RT_THREADS) sel_e[i] = c.topk_idx[i];
    for (int i = tid; i < c.n_blocks * c.n_routed; i += RT_THREADS) hist[i] = 0;
    __syncthreads();
    for (int p = tid; p < n_pairs; p += RT_THREADS) {
      const int blk = p / per_block, e = sel_e[p];
      int rank = 0;
      for (int q = blk * per_block; q < p; ++q) rank += sel_e[q] == e;
      c.local_rank[p] = rank;
      atomicAdd(&hist[blk * c.n_routed + e], 1);
    }
    __syncthreads();
    // exclusive scan of every routed expert's per-block counts over the blocks, as k_block_scan
    for (int e = tid; e < c.n_routed; e += RT_THREADS) {
      int run = 0;
      for (int b = 0; b < c.n_blocks; ++b) {
        c.block_hist[(size_t)b * c.n_routed + e] = run;
        run += hist[b * c.n_routed + e];
      }
      c.counts[e] = run;
    }
    __syncthreads();
  }
  if (tid < 32) plan_body(c, tid);
}

// Token t's row to its place in each of its experts' lists, one CTA per token (a row is a few KB: its pieces are
// copied side by side instead of one after the other); the CTAs past the tokens pad the routed experts' lists.
__global__ void __launch_bounds__(RT_THREADS) k_permute_small(ScoreCtx c, int row_bytes) {
  __shared__ int pos[MAX_TOPK];
  const int nvec = row_bytes / 16, k = c.top_k;
  if ((int)blockIdx.x >= c.n_tokens) {
    const ExpertDyn dy = c.edyn[blockIdx.x - c.n_tokens];
    const int end = (dy.rows + ROW_ALIGN - 1) / ROW_ALIGN * ROW_ALIGN;
    for (int r = dy.rows; r < end; ++r) {
      const size_t row = (size_t)dy.row_base + r;
      uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(c.x_perm) + row * row_bytes);
      for (int v = threadIdx.x; v < nvec; v += blockDim.x) dst[v] = make_uint4(0, 0, 0, 0);
      if (threadIdx.x == 0) c.perm_w[row] = 0.f;
    }
    return;
  }
  const int t = blockIdx.x;
  if ((int)threadIdx.x < k) {
    const int e = c.topk_idx[(size_t)t * k + threadIdx.x];
    int p = -1;
    if (e >= 0 && e < c.n_routed) {
      p = c.edyn[e].row_base + c.block_hist[(size_t)(t / ROUTER_TOK) * c.n_routed + e] + c.local_rank[(size_t)t * k + threadIdx.x];
      if (p < 0 || p >= c.max_rows_perm) p = -1;
    }
    if (p >= 0) c.perm_w[p] = c.topk_w[(size_t)t * k + threadIdx.x];
    else atomicExch(&c.totals->status, (int)CAMERA_ERR_INVALID_ARG);
    pos[threadIdx.x] = p;
  }
  __syncthreads();
  const uint4* src = reinterpret_cast<const uint4*>(static_cast<const char*>(c.x) + (size_t)t * row_bytes);
  for (int v = threadIdx.x; v < nvec; v += RT_THREADS) {
    const uint4 val = __ldg(src + v);
    for (int s = 0; s < k; ++s)
      if (pos[s] >= 0) reinterpret_cast<uint4*>(static_cast<char*>(c.x_perm) + (size_t)pos[s] * row_bytes)[v] = val;
  }
}

// One warp per token: copies the token's hidden state to its row in every chosen expert's list.
__global__ void __launch_bounds__(256) k_permute(ScoreCtx c, int row_bytes) {
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= c.n_tokens) return;
  const int k = c.top_k;
  int pos_l = 0;
  if (lane < k) {
    const int e = c.topk_idx[(size_t)t * k + lane];
    pos_l = -1;
    if (e >= 0 && e < c.n_routed) {
      pos_l = c.edyn[e].row_base + c.block_hist[(size_t)(t / ROUTER_TOK) * c.n_routed + e] +
              c.local_rank[(size_t)t * k + lane];
      if (pos_l < 0 || pos_l >= c.max_rows_perm) pos_l = -1;
    }
    // the routers only write pairs that pass this; a pair that does not is skipped and reported, never written
    if (pos_l >= 0) c.perm_w[pos_l] = c.topk_w[(size_t)t * k + lane];
    else atomicExch(&c.totals->status, (int)CAMERA_ERR_INVALID_ARG);
  }
  int pos[MAX_TOPK];
#pragma unroll
  for (int s = 0; s < MAX_TOPK; ++s) pos[s] = __shfl_sync(0xffffffffu, pos_l, s);
  const uint4* src = reinterpret_cast<const uint4*>(static_cast<const char*>(c.x) + (size_t)t * row_bytes);
  const int nvec = row_bytes / 16;
  for (int v = lane; v < nvec; v += 32) {
    const uint4 val = __ldg(src + v);
#pragma unroll
    for (int s = 0; s < MAX_TOPK; ++s)
      if (s < k && pos[s] >= 0)
        reinterpret_cast<uint4*>(static_cast<char*>(c.x_perm) + (size_t)pos[s] * row_bytes)[v] = val;
  }
}

// One CTA per routed expert: zero rows and zero weights for the padding behind its token list.
__global__ void __launch_bounds__(128) k_pad_rows(ScoreCtx c, int row_bytes) {
  const ExpertDyn dy = c.edyn[blockIdx.x];
  const int end = (dy.rows + ROW_ALIGN - 1) / ROW_ALIGN * ROW_ALIGN;
  const int nvec = row_bytes / 16;
  for (int r = dy.rows; r < end; ++r) {
    const size_t row = (size_t)dy.row_base + r;
    uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(c.x_perm) + row * row_bytes);
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) dst[v] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) c.perm_w[row] = 0.f;
  }
}

size_t router_smem_bytes(const ScoreCtx& c) {
  const int n_gated = (c.flags & CAMERA_SHARED_GATE_SIGMOID) ? c.n_shared : 0;
  const int nc = c.n_routed + n_gated;
  const int nc_pad = ((nc + RT_COLS - 1) / RT_COLS) * RT_COLS;
  return sizeof(float) * (2 * RT_KC * RT_LD + RT_TOK * (nc_pad + 1)) + sizeof(int) * RT_TOK * MAX_TOPK;
}

}  // namespace

cudaError_t launch_routing_from_input(const ScoreCtx& c, const int32_t* idx_in, const float* w_in, cudaStream_t st) {
  if (c.n_blocks == 0) return cudaSuccess;
  const size_t smem = router_smem_bytes(c);
  const int grid = (c.n_tokens + RT_TOK - 1) / RT_TOK;
  if (c.dtype == CAMERA_BF16) {
    cudaError_t e = cudaFuncSetAttribute(k_router<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_router<__nv_bfloat16><<<grid, RT_THREADS, smem, st>>>(c, idx_in, w_in);
  } else {
    cudaError_t e = cudaFuncSetAttribute(k_router<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_router<float><<<grid, RT_THREADS, smem, st>>>(c, idx_in, w_in);
  }
  return cudaGetLastError();
}

cudaError_t launch_router(const ScoreCtx& c, cudaStream_t st) {
  return launch_routing_from_input(c, nullptr, nullptr, st);
}

bool front_small_ok(const ScoreCtx& c) {
  const int n_gated = (c.flags & CAMERA_SHARED_GATE_SIGMOID) ? c.n_shared : 0;
  const int nc = c.n_routed + n_gated;
  return c.n_tokens > 0 && c.n_tokens <= RS_MAX_TOK && nc >= 1 && nc <= RS_MAX_COLS;
}

size_t front_small_scratch_bytes(int d_model, int64_t n_tokens) {
  (void)d_model;
  if (n_tokens <= 0 || n_tokens > RS_MAX_TOK) return 0;
  return sizeof(float) * (size_t)n_tokens * RS_MAX_COLS;
}

// Router, counting sort and plan of a small batch.
cudaError_t launch_route_small(const ScoreCtx& c, const int32_t* idx_in, const float* w_in, float* scratch, cudaStream_t st) {
  const int n_gated = (c.flags & CAMERA_SHARED_GATE_SIGMOID) ? c.n_shared : 0;
  const int nc = c.n_routed + n_gated, nc_ld = (nc + 3) & ~3;
  const bool need_logits = n_gated > 0 || (c.n_routed > 0 && idx_in == nullptr);
  if (need_logits) {
    const int grid = ((c.n_tokens + RS_TOK - 1) / RS_TOK) * ((nc + RS_COLS - 1) / RS_COLS);
    if (c.dtype == CAMERA_BF16) k_router_logits_small<__nv_bfloat16><<<grid, 32 * RS_WARPS, 0, st>>>(c, scratch, nc, nc_ld);
    else k_router_logits_small<float><<<grid, 32 * RS_WARPS, 0, st>>>(c, scratch, nc, nc_ld);
  }
  const int per_cta = RT_THREADS / 32;
  k_route_tokens_small<<<(c.n_tokens + per_cta - 1) / per_cta, RT_THREADS, 0, st>>>(c, idx_in, w_in, scratch, nc_ld);
  k_rank_plan_small<<<1, RT_THREADS, 0, st>>>(c);
  return cudaGetLastError();
}

cudaError_t launch_permute_small(const ScoreCtx& c, cudaStream_t st) {
  if (c.n_routed == 0 || c.n_tokens == 0) return cudaSuccess;
  const int row_bytes = c.d_model * (c.dtype == CAMERA_BF16 ? 2 : 4);
  k_permute_small<<<c.n_tokens + c.n_routed, RT_THREADS, 0, st>>>(c, row_bytes);
  return cudaGetLastError();
}

cudaError_t launch_plan(const ScoreCtx& c, cudaStream_t st) {
  if (c.n_routed > 0 && c.n_blocks > 0) k_block_scan<<<c.n_routed, 256, 0, st>>>(c);
  k_plan<<<1, 32, 0, st>>>(c);
  return cudaGetLastError();
}

cudaError_t launch_permute(const ScoreCtx& c, cudaStream_t st) {
  if (c.n_routed == 0 || c.n_tokens == 0) return cudaSuccess;
  const int row_bytes = c.d_model * (c.dtype == CAMERA_BF16 ? 2 : 4);
  k_permute<<<(c.n_tokens + 7) / 8, 256, 0, st>>>(c, row_bytes);
  k_pad_rows<<<c.n_routed, 128, 0, st>>>(c, row_bytes);
  return cudaGetLastError();
}

}  // namespace camera
