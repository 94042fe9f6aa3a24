// omega^2_i = ||w_i||_2^2 over the W_down of every expert (Algorithm 1, the ColumnSum of W_down * W_down).  Pure HBM stream:
// every element of W_down is read exactly once with 16-byte loads, sums in fp32.
#include "common.cuh"

namespace camera {

namespace {

constexpr int NORM_THREADS = 256;
constexpr int NORM_WARPS = NORM_THREADS / 32;
constexpr int NORM_ROWS_PER_CTA = 32;   // ME-major layout: micro-experts per CTA

// CAMERA_DOWN_HF, W_down = [d_model, d_ff]: micro-expert i is column i.  A CTA owns 32 * VN
// consecutive columns; each of its warps walks a strided share of the d_model rows with one
// 16-byte load per lane per row, keeping VN running sums; the 8 warps are then added in a fixed
// order through shared memory.
template <typename T>
__global__ void __launch_bounds__(NORM_THREADS) k_colnorm_hf(ScoreCtx c) {
  constexpr int VN = Vec16<T>::N;
  __shared__ float red[NORM_WARPS][32 * VN + 1];
  // which expert does this CTA belong to
  int lo = 0, hi = c.n_experts;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (c.est[mid].norm_blk_begin <= (int)blockIdx.x) lo = mid; else hi = mid;
  }
  const ExpertStatic es = c.est[lo];
  const int f = es.d_ff, d = c.d_model, ld = es.down_ld;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col = ((int)blockIdx.x - es.norm_blk_begin) * 32 * VN + lane * VN;
  const T* W = static_cast<const T*>(es.w_down);
  float s[VN];
#pragma unroll
  for (int i = 0; i < VN; ++i) s[i] = 0.f;
  if (col < f) {   // d_ff is a multiple of VN, so a vector is entirely inside or outside
    int r = warp;
    for (; r + 3 * NORM_WARPS < d; r += 4 * NORM_WARPS) {
      float v[4][VN];
#pragma unroll
      for (int u = 0; u < 4; ++u) Vec16<T>::load(W + (size_t)(r + u * NORM_WARPS) * ld + col, v[u]);
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int i = 0; i < VN; ++i) s[i] = fmaf(v[u][i], v[u][i], s[i]);
    }
    for (; r < d; r += NORM_WARPS) {
      float v[VN];
      Vec16<T>::load(W + (size_t)r * ld + col, v);
#pragma unroll
      for (int i = 0; i < VN; ++i) s[i] = fmaf(v[i], v[i], s[i]);
    }
  }
#pragma unroll
  for (int i = 0; i < VN; ++i) red[warp][lane * VN + i] = s[i];
  __syncthreads();
  for (int j = threadIdx.x; j < 32 * VN; j += NORM_THREADS) {
    const int cj = ((int)blockIdx.x - es.norm_blk_begin) * 32 * VN + j;
    if (cj < f) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < NORM_WARPS; ++w) t += red[w][j];
      c.omega2[es.me_off + cj] = t;
    }
  }
}

// CAMERA_DOWN_ME_MAJOR, W_down = [d_ff, d_model]: micro-expert i is row i.  One warp per row,
// 16-byte loads, warp-shuffle reduction.
template <typename T>
__global__ void __launch_bounds__(NORM_THREADS) k_rownorm_me(ScoreCtx c) {
  constexpr int VN = Vec16<T>::N;
  int lo = 0, hi = c.n_experts;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (c.est[mid].norm_blk_begin <= (int)blockIdx.x) lo = mid; else hi = mid;
  }
  const ExpertStatic es = c.est[lo];
  const int d = c.d_model, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row0 = ((int)blockIdx.x - es.norm_blk_begin) * NORM_ROWS_PER_CTA;
  const T* W = static_cast<const T*>(es.w_down);
  for (int r = row0 + warp; r < row0 + NORM_ROWS_PER_CTA && r < es.d_ff; r += NORM_WARPS) {
    const T* src = W + (size_t)r * d;
    float s = 0.f;
    for (int k = lane * VN; k < d; k += 32 * VN) {
      float v[VN];
      Vec16<T>::load(src + k, v);
#pragma unroll
      for (int i = 0; i < VN; ++i) s = fmaf(v[i], v[i], s);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) c.omega2[es.me_off + r] = s;
  }
}

}  // namespace

// CTAs of the row-norm grid that expert e (d_ff = f) needs; used by the host planner too.
int rownorm_blocks(int down_layout, int dtype, int f) {
  if (down_layout == CAMERA_DOWN_HF) {
    const int cols = 32 * (dtype == CAMERA_BF16 ? 8 : 4);
    return (f + cols - 1) / cols;
  }
  return (f + NORM_ROWS_PER_CTA - 1) / NORM_ROWS_PER_CTA;
}

cudaError_t launch_rownorm(const ScoreCtx& c, int n_norm_blocks, cudaStream_t st) {
  if (n_norm_blocks == 0) return cudaSuccess;
  if (c.down_layout == CAMERA_DOWN_HF) {
    if (c.dtype == CAMERA_BF16) k_colnorm_hf<__nv_bfloat16><<<n_norm_blocks, NORM_THREADS, 0, st>>>(c);
    else k_colnorm_hf<float><<<n_norm_blocks, NORM_THREADS, 0, st>>>(c);
  } else {
    if (c.dtype == CAMERA_BF16) k_rownorm_me<__nv_bfloat16><<<n_norm_blocks, NORM_THREADS, 0, st>>>(c);
    else k_rownorm_me<float><<<n_norm_blocks, NORM_THREADS, 0, st>>>(c);
  }
  return cudaGetLastError();
}

}  // namespace camera
