// fp32-FMA scoring kernel (Algorithm 1's Lambda, ColumnSum and ColumnMax steps with Lambda kept in registers) and the final
// combine (the energy step, Eq. 11).  This kernel serves fp32 layers and shapes the tensor-core kernel
// does not take; it uses the same work units and partial layout as the tensor-core kernel.
#include "common.cuh"

namespace camera {

namespace {

constexpr int SS_THREADS = 256;
constexpr int SS_TOK = 64;
constexpr int SS_KC = 16;
constexpr int SS_LD = 68;
constexpr int SS_CH = 64;           // channels per pass

// Work unit = (expert, tile of ch_tile channels, chunk of chunk_tokens tokens), handled as
// ch_tile / 64 passes of 64 channels.  For every token tile the CTA forms g = W_gate x and
// u = W_up x for 64 tokens x 64 channels in fp32,
// then lambda = a_t * SiLU(g) * u and folds lambda^2 / |lambda| into per-channel running sum / max.
// One partial (sum, max) per channel and chunk goes to the workspace; chunks are added later in
// a fixed order, so results do not depend on scheduling.
template <typename T>
__global__ void __launch_bounds__(SS_THREADS) k_score_simt(ScoreCtx c) {
  __shared__ __align__(16) float Xs[SS_KC][SS_LD];
  __shared__ __align__(16) float Gs[SS_KC][SS_LD];
  __shared__ __align__(16) float Us[SS_KC][SS_LD];
  __shared__ float red_s[16][SS_CH];
  __shared__ float red_m[16][SS_CH];
  constexpr int VN = Vec16<T>::N;
  constexpr int VPR = SS_KC / VN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int d = c.d_model;
  const int total_units = c.totals->total_units;

  const int passes = c.ch_tile / SS_CH;
  for (int work = blockIdx.x; work < total_units * passes; work += gridDim.x) {
    const UnitInfo u = decode_unit(c, work / passes);
    const ExpertStatic es = c.est[u.e];
    const int pass_off = (work % passes) * SS_CH;
    const int f = u.f, ch0 = u.ch0 + pass_off, rows = u.rows;
    if (ch0 >= f) continue;
    const T* Xsrc = (es.shared_idx < 0 ? static_cast<const T*>(c.x_perm) : static_cast<const T*>(c.x)) +
                    (size_t)u.row0 * d;
    const float* wsrc = (es.shared_idx < 0 ? c.perm_w : c.shared_w + (size_t)es.shared_idx * c.shared_ld) + u.row0;
    const T* Wg = static_cast<const T*>(es.w_gate);
    const T* Wu = static_cast<const T*>(es.w_up);

    float s[4] = {0.f, 0.f, 0.f, 0.f}, m[4] = {0.f, 0.f, 0.f, 0.f};
    for (int r0 = 0; r0 < rows; r0 += SS_TOK) {
      float ag[4][4], au[4][4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { ag[i][j] = 0.f; au[i][j] = 0.f; }
      for (int k0 = 0; k0 < d; k0 += SS_KC) {
        __syncthreads();
        for (int v = tid; v < 3 * SS_TOK * VPR; v += SS_THREADS) {
          const int which = v / (SS_TOK * VPR), w = v % (SS_TOK * VPR);
          const int row = w / VPR, kv = (w % VPR) * VN;
          float fv[VN];
#pragma unroll
          for (int i = 0; i < VN; ++i) fv[i] = 0.f;
          if (k0 + kv < d) {
            if (which == 0) {
              if (r0 + row < rows) Vec16<T>::load(Xsrc + (size_t)(r0 + row) * d + k0 + kv, fv);
            } else if (ch0 + row < f) {
              Vec16<T>::load((which == 1 ? Wg : Wu) + (size_t)(ch0 + row) * d + k0 + kv, fv);
            }
          }
          float* dst = which == 0 ? &Xs[0][0] : (which == 1 ? &Gs[0][0] : &Us[0][0]);
#pragma unroll
          for (int i = 0; i < VN; ++i) dst[(kv + i) * SS_LD + row] = fv[i];
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < SS_KC; ++k) {
          const float4 a = *reinterpret_cast<const float4*>(&Xs[k][ty * 4]);
          const float4 g = *reinterpret_cast<const float4*>(&Gs[k][tx * 4]);
          const float4 u = *reinterpret_cast<const float4*>(&Us[k][tx * 4]);
          const float av[4] = {a.x, a.y, a.z, a.w}, gv[4] = {g.x, g.y, g.z, g.w}, uv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              ag[i][j] = fmaf(av[i], gv[j], ag[i][j]);
              au[i][j] = fmaf(av[i], uv[j], au[i][j]);
            }
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int row = r0 + ty * 4 + i;
        const float a_t = row < rows ? wsrc[row] : 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float g = ag[i][j];
          const float lam = a_t * (g / (1.f + expf(-g))) * au[i][j];
          s[j] = fmaf(lam, lam, s[j]);
          m[j] = fmaxf(m[j], fabsf(lam));
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 4; ++j) { red_s[ty][tx * 4 + j] = s[j]; red_m[ty][tx * 4 + j] = m[j]; }
    __syncthreads();
    if (tid < SS_CH && ch0 + tid < f) {
      float ts = 0.f, tm = 0.f;
#pragma unroll
      for (int y = 0; y < 16; ++y) { ts += red_s[y][tid]; tm = fmaxf(tm, red_m[y][tid]); }
      const size_t slot = (size_t)u.part_slot + pass_off + tid;
      c.part_sum[slot] = ts;
      c.part_max[slot] = tm;
    }
  }
}

// Adds the chunk partials of every micro-expert (fp64, fixed order: eight interleaved running sums, then those in
// order), squares the max and blends: E_i = [(1-alpha) phi2_i + alpha phi_inf_i] * omega2_i   (Eq. 11).
// Block = 32 micro-experts x 8 chunk lanes, so that eight loads per micro-expert are in flight.
constexpr int CB_X = 32, CB_Y = 8;
__global__ void __launch_bounds__(CB_X * CB_Y) k_combine(ScoreCtx c) {
  __shared__ double ssum[CB_Y][CB_X];
  __shared__ float smax[CB_Y][CB_X];
  const int i = blockIdx.x * CB_X + threadIdx.x;
  double s = 0.0;
  float m = 0.f;
  if (i < c.n_me) {
    const int e = upper_segment(c.me_prefix, c.n_experts, i);
    const int ch = i - c.me_prefix[e];
    const ExpertDyn dy = c.edyn[e];
    const int f = c.est[e].d_ff;
    for (int j = threadIdx.y; j < dy.n_chunks; j += CB_Y) {
      const size_t slot = (size_t)dy.part_begin + (size_t)j * f + ch;
      s += (double)c.part_sum[slot];
      m = fmaxf(m, c.part_max[slot]);
    }
  }
  ssum[threadIdx.y][threadIdx.x] = s;
  smax[threadIdx.y][threadIdx.x] = m;
  __syncthreads();
  if (threadIdx.y != 0 || i >= c.n_me) return;
  s = 0.0; m = 0.f;
#pragma unroll
  for (int y = 0; y < CB_Y; ++y) { s += ssum[y][threadIdx.x]; m = fmaxf(m, smax[y][threadIdx.x]); }
  double m2 = (double)m * (double)m;
  if (c.accumulate) {     // earlier batches of tokens: sums add, maxima take the maximum
    s += (double)c.phi2[i];
    m2 = fmax(m2, (double)c.phi_inf_sq[i]);
  }
  const double a = (double)c.alpha;
  c.phi2[i] = (float)s;
  c.phi_inf_sq[i] = (float)m2;
  c.energy[i] = (float)(((1.0 - a) * s + a * m2) * (double)c.omega2[i]);
}

}  // namespace

cudaError_t launch_score_simt(const ScoreCtx& c, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = sms * 4;
  if (c.dtype == CAMERA_BF16) k_score_simt<__nv_bfloat16><<<grid, SS_THREADS, 0, st>>>(c);
  else k_score_simt<float><<<grid, SS_THREADS, 0, st>>>(c);
  return cudaGetLastError();
}

cudaError_t launch_combine(const ScoreCtx& c, cudaStream_t st) {
  if (c.n_me == 0) return cudaSuccess;
  k_combine<<<(c.n_me + CB_X - 1) / CB_X, dim3(CB_X, CB_Y), 0, st>>>(c);
  return cudaGetLastError();
}

}  // namespace camera
