// Applying a selection to the weights: the per-expert index lists (GetSubIndex, Algorithm 3;
// the retained sets of Algorithm 2) and the gathers W_up[S,:], W_gate[S,:], W_down[:,S]
// (Algorithm 2, the slicing step).  Pure data movement: every kernel is bound by HBM bandwidth.
#include <string.h>

#include <vector>

#include "common.cuh"

namespace camera {

namespace {

constexpr int SUB_THREADS = 256;
constexpr int GR_THREADS = 256;
constexpr int GR_ROWS = GR_THREADS / 32;     // destination rows per CTA of the row gather (one warp each)
constexpr int GC_ROWS = 8;                   // d_model rows per CTA of the column gather

struct LabelOrder { unsigned char v[MAX_LEVELS]; };

struct CompactExpert {
  const void *src_gate, *src_up, *src_down;
  void *dst_gate, *dst_up, *dst_down;
  int32_t d_ff, me_off, down_ld;
  int32_t row_blk_begin;     // first CTA of the row-gather grid that belongs to this expert
  int32_t col_blk_begin;     // first CTA of the column-gather grid that belongs to this expert
  int32_t pad;
};

// One CTA per expert.  For each label value of `order` in turn, the expert's channels that carry it
// are appended to the expert's list in ascending channel order (a stable partition by label).
__global__ void __launch_bounds__(SUB_THREADS)
k_sub_index(const unsigned char* __restrict__ labels, const long long* __restrict__ expert_off, LabelOrder order,
            int n_labels, int* __restrict__ sub_index, int* __restrict__ counts) {
  __shared__ int wcount[SUB_THREADS / 32];
  const int e = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long b = expert_off[e];
  const int n = (int)(expert_off[e + 1] - b);
  int run = 0;
  for (int j = 0; j < n_labels; ++j) {
    const unsigned char v = order.v[j];
    const int before = run;
    for (int i0 = 0; i0 < n; i0 += SUB_THREADS) {
      const int i = i0 + tid;
      const bool m = i < n && labels[b + i] == v;
      const unsigned bal = __ballot_sync(0xffffffffu, m);
      if (lane == 0) wcount[warp] = __popc(bal);
      __syncthreads();
      int woff = 0, total = 0;
#pragma unroll
      for (int w = 0; w < SUB_THREADS / 32; ++w) {
        const int cw = wcount[w];
        woff += w < warp ? cw : 0;
        total += cw;
      }
      if (m) sub_index[b + run + woff + __popc(bal & ((1u << lane) - 1u))] = i;
      __syncthreads();
      run += total;
    }
    if (tid == 0) counts[(size_t)e * n_labels + j] = run - before;
  }
}

__device__ __forceinline__ int expert_of_block(const CompactExpert* tab, int n_experts, int blk, bool col) {
  int lo = 0, hi = n_experts;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if ((col ? tab[mid].col_blk_begin : tab[mid].row_blk_begin) <= blk) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ int rows_taken(const int* counts, int e, int n_labels, int n_take) {
  int m = 0;
  for (int j = 0; j < n_take; ++j) m += counts[(size_t)e * n_labels + j];
  return m;
}

// Destination row r of an expert <- source row sub_index[r], for W_gate, W_up and (micro-expert-major
// layout) W_down.  One warp per destination row, 16-byte copies.
__global__ void __launch_bounds__(GR_THREADS)
k_gather_rows(const CompactExpert* __restrict__ tab, int n_experts, const int* __restrict__ sub_index,
              const int* __restrict__ counts, int n_labels, int n_take, int row_bytes, int down_rows) {
  const int e = expert_of_block(tab, n_experts, blockIdx.x, false);
  const CompactExpert ce = tab[e];
  const int r = ((int)blockIdx.x - ce.row_blk_begin) * GR_ROWS + (threadIdx.x >> 5);
  if (r >= rows_taken(counts, e, n_labels, n_take)) return;
  const int src = sub_index[ce.me_off + r];
  const int lane = threadIdx.x & 31, nvec = row_bytes / 16;
  const size_t so = (size_t)src * row_bytes, dof = (size_t)r * row_bytes;
  const uint4* sg = reinterpret_cast<const uint4*>(static_cast<const char*>(ce.src_gate) + so);
  const uint4* su = reinterpret_cast<const uint4*>(static_cast<const char*>(ce.src_up) + so);
  uint4* dg = reinterpret_cast<uint4*>(static_cast<char*>(ce.dst_gate) + dof);
  uint4* du = reinterpret_cast<uint4*>(static_cast<char*>(ce.dst_up) + dof);
  for (int v = lane; v < nvec; v += 32) { dg[v] = __ldg(sg + v); du[v] = __ldg(su + v); }
  if (down_rows) {
    const uint4* sd = reinterpret_cast<const uint4*>(static_cast<const char*>(ce.src_down) + so);
    uint4* dd = reinterpret_cast<uint4*>(static_cast<char*>(ce.dst_down) + dof);
    for (int v = lane; v < nvec; v += 32) dd[v] = __ldg(sd + v);
  }
}

// Paper layout W_down [d_model, d_ff]: destination column j <- source column sub_index[j], for GC_ROWS rows of
// d_model per CTA.  A thread takes two neighbouring destination columns: their indices are read once and used for all
// of the CTA's rows, the 2 * GC_ROWS loads are independent, and every store writes both columns at once.
template <typename T> struct Pair;
template <> struct Pair<__nv_bfloat16> { typedef __nv_bfloat162 type; };
template <> struct Pair<float> { typedef float2 type; };

template <typename T>
__global__ void __launch_bounds__(GR_THREADS)
k_gather_cols(const CompactExpert* __restrict__ tab, int n_experts, const int* __restrict__ sub_index,
              const int* __restrict__ counts, int n_labels, int n_take, int d_model) {
  typedef typename Pair<T>::type T2;
  const int e = expert_of_block(tab, n_experts, blockIdx.x, true);
  const CompactExpert ce = tab[e];
  const int c0 = ((int)blockIdx.x - ce.col_blk_begin) * GC_ROWS;
  const int m = rows_taken(counts, e, n_labels, n_take);
  const int rows = min(GC_ROWS, d_model - c0);
  const T* src = static_cast<const T*>(ce.src_down) + (size_t)c0 * ce.d_ff;
  T* dst = static_cast<T*>(ce.dst_down) + (size_t)c0 * ce.down_ld;
  const int* idx = sub_index + ce.me_off;
  const bool pair_ok = (ce.down_ld & 1) == 0 && (ce.me_off & 1) == 0 &&
                       (reinterpret_cast<uintptr_t>(ce.dst_down) & (2 * sizeof(T) - 1)) == 0;
  for (int j = 2 * threadIdx.x; j < m; j += 2 * GR_THREADS) {
    if (pair_ok && j + 1 < m) {
      const int2 s = *reinterpret_cast<const int2*>(idx + j);
      T a[GC_ROWS], b[GC_ROWS];
#pragma unroll
      for (int r = 0; r < GC_ROWS; ++r)
        if (r < rows) { a[r] = src[(size_t)r * ce.d_ff + s.x]; b[r] = src[(size_t)r * ce.d_ff + s.y]; }
#pragma unroll
      for (int r = 0; r < GC_ROWS; ++r)
        if (r < rows) {
          T2 v; v.x = a[r]; v.y = b[r];
          *reinterpret_cast<T2*>(dst + (size_t)r * ce.down_ld + j) = v;
        }
    } else {
      for (int jj = j; jj < min(j + 2, m); ++jj) {
        const int s = idx[jj];
        for (int r = 0; r < rows; ++r) dst[(size_t)r * ce.down_ld + jj] = src[(size_t)r * ce.d_ff + s];
      }
    }
  }
}

}  // namespace
}  // namespace camera

using namespace camera;

extern "C" int camera_sub_index(const uint8_t* labels, const int64_t* expert_offsets, int32_t n_experts,
                                const int32_t* label_order, int32_t n_labels, int32_t* sub_index, int32_t* counts,
                                void* cuda_stream) {
  if (labels == nullptr || expert_offsets == nullptr || n_experts < 1 || label_order == nullptr || n_labels < 1 ||
      n_labels > MAX_LEVELS || sub_index == nullptr || counts == nullptr)
    return CAMERA_ERR_INVALID_ARG;
  LabelOrder lo;
  memset(&lo, 0, sizeof(lo));
  for (int j = 0; j < n_labels; ++j) {
    if (label_order[j] < 0 || label_order[j] > 255) return CAMERA_ERR_INVALID_ARG;
    for (int i = 0; i < j; ++i)
      if (label_order[i] == label_order[j]) return CAMERA_ERR_INVALID_ARG;
    lo.v[j] = (unsigned char)label_order[j];
  }
  k_sub_index<<<n_experts, SUB_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      labels, reinterpret_cast<const long long*>(expert_offsets), lo, n_labels, sub_index, counts);
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}

extern "C" size_t camera_compact_workspace_bytes(int32_t n_experts) {
  return n_experts < 1 ? 0 : ((sizeof(CompactExpert) * (size_t)n_experts + 255) & ~(size_t)255);
}

extern "C" int camera_compact_weights(const camera_layer_t* L, const int32_t* sub_index, const int32_t* counts,
                                      int32_t n_labels, int32_t n_take, void* const* w_gate_out, void* const* w_up_out,
                                      void* const* w_down_out, const int32_t* down_ld, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream) {
  if (L == nullptr || L->d_ff == nullptr || L->w_gate == nullptr || L->w_up == nullptr || L->w_down == nullptr ||
      sub_index == nullptr || counts == nullptr || w_gate_out == nullptr || w_up_out == nullptr || w_down_out == nullptr ||
      n_labels < 1 || n_labels > MAX_LEVELS || n_take < 1 || n_take > n_labels)
    return CAMERA_ERR_INVALID_ARG;
  if (L->dtype != CAMERA_F32 && L->dtype != CAMERA_BF16) return CAMERA_ERR_INVALID_ARG;
  if (L->down_layout != CAMERA_DOWN_HF && L->down_layout != CAMERA_DOWN_ME_MAJOR) return CAMERA_ERR_INVALID_ARG;
  const int E = L->n_routed + L->n_shared;
  if (E < 1 || L->n_routed < 0 || L->n_shared < 0) return CAMERA_ERR_INVALID_ARG;
  if (L->d_model < 8 || L->d_model % 8 != 0) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  if (workspace == nullptr || workspace_bytes < camera_compact_workspace_bytes(E) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CAMERA_ERR_WORKSPACE;
  std::vector<CompactExpert> tab(E);
  long long me = 0, row_blocks = 0, col_blocks = 0;
  const bool hf = L->down_layout == CAMERA_DOWN_HF;
  for (int e = 0; e < E; ++e) {
    const int f = L->d_ff[e];
    if (f < 1) return CAMERA_ERR_UNSUPPORTED_SHAPE;
    const void* ptrs[6] = {L->w_gate[e], L->w_up[e], L->w_down[e], w_gate_out[e], w_up_out[e], w_down_out[e]};
    for (int i = 0; i < 6; ++i)
      if (ptrs[i] == nullptr || (reinterpret_cast<uintptr_t>(ptrs[i]) & 15)) return CAMERA_ERR_INVALID_ARG;
    CompactExpert& c = tab[e];
    memset(&c, 0, sizeof(c));
    c.src_gate = L->w_gate[e]; c.src_up = L->w_up[e]; c.src_down = L->w_down[e];
    c.dst_gate = w_gate_out[e]; c.dst_up = w_up_out[e]; c.dst_down = w_down_out[e];
    c.d_ff = f; c.me_off = (int32_t)me;
    c.down_ld = down_ld ? down_ld[e] : f;
    if (c.down_ld < 1) return CAMERA_ERR_INVALID_ARG;
    c.row_blk_begin = (int32_t)row_blocks; c.col_blk_begin = (int32_t)col_blocks;
    me += f;
    row_blocks += (f + GR_ROWS - 1) / GR_ROWS;
    col_blocks += (L->d_model + GC_ROWS - 1) / GC_ROWS;
    if (me >= (1ll << 31) || row_blocks >= (1ll << 31) || col_blocks >= (1ll << 31)) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CompactExpert* d_tab = static_cast<CompactExpert*>(workspace);
  if (cudaMemcpyAsync(d_tab, tab.data(), sizeof(CompactExpert) * E, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return CAMERA_ERR_CUDA;
  }
  const int esz = L->dtype == CAMERA_BF16 ? 2 : 4;
  k_gather_rows<<<(unsigned)row_blocks, GR_THREADS, 0, st>>>(d_tab, E, sub_index, counts, n_labels, n_take,
                                                              L->d_model * esz, hf ? 0 : 1);
  if (hf) {
    if (L->dtype == CAMERA_BF16)
      k_gather_cols<__nv_bfloat16><<<(unsigned)col_blocks, GR_THREADS, 0, st>>>(d_tab, E, sub_index, counts, n_labels,
                                                                                 n_take, L->d_model);
    else
      k_gather_cols<float><<<(unsigned)col_blocks, GR_THREADS, 0, st>>>(d_tab, E, sub_index, counts, n_labels, n_take,
                                                                         L->d_model);
  }
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}
