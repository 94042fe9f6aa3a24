// Device-wide segmented rank selection for CAMERA-P (Algorithm 2, TopSelect) and CAMERA-Q
// (Algorithm 3, ListSplitByRatio / GetSubIndex).
//
// Every micro-expert gets the 64-bit key (order-preserving image of its fp32 energy) << 32 | index
// within its segment.  Keys are unique, so "the r-th smallest key" is unambiguous and equal
// energies are ordered by index.  The key of rank r is found by a most-significant-digit radix
// select: 8 passes of 8 bits, each pass a histogram (shared-memory bins, flushed with integer
// atomics, hence deterministic) of the digit among the keys that match the prefix found so far.
// Several ranks per segment (the class boundaries) are selected in the same passes.
#include <math.h>
#include <string.h>

#include <vector>

#include "common.cuh"

namespace camera {

namespace {

constexpr int SEL_THREADS = 256;
constexpr int SEL_PASSES = 8;
constexpr int MAX_THR = MAX_LEVELS - 1;

struct SelState {
  unsigned long long prefix;   // digits fixed so far, in place
  long long rank;              // rank still to find among the keys that match; < 0 = no such element
};

__device__ __forceinline__ unsigned long long make_key(float e, unsigned idx) {
  unsigned b = __float_as_uint(e);
  b ^= (b >> 31) ? 0xffffffffu : 0x80000000u;
  return ((unsigned long long)b << 32) | idx;
}

__device__ __forceinline__ float key_energy(unsigned long long key) {
  unsigned b = (unsigned)(key >> 32);
  b = (b & 0x80000000u) ? (b ^ 0x80000000u) : ~b;
  return __uint_as_float(b);
}

// State after `pass` passes for (segment seg, threshold j), computed by warp j of every CTA from
// the state after pass-1 passes and the (complete) histogram of pass-1.  Result in shared st[j].
__device__ void advance_state(int pass, int seg, int n_thr, long long seg_len, const long long* ranks,
                              const SelState* S, const unsigned* hist, int n_seg, SelState* st) {
  const int lane = threadIdx.x & 31, j = threadIdx.x >> 5;
  if (j >= n_thr) return;
  SelState cur;
  if (pass <= 1) {
    cur.prefix = 0ull;
    cur.rank = ranks[seg * n_thr + j];
    if (cur.rank >= seg_len) cur.rank = -1;
  } else {
    cur = S[((size_t)(pass - 2) * n_seg + seg) * n_thr + j];
  }
  if (pass >= 1 && cur.rank >= 0) {
    const unsigned* h = hist + (((size_t)(pass - 1) * n_seg + seg) * n_thr + j) * 256;
    // lane owns bins [8*lane, 8*lane+8)
    unsigned v[8];
    long long mine = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { v[i] = h[lane * 8 + i]; mine += v[i]; }
    long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    long long before = incl - mine;
    const bool here = cur.rank >= before && cur.rank < incl;
    int bin = -1;
    long long newrank = 0;
    if (here) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (bin < 0 && cur.rank < before + (long long)v[i]) { bin = lane * 8 + i; newrank = cur.rank - before; }
        before += v[i];
      }
    }
    const unsigned who = __ballot_sync(0xffffffffu, here);
    if (who == 0u) {
      cur.rank = -1;    // cannot happen for a rank inside the segment
    } else {
      const int src = __ffs(who) - 1;
      bin = __shfl_sync(0xffffffffu, bin, src);
      newrank = __shfl_sync(0xffffffffu, newrank, src);
      cur.prefix |= (unsigned long long)bin << (56 - 8 * (pass - 1));
      cur.rank = newrank;
    }
  }
  if (lane == 0) st[j] = cur;
}

__global__ void __launch_bounds__(SEL_THREADS)
k_select_hist(int pass, const float* __restrict__ energy, const long long* seg_off, const long long* ranks,
              SelState* S, unsigned* hist, int n_seg, int n_thr) {
  __shared__ SelState st[MAX_THR];
  __shared__ unsigned bins[MAX_THR][256];
  const int seg = blockIdx.y;
  const long long begin = seg_off[seg], len = seg_off[seg + 1] - begin;
  for (int i = threadIdx.x; i < n_thr * 256; i += SEL_THREADS) (&bins[0][0])[i] = 0u;
  advance_state(pass, seg, n_thr, len, ranks, S, hist, n_seg, st);
  __syncthreads();
  if (pass >= 1 && blockIdx.x == 0 && threadIdx.x < n_thr)
    S[((size_t)(pass - 1) * n_seg + seg) * n_thr + threadIdx.x] = st[threadIdx.x];
  const int shift = 56 - 8 * pass;
  for (long long i = (long long)blockIdx.x * SEL_THREADS + threadIdx.x; i < len; i += (long long)gridDim.x * SEL_THREADS) {
    const unsigned long long key = make_key(energy[begin + i], (unsigned)i);
    const unsigned digit = (unsigned)(key >> shift) & 0xffu;
    for (int j = 0; j < n_thr; ++j) {
      if (st[j].rank < 0) continue;
      if (pass == 0 || (key >> (shift + 8)) == (st[j].prefix >> (shift + 8))) atomicAdd(&bins[j][digit], 1u);
    }
  }
  __syncthreads();
  unsigned* h = hist + (((size_t)pass * n_seg + seg) * n_thr) * 256;
  for (int i = threadIdx.x; i < n_thr * 256; i += SEL_THREADS) {
    const unsigned v = (&bins[0][0])[i];
    if (v) atomicAdd(h + i, v);
  }
}

struct LevelValues { unsigned char v[MAX_LEVELS]; };

// Labels every element with the value of its class: class = (n_thr - number of thresholds the
// key is at or above), thresholds being the selected keys.
__global__ void __launch_bounds__(SEL_THREADS)
k_select_mark(const float* __restrict__ energy, const long long* seg_off, const long long* ranks, SelState* S,
              const unsigned* hist, int n_seg, int n_thr, LevelValues lv, unsigned char* out, float* thresholds) {
  __shared__ SelState st[MAX_THR];
  const int seg = blockIdx.y;
  const long long begin = seg_off[seg], len = seg_off[seg + 1] - begin;
  advance_state(SEL_PASSES, seg, n_thr, len, ranks, S, hist, n_seg, st);
  __syncthreads();
  if (blockIdx.x == 0 && threadIdx.x < n_thr) {
    S[((size_t)(SEL_PASSES - 1) * n_seg + seg) * n_thr + threadIdx.x] = st[threadIdx.x];
    if (thresholds != nullptr && threadIdx.x == 0)
      thresholds[seg] = st[0].rank >= 0 ? key_energy(st[0].prefix) : INFINITY;
  }
  for (long long i = (long long)blockIdx.x * SEL_THREADS + threadIdx.x; i < len; i += (long long)gridDim.x * SEL_THREADS) {
    const unsigned long long key = make_key(energy[begin + i], (unsigned)i);
    int above = 0;
    for (int j = 0; j < n_thr; ++j) above += (st[j].rank >= 0 && key >= st[j].prefix) ? 1 : 0;
    out[begin + i] = lv.v[n_thr - above];
  }
}

// The mark pass of camera_select_all: thresholds 0 .. n_prune-1 each give a keep mask of their own, the remaining
// n_thr - n_prune thresholds are the class boundaries of the bit-width allocation.
__global__ void __launch_bounds__(SEL_THREADS)
k_select_mark_all(const float* __restrict__ energy, const long long* seg_off, const long long* ranks, SelState* S,
                  const unsigned* hist, int n_seg, int n_thr, int n_prune, LevelValues lv, long long n_total,
                  unsigned char* keep_out, unsigned char* bits_out) {
  __shared__ SelState st[MAX_THR];
  const int seg = blockIdx.y;
  const long long begin = seg_off[seg], len = seg_off[seg + 1] - begin;
  advance_state(SEL_PASSES, seg, n_thr, len, ranks, S, hist, n_seg, st);
  __syncthreads();
  if (blockIdx.x == 0 && threadIdx.x < n_thr)
    S[((size_t)(SEL_PASSES - 1) * n_seg + seg) * n_thr + threadIdx.x] = st[threadIdx.x];
  const int n_bounds = n_thr - n_prune;
  for (long long i = (long long)blockIdx.x * SEL_THREADS + threadIdx.x; i < len; i += (long long)gridDim.x * SEL_THREADS) {
    const unsigned long long key = make_key(energy[begin + i], (unsigned)i);
    for (int j = 0; j < n_prune; ++j)
      keep_out[(size_t)j * n_total + begin + i] = (st[j].rank >= 0 && key >= st[j].prefix) ? 1 : 0;
    if (bits_out != nullptr) {
      int above = 0;
      for (int j = n_prune; j < n_thr; ++j) above += (st[j].rank >= 0 && key >= st[j].prefix) ? 1 : 0;
      bits_out[begin + i] = lv.v[n_bounds - above];
    }
  }
}

// One CTA per expert: how many of its micro-experts fall in each class (or are retained).
__global__ void __launch_bounds__(SEL_THREADS)
k_class_counts(const float* __restrict__ energy, const long long* seg_off, const SelState* S, int n_seg, int n_thr,
               const long long* expert_off, int n_classes_out, int* counts) {
  __shared__ int cnt[MAX_LEVELS];
  const int e = blockIdx.x;
  const long long b = expert_off[e], en = expert_off[e + 1];
  if (threadIdx.x < MAX_LEVELS) cnt[threadIdx.x] = 0;
  __syncthreads();
  if (en > b) {
    const int seg = upper_segment(seg_off, n_seg, b);
    const SelState* fin = S + ((size_t)(SEL_PASSES - 1) * n_seg + seg) * n_thr;
    int local[MAX_LEVELS];
#pragma unroll
    for (int j = 0; j < MAX_LEVELS; ++j) local[j] = 0;
    for (long long i = b + threadIdx.x; i < en; i += SEL_THREADS) {
      const unsigned long long key = make_key(energy[i], (unsigned)(i - seg_off[seg]));
      int above = 0;
      for (int j = 0; j < n_thr; ++j) above += (fin[j].rank >= 0 && key >= fin[j].prefix) ? 1 : 0;
      const int cls = n_thr - above;
#pragma unroll
      for (int j = 0; j < MAX_LEVELS; ++j) local[j] += (cls == j);
    }
#pragma unroll
    for (int j = 0; j < MAX_LEVELS; ++j)
      if (local[j]) atomicAdd(&cnt[j], local[j]);
  }
  __syncthreads();
  if (threadIdx.x < n_classes_out) counts[(size_t)e * n_classes_out + threadIdx.x] = cnt[threadIdx.x];
}

struct SelLayout {
  size_t seg_off, ranks, state, hist, total;
};

SelLayout sel_layout(int n_seg, int n_thr) {
  auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
  SelLayout L;
  size_t o = 0;
  L.seg_off = o; o = up(o + sizeof(long long) * (n_seg + 1));
  L.ranks = o;   o = up(o + sizeof(long long) * (size_t)n_seg * n_thr);
  L.state = o;   o = up(o + sizeof(SelState) * (size_t)SEL_PASSES * n_seg * n_thr);
  L.hist = o;    o = up(o + sizeof(unsigned) * (size_t)SEL_PASSES * n_seg * n_thr * 256);
  L.total = o;
  return L;
}

long long floor_count(double ratio, long long n) { return (long long)floor(ratio * (double)n + 1e-9); }

// ranks_host: [n_seg * n_thr] target ascending ranks (a rank >= the segment length selects nothing).
// n_prune >= 0 selects the mark pass of camera_select_all: `out` then holds n_prune masks of seg_offsets[n_seg] bytes
// and bits_out (may be null) gets the class values.
int select_core(const float* energy, const int64_t* seg_offsets, int n_seg, int n_thr, const long long* ranks_host,
                LevelValues lv, const int64_t* expert_offsets, int n_experts, int n_classes_out, unsigned char* out,
                int* counts, float* thresholds, void* ws, size_t ws_bytes, cudaStream_t st, int n_prune = -1,
                unsigned char* bits_out = nullptr) {
  const SelLayout L = sel_layout(n_seg, n_thr);
  if (ws == nullptr || ws_bytes < L.total) return CAMERA_ERR_WORKSPACE;
  char* base = static_cast<char*>(ws);
  long long* d_seg = reinterpret_cast<long long*>(base + L.seg_off);
  long long* d_ranks = reinterpret_cast<long long*>(base + L.ranks);
  SelState* d_state = reinterpret_cast<SelState*>(base + L.state);
  unsigned* d_hist = reinterpret_cast<unsigned*>(base + L.hist);
  long long max_len = 0;
  for (int s = 0; s < n_seg; ++s) max_len = seg_offsets[s + 1] - seg_offsets[s] > max_len ? seg_offsets[s + 1] - seg_offsets[s] : max_len;
  if (cudaMemcpyAsync(d_seg, seg_offsets, sizeof(long long) * (n_seg + 1), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(d_ranks, ranks_host, sizeof(long long) * (size_t)n_seg * n_thr, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemsetAsync(d_hist, 0, sizeof(unsigned) * (size_t)SEL_PASSES * n_seg * n_thr * 256, st) != cudaSuccess)
    return CAMERA_ERR_CUDA;
  if (max_len > 0) {
    long long gx = (max_len + SEL_THREADS * 8 - 1) / (SEL_THREADS * 8);
    if (gx > 1184) gx = 1184;
    if (gx < 1) gx = 1;
    const dim3 grid((unsigned)gx, (unsigned)n_seg);
    for (int p = 0; p < SEL_PASSES; ++p)
      k_select_hist<<<grid, SEL_THREADS, 0, st>>>(p, energy, d_seg, d_ranks, d_state, d_hist, n_seg, n_thr);
    if (n_prune >= 0)
      k_select_mark_all<<<grid, SEL_THREADS, 0, st>>>(energy, d_seg, d_ranks, d_state, d_hist, n_seg, n_thr, n_prune, lv,
                                                      (long long)seg_offsets[n_seg], out, bits_out);
    else
      k_select_mark<<<grid, SEL_THREADS, 0, st>>>(energy, d_seg, d_ranks, d_state, d_hist, n_seg, n_thr, lv, out, thresholds);
  }
  if (counts != nullptr && expert_offsets != nullptr && n_experts > 0) {
    if (max_len > 0)
      k_class_counts<<<n_experts, SEL_THREADS, 0, st>>>(energy, d_seg, d_state, n_seg, n_thr,
                                                        reinterpret_cast<const long long*>(expert_offsets), n_classes_out, counts);
    else if (cudaMemsetAsync(counts, 0, sizeof(int) * (size_t)n_experts * n_classes_out, st) != cudaSuccess)
      return CAMERA_ERR_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}

bool segments_ok(const int64_t* seg, int n_seg) {
  if (seg == nullptr || n_seg < 1 || n_seg > 65535 || seg[0] != 0) return false;
  for (int s = 0; s < n_seg; ++s)
    if (seg[s + 1] < seg[s] || seg[s + 1] - seg[s] > 0xffffffffll) return false;
  return true;
}

}  // namespace
}  // namespace camera

using namespace camera;

extern "C" size_t camera_select_workspace_bytes(int64_t n_total, int32_t n_segments, int32_t n_levels) {
  if (n_total < 0 || n_segments < 1 || n_levels < 2 || n_levels > MAX_LEVELS) return 0;
  return sel_layout(n_segments, n_levels - 1).total;
}

extern "C" int camera_select_prune(const float* energy, const int64_t* seg_offsets, int32_t n_segments,
                                   double prune_ratio, const int64_t* expert_offsets, int32_t n_experts_total,
                                   uint8_t* keep_mask, int32_t* kept_per_expert, float* thresholds,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!segments_ok(seg_offsets, n_segments) || !(prune_ratio >= 0.0 && prune_ratio < 1.0) || keep_mask == nullptr)
    return CAMERA_ERR_INVALID_ARG;
  if (seg_offsets[n_segments] > 0 && energy == nullptr) return CAMERA_ERR_INVALID_ARG;
  if (kept_per_expert != nullptr && (expert_offsets == nullptr || n_experts_total < 1)) return CAMERA_ERR_INVALID_ARG;
  long long* ranks = new long long[n_segments];
  for (int s = 0; s < n_segments; ++s) ranks[s] = floor_count(prune_ratio, seg_offsets[s + 1] - seg_offsets[s]);
  LevelValues lv;
  memset(&lv, 0, sizeof(lv));
  lv.v[0] = 1;   // class 0 = at or above the threshold = retained
  lv.v[1] = 0;
  const int rc = select_core(energy, seg_offsets, n_segments, 1, ranks, lv, expert_offsets, n_experts_total, 1, keep_mask,
                             kept_per_expert, thresholds, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
  delete[] ranks;
  return rc;
}

extern "C" int camera_alloc_bits(const float* energy, const int64_t* seg_offsets, int32_t n_segments,
                                 const double* ratios, const int32_t* bits, int32_t n_levels,
                                 const int64_t* expert_offsets, int32_t n_experts_total,
                                 uint8_t* bits_out, int32_t* class_counts,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!segments_ok(seg_offsets, n_segments) || ratios == nullptr || bits == nullptr || n_levels < 2 ||
      n_levels > MAX_LEVELS || bits_out == nullptr)
    return CAMERA_ERR_INVALID_ARG;
  if (seg_offsets[n_segments] > 0 && energy == nullptr) return CAMERA_ERR_INVALID_ARG;
  if (class_counts != nullptr && (expert_offsets == nullptr || n_experts_total < 1)) return CAMERA_ERR_INVALID_ARG;
  double sum = 0.0;
  LevelValues lv;
  memset(&lv, 0, sizeof(lv));
  for (int j = 0; j < n_levels; ++j) {
    if (!(ratios[j] >= 0.0) || bits[j] < 0 || bits[j] > 255) return CAMERA_ERR_INVALID_ARG;
    sum += ratios[j];
    lv.v[j] = (unsigned char)bits[j];
  }
  if (fabs(sum - 1.0) > 1e-9) return CAMERA_ERR_INVALID_ARG;
  const int n_thr = n_levels - 1;
  long long* ranks = new long long[(size_t)n_segments * n_thr];
  for (int s = 0; s < n_segments; ++s) {
    const long long n = seg_offsets[s + 1] - seg_offsets[s];
    double acc = 0.0;
    for (int m = 1; m <= n_thr; ++m) {      // threshold m separates classes m-1 and m
      acc += ratios[m - 1];
      long long cm = floor_count(acc, n);
      if (cm > n) cm = n;
      ranks[(size_t)s * n_thr + (m - 1)] = n - cm;   // ascending rank of the lowest key of classes < m
    }
  }
  const int rc = select_core(energy, seg_offsets, n_segments, n_thr, ranks, lv, expert_offsets, n_experts_total, n_levels,
                             bits_out, class_counts, nullptr, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
  delete[] ranks;
  return rc;
}

extern "C" int camera_select_all(const float* energy, const int64_t* seg_offsets, int32_t n_segments,
                                 const double* prune_ratios, int32_t n_prune, uint8_t* keep_masks, const double* ratios,
                                 const int32_t* bits, int32_t n_levels, uint8_t* bits_out, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
  if (!segments_ok(seg_offsets, n_segments) || n_prune < 0 || (n_prune > 0 && (prune_ratios == nullptr || keep_masks == nullptr)))
    return CAMERA_ERR_INVALID_ARG;
  if (bits_out != nullptr && (ratios == nullptr || bits == nullptr || n_levels < 2 || n_levels > MAX_LEVELS))
    return CAMERA_ERR_INVALID_ARG;
  const int n_bounds = bits_out != nullptr ? n_levels - 1 : 0;
  const int n_thr = n_prune + n_bounds;
  if (n_thr < 1 || n_thr > MAX_THR) return CAMERA_ERR_INVALID_ARG;
  if (seg_offsets[n_segments] > 0 && energy == nullptr) return CAMERA_ERR_INVALID_ARG;
  for (int p = 0; p < n_prune; ++p)
    if (!(prune_ratios[p] >= 0.0 && prune_ratios[p] < 1.0)) return CAMERA_ERR_INVALID_ARG;
  LevelValues lv;
  memset(&lv, 0, sizeof(lv));
  if (bits_out != nullptr) {
    double sum = 0.0;
    for (int j = 0; j < n_levels; ++j) {
      if (!(ratios[j] >= 0.0) || bits[j] < 0 || bits[j] > 255) return CAMERA_ERR_INVALID_ARG;
      sum += ratios[j];
      lv.v[j] = (unsigned char)bits[j];
    }
    if (fabs(sum - 1.0) > 1e-9) return CAMERA_ERR_INVALID_ARG;
  }
  std::vector<long long> ranks((size_t)n_segments * n_thr);
  for (int s = 0; s < n_segments; ++s) {
    const long long n = seg_offsets[s + 1] - seg_offsets[s];
    for (int p = 0; p < n_prune; ++p) ranks[(size_t)s * n_thr + p] = floor_count(prune_ratios[p], n);   // as camera_select_prune
    double acc = 0.0;
    for (int m = 1; m <= n_bounds; ++m) {                                                              // as camera_alloc_bits
      acc += ratios[m - 1];
      long long cm = floor_count(acc, n);
      if (cm > n) cm = n;
      ranks[(size_t)s * n_thr + n_prune + (m - 1)] = n - cm;
    }
  }
  return select_core(energy, seg_offsets, n_segments, n_thr, ranks.data(), lv, nullptr, 0, 0, keep_masks, nullptr, nullptr,
                     workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream), n_prune, bits_out);
}

// ---------------------------------------------------------------------------------------------
// camera_select_prune_static: the same selection with its scratch in a fixed device array that is
// part of the library image, for callers that have no way to hand over a workspace.
// ---------------------------------------------------------------------------------------------
namespace camera {
namespace {

constexpr int STATIC_MAX_SEGMENTS = 32;
constexpr size_t STATIC_SCRATCH_BYTES = 288 * 1024;   // room for 32 segments (checked on every call)

// Lives in every GPU's memory from the moment the library is loaded there until the process ends.
static __device__ __align__(256) unsigned char g_select_scratch[STATIC_SCRATCH_BYTES];

constexpr int STATIC_MAX_DEVICES = 64;
void* g_scratch_ptr[STATIC_MAX_DEVICES];     // device address of g_select_scratch, per device ordinal
bool g_scratch_ready[STATIC_MAX_DEVICES];

// In host code `g_select_scratch` is only a handle; the address kernels can use has to be asked for,
// once per device, while that device is current.
int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return CAMERA_ERR_CUDA;
  if (!g_scratch_ready[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return CAMERA_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
    g_scratch_ready[dev] = true;
  }
  *out = g_scratch_ptr[dev];
  return CAMERA_OK;
}

}  // namespace
}  // namespace camera

extern "C" int camera_select_prune_static(const float* energy, const int64_t* seg_offsets, int32_t n_segments,
                                          double prune_ratio, uint8_t* keep_mask, float* thresholds,
                                          void* cuda_stream) {
  if (!segments_ok(seg_offsets, n_segments) || !(prune_ratio >= 0.0 && prune_ratio < 1.0) || keep_mask == nullptr)
    return CAMERA_ERR_INVALID_ARG;
  if (seg_offsets[n_segments] > 0 && energy == nullptr) return CAMERA_ERR_INVALID_ARG;
  if (n_segments > STATIC_MAX_SEGMENTS || sel_layout(n_segments, 1).total > STATIC_SCRATCH_BYTES)
    return CAMERA_ERR_UNSUPPORTED_SHAPE;
  void* scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != CAMERA_OK) return rc;
  long long ranks[STATIC_MAX_SEGMENTS];
  for (int s = 0; s < n_segments; ++s) ranks[s] = floor_count(prune_ratio, seg_offsets[s + 1] - seg_offsets[s]);
  LevelValues lv;
  memset(&lv, 0, sizeof(lv));
  lv.v[0] = 1;
  lv.v[1] = 0;
  // select_core clears the histograms it counts into on every call; nothing else in the array has to start at zero
  return select_core(energy, seg_offsets, n_segments, 1, ranks, lv, nullptr, 0, 1, keep_mask, nullptr, thresholds, scratch,
                     STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(cuda_stream));
}
