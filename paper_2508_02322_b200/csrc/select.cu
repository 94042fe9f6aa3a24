// Device-wide segmented rank selection for CAMERA-P (Algorithm 2, TopSelect) and CAMERA-Q
// (Algorithm 3, ListSplitByRatio / GetSubIndex).
//
// Every micro-expert has the key (order-preserving image of its fp32 energy, index within its
// segment), compared lexicographically: keys are unique, "the r-th smallest key" is unambiguous and
// equal energies are ordered by index.  The key of rank r is found by a most-significant-digit radix
// select over the 32 energy bits, 4 digits of 8 bits: each pass builds a histogram (shared-memory
// bins, flushed with integer atomics, hence deterministic) of the next digit among the keys that
// match the digits found so far.  The index part only matters among the keys whose energy equals
// the threshold's, and only when some of them fall below it: then every CTA counts its share of them
// and the one CTA that holds the boundary finds it with an ordered scan.  Several ranks per segment
// (prune thresholds of several ratios, class boundaries) are selected in the same passes.
//
// All of it is ONE launch.  A segment is split over gridDim.x CTAs that keep their keys in shared
// memory and meet after every pass at a counter in global memory (five meetings at most).  CTAs that
// wait on one another must be resident together, so the kernel is launched cooperatively whenever a
// segment has more than one CTA, with a grid no larger than what fits the device at once; rows of
// CTAs walk over the segments.  The waits are bounded: one that runs out records
// CAMERA_ERR_DEVICE_TIMEOUT in the scratch's status word and the kernel returns.
#include <math.h>
#include <string.h>

#include <atomic>
#include <vector>

#include "common.cuh"
#include "umma.cuh"

namespace camera {

namespace {

constexpr int SEL_THREADS = 256;
constexpr int SEL_PASSES = 4;
constexpr int MAX_THR = MAX_LEVELS - 1;
constexpr int SEL_CTA_KEYS = 2048;        // keys a CTA takes when the device has CTAs to spare
constexpr int SEL_CACHE_KEYS = 6144;      // most keys a CTA keeps in shared memory (longer shares are re-read from L2);
                                          // six CTAs of 24 KB + 7 KB fit an SM
constexpr int SEL_MAX_GX = 2048;          // bound on CTAs per segment that the scratch is sized for
constexpr int SEL_PARAM_SEGS = 32;        // up to this many segments the offsets and ranks travel as kernel arguments
constexpr int SEL_BARS = 8;               // meeting counters per segment (5 used)

// First bytes of the scratch, laid out like the scoring workspace's so that camera_read_status reads either.
struct SelHeader {
  int32_t r0, r1;
  int32_t status;
  int32_t abort;      // set with the status: the other CTAs stop waiting
  int32_t pad[4];
};

// The selected key of one (segment, threshold): an element is at or above it when
// (bits, index) >= (bits, index) lexicographically; valid == 0: nothing is.
struct SelFinal {
  unsigned bits;
  unsigned index;
  int valid;
  int pad;
};

struct LevelValues { unsigned char v[MAX_LEVELS]; };

struct SelParams {
  long long seg_off[SEL_PARAM_SEGS + 1];
  long long ranks[SEL_PARAM_SEGS * MAX_THR];
};

struct SelArgs {
  const float* energy;
  const long long* seg_off;     // DEVICE copies when there are more than SEL_PARAM_SEGS segments, else null
  const long long* ranks;
  SelHeader* hdr;
  unsigned* bars;               // [n_seg][SEL_BARS], zero at launch
  unsigned* hist;               // [n_seg][SEL_PASSES][n_thr][256], zero at launch
  unsigned* eqcnt;              // [n_seg][n_thr][gridDim.x]
  SelFinal* fin;                // [n_seg][n_thr]
  int n_seg, n_thr;
  int n_prune;                  // >= 0: thresholds 0 .. n_prune-1 give keep masks, the rest class boundaries
  LevelValues lv;
  long long n_total;
  unsigned char* out;           // n_prune < 0: the label of every element; else n_prune masks of n_total bytes
  unsigned char* bits_out;      // n_prune >= 0: class values, or null
  float* thresholds;            // [n_seg] energy of threshold 0, or null
  unsigned long long wait_limit_ns;
};

__device__ __forceinline__ unsigned key_bits(float e) {
  const unsigned b = __float_as_uint(e);
  return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float bits_energy(unsigned b) {
  return __uint_as_float((b & 0x80000000u) ? (b ^ 0x80000000u) : ~b);
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// The CTAs of a segment meet: everything they wrote before is visible to all of them after.  Bounded: returns false
// (for the whole CTA) when the limit ran out here or in another CTA.
__device__ bool seg_meet(unsigned* counter, unsigned expected, const SelArgs& a, int* s_abort) {
  __syncthreads();
  if (threadIdx.x == 0) {
    if (expected > 1u) {
      __threadfence();
      atomicAdd(counter, 1u);
      const unsigned long long t0 = globaltimer_ns();
      unsigned spins = 0;
      while (ld_acquire_u32(counter) < expected) {
        if ((++spins & 15u) == 0u) {
          if (*reinterpret_cast<volatile int*>(&a.hdr->abort)) { *s_abort = 1; break; }
          if (globaltimer_ns() - t0 > a.wait_limit_ns) {
            atomicExch(&a.hdr->status, (int)CAMERA_ERR_DEVICE_TIMEOUT);
            atomicExch(&a.hdr->abort, 1);
            *s_abort = 1;
            break;
          }
        }
      }
      __threadfence();
    }
  }
  __syncthreads();
  return *s_abort == 0;
}

struct ThrState {
  unsigned prefix;      // digits found so far, in place
  int valid;            // 0: the rank is past the segment, nothing is at or above
  long long rank;       // rank still to find among the keys that match the prefix
};

__global__ void __launch_bounds__(SEL_THREADS, 6)
k_select_fused(const __grid_constant__ SelArgs a, const __grid_constant__ SelParams prm) {
  extern __shared__ unsigned skeys[];                 // [SEL_CACHE_KEYS] when the grid's shares fit, else unused
  __shared__ unsigned bins[MAX_THR][256];
  __shared__ ThrState st[MAX_THR];
  __shared__ unsigned eq_mine[MAX_THR];               // this CTA's keys whose energy equals the threshold's
  __shared__ unsigned first_above[MAX_THR];           // local index from which such keys are at or above the threshold
  __shared__ int boundary[MAX_THR];
  __shared__ int rep[MAX_THR];
  __shared__ unsigned lut[256];                       // by a key's last fixed digit: the thresholds it may match
  __shared__ unsigned pre_s[MAX_THR];
  __shared__ unsigned boundary_skip[MAX_THR];
  __shared__ unsigned wtot[SEL_THREADS / 32];
  __shared__ int s_abort;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_thr = a.n_thr;
  const unsigned gx = gridDim.x, bx = blockIdx.x;
  if (tid == 0) s_abort = 0;

  for (int seg = blockIdx.y; seg < a.n_seg; seg += gridDim.y) {
    const long long begin = a.seg_off ? a.seg_off[seg] : prm.seg_off[seg];
    const long long len = (a.seg_off ? a.seg_off[seg + 1] : prm.seg_off[seg + 1]) - begin;
    if (len == 0) {                                    // the same for every CTA of the row: nothing to select from
      if (bx == 0 && tid < n_thr) {
        SelFinal f;
        f.bits = 0u; f.index = 0u; f.valid = 0; f.pad = 0;
        a.fin[(size_t)seg * n_thr + tid] = f;
        if (tid == 0 && a.thresholds != nullptr) a.thresholds[seg] = INFINITY;
      }
      continue;
    }
    const long long per = ((len + gx - 1) / gx + 3) & ~3ll;          // shares start on multiples of 4 keys
    const long long c0 = per * bx < len ? per * bx : len;
    const int n = (int)((c0 + per < len ? c0 + per : len) - c0);       // this CTA's share: [c0, c0 + n) of the segment
    const bool cached = per <= SEL_CACHE_KEYS;
    const float* src = a.energy + begin + c0;
    if (cached)
      for (int i = tid; i < n; i += SEL_THREADS) skeys[i] = key_bits(src[i]);
    if (tid < n_thr) {
      const long long r = a.ranks ? a.ranks[(size_t)seg * n_thr + tid] : prm.ranks[seg * n_thr + tid];
      st[tid].prefix = 0u;
      st[tid].valid = r >= 0 && r < len;
      st[tid].rank = r;
      eq_mine[tid] = 0u;
      first_above[tid] = 0u;
      boundary[tid] = 0;
      rep[tid] = tid;
    }
    unsigned* const hseg = a.hist + (size_t)seg * SEL_PASSES * n_thr * 256;
    unsigned* const bseg = a.bars + (size_t)seg * SEL_BARS;

    for (int pass = 0; pass < SEL_PASSES; ++pass) {
      const int nh = pass == 0 ? 1 : n_thr;            // the first digit's histogram serves every threshold
      for (int i = tid; i < nh * 256; i += SEL_THREADS) (&bins[0][0])[i] = 0u;
      __syncthreads();
      const int shift = 24 - 8 * pass;
      if (pass == 0) {
        // energies of one layer share their leading bits: a thread counts runs of equal digits in a register and
        // touches the bin once per run, not once per key
        unsigned run_digit = 0u, run_len = 0u;
        auto count_first = [&](unsigned b) {
          const unsigned digit = b >> 24;
          if (digit != run_digit) {
            if (run_len) atomicAdd(&bins[0][run_digit], run_len);
            run_digit = digit;
            run_len = 0u;
          }
          ++run_len;
        };
        if (cached) {
          const uint4* k4 = reinterpret_cast<const uint4*>(skeys);
          for (int q = tid; 4 * q < n; q += SEL_THREADS) {
            const uint4 kk = k4[q];
            count_first(kk.x);
            if (4 * q + 1 < n) count_first(kk.y);
            if (4 * q + 2 < n) count_first(kk.z);
            if (4 * q + 3 < n) count_first(kk.w);
          }
        } else {
          for (int i = tid; i < n; i += SEL_THREADS) count_first(key_bits(src[i]));
        }
        if (run_len) atomicAdd(&bins[0][run_digit], run_len);
      } else {
        // Thresholds whose digits so far agree share one histogram (that of the lowest-numbered among them).  Most
        // keys match none: a table on the last digit found says which thresholds a key can match at all.
        for (int i = tid; i < 256; i += SEL_THREADS) lut[i] = 0u;
        __syncthreads();
        if (tid < n_thr && st[tid].valid && rep[tid] == tid) {
          pre_s[tid] = st[tid].prefix >> (shift + 8);
          atomicOr(&lut[pre_s[tid] & 0xffu], 1u << tid);
        }
        __syncthreads();
        // the thresholds that count in this pass, in order; with one or two of them (the rule while the thresholds'
        // leading digits still agree, when every key of a narrow energy range is a candidate) a key is compared with
        // them directly
        int n_act = 0, j0 = 0, j1 = 0;
        unsigned p0 = 0xffffffffu, p1 = 0xffffffffu;
        for (int j = 0; j < n_thr; ++j)
          if (st[j].valid && rep[j] == j) {
            if (n_act == 0) { j0 = j; p0 = st[j].prefix >> (shift + 8); }
            else if (n_act == 1) { j1 = j; p1 = st[j].prefix >> (shift + 8); }
            ++n_act;
          }
        const bool few = n_act <= 2;
        auto count_key = [&](unsigned b) {
          const unsigned hi = b >> (shift + 8), digit = (b >> shift) & 0xffu;
          if (few) {
            if (hi == p0) atomicAdd(&bins[j0][digit], 1u);
            else if (hi == p1) atomicAdd(&bins[j1][digit], 1u);
            return;
          }
          unsigned cand = lut[hi & 0xffu];
          while (cand) {
            const int j = __ffs(cand) - 1;
            cand &= cand - 1u;
            if (hi == pre_s[j]) atomicAdd(&bins[j][digit], 1u);
          }
        };
        if (cached) {
          const uint4* k4 = reinterpret_cast<const uint4*>(skeys);
          for (int q = tid; 4 * q < n; q += SEL_THREADS) {
            const uint4 kk = k4[q];
            count_key(kk.x);
            if (4 * q + 1 < n) count_key(kk.y);
            if (4 * q + 2 < n) count_key(kk.z);
            if (4 * q + 3 < n) count_key(kk.w);
          }
        } else {
          for (int i = tid; i < n; i += SEL_THREADS) count_key(key_bits(src[i]));
        }
      }
      __syncthreads();
      for (int i = tid; i < nh * 256; i += SEL_THREADS) {
        const unsigned v = (&bins[0][0])[i];
        if (v) atomicAdd(hseg + (size_t)pass * n_thr * 256 + i, v);
      }
      if (!seg_meet(bseg + pass, gx, a, &s_abort)) return;
      // warp j: the bin of threshold j's rank in the segment's histogram of this digit
      if (warp < n_thr && st[warp].valid) {
        const unsigned* h = hseg + ((size_t)pass * n_thr + (pass == 0 ? 0 : rep[warp])) * 256;
        unsigned v[8];
        long long mine = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { v[i] = __ldcg(h + lane * 8 + i); mine += v[i]; }     // lane owns bins [8 lane, 8 lane + 8)
        long long incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const long long t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        long long before = incl - mine;
        const long long rank = st[warp].rank;
        if (rank >= before && rank < incl) {           // exactly one lane, for a rank inside the segment
          int bin = lane * 8;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (rank >= before + (long long)v[i]) { before += v[i]; bin = lane * 8 + i + 1; }
            else break;
          }
          st[warp].prefix |= (unsigned)bin << shift;
          st[warp].rank = rank - before;
        }
      }
      __syncthreads();
      if (tid < n_thr && pass + 1 < SEL_PASSES) {       // whose histogram threshold tid reads in the next pass
        int r = tid;
        for (int j = tid - 1; j >= 0; --j)
          if (st[j].valid && st[tid].valid && st[j].prefix == st[tid].prefix) r = j;
        rep[tid] = r;
      }
      // (the barrier after the bins are cleared orders this before the next pass reads it)
    }

    // Keys whose energy equals a threshold's: the st.rank lowest-indexed of them are below it.  With rank 0 (always,
    // when the threshold's energy occurs once) all are at or above and nothing more is needed.  Otherwise the CTAs
    // count theirs, and the one CTA whose share holds the first such key at or above the threshold looks it up.
    bool ties = false;
    for (int j = 0; j < n_thr; ++j) ties = ties || (st[j].valid && st[j].rank > 0);
    if (ties) {
      // how many such keys this CTA holds: its own count of the threshold's last digit in the last pass (the bins still
      // hold the CTA's counts; `rep` still says whose bins a threshold counted into)
      if (tid < n_thr) eq_mine[tid] = st[tid].valid ? bins[rep[tid]][st[tid].prefix & 0xffu] : 0u;
      __syncthreads();
      if (tid < n_thr) a.eqcnt[((size_t)seg * n_thr + tid) * gx + bx] = eq_mine[tid];
      if (!seg_meet(bseg + SEL_PASSES, gx, a, &s_abort)) return;
      if (warp < n_thr && st[warp].valid && st[warp].rank > 0) {
        const unsigned* ec = a.eqcnt + ((size_t)seg * n_thr + warp) * gx;
        long long base = 0;                            // such keys in the CTAs before this one
        for (unsigned c = lane; c < bx; c += 32) base += __ldcg(ec + c);
#pragma unroll
        for (int o = 16; o; o >>= 1) base += __shfl_xor_sync(0xffffffffu, base, o);
        if (lane == 0) {
          const long long r = st[warp].rank, mine = eq_mine[warp];
          if (base + mine <= r) first_above[warp] = 0xffffffffu;       // all of this CTA's are below
          else if (base > r) first_above[warp] = 0u;                   // all are at or above
          else { boundary[warp] = 1; boundary_skip[warp] = (unsigned)(r - base); }   // it holds the first one at or above
        }
      }
      __syncthreads();
      // the one CTA that holds the boundary: the local index of its boundary_skip-th such key.  A thread counts the
      // matches in its own run of consecutive keys, one scan over the threads orders the runs, and the thread whose
      // run holds the key walks to it.
      for (int j = 0; j < n_thr; ++j) {
        if (!boundary[j]) continue;                    // the same for every thread
        const unsigned want = boundary_skip[j], tau = st[j].prefix;
        const int run_len = (n + SEL_THREADS - 1) / SEL_THREADS;
        const int i0 = min(n, tid * run_len), i1 = min(n, i0 + run_len);
        unsigned c = 0u;
        for (int i = i0; i < i1; ++i) c += (cached ? skeys[i] : key_bits(src[i])) == tau;
        unsigned incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        if (lane == 31) wtot[warp] = incl;
        __syncthreads();
        unsigned before = incl - c;
#pragma unroll
        for (int w = 0; w < SEL_THREADS / 32; ++w) before += w < warp ? wtot[w] : 0u;
        if (before <= want && want < before + c) {     // exactly one thread
          unsigned seen = before;
          for (int i = i0; i < i1; ++i)
            if ((cached ? skeys[i] : key_bits(src[i])) == tau && seen++ == want) { first_above[j] = (unsigned)i; break; }
        }
        __syncthreads();
      }
    }

    // the selected keys, for the per-expert counts and the thresholds' energies
    if (tid < n_thr) {
      const bool writer = st[tid].valid && st[tid].rank > 0 ? boundary[tid] != 0 : bx == 0;
      if (writer) {
        SelFinal f;
        f.bits = st[tid].prefix;
        f.index = st[tid].valid ? (unsigned)(c0 + (boundary[tid] ? first_above[tid] : 0u)) : 0u;
        f.valid = st[tid].valid;
        f.pad = 0;
        a.fin[(size_t)seg * n_thr + tid] = f;
      }
      if (tid == 0 && bx == 0 && a.thresholds != nullptr)
        a.thresholds[seg] = st[0].valid ? bits_energy(st[0].prefix) : INFINITY;
    }

    // labels
    unsigned tau[MAX_THR];
    unsigned valid_mask = 0u;
    bool any_first = false;                            // some threshold cuts through a run of equal energies
#pragma unroll
    for (int j = 0; j < MAX_THR; ++j) {
      const bool v = j < n_thr && st[j].valid;
      tau[j] = v ? st[j].prefix : 0xffffffffu;
      valid_mask |= (unsigned)v << j;
      any_first = any_first || (v && first_above[j] != 0u);
    }
    const int n_prune = a.n_prune, n_bounds = n_thr - (n_prune < 0 ? 0 : n_prune);
    // bit j of the result: the key at local index i is at or above threshold j
    auto at_of = [&](unsigned b, int i) {
      unsigned at = 0u;
#pragma unroll
      for (int j = 0; j < MAX_THR; ++j) at |= (unsigned)(b >= tau[j]) << j;
      at &= valid_mask;
      if (any_first) {                                 // keys equal to a threshold's energy: below it before `first_above`
#pragma unroll
        for (int j = 0; j < MAX_THR; ++j)
          if (b == tau[j] && (unsigned)i < first_above[j]) at &= ~(1u << j);
      }
      return at;
    };
    const size_t g0 = (size_t)(begin + c0);
    const bool words = cached && (g0 % 4 == 0) && (a.n_total % 4 == 0) && (reinterpret_cast<uintptr_t>(a.out) % 4 == 0) &&
                       (a.bits_out == nullptr || reinterpret_cast<uintptr_t>(a.bits_out) % 4 == 0);
    if (words) {       // four keys per step, their labels in one 32-bit store per output
      // label table by the number c of boundaries a key is at or above: byte c = lv[(boundaries) - c]
      const int n_b = n_prune < 0 ? n_thr : n_bounds;
      unsigned lab_lo = 0u, lab_hi = 0u;
      for (int cnt = 0; cnt <= n_b; ++cnt) {
        const unsigned v = a.lv.v[n_b - cnt];
        if (cnt < 4) lab_lo |= v << (8 * cnt); else lab_hi |= v << (8 * (cnt - 4));
      }
      const unsigned bound_bits4 = ((1u << n_bounds) - 1u) * 0x01010101u;
      const uint4* k4 = reinterpret_cast<const uint4*>(skeys);
      for (int q = tid; 4 * q < n; q += SEL_THREADS) {
        const uint4 kk = k4[q];
        const int i = 4 * q;
        const unsigned at0 = at_of(kk.x, i), at1 = at_of(kk.y, i + 1), at2 = at_of(kk.z, i + 2), at3 = at_of(kk.w, i + 3);
        const bool full = i + 3 < n;
        const size_t g = g0 + i;
        auto put = [&](unsigned char* base, unsigned w) {
          if (full) *reinterpret_cast<unsigned*>(base + g) = w;
          else
            for (int r = 0; i + r < n; ++r) base[g + r] = (unsigned char)(w >> (8 * r));
        };
        // the four keys' bits side by side, one byte per key: mask j is bit j of every byte, the class of a key the
        // number of its boundary bits (counted in all four bytes at once), the label a byte picked from the table
        const unsigned w4 = at0 | (at1 << 8) | (at2 << 16) | (at3 << 24);
        auto labels_of = [&](unsigned bits4) {       // per byte: lv[(number of boundaries) - popcount(byte)]
          unsigned x = bits4;
          x -= (x >> 1) & 0x55555555u;
          x = (x & 0x33333333u) + ((x >> 2) & 0x33333333u);
          x = (x + (x >> 4)) & 0x0f0f0f0fu;
          const unsigned sel = (x & 0xfu) | ((x >> 4) & 0xf0u) | ((x >> 8) & 0xf00u) | ((x >> 12) & 0xf000u);
          return __byte_perm(lab_lo, lab_hi, sel);
        };
        if (n_prune < 0) {
          put(a.out, labels_of(w4));
        } else {
          for (int j = 0; j < n_prune; ++j) put(a.out + (size_t)j * a.n_total, (w4 >> j) & 0x01010101u);
          if (a.bits_out != nullptr) put(a.bits_out, labels_of((w4 >> n_prune) & bound_bits4));
        }
      }
    } else {
      for (int i = tid; i < n; i += SEL_THREADS) {
        const unsigned at = at_of(cached ? skeys[i] : key_bits(src[i]), i);
        const size_t g = g0 + i;
        if (n_prune < 0) {
          a.out[g] = a.lv.v[n_thr - __popc(at)];
        } else {
          for (int j = 0; j < n_prune; ++j) a.out[(size_t)j * a.n_total + g] = (at >> j) & 1u;
          if (a.bits_out != nullptr) a.bits_out[g] = a.lv.v[n_bounds - __popc(at >> n_prune)];
        }
      }
    }
    __syncthreads();       // the next segment reuses the shared arrays
  }
}

// One CTA per expert: how many of its micro-experts fall in each class (or are retained).
__global__ void __launch_bounds__(SEL_THREADS)
k_class_counts(const float* __restrict__ energy, const long long* seg_off, const SelFinal* fin, int n_seg, int n_thr,
               const long long* expert_off, int n_classes_out, int* counts) {
  __shared__ int cnt[MAX_LEVELS];
  const int e = blockIdx.x;
  const long long b = expert_off[e], en = expert_off[e + 1];
  if (threadIdx.x < MAX_LEVELS) cnt[threadIdx.x] = 0;
  __syncthreads();
  if (en > b) {
    const int seg = upper_segment(seg_off, n_seg, b);
    const SelFinal* f = fin + (size_t)seg * n_thr;
    int local[MAX_LEVELS];
#pragma unroll
    for (int j = 0; j < MAX_LEVELS; ++j) local[j] = 0;
    for (long long i = b + threadIdx.x; i < en; i += SEL_THREADS) {
      const unsigned kb = key_bits(energy[i]), idx = (unsigned)(i - seg_off[seg]);
      int above = 0;
      for (int j = 0; j < n_thr; ++j)
        above += (f[j].valid && (kb > f[j].bits || (kb == f[j].bits && idx >= f[j].index))) ? 1 : 0;
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

// CTAs per segment the scratch has room for: never more than the kernel is given.
int sel_gx_bound(long long n_total, int n_seg) {
  long long by_keys = (n_total + SEL_CTA_KEYS - 1) / SEL_CTA_KEYS;
  long long by_segs = SEL_MAX_GX / (n_seg < SEL_MAX_GX ? n_seg : SEL_MAX_GX);
  long long g = by_keys < by_segs ? by_keys : by_segs;
  return (int)(g < 1 ? 1 : g);
}

struct SelLayout {
  size_t hdr, bars, hist, zero_bytes, fin, eqcnt, seg_off, ranks, total;
};

SelLayout sel_layout(long long n_total, int n_seg, int n_thr) {
  auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
  SelLayout L;
  size_t o = 0;
  L.hdr = o;     o = up(o + sizeof(SelHeader));
  L.bars = o;    o = up(o + sizeof(unsigned) * (size_t)n_seg * SEL_BARS);
  L.hist = o;    o = up(o + sizeof(unsigned) * (size_t)SEL_PASSES * n_seg * n_thr * 256);
  L.zero_bytes = o;                                   // everything up to here starts at zero, in one memset
  L.fin = o;     o = up(o + sizeof(SelFinal) * (size_t)n_seg * n_thr);
  L.eqcnt = o;   o = up(o + sizeof(unsigned) * (size_t)n_seg * n_thr * sel_gx_bound(n_total, n_seg));
  L.seg_off = o; o = up(o + sizeof(long long) * (n_seg + 1));
  L.ranks = o;   o = up(o + sizeof(long long) * (size_t)n_seg * n_thr);
  L.total = o;
  return L;
}

long long floor_count(double ratio, long long n) { return (long long)floor(ratio * (double)n + 1e-9); }

// CTAs of k_select_fused that are resident at once on the current device (0 on error); asked once per device.
int resident_ctas(size_t smem) {
  constexpr int MAX_DEV = 64;
  static int cache[MAX_DEV];      // 0 = not asked yet
  int dev = 0, sms = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
  if (dev >= 0 && dev < MAX_DEV && cache[dev] > 0) return cache[dev];
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaFuncSetAttribute(k_select_fused, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_select_fused, SEL_THREADS, smem) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  if (dev >= 0 && dev < MAX_DEV) cache[dev] = sms * per_sm;
  return sms * per_sm;
}

// ranks_host: [n_seg * n_thr] target ascending ranks (a rank >= the segment length selects nothing).
// n_prune >= 0 selects the labelling of camera_select_all: `out` then holds n_prune masks of seg_offsets[n_seg] bytes
// and bits_out (may be null) gets the class values.
int select_core(const float* energy, const int64_t* seg_offsets, int n_seg, int n_thr, const long long* ranks_host,
                LevelValues lv, const int64_t* expert_offsets, int n_experts, int n_classes_out, unsigned char* out,
                int* counts, float* thresholds, void* ws, size_t ws_bytes, cudaStream_t st, int n_prune = -1,
                unsigned char* bits_out = nullptr) {
  const long long n_total = seg_offsets[n_seg];
  const SelLayout L = sel_layout(n_total, n_seg, n_thr);
  if (ws == nullptr || ws_bytes < L.total || (reinterpret_cast<uintptr_t>(ws) & 255)) return CAMERA_ERR_WORKSPACE;
  char* base = static_cast<char*>(ws);
  long long max_len = 0;
  for (int s = 0; s < n_seg; ++s) max_len = seg_offsets[s + 1] - seg_offsets[s] > max_len ? seg_offsets[s + 1] - seg_offsets[s] : max_len;

  SelArgs a;
  memset(&a, 0, sizeof(a));
  SelParams prm;
  memset(&prm, 0, sizeof(prm));
  a.energy = energy;
  a.hdr = reinterpret_cast<SelHeader*>(base + L.hdr);
  a.bars = reinterpret_cast<unsigned*>(base + L.bars);
  a.hist = reinterpret_cast<unsigned*>(base + L.hist);
  a.eqcnt = reinterpret_cast<unsigned*>(base + L.eqcnt);
  a.fin = reinterpret_cast<SelFinal*>(base + L.fin);
  a.n_seg = n_seg; a.n_thr = n_thr; a.n_prune = n_prune; a.lv = lv; a.n_total = n_total;
  a.out = out; a.bits_out = bits_out; a.thresholds = thresholds;
  a.wait_limit_ns = current_wait_limit_ns();
  long long* d_seg = reinterpret_cast<long long*>(base + L.seg_off);
  if (n_seg <= SEL_PARAM_SEGS) {
    for (int s = 0; s <= n_seg; ++s) prm.seg_off[s] = seg_offsets[s];
    for (int i = 0; i < n_seg * n_thr; ++i) prm.ranks[i] = ranks_host[i];
  } else {
    a.seg_off = d_seg;
    a.ranks = reinterpret_cast<long long*>(base + L.ranks);
    if (cudaMemcpyAsync(d_seg, seg_offsets, sizeof(long long) * (n_seg + 1), cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(const_cast<long long*>(a.ranks), ranks_host, sizeof(long long) * (size_t)n_seg * n_thr,
                        cudaMemcpyHostToDevice, st) != cudaSuccess) {
      cudaGetLastError();
      return CAMERA_ERR_CUDA;
    }
  }
  if (cudaMemsetAsync(base, 0, L.zero_bytes, st) != cudaSuccess) { cudaGetLastError(); return CAMERA_ERR_CUDA; }

  {   // empty segments get their thresholds (infinity) from the kernel too
    const size_t smem = sizeof(unsigned) * SEL_CACHE_KEYS;
    const int resident = resident_ctas(smem);
    if (resident < 1) return CAMERA_ERR_CUDA;
    // CTAs per segment: shares of SEL_CTA_KEYS keys while the device has room, never more than the scratch holds
    long long gx = (max_len + SEL_CTA_KEYS - 1) / SEL_CTA_KEYS;
    const int rows_wanted = n_seg < resident ? n_seg : resident;
    if (gx > resident / rows_wanted) gx = resident / rows_wanted;
    const int bound = sel_gx_bound(n_total, n_seg);
    if (gx > bound) gx = bound;
    if (gx < 1) gx = 1;
    long long gy = resident / gx;
    if (gy > n_seg) gy = n_seg;
    if (gy > 65535) gy = 65535;
    bool launched = false;
    if (gx > 1) {     // CTAs of a segment wait for one another: they must all be resident
      void* args[2] = {&a, &prm};
      launched = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(k_select_fused), dim3((unsigned)gx, (unsigned)gy),
                                             dim3(SEL_THREADS), args, smem, st) == cudaSuccess;
      if (!launched) {      // a context without cooperative launches: one CTA per segment, which waits for nobody
        cudaGetLastError();
        gx = 1;
        gy = n_seg < 65535 ? n_seg : 65535;
      }
    }
    if (!launched) k_select_fused<<<dim3((unsigned)gx, (unsigned)gy), SEL_THREADS, smem, st>>>(a, prm);
  }
  if (counts != nullptr && expert_offsets != nullptr && n_experts > 0) {
    if (max_len > 0) {
      if (a.seg_off == nullptr &&
          cudaMemcpyAsync(d_seg, seg_offsets, sizeof(long long) * (n_seg + 1), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return CAMERA_ERR_CUDA;
      }
      k_class_counts<<<n_experts, SEL_THREADS, 0, st>>>(energy, d_seg, a.fin, n_seg, n_thr,
                                                        reinterpret_cast<const long long*>(expert_offsets), n_classes_out, counts);
    } else if (cudaMemsetAsync(counts, 0, sizeof(int) * (size_t)n_experts * n_classes_out, st) != cudaSuccess) {
      cudaGetLastError();
      return CAMERA_ERR_CUDA;
    }
  }
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}

bool segments_ok(const int64_t* seg, int n_seg) {
  if (seg == nullptr || n_seg < 1 || n_seg > 65535 || seg[0] != 0) return false;
  for (int s = 0; s < n_seg; ++s)
    if (seg[s + 1] < seg[s] || seg[s + 1] - seg[s] > 0x7fff0000ll) return false;
  return true;
}

}  // namespace
}  // namespace camera

using namespace camera;

extern "C" size_t camera_select_workspace_bytes(int64_t n_total, int32_t n_segments, int32_t n_levels) {
  if (n_total < 0 || n_segments < 1 || n_segments > 65535 || n_levels < 2 || n_levels > MAX_LEVELS) return 0;
  return sel_layout(n_total, n_segments, n_levels - 1).total;
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
std::atomic<void*> g_scratch_ptr[STATIC_MAX_DEVICES];     // device address of g_select_scratch per device ordinal; null = not asked yet

// In host code `g_select_scratch` is only a handle; the address kernels can use has to be asked for,
// once per device, while that device is current.  Two host threads that ask at the same time get the same answer.
int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return CAMERA_ERR_CUDA;
  void* p = g_scratch_ptr[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return CAMERA_ERR_CUDA;
    }
    g_scratch_ptr[dev].store(p, std::memory_order_release);
  }
  *out = p;
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
  if (n_segments > STATIC_MAX_SEGMENTS || sel_layout(seg_offsets[n_segments], n_segments, 1).total > STATIC_SCRATCH_BYTES)
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
  // select_core clears what has to start at zero (status word, meeting counters, histograms) on the stream, every call
  return select_core(energy, seg_offsets, n_segments, 1, ranks, lv, nullptr, 0, 1, keep_mask, nullptr, thresholds, scratch,
                     STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(cuda_stream));
}
