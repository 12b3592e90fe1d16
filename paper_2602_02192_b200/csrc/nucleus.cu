// Nucleus (top-p) cut of a logits row (Section 5.1 samples with top-p 0.95).
//
// The nucleus of a row is the shortest prefix, in order of decreasing score s = z / T (equal
// scores: increasing id), whose softmax mass reaches top_p.  This kernel finds the LAST member of
// that prefix, the "cut" (its score as an order-preserving 32-bit key, and its id); the sampler
// then keeps exactly the ids that rank at or before the cut.  No sort of the vocabulary:
//   pass 0   max, min and sum of exp over the row;
//   level l  a histogram of probability mass (fixed point) over 2048 equal score bins of the current interval
//            (shared-memory atomics), a block-wide scan for the bin in which the cumulative mass
//            crosses top_p, and the interval shrinks to that bin - until the bin holds at most
//            kCand ids (one level for a vocabulary of 150k with spread-out logits);
//   finish   the ids of that bin are gathered, sorted by (score descending, id ascending) in shared
//            memory, and one thread walks them adding mass until the target is reached.
// Rows whose boundary bin cannot be resolved by score (more than kCand ids with one and the same
// score, e.g. an all-equal row) are cut by id: the k lowest ids of the tied set that are still
// needed, found with the same histogram-and-shrink scheme over the id range.
// One CTA of 1024 threads per logits row.

#include "common.cuh"

namespace echo {

namespace {

constexpr int kNucThreads = 1024;
constexpr int kNucBins = 2048;                 // bins per level (2 per thread)
constexpr int kPerThread = kNucBins / kNucThreads;
// Probability mass is summed in 2^-40 fixed point: tens of thousands of equal addends per bin make
// a float sum drift by 1e-4 of the total, more than one vocabulary entry weighs.
constexpr double kFix = 1099511627776.0;       // 2^40
__device__ __forceinline__ unsigned long long to_fix(float e) {
  return static_cast<unsigned long long>(static_cast<double>(e) * kFix);
}
constexpr int kCand = 1024;                    // ids sorted in shared memory at the end
constexpr int kMaxLevels = 6;

__device__ __forceinline__ float key_to_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

struct Levels {
  float hi[kMaxLevels], width[kMaxLevels];
  int pick[kMaxLevels];
  int n;
};
// bin of score s at level l (bin 0 holds the highest scores)
__device__ __forceinline__ int level_bin(const Levels &L, int l, float s) {
  const int b = static_cast<int>((L.hi[l] - s) / L.width[l]);
  return b < 0 ? 0 : (b >= kNucBins ? kNucBins - 1 : b);
}
// -1: s ranks above the current interval (already counted), 0: inside it, +1: below it
__device__ __forceinline__ int locate(const Levels &L, float s) {
  for (int l = 0; l < L.n; ++l) {
    const int b = level_bin(L, l, s);
    if (b != L.pick[l]) return b < L.pick[l] ? -1 : 1;
  }
  return 0;
}

// Block-wide: first non-empty bin b with base + (hist[0] + ... + hist[b]) >= target; returns it and
// the mass before it.  When rounding leaves the total short of the target, the last non-empty bin.
__device__ void find_crossing(const unsigned long long *hist, const int *cnt, unsigned long long base,
                              unsigned long long target, unsigned long long *scratch, int *out_bin,
                              unsigned long long *out_before) {
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  __shared__ int s_best, s_last;
  unsigned long long v[kPerThread], sum = 0;
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    v[i] = hist[kPerThread * t + i];
    sum += v[i];
  }
  unsigned long long incl = sum;                         // inclusive scan of per-thread sums
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) scratch[warp] = incl;
  if (t == 0) {
    s_best = kNucBins;
    s_last = -1;
  }
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = scratch[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long n = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += n;
    }
    scratch[32 + lane] = w;                              // inclusive scan of warp totals
  }
  __syncthreads();
  const unsigned long long before_thread = base + (warp ? scratch[32 + warp - 1] : 0ull) + (incl - sum);
  unsigned long long run = before_thread;
  int mine = kNucBins;
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    if (cnt[kPerThread * t + i] > 0) atomicMax(&s_last, kPerThread * t + i);
    if (mine == kNucBins && run + v[i] >= target && cnt[kPerThread * t + i] > 0) mine = kPerThread * t + i;
    if (mine == kNucBins) run += v[i];
  }
  if (mine < kNucBins) atomicMin(&s_best, mine);
  __syncthreads();
  const int best = s_best < kNucBins ? s_best : (s_last < 0 ? 0 : s_last);
  if (best / kPerThread == t) {
    unsigned long long b = before_thread;
    for (int i = 0; i < best % kPerThread; ++i) b += v[i];
    *out_before = b;
    *out_bin = best;
  }
  __syncthreads();
}


__device__ __forceinline__ void lse_join(float &m, float &l, float m2, float l2) {
  if (m2 == -INFINITY) return;
  if (m == -INFINITY) {
    m = m2;
    l = l2;
    return;
  }
  const float mm = fmaxf(m, m2);
  l = l * __expf(m - mm) + l2 * __expf(m2 - mm);
  m = mm;
}

// Sorts keys[0, n_pow2) ascending in shared memory (bitonic; n_pow2 a power of two <= 2 * blockDim).
__device__ void sort_shared(unsigned long long *keys, int n_pow2) {
  for (int k = 2; k <= n_pow2; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = threadIdx.x; i < n_pow2; i += blockDim.x) {
        const int ixj = i ^ j;
        if (ixj > i) {
          const unsigned long long a = keys[i], b = keys[ixj];
          const bool up = (i & k) == 0;
          if ((a > b) == up) {
            keys[i] = b;
            keys[ixj] = a;
          }
        }
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(kNucThreads)
nucleus_cut_kernel(const float *__restrict__ logits, int V, float inv_temperature, float top_p,
                   uint2 *__restrict__ cut) {
  __shared__ unsigned long long hist[kNucBins];
  __shared__ int cnt[kNucBins];
  __shared__ unsigned long long cand[kCand];
  __shared__ unsigned long long scratch[64];
  __shared__ float red_m[32], red_l[32], red_min[32];
  __shared__ int s_bin, s_n;
  __shared__ unsigned long long s_before;
  early_start_sync();
  const float *z = logits + static_cast<size_t>(blockIdx.x) * V;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;

  // ---- pass 0: max, sum of exp, min ------------------------------------------------------------
  float m = -INFINITY, l = 0.f, smin = INFINITY;
  for (int v = t; v < V; v += kNucThreads) {
    const float s = z[v] * inv_temperature;
    if (s > m) {
      l = l * __expf(m - s) + 1.0f;
      m = s;
    } else {
      l += __expf(s - m);
    }
    smin = fminf(smin, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lse_join(m, l, __shfl_xor_sync(0xffffffffu, m, o), __shfl_xor_sync(0xffffffffu, l, o));
    smin = fminf(smin, __shfl_xor_sync(0xffffffffu, smin, o));
  }
  if (lane == 0) {
    red_m[warp] = m;
    red_l[warp] = l;
    red_min[warp] = smin;
  }
  __syncthreads();
  m = -INFINITY, l = 0.f, smin = INFINITY;
  for (int w = 0; w < kNucThreads / 32; ++w) {          // same order in every thread
    lse_join(m, l, red_m[w], red_l[w]);
    smin = fminf(smin, red_min[w]);
  }
  // mass in units of exp(s - m), fixed point
  const unsigned long long target = static_cast<unsigned long long>(static_cast<double>(top_p) * l * kFix);

  // ---- shrink the score interval until the boundary bin is small -------------------------------
  Levels L;
  L.n = 0;
  unsigned long long mass_above = 0;
  float hi = m, width = (m - smin) / kNucBins;
  int members = V;
  bool tied = !(width > 0.f);                            // the whole row is one score
  while (!tied && members > kCand && L.n < kMaxLevels) {
    const int lv = L.n;
    L.hi[lv] = hi;
    L.width[lv] = width;
    for (int i = t; i < kNucBins; i += kNucThreads) {
      hist[i] = 0ull;
      cnt[i] = 0;
    }
    __syncthreads();
    for (int v = t; v < V; v += kNucThreads) {
      const float s = z[v] * inv_temperature;
      if (locate(L, s) == 0) {
        const int b = level_bin(L, lv, s);
        atomicAdd(&hist[b], to_fix(__expf(s - m)));
        atomicAdd(&cnt[b], 1);
      }
    }
    __syncthreads();
    find_crossing(hist, cnt, mass_above, target, scratch, &s_bin, &s_before);
    L.pick[lv] = s_bin;
    L.n = lv + 1;
    mass_above = s_before;
    members = cnt[s_bin];
    hi = hi - s_bin * width;
    const float w2 = width / kNucBins;
    tied = !(w2 > 0.f) || !(hi - w2 < hi);               // the bin cannot be divided any further
    width = w2;
    __syncthreads();
  }

  if (members <= kCand) {
    // ---- gather the boundary bin, sort it, walk it ---------------------------------------------
    if (t == 0) s_n = 0;
    for (int i = t; i < kCand; i += kNucThreads) cand[i] = ~0ull;
    __syncthreads();
    for (int v = t; v < V; v += kNucThreads) {
      const float s = z[v] * inv_temperature;
      if (locate(L, s) == 0) {
        const int slot = atomicAdd(&s_n, 1);
        if (slot < kCand)                                  // (descending score, ascending id) as one ascending key
          cand[slot] = (static_cast<unsigned long long>(~order_key(s)) << 32) | static_cast<uint32_t>(v);
      }
    }
    __syncthreads();
    sort_shared(cand, kCand);
    if (t == 0) {
      const int n = s_n < kCand ? s_n : kCand;
      unsigned long long acc = mass_above;
      uint2 c = make_uint2(0u, 0x7fffffffu);             // nothing gathered: keep every id
      for (int i = 0; i < n; ++i) {
        const uint32_t key = ~static_cast<uint32_t>(cand[i] >> 32);
        c = make_uint2(key, static_cast<uint32_t>(cand[i] & 0xffffffffu));
        acc += to_fix(__expf(key_to_float(key) - m));
        if (acc >= target) break;
      }
      cut[blockIdx.x] = c;
    }
    return;
  }

  // ---- more than kCand ids share the boundary score: cut by id ---------------------------------
  // the tied set = ids inside the current interval; its score = the highest one in it
  float s_tie = -INFINITY;
  for (int v = t; v < V; v += kNucThreads) {
    const float s = z[v] * inv_temperature;
    if (locate(L, s) == 0) s_tie = fmaxf(s_tie, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s_tie = fmaxf(s_tie, __shfl_xor_sync(0xffffffffu, s_tie, o));
  if (lane == 0) red_m[warp] = s_tie;
  __syncthreads();
  for (int w = 0; w < kNucThreads / 32; ++w) s_tie = fmaxf(s_tie, red_m[w]);
  const unsigned long long each = to_fix(__expf(s_tie - m));
  // ids of the tied set still needed
  long need = target > mass_above && each > 0 ? static_cast<long>((target - mass_above + each - 1) / each) : 1;
  if (need < 1) need = 1;
  if (need >= members) {
    if (t == 0) cut[blockIdx.x] = make_uint2(order_key(s_tie), 0x7fffffffu);
    return;
  }
  // the need-th lowest id of the tied set: histogram of counts over id ranges, shrink, repeat
  int id_lo = 0, id_hi = V;                                // [id_lo, id_hi)
  long before = 0;
  for (int round = 0; round < 4; ++round) {
    const int span = id_hi - id_lo;
    const int wid = (span + kNucBins - 1) / kNucBins;
    for (int i = t; i < kNucBins; i += kNucThreads) cnt[i] = 0;
    __syncthreads();
    for (int v = id_lo + t; v < id_hi; v += kNucThreads) {
      const float s = z[v] * inv_temperature;
      if (locate(L, s) == 0) atomicAdd(&cnt[(v - id_lo) / wid], 1);
    }
    __syncthreads();
    if (t == 0) {
      long run = before;
      int b = 0;
      for (; b < kNucBins - 1; ++b) {
        if (run + cnt[b] >= need) break;
        run += cnt[b];
      }
      s_bin = b;
      s_n = static_cast<int>(run - before);
    }
    __syncthreads();
    before += s_n;
    id_lo = id_lo + s_bin * wid;
    id_hi = min(id_hi, id_lo + wid);
    __syncthreads();
    if (wid == 1) break;
  }
  // [id_lo, id_hi) now holds one id (wid == 1) or a short range: the cut id is the (need - before)-th
  // tied id in it
  if (t == 0) {
    long k = need - before;
    int id_cut = id_hi - 1;
    for (int v = id_lo; v < id_hi; ++v) {
      const float s = z[v] * inv_temperature;
      if (locate(L, s) == 0 && --k <= 0) {
        id_cut = v;
        break;
      }
    }
    cut[blockIdx.x] = make_uint2(order_key(s_tie), static_cast<uint32_t>(id_cut));
  }
}

}  // namespace

cudaError_t nucleus_cut_launch(const float *logits, int rows, int V, float temperature, float top_p, uint2 *cut,
                               cudaStream_t s) {
  if (rows == 0) return cudaSuccess;
  return launch_early(nucleus_cut_kernel, dim3(rows), dim3(kNucThreads), 0, s, logits, V, 1.0f / temperature, top_p,
                      cut);
}

}  // namespace echo
