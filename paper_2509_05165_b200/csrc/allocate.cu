// Layer-adaptive budget allocation (Eqs. 20-22).
//
// Per sequence, the pool P holds the L * N composite scores; the B largest are kept and N_l is
// how many of them lie in layer l.  Because composite[l, :] is non-increasing, the kept set of a
// layer is a prefix, so the answer is fixed by the B-th largest pooled value T:
//   N_l = #{k : I[l, k] > T}  +  (a share of the entries equal to T, handed out in layer order
//                                 until the budget is met -- the total order (I desc, l asc, k asc)).
// Two ways to T, both over the 32-bit order-preserving keys:
//   * pools of up to 128 rows: one kernel, one CTA per sequence, which only ever looks at a few
//     thousand entries.  Every row keeps a window of positions that must hold its boundary; per
//     round the CTA samples each window at equal distances, sorts the samples with their block
//     sizes as weights, and the weighted ranks bracket T between two sample values, which cuts
//     every window to the blocks between them (about a sixteenth per round).  A value with so many
//     copies that the windows stop shrinking is located exactly in every row (32-way searches) and
//     either is T or leaves the windows; when at most 1024 entries are left they are sorted and T
//     is read off.  The rounds are bounded; past the bound T is found by bisection over the key
//     range with exact counts.
//   * larger pools: a most-significant-digit radix select -- four histogram passes over the pool
//     (each CTA re-derives the prefix chosen so far from the previous passes' global histograms),
//     then one small kernel does the per-row searches and the tie hand-out.
//
// The rows of the pool are the layers (Eqs. 20-22) or, for the unstructured variant of App. A.2,
// the (layer, head) pairs with the heads' sorted scores as rows.  With a per-layer minimum m the
// first m entries of every row are kept outright and stay out of the pool.
#include <atomic>

#include "kvc_internal.cuh"

namespace kvc {
namespace {

constexpr int kRadix = 256;
constexpr int kHistThreads = 256;
constexpr int kItemsPerThread = 16;

// Select state after `passes` completed passes: the key prefix (high bits) and the rank that is
// still to be located inside that prefix bucket.  rank is 1-based among ascending keys.
// Where row r of sequence b starts: rows are layers of composite [L, Bt, N] (heads_per_row = 1) or
// (layer, head) pairs of sorted scores [L, Bt, Hkv, N] (heads_per_row = Hkv).
__device__ __forceinline__ long long row_start(long long r, int b, int Bt, int hpr, long long N) {
  const long long l = r / hpr, h = r - l * hpr;
  return ((l * Bt + b) * hpr + h) * N;
}

struct SelectState {
  uint32_t prefix;
  unsigned long long rank;
};

// hist: [4][256] counts of digit (MSD first) among keys whose higher digits equal the prefix.
// Walks the completed passes: in each, the digit whose cumulative count first reaches the rank.
// Cooperative: the first 256 threads of the block take one bin each (blockDim.x >= 256); the
// result is valid in every thread after the call.  `scratch` is 16 words of shared memory.
__device__ inline SelectState derive_state(const unsigned int* __restrict__ hist_b, int passes,
                                           unsigned long long rank0, unsigned long long* scratch) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  SelectState s;
  s.prefix = 0;
  s.rank = rank0;
  for (int p = 0; p < passes; ++p) {
    unsigned long long c = 0, incl = 0;
    if (tid < kRadix) {
      c = hist_b[p * kRadix + tid];
      incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (lane == 31) scratch[warp] = incl;
    }
    __syncthreads();
    if (tid == 0) { scratch[8] = kRadix - 1; scratch[9] = 0; }     // default: the last digit
    __syncthreads();
    if (tid < kRadix) {
      unsigned long long before = 0;
      for (int wv = 0; wv < warp; ++wv) before += scratch[wv];
      incl += before;
      const unsigned long long excl = incl - c;
      if (excl < s.rank && s.rank <= incl) { scratch[8] = (unsigned long long)tid; scratch[9] = excl; }
    }
    __syncthreads();
    if (s.rank > 0) {
      const unsigned long long total_last = scratch[9];
      s.prefix |= (uint32_t)scratch[8] << (24 - 8 * p);
      // when the rank lies beyond the total (cannot happen for a valid budget) the last digit
      // was kept with nothing subtracted
      s.rank -= total_last;
    }
    __syncthreads();
  }
  return s;
}

// Clears the histograms of all passes (a kernel rather than a memset, so that it can be launched
// as a programmatic dependent of whatever ran before).
__global__ void __launch_bounds__(1024)
select_clear_kernel(unsigned int* __restrict__ hist) {
  grid_dependency_wait();
  hist[(size_t)blockIdx.x * 4 * kRadix + threadIdx.x] = 0u;
}

// R rows per sequence, each of N entries of which the first `floor` are out of the pool; `budget`
// is what is left to hand out among the others.
__global__ void __launch_bounds__(kHistThreads)
select_hist_kernel(const float* __restrict__ composite, unsigned int* __restrict__ hist, int pass,
                   int R, int Bt, int hpr, long long N, long long floor, long long budget) {
  __shared__ unsigned int sh[kRadix];
  __shared__ unsigned long long scratch[16];
  grid_dependency_wait();
  const int b = blockIdx.y;
  unsigned int* hist_b = hist + (size_t)b * 4 * kRadix;
  for (int i = threadIdx.x; i < kRadix; i += kHistThreads) sh[i] = 0;
  const SelectState st = derive_state(hist_b, pass, (unsigned long long)budget, scratch);
  __syncthreads();
  const uint32_t prefix = st.prefix;
  const int shift = 24 - 8 * pass;
  const uint32_t hi_mask = (pass == 0) ? 0u : (0xffffffffu << (shift + 8));
  const long long M = N - floor;                       // pooled entries per row
  const long long total = (long long)R * M;
  const long long tile = (long long)kHistThreads * kItemsPerThread;
  for (long long t0 = (long long)blockIdx.x * tile; t0 < total; t0 += (long long)gridDim.x * tile) {
    // pooled index -> (row, position) once per tile, then by steps of the block width
    long long i = t0 + threadIdx.x;
    long long r = i / M, kk = i - r * M;
    long long base = row_start(r, b, Bt, hpr, N) + floor;      // (recomputed only when the row changes)
    // all of the thread's loads first ...
    float v[kItemsPerThread];
#pragma unroll
    for (int it = 0; it < kItemsPerThread; ++it) {
      v[it] = 0.f;
      if (i < total) v[it] = composite[base + kk];
      i += kHistThreads;
      kk += kHistThreads;
      if (kk >= M) {
        while (kk >= M) { kk -= M; ++r; }
        base = row_start(r, b, Bt, hpr, N) + floor;
      }
    }
    // ... then the bins.  Consecutive lanes hold consecutive entries of a non-increasing row: equal digits
    // come in runs, and only the first lane of a run adds (its length) to the bin.
    i = t0 + threadIdx.x;
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int it = 0; it < kItemsPerThread; ++it, i += kHistThreads) {
      uint32_t digit = 0x100u;                                  // not in the bucket / beyond the pool
      if (i < total) {
        const uint32_t key = score_to_key(v[it]);
        if ((key & hi_mask) == prefix) digit = (key >> shift) & 0xffu;
      }
      const uint32_t prev = __shfl_up_sync(0xffffffffu, digit, 1);
      const bool head = lane == 0 || prev != digit;
      const uint32_t heads = __ballot_sync(0xffffffffu, head);
      if (head && digit < 0x100u) {
        const uint32_t later = lane == 31 ? 0u : (heads >> (lane + 1));
        atomicAdd(&sh[digit], (unsigned int)(later ? __ffs(later) : 32 - lane));
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kRadix; i += kHistThreads)
    if (sh[i]) atomicAdd(&hist_b[pass * kRadix + i], sh[i]);
}

// One warp per layer: number of entries of the non-increasing row with key < T (strictly better)
// and with key <= T, by a 32-way search (every step probes 32 positions at once).
__device__ inline void count_layer_warp(const float* __restrict__ row, long long N, uint32_t T,
                                        long long* gt, long long* ge) {
  const int lane = threadIdx.x & 31;
  // first index with key >= T, then first index with key > T: the same search with two predicates
  long long res[2];
#pragma unroll
  for (int which = 0; which < 2; ++which) {
    long long lo = 0, hi = N;                  // the answer lies in [lo, hi]
    while (hi - lo > 0) {
      const long long span = hi - lo;
      const long long step = (span + 31) / 32;                 // probe lo + (lane + 1) * step - 1
      const long long pos = lo + (lane + 1) * step - 1;
      bool before = false;                                     // "row[pos] sorts before the boundary"
      if (pos < hi) {
        const uint32_t key = score_to_key(row[pos]);
        before = which == 0 ? (key < T) : (key <= T);
      }
      const uint32_t m = __ballot_sync(0xffffffffu, before);   // a prefix of the lanes (the row is sorted)
      const int n_before = __popc(m);
      // the boundary lies after probe n_before - 1 and at or before probe n_before
      const long long new_lo = n_before == 0 ? lo : min(hi, lo + (long long)n_before * step);
      const long long new_hi = n_before == 32 ? hi : min(hi, lo + (long long)(n_before + 1) * step - 1);
      lo = new_lo;
      hi = new_hi;
    }
    res[which] = lo;
  }
  *gt = res[0];
  *ge = res[1];
}

// `budget` is again what is left to hand out beyond the rows' first `floor` entries.
__global__ void __launch_bounds__(1024)
select_finish_kernel(const float* __restrict__ composite,
                     const unsigned int* __restrict__ hist, int R, int Bt, int hpr, long long N,
                     long long floor, long long budget, int32_t* __restrict__ n_keep,
                     long long* __restrict__ offsets) {
  extern __shared__ long long s_cnt[];               // [R] strictly better than T, [R] at least as good
  long long* s_gt = s_cnt;
  long long* s_ge = s_cnt + R;
  __shared__ unsigned long long scratch[16];
  grid_dependency_wait();
  const int b = blockIdx.x;
  const SelectState st = derive_state(hist + (size_t)b * 4 * kRadix, 4, (unsigned long long)budget, scratch);
  const uint32_t T = st.prefix;
  const int warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int r = warp; r < R; r += n_warps) {
    long long gt = 0, ge = 0;
    if (budget > 0) count_layer_warp(composite + row_start(r, b, Bt, hpr, N) + floor, N - floor, T, &gt, &ge);
    if ((threadIdx.x & 31) == 0) { s_gt[r] = gt; s_ge[r] = ge; }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    long long used = 0;
    for (int r = 0; r < R; ++r) used += s_gt[r];
    long long rem = budget - used;     // entries equal to T still to hand out, in row order
    long long off = 0;
    for (int r = 0; r < R; ++r) {
      long long take = s_ge[r] - s_gt[r];
      if (take > rem) take = rem;
      if (take < 0) take = 0;
      rem -= take;
      const long long n = floor + s_gt[r] + take;
      n_keep[(long long)b * R + r] = (int32_t)n;
      offsets[(long long)b * (R + 1) + r] = off;
      off += n;
    }
    offsets[(long long)b * (R + 1) + R] = off;
  }
}


// ------------------------------------------------------------------------------------------------
// Selection on the sorted rows themselves: one CTA per sequence, no scratch in global memory.
// ------------------------------------------------------------------------------------------------
constexpr int kSelThreads = 1024;
constexpr int kSelMaxRows = 128;          // rows of a pool this kernel takes (fewer samples per row as the rows grow)
constexpr int kSelDefaultRounds = 40;     // sampling rounds and exact steps together, before the bisection takes over

struct SelectShared {
  uint32_t sortbuf[2][kSelThreads];             // exchange buffers of the sort
  unsigned long long pref[kSelThreads];         // weighted inclusive ranks, in sorted order
  long long wt[kSelThreads];                    // block size behind every sample
  uint32_t skey[kSelThreads];                   // the samples' shortened keys in sorted order
  uint32_t fkey[kSelThreads];                   // the samples' keys
  long long lo[kSelMaxRows], hi[kSelMaxRows];   // the rows' windows: positions < lo are better than T, >= hi worse
  long long gt[kSelMaxRows], ge[kSelMaxRows];   // the answer: entries better than T, and at least as good
  long long off[kSelMaxRows + 1];               // running sum of the window lengths (last step)
  long long row_a[kSelMaxRows], row_b[kSelMaxRows];   // per-row terms of the sums below
  int clt[kSelMaxRows], cle[kSelMaxRows];
  unsigned long long warp_tot[32];
  long long rank, width;                        // T is the rank-th best entry inside the windows (1-based); their total length
  long long slack, new_width;
  unsigned long long tot_lt, tot_le;
  uint32_t khi, khi_key;                        // upper bracket: shortened key, and the key of the sample it came from
  uint32_t kmin, kmax;                          // range of the round's sample keys
  int ilo;
};

// Bitonic sort of 1024 32-bit values, one per thread; returns the value of rank threadIdx.x (ascending).
// K0 = 2 for any input; K0 = 2 m when the values arrive as runs of m neighbours that are already
// sorted, ascending where (threadIdx.x & m) == 0 and descending elsewhere: the stages that would
// build such runs are left out.  Exchanges closer than a warp go through shuffles, the others
// through shared memory (two buffers in turn: one barrier per step).  Fully unrolled: every
// step's partner and direction are constants.
template <int K0>
__device__ __forceinline__ uint32_t block_sort(uint32_t v, SelectShared& sh) {
  const int i = threadIdx.x;
  int which = 0;
#pragma unroll
  for (int k = K0; k <= kSelThreads; k <<= 1) {
    const bool asc = (i & k) == 0;
#pragma unroll
    for (int j = k >> 1; j > 0; j >>= 1) {
      uint32_t other;
      if (j >= 32) {
        sh.sortbuf[which][i] = v;
        __syncthreads();
        other = sh.sortbuf[which][i ^ j];
        which ^= 1;
      } else {
        other = __shfl_xor_sync(0xffffffffu, v, j);
      }
      const bool take_min = ((i & j) == 0) == asc;
      if ((other < v) == take_min) v = other;
    }
  }
  return v;
}

// Inclusive sum over the block in thread order.
__device__ inline unsigned long long block_scan(unsigned long long v, SelectShared& sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long n = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += n;
  }
  if (lane == 31) sh.warp_tot[warp] = v;    // (last read before the barriers of the sort that precedes every scan)
  __syncthreads();
  if (warp == 0) {
    const unsigned long long t = sh.warp_tot[lane];
    unsigned long long incl = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    sh.warp_tot[lane] = incl - t;
  }
  __syncthreads();
  return v + sh.warp_tot[warp];
}

// Sum of a per-row array (kSelMaxRows entries, zeros beyond the rows in use); call with the whole first warp.
__device__ inline long long warp_sum_rows(const long long* a) {
  const int lane = threadIdx.x & 31;
  long long v = a[lane] + a[lane + 32] + a[lane + 64] + a[lane + 96];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Exact position of key T in every row's window (32-way searches, one warp per row): gt / ge of
// the row as absolute pool positions, and their sums over the rows relative to the windows.
__device__ inline void locate_in_windows(const float* __restrict__ composite, SelectShared& sh, int R, int b, int Bt,
                                         int hpr, long long N, long long floor, uint32_t T) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) { sh.tot_lt = 0; sh.tot_le = 0; }
  __syncthreads();
  for (int r = warp; r < R; r += kSelThreads / 32) {
    const long long lo = sh.lo[r], w = sh.hi[r] - lo;
    long long lt = 0, le = 0;
    if (w > 0) count_layer_warp(composite + row_start(r, b, Bt, hpr, N) + floor + lo, w, T, &lt, &le);
    if (lane == 0) {
      sh.gt[r] = lo + lt;
      sh.ge[r] = lo + le;
      atomicAdd(&sh.tot_lt, (unsigned long long)lt);
      atomicAdd(&sh.tot_le, (unsigned long long)le);
    }
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kSelThreads)
select_sorted_kernel(const float* __restrict__ composite, int R, int Bt, int hpr, long long N, long long floor,
                     long long budget, int max_rounds, int32_t* __restrict__ n_keep,
                     long long* __restrict__ offsets) {
  __shared__ SelectShared sh;
  grid_dependency_wait();
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const long long M = N - floor;                       // pooled entries per row
  // samples per row and round: 32 for up to 32 rows, 16 for up to 64, 8 beyond
  const int sshift = R <= 32 ? 5 : (R <= 64 ? 4 : 3);
  const int S = 1 << sshift;
  const int r = tid >> sshift, k = tid & (S - 1);      // this thread's row and its place among the row's threads
  // the row's samples are sorted already: every other row takes them in reverse, so that the sort can
  // start from runs of S
  const int ks = (tid & S) ? S - 1 - k : k;            // which sample of the row this thread takes
  const unsigned int sample_id = (unsigned int)((r << sshift) | ks);
  const int rr0 = r < R ? r : 0, rl = rr0 / hpr;       // (32-bit: the 64-bit division of row_start is slow)
  const float* row = composite + (((long long)rl * Bt + b) * hpr + (rr0 - rl * hpr)) * N + floor;
  if (tid < R) { sh.lo[tid] = 0; sh.hi[tid] = M; sh.gt[tid] = 0; sh.ge[tid] = 0; }
  if (tid < kSelMaxRows) { sh.row_a[tid] = 0; sh.row_b[tid] = 0; }
  if (tid == 0) {
    sh.width = (long long)R * M;
    sh.rank = budget < sh.width ? budget : sh.width;
    sh.kmin = 0xffffffffu;
    sh.kmax = 0u;
  }
  __syncthreads();
  if (budget > 0 && M > 0) {
    bool found = false;                                // sh.gt / sh.ge hold the answer
    for (int round = 0; round < max_rounds; ++round) {
      const long long width = sh.width, rank = sh.rank;
      if (width <= kSelThreads) break;
      __syncthreads();                                 // (everyone has read width and rank)
      if (tid == 0) sh.ilo = 0;
      // this thread's sample: the last (worst) entry of block k of its row's window
      long long lo = 0, w = 0, s = 0, wgt = 0;
      uint32_t key = 0xffffffffu;
      if (r < R) {
        lo = sh.lo[r];
        w = sh.hi[r] - lo;
        if (w > 0) {
          s = (w + S - 1) >> sshift;
          const long long b0 = ks * s;
          if (b0 < w) {
            const long long b1 = b0 + s < w ? b0 + s : w;
            wgt = b1 - b0;
            key = score_to_key(row[lo + b1 - 1]);
          }
        }
        if (k == 0) sh.row_a[r] = w > 0 ? s - 1 : 0;   // what a partial block can hide
      }
      sh.wt[sample_id] = wgt;
      sh.fkey[sample_id] = key;
      // The samples are sorted as 32-bit words: the key, taken relative to the smallest sample key and
      // shortened to its leading 22 bits of the samples' range, above the sample's number (which breaks
      // ties so that the rows' runs stay sorted).  Shortening is monotone, so every bound below holds
      // for the shortened keys as it would for the keys; samples that fall together just make the
      // brackets a little wider.
      const bool real = wgt > 0;
      {
        const uint32_t wmin = __reduce_min_sync(0xffffffffu, real ? key : 0xffffffffu);
        const uint32_t wmax = __reduce_max_sync(0xffffffffu, real ? key : 0u);
        if (lane == 0) { atomicMin(&sh.kmin, wmin); atomicMax(&sh.kmax, wmax); }
      }
      __syncthreads();
      const uint32_t base = sh.kmin, span = sh.kmax - base;
      const int cut = (span >> 22) ? (32 - __clz(span)) - 22 : 0;
      const uint32_t tkey = real ? ((key - base) >> cut) : 0x3fffffu;
      const uint32_t packed = (tkey << 10) | sample_id;
      const uint32_t e = sshift == 5 ? block_sort<64>(packed, sh)
                       : sshift == 4 ? block_sort<32>(packed, sh) : block_sort<16>(packed, sh);
      const uint32_t ekey = e >> 10;
      // weighted rank: entries known to be at least as good as this sample (whole blocks only)
      const unsigned long long P = block_scan((unsigned long long)sh.wt[e & 1023u], sh);
      sh.skey[tid] = ekey;
      sh.pref[tid] = P;
      if (tid < 32) { const long long v = warp_sum_rows(sh.row_a); if (tid == 0) sh.slack = v; }
      __syncthreads();
      // upper bracket: the first sample whose whole blocks already hold `rank` entries: T is at least as good.
      // lower bracket: the last sample value v for which even whole blocks plus one partial block per row
      // hold fewer than `rank` entries at least as good as v: T is worse than v.
      const unsigned long long Pprev = tid ? sh.pref[tid - 1] : 0ull;
      if (Pprev < (unsigned long long)rank && (unsigned long long)rank <= P) { sh.khi = ekey; sh.khi_key = sh.fkey[e & 1023u]; }
      const long long bound = rank - sh.slack - 1;
      const bool last_of_value = tid == kSelThreads - 1 || sh.skey[tid + 1] != ekey;
      if (last_of_value && (long long)P <= bound) atomicMax(&sh.ilo, tid + 1);
      __syncthreads();
      const uint32_t khi = sh.khi;
      const int ilo = sh.ilo;
      const uint32_t klo = ilo ? sh.skey[ilo - 1] : 0u;
      // samples of the row on the good side of either bracket (the lanes of a row are neighbours)
      const uint32_t mlo = __ballot_sync(0xffffffffu, real && ilo > 0 && tkey <= klo);
      const uint32_t mhi = __ballot_sync(0xffffffffu, real && tkey <= khi);
      if (r < R && k == 0) {
        long long nlo = lo, nhi = lo;
        if (w > 0) {
          const uint32_t gmask = (S == 32 ? 0xffffffffu : ((1u << S) - 1u)) << (lane & ~(S - 1));
          const long long jlo = __popc(mlo & gmask), jhi = __popc(mhi & gmask);
          nlo = lo + (s * jlo < w ? s * jlo : w);
          nhi = lo + (s * (jhi + 1) < w ? s * (jhi + 1) : w);
          sh.lo[r] = nlo;
          sh.hi[r] = nhi;
        }
        sh.row_a[r] = nlo - lo;                        // entries now known to be better than T
        sh.row_b[r] = nhi - nlo;
      }
      __syncthreads();
      if (tid < 32) {
        const long long taken = warp_sum_rows(sh.row_a), nw = warp_sum_rows(sh.row_b);
        if (tid == 0) { sh.rank = rank - taken; sh.width = nw; sh.new_width = nw; sh.kmin = 0xffffffffu; sh.kmax = 0u; }
      }
      __syncthreads();
      const long long new_width = sh.new_width;
      if (new_width > width / 2) {
        // the windows did not shrink: some value has very many copies (or many keys fell together when
        // they were shortened).  Locate the key of the upper bracket's sample exactly.
        locate_in_windows(composite, sh, R, b, Bt, hpr, N, floor, sh.khi_key);
        const long long rk = sh.rank, lt = (long long)sh.tot_lt, le = (long long)sh.tot_le;
        __syncthreads();
        if (rk > lt && rk <= le) { found = true; break; }            // it is T
        if (rk <= lt) {                                               // T is better: the copies leave the windows
          if (tid < R) sh.hi[tid] = sh.gt[tid];
          if (tid == 0) sh.width = lt;
        } else {                                                      // T is worse (only among keys that were shortened alike)
          if (tid < R) sh.lo[tid] = sh.ge[tid];
          if (tid == 0) { sh.rank = rk - le; sh.width = new_width - le; }
        }
        __syncthreads();
      }
    }
    if (!found) {
      __syncthreads();
      const long long width = sh.width, rank = sh.rank;
      uint32_t T;
      if (width <= kSelThreads) {
        // few enough entries left: sort them all, T is the rank-th
        if (tid < 32) {
          long long a[4], sum = 0;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int rr = 4 * tid + i;
            a[i] = rr < R ? sh.hi[rr] - sh.lo[rr] : 0;
            sum += a[i];
          }
          long long incl = sum;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const long long n = __shfl_up_sync(0xffffffffu, incl, o);
            if (tid >= o) incl += n;
          }
          long long run = incl - sum;
#pragma unroll
          for (int i = 0; i < 4; ++i) { sh.off[4 * tid + i] = run; run += a[i]; }
          if (tid == 31) sh.off[kSelMaxRows] = run;
        }
        if (tid < kSelMaxRows) { sh.clt[tid] = 0; sh.cle[tid] = 0; }
        __syncthreads();
        uint32_t key = 0xffffffffu;
        int rr = 0;
        if (tid < width) {
          int a = 0, c = R - 1;                        // the row with off[rr] <= tid < off[rr + 1]
          while (a < c) {
            const int m = (a + c) >> 1;
            if (sh.off[m + 1] > tid) c = m; else a = m + 1;
          }
          rr = a;
          key = score_to_key(composite[row_start(rr, b, Bt, hpr, N) + floor + sh.lo[rr] + (tid - sh.off[rr])]);
        }
        const uint32_t e = block_sort<2>(tid < width ? key : 0xffffffffu, sh);    // (keys alone: T is a value)
        if (tid == rank - 1) sh.khi = e;
        __syncthreads();
        T = sh.khi;
        if (tid < width) {
          if (key < T) atomicAdd(&sh.clt[rr], 1);
          if (key <= T) atomicAdd(&sh.cle[rr], 1);
        }
        __syncthreads();
        if (tid < R) { sh.gt[tid] = sh.lo[tid] + sh.clt[tid]; sh.ge[tid] = sh.lo[tid] + sh.cle[tid]; }
      } else {
        // out of rounds: bisection over the keys, exact counts inside the windows
        uint32_t a = 0u, c = 0xffffffffu;              // T lies in [a, c]
        for (int it = 0; it < 32 && a < c; ++it) {
          const uint32_t mid = a + (c - a) / 2;
          locate_in_windows(composite, sh, R, b, Bt, hpr, N, floor, mid);
          const long long le = (long long)sh.tot_le;
          __syncthreads();
          if (le >= rank) c = mid; else a = mid + 1;
        }
        T = a;
        locate_in_windows(composite, sh, R, b, Bt, hpr, N, floor, T);
      }
    }
  }
  __syncthreads();
  if (tid < 32) {
    // the entries equal to T go to the rows in row order until the budget is met; lane i has rows 4i .. 4i + 3
    long long g[4], tie[4], gsum = 0, tsum = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int rr = 4 * tid + i;
      g[i] = rr < R ? sh.gt[rr] : 0;
      tie[i] = rr < R ? sh.ge[rr] - sh.gt[rr] : 0;
      gsum += g[i];
      tsum += tie[i];
    }
    long long used = gsum, ties_before = tsum;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) used += __shfl_xor_sync(0xffffffffu, used, o);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long n = __shfl_up_sync(0xffffffffu, ties_before, o);
      if (tid >= o) ties_before += n;
    }
    ties_before -= tsum;                               // ties in the rows before this lane's
    long long rem = budget - used - ties_before;       // what is left when this lane's rows are served
    long long n[4], nsum = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      long long take = tie[i];
      if (take > rem) take = rem;
      if (take < 0) take = 0;
      rem -= tie[i];
      n[i] = floor + g[i] + take;
      if (4 * tid + i >= R) n[i] = 0;
      nsum += n[i];
    }
    long long off = nsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long v = __shfl_up_sync(0xffffffffu, off, o);
      if (tid >= o) off += v;
    }
    const long long total = __shfl_sync(0xffffffffu, off, 31);
    off -= nsum;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int rr = 4 * tid + i;
      if (rr < R) {
        n_keep[(long long)b * R + rr] = (int32_t)n[i];
        offsets[(long long)b * (R + 1) + rr] = off;
      }
      off += n[i];
    }
    if (tid == 0) offsets[(long long)b * (R + 1) + R] = total;
  }
}

// Test hooks (see kvc_debug_select_hooks).
std::atomic<int> g_select_path{0};
std::atomic<int> g_select_rounds{-1};

}  // namespace

size_t allocate_workspace_bytes(const Problem& P) {
  return align_up((size_t)P.Bt * 4 * kRadix * sizeof(unsigned int));
}

void set_select_hooks(int path, int max_rounds) {
  g_select_path.store(path);
  g_select_rounds.store(max_rounds);
}

kvc_status launch_allocate(const Problem& P, const float* composite, long long budget, int heads_per_row,
                           long long min_keep, int32_t* n_keep, long long* offsets, void* ws,
                           size_t ws_bytes, cudaStream_t st, SelectPath path) {
  if (ws_bytes < allocate_workspace_bytes(P)) {
    set_error("allocate: workspace too small");
    return KVC_ERR_WORKSPACE;
  }
  const int R = P.L * heads_per_row;
  if (R > kMaxSelectRows) {
    set_error("allocate: %d rows in the pool, at most %d supported", R, kMaxSelectRows);
    return KVC_ERR_UNSUPPORTED;
  }
  if (min_keep < 0 || min_keep > P.N || (long long)R * min_keep > budget) {
    set_error("allocate: per-layer minimum %lld does not fit (N = %lld, rows * minimum <= budget = %lld required)",
              min_keep, P.N, budget);
    return KVC_ERR_INVALID_ARG;
  }
  const long long rest = budget - (long long)R * min_keep;     // handed out beyond the minimum
  if (path == SelectPath::kAuto) {
    const int hook = g_select_path.load();
    if (hook == 1) path = SelectPath::kHistograms;
    if (hook == 2) path = SelectPath::kSortedRows;
  }
  if (path != SelectPath::kHistograms && R <= kSelMaxRows) {
    const int hook_rounds = g_select_rounds.load();
    const int rounds = hook_rounds >= 0 ? hook_rounds : kSelDefaultRounds;
    KVC_CUDA(launch_dependent(select_sorted_kernel, dim3(P.Bt), dim3(kSelThreads), 0, st, composite, R, P.Bt,
                              heads_per_row, P.N, min_keep, rest, rounds, n_keep, offsets));
    KVC_LAUNCH_CHECK("select_sorted_kernel");
    return KVC_OK;
  }
  unsigned int* hist = reinterpret_cast<unsigned int*>(ws);
  KVC_CUDA(launch_dependent(select_clear_kernel, dim3(P.Bt), dim3(4 * kRadix), 0, st, hist));
  KVC_LAUNCH_CHECK("select_clear_kernel");
  const long long total = (long long)R * (P.N - min_keep);
  const long long tile = (long long)kHistThreads * kItemsPerThread;
  long long blocks = (total + tile - 1) / tile;
  int dev = 0, sms = 0;
  KVC_CUDA(cudaGetDevice(&dev));
  KVC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (blocks > 4LL * sms) blocks = 4LL * sms;
  if (blocks < 1) blocks = 1;
  if (rest > 0) {
    for (int pass = 0; pass < 4; ++pass) {
      KVC_CUDA(launch_dependent(select_hist_kernel, dim3((unsigned)blocks, P.Bt), dim3(kHistThreads), 0, st,
                                composite, hist, pass, R, P.Bt, heads_per_row, P.N, min_keep, rest));
      KVC_LAUNCH_CHECK("select_hist_kernel");
    }
  }
  KVC_CUDA(launch_dependent(select_finish_kernel, dim3(P.Bt), dim3(1024), (size_t)R * 2 * sizeof(long long), st,
                            composite, hist, R, P.Bt, heads_per_row, P.N, min_keep, rest, n_keep, offsets));
  KVC_LAUNCH_CHECK("select_finish_kernel");
  return KVC_OK;
}

}  // namespace kvc

// Test hook: which way the allocation finds its threshold (0: the library chooses, 1: the histogram
// passes, 2: the sorted-rows kernel wherever the pool has few enough rows) and how many rounds the
// sorted-rows kernel may take before it bisects (< 0: the default; 0: bisect at once).  Process-wide;
// takes effect at the next call.  kvc_allocate_static always takes the histogram passes.
extern "C" __attribute__((visibility("default"))) void kvc_debug_select_hooks(int32_t path, int32_t max_rounds) {
  kvc::set_select_hooks(path, max_rounds);
}
