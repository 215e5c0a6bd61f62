// Layer-adaptive budget allocation (Eqs. 20-22).
//
// Per sequence, the pool P holds the L * N composite scores; the B largest are kept and N_l is
// how many of them lie in layer l.  Because composite[l, :] is non-increasing, the kept set of a
// layer is a prefix, so the answer is fixed by the B-th largest pooled value T:
//   N_l = #{k : I[l, k] > T}  +  (a share of the entries equal to T, handed out in layer order
//                                 until the budget is met -- the total order (I desc, l asc, k asc)).
// T is found by a most-significant-digit radix select over the 32-bit order-preserving keys:
// four histogram passes over the pool (each CTA re-derives the prefix chosen so far from the
// previous passes' global histograms), then one small kernel does the per-layer binary searches
// and the tie hand-out.
//
// The rows of the pool are the layers (Eqs. 20-22) or, for the unstructured variant of App. A.2,
// the (layer, head) pairs with the heads' sorted scores as rows.  With a per-layer minimum m the
// first m entries of every row are kept outright and stay out of the pool.
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

}  // namespace

size_t allocate_workspace_bytes(const Problem& P) {
  return align_up((size_t)P.Bt * 4 * kRadix * sizeof(unsigned int));
}

kvc_status launch_allocate(const Problem& P, const float* composite, long long budget, int heads_per_row,
                           long long min_keep, int32_t* n_keep, long long* offsets, void* ws,
                           size_t ws_bytes, cudaStream_t st) {
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
