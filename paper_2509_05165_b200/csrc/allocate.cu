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
#include "kvc_internal.cuh"

namespace kvc {
namespace {

constexpr int kRadix = 256;
constexpr int kHistThreads = 256;
constexpr int kItemsPerThread = 16;

// Select state after `passes` completed passes: the key prefix (high bits) and the rank that is
// still to be located inside that prefix bucket.  rank is 1-based among ascending keys.
struct SelectState {
  uint32_t prefix;
  unsigned long long rank;
};

// hist: [Bt][4][256] counts of digit (MSD first) among keys whose higher digits equal the prefix.
__device__ inline SelectState derive_state(const unsigned int* __restrict__ hist_b, int passes,
                                           unsigned long long rank0) {
  SelectState s;
  s.prefix = 0;
  s.rank = rank0;
  for (int p = 0; p < passes; ++p) {
    const unsigned int* h = hist_b + p * kRadix;
    unsigned long long cum = 0;
    int dsel = kRadix - 1;
    for (int dgt = 0; dgt < kRadix; ++dgt) {
      const unsigned long long c = h[dgt];
      if (cum + c >= s.rank) { dsel = dgt; break; }
      cum += c;
    }
    s.rank -= cum;
    s.prefix |= (uint32_t)dsel << (24 - 8 * p);
  }
  return s;
}

__global__ void __launch_bounds__(kHistThreads)
select_hist_kernel(const float* __restrict__ composite, unsigned int* __restrict__ hist, int pass,
                   int L, int Bt, long long N, long long budget) {
  __shared__ unsigned int sh[kRadix];
  __shared__ SelectState st;
  const int b = blockIdx.y;
  unsigned int* hist_b = hist + (size_t)b * 4 * kRadix;
  for (int i = threadIdx.x; i < kRadix; i += kHistThreads) sh[i] = 0;
  if (threadIdx.x == 0) st = derive_state(hist_b, pass, (unsigned long long)budget);
  __syncthreads();
  const uint32_t prefix = st.prefix;
  const int shift = 24 - 8 * pass;
  const uint32_t hi_mask = (pass == 0) ? 0u : (0xffffffffu << (shift + 8));
  const long long total = (long long)L * N;
  const long long tile = (long long)kHistThreads * kItemsPerThread;
  for (long long t0 = (long long)blockIdx.x * tile; t0 < total; t0 += (long long)gridDim.x * tile) {
#pragma unroll 4
    for (int it = 0; it < kItemsPerThread; ++it) {
      const long long i = t0 + (long long)it * kHistThreads + threadIdx.x;
      if (i < total) {
        const long long l = i / N, kk = i - l * N;
        const uint32_t key = score_to_key(composite[(l * Bt + b) * N + kk]);
        if ((key & hi_mask) == prefix) atomicAdd(&sh[(key >> shift) & 0xffu], 1u);
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kRadix; i += kHistThreads)
    if (sh[i]) atomicAdd(&hist_b[pass * kRadix + i], sh[i]);
}

// Number of entries of the non-increasing row with key < T (strictly better) and <= T.
__device__ inline void count_layer(const float* __restrict__ row, long long N, uint32_t T,
                                   long long* gt, long long* ge) {
  long long lo = 0, hi = N;           // first index with key >= T
  while (lo < hi) {
    const long long mid = (lo + hi) >> 1;
    if (score_to_key(row[mid]) < T) lo = mid + 1; else hi = mid;
  }
  *gt = lo;
  hi = N;                              // first index with key > T
  while (lo < hi) {
    const long long mid = (lo + hi) >> 1;
    if (score_to_key(row[mid]) <= T) lo = mid + 1; else hi = mid;
  }
  *ge = lo;
}

__global__ void select_finish_kernel(const float* __restrict__ composite,
                                     const unsigned int* __restrict__ hist, int L, int Bt, long long N,
                                     long long budget, int32_t* __restrict__ n_keep,
                                     long long* __restrict__ offsets) {
  __shared__ long long s_gt[KVC_MAX_LAYERS];
  __shared__ long long s_ge[KVC_MAX_LAYERS];
  __shared__ uint32_t s_T;
  const int b = blockIdx.x;
  if (threadIdx.x == 0) s_T = derive_state(hist + (size_t)b * 4 * kRadix, 4, (unsigned long long)budget).prefix;
  __syncthreads();
  const uint32_t T = s_T;
  for (int l = threadIdx.x; l < L; l += blockDim.x) {
    if (budget == 0) { s_gt[l] = 0; s_ge[l] = 0; }
    else count_layer(composite + ((long long)l * Bt + b) * N, N, T, &s_gt[l], &s_ge[l]);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    long long used = 0;
    for (int l = 0; l < L; ++l) used += s_gt[l];
    long long rem = budget - used;     // entries equal to T still to hand out, in layer order
    long long off = 0;
    for (int l = 0; l < L; ++l) {
      long long take = s_ge[l] - s_gt[l];
      if (take > rem) take = rem;
      if (take < 0) take = 0;
      rem -= take;
      const long long n = s_gt[l] + take;
      n_keep[(long long)b * L + l] = (int32_t)n;
      offsets[(long long)b * (L + 1) + l] = off;
      off += n;
    }
    offsets[(long long)b * (L + 1) + L] = off;
  }
}

}  // namespace

size_t allocate_workspace_bytes(const Problem& P) {
  return align_up((size_t)P.Bt * 4 * kRadix * sizeof(unsigned int));
}

kvc_status launch_allocate(const Problem& P, const float* composite, long long budget,
                           int32_t* n_keep, long long* offsets, void* ws, size_t ws_bytes,
                           cudaStream_t st) {
  if (ws_bytes < allocate_workspace_bytes(P)) {
    set_error("allocate: workspace too small");
    return KVC_ERR_WORKSPACE;
  }
  unsigned int* hist = reinterpret_cast<unsigned int*>(ws);
  KVC_CUDA(cudaMemsetAsync(hist, 0, (size_t)P.Bt * 4 * kRadix * sizeof(unsigned int), st));
  const long long total = (long long)P.L * P.N;
  const long long tile = (long long)kHistThreads * kItemsPerThread;
  long long blocks = (total + tile - 1) / tile;
  if (blocks > 592) blocks = 592;
  if (blocks < 1) blocks = 1;
  if (budget > 0) {
    for (int pass = 0; pass < 4; ++pass) {
      select_hist_kernel<<<dim3((unsigned)blocks, P.Bt), kHistThreads, 0, st>>>(
          composite, hist, pass, P.L, P.Bt, P.N, budget);
      KVC_LAUNCH_CHECK("select_hist_kernel");
    }
  }
  select_finish_kernel<<<P.Bt, 128, 0, st>>>(composite, hist, P.L, P.Bt, P.N, budget, n_keep, offsets);
  KVC_LAUNCH_CHECK("select_finish_kernel");
  return KVC_OK;
}

}  // namespace kvc
