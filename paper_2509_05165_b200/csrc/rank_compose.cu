// Per-head ranking (Eq. 17), sorted scores (Eq. 18) and composite scores (Eq. 19).
//
// Every (layer, sequence, KV head) is one segment of N (score, position) pairs that must come
// out in descending score order with equal scores in ascending position.  Scores are mapped to
// 32-bit keys whose ascending order is the wanted order, and each segment is sorted by one CTA
// with a stable least-significant-digit radix sort (8-bit digits, 4 passes) that ping-pongs
// between two scratch buffers; a segment's working set (8 bytes per token per buffer) stays in
// L2 between passes.  The last pass writes the positions straight into idx and leaves the sorted
// keys for the composite kernel, which turns them back into scores and reduces over the heads.
#include "kvc_internal.cuh"

namespace kvc {
namespace {

constexpr int kSortThreads = 1024;
constexpr int kWarps = kSortThreads / 32;
constexpr int kRadix = 256;

struct SortBuffers {
  uint32_t* keys_a; int32_t* vals_a;
  uint32_t* keys_b; int32_t* vals_b;
};

__global__ void __launch_bounds__(kSortThreads)
segment_sort_kernel(const float* __restrict__ scores, int32_t* __restrict__ idx_out,
                    SortBuffers buf, long long N) {
  __shared__ uint32_t hist4[4][kRadix];
  __shared__ uint32_t base[kRadix];
  __shared__ uint16_t warp_cnt[kWarps][kRadix];   // per tile: count, then exclusive offset
  __shared__ uint32_t scan_tmp[kRadix / 32];

  const long long seg = blockIdx.x;
  const float* s_in = scores + seg * N;
  uint32_t* ka = buf.keys_a + seg * N; int32_t* va = buf.vals_a + seg * N;
  uint32_t* kb = buf.keys_b + seg * N; int32_t* vb = buf.vals_b + seg * N;
  int32_t* out_idx = idx_out + seg * N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;

  // ---- digit histograms of all four passes in one sweep (the multiset of keys never changes)
  for (int i = tid; i < 4 * kRadix; i += kSortThreads) (&hist4[0][0])[i] = 0;
  __syncthreads();
  for (long long t0 = 0; t0 < N; t0 += kSortThreads) {
    const long long i = t0 + tid;
    const bool valid = i < N;
    const uint32_t key = valid ? score_to_key(s_in[i]) : 0u;
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const uint32_t digit = valid ? ((key >> (8 * pass)) & 0xffu) : 0x100u;
      const uint32_t peers = __match_any_sync(0xffffffffu, digit);
      if (valid && (peers & lt_mask) == 0) atomicAdd(&hist4[pass][digit], (uint32_t)__popc(peers));
    }
  }
  __syncthreads();

  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 8 * pass;
    // pass 0: scores -> A;  1: A -> B;  2: B -> A;  3: A -> (keys_b, idx)
    const uint32_t* src_k = (pass == 2) ? kb : ka;
    const int32_t* src_v = (pass == 2) ? vb : va;
    uint32_t* dst_k = (pass == 0 || pass == 2) ? ka : kb;
    int32_t* dst_v = (pass == 0 || pass == 2) ? va : (pass == 3 ? out_idx : vb);
    uint32_t* hist = hist4[pass];

    // ---- exclusive scan of the 256 bins -> base
    if (tid < kRadix) {
      uint32_t v = hist[tid];
      uint32_t incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (lane == 31) scan_tmp[warp] = incl;
      base[tid] = incl - v;
    }
    __syncthreads();
    if (tid < kRadix) {
      uint32_t add = 0;
      for (int wv = 0; wv < warp; ++wv) add += scan_tmp[wv];
      base[tid] += add;
    }
    __syncthreads();

    // ---- stable scatter, one tile of kSortThreads items at a time, tiles in order
    for (long long t0 = 0; t0 < N; t0 += kSortThreads) {
      const long long i = t0 + tid;
      const bool valid = i < N;
      uint32_t key = 0; int32_t val = 0;
      if (valid) {
        if (pass == 0) { key = score_to_key(s_in[i]); val = (int32_t)i; }
        else { key = src_k[i]; val = src_v[i]; }
      }
      const uint32_t digit = valid ? ((key >> shift) & 0xffu) : 0x100u;
      // clear this warp's counters, then count per (warp, digit)
      for (int dgt = lane; dgt < kRadix; dgt += 32) warp_cnt[warp][dgt] = 0;
      __syncwarp();
      const uint32_t peers = __match_any_sync(0xffffffffu, digit);
      const int rank_in_warp = __popc(peers & lt_mask);
      if (valid && rank_in_warp == 0) warp_cnt[warp][digit] = (uint16_t)__popc(peers);
      __syncthreads();
      // per digit: exclusive scan over the warps, then advance the digit's base
      if (tid < kRadix) {
        uint32_t run = 0;
#pragma unroll 8
        for (int wv = 0; wv < kWarps; ++wv) {
          const uint32_t cnt = warp_cnt[wv][tid];
          warp_cnt[wv][tid] = (uint16_t)run;
          run += cnt;
        }
        hist[tid] = base[tid];      // start of this tile's run of the digit
        base[tid] += run;
      }
      __syncthreads();
      if (valid) {
        const uint32_t pos = hist[digit] + warp_cnt[warp][digit] + rank_in_warp;
        dst_k[pos] = key;
        dst_v[pos] = val;
      }
      __syncthreads();
    }
    __threadfence_block();
    __syncthreads();
  }
}

// Eq. 19 over the sorted keys: composite[lb, k] = agg_head_h score(keys[lb, h, k]).
// Mean: heads added in ascending order in fp32, one division at the end.
__global__ void compose_kernel(const uint32_t* __restrict__ keys, float* __restrict__ composite,
                               int Hkv, long long N, long long total, int agg_head) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const long long lb = i / N, kk = i - lb * N;
  const uint32_t* p = keys + lb * Hkv * N + kk;
  float acc = key_to_score(p[0]);
  for (int h = 1; h < Hkv; ++h) {
    const float a = key_to_score(p[(long long)h * N]);
    acc = (agg_head == KVC_AGG_MAX) ? fmaxf(acc, a) : __fadd_rn(acc, a);
  }
  if (agg_head == KVC_AGG_MEAN) acc = __fdiv_rn(acc, (float)Hkv);
  composite[i] = acc;
}

}  // namespace

size_t compose_workspace_bytes(const Problem& P) {
  const size_t items = (size_t)P.L * P.Bt * P.Hkv * P.N;
  return 4 * align_up(items * 4);
}

kvc_status launch_compose(const Problem& P, const float* scores, int32_t* idx, float* composite,
                          void* ws, size_t ws_bytes, cudaStream_t st) {
  if (ws_bytes < compose_workspace_bytes(P)) {
    set_error("compose: workspace too small");
    return KVC_ERR_WORKSPACE;
  }
  const size_t items = (size_t)P.L * P.Bt * P.Hkv * P.N;
  const size_t region = align_up(items * 4);
  char* w = reinterpret_cast<char*>(ws);
  SortBuffers buf;
  buf.keys_a = reinterpret_cast<uint32_t*>(w);
  buf.vals_a = reinterpret_cast<int32_t*>(w + region);
  buf.keys_b = reinterpret_cast<uint32_t*>(w + 2 * region);
  buf.vals_b = reinterpret_cast<int32_t*>(w + 3 * region);
  const long long segments = (long long)P.L * P.Bt * P.Hkv;
  segment_sort_kernel<<<(unsigned)segments, kSortThreads, 0, st>>>(scores, idx, buf, P.N);
  KVC_LAUNCH_CHECK("segment_sort_kernel");
  const long long total = (long long)P.L * P.Bt * P.N;
  compose_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(buf.keys_b, composite, P.Hkv, P.N,
                                                                 total, P.agg_head);
  KVC_LAUNCH_CHECK("compose_kernel");
  return KVC_OK;
}

}  // namespace kvc
