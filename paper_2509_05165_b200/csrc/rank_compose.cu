// Per-head ranking (Eq. 17), sorted scores (Eq. 18) and composite scores (Eq. 19).
//
// Every (layer, sequence, KV head) is one segment of N (score, position) pairs that must come
// out in descending score order with equal scores in ascending position.  Scores are mapped to
// 32-bit keys whose ascending order is the wanted order, and each segment is sorted by one CTA
// with a stable least-significant-digit radix sort (8-bit digits, 4 passes, tiles of 8192
// elements with eight per thread so that the loads of a tile are in flight together) that
// ping-pongs between two scratch buffers; a segment's working set (8 bytes per token per buffer)
// stays in L2 between passes.  The last pass writes the positions straight into idx and leaves the sorted
// keys for the composite kernel, which turns them back into scores and reduces over the heads.
#include "kvc_internal.cuh"

namespace kvc {
namespace {

constexpr int kSortThreads = 512;            // two CTAs per SM: all 256 segments of the 8B shape are resident at once
constexpr int kWarps = kSortThreads / 32;
constexpr int kRadix = 256;
constexpr int kItems = 8;                               // elements per thread per tile
constexpr int kTileItems = kSortThreads * kItems;       // 8192 elements per tile
constexpr int kWarpItems = 32 * kItems;                 // a warp owns 256 consecutive elements of a tile

struct SortBuffers {
  uint32_t* keys_a; int32_t* vals_a;
  uint32_t* keys_b; int32_t* vals_b;
};

// Lanes of the warp whose 8-bit digit equals this lane's (0 for a lane without an element).
// Eight ballots: the cost does not depend on how many different digits the warp holds.
__device__ __forceinline__ uint32_t same_digit_lanes(uint32_t digit, bool valid) {
  uint32_t peers = __ballot_sync(0xffffffffu, valid);
#pragma unroll
  for (int b = 0; b < 8; ++b) {
    const bool bit = (digit >> b) & 1u;
    const uint32_t m = __ballot_sync(0xffffffffu, bit);
    peers &= bit ? m : ~m;
  }
  return valid ? peers : 0u;
}

__global__ void __launch_bounds__(kSortThreads, 2)
segment_sort_kernel(const float* __restrict__ scores, int32_t* __restrict__ idx_out,
                    SortBuffers buf, long long N) {
  __shared__ uint32_t hist4[4][kRadix];
  __shared__ uint32_t base[kRadix];               // running start of every digit's output range
  __shared__ uint32_t tile_base[kRadix];          // ... as it was when the current tile began
  __shared__ uint16_t warp_cnt[kWarps][kRadix];   // per tile: count, then exclusive offset, per (warp, digit)
  __shared__ uint32_t scan_tmp[kRadix / 32];
  __shared__ uint32_t tile_start[kRadix];         // first slot of every digit inside the reordered tile
  __shared__ uint32_t stage_k[kTileItems];        // the tile, reordered by digit, before it goes out
  __shared__ int32_t stage_v[kTileItems];

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
  for (long long t0 = 0; t0 < N; t0 += kTileItems) {
    uint32_t key[kItems];
    bool valid[kItems];
#pragma unroll
    for (int k = 0; k < kItems; ++k) {
      const long long i = t0 + (long long)warp * kWarpItems + k * 32 + lane;
      valid[k] = i < N;
      key[k] = valid[k] ? score_to_key(s_in[i]) : 0u;
    }
#pragma unroll
    for (int k = 0; k < kItems; ++k) {
      // the three low digits are spread over their 256 bins: plain shared-memory atomics hardly
      // collide.  The top digit (sign and high exponent bits) takes a handful of values, so the
      // warp adds its lanes up first.
#pragma unroll
      for (int pass = 0; pass < 3; ++pass)
        if (valid[k]) atomicAdd(&hist4[pass][(key[k] >> (8 * pass)) & 0xffu], 1u);
      const uint32_t digit = key[k] >> 24;
      const uint32_t peers = same_digit_lanes(digit, valid[k]);
      if (valid[k] && (peers & lt_mask) == 0) atomicAdd(&hist4[3][digit], (uint32_t)__popc(peers));
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
    const uint32_t* hist = hist4[pass];

    // ---- exclusive scan of the 256 bins -> base
    if (tid < kRadix) {
      const uint32_t v = hist[tid];
      uint32_t incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
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

    // ---- stable scatter, one tile of 8192 elements at a time, tiles in order.  Inside a tile
    //      the order is (warp, item, lane), which is the order of the positions.
    for (long long t0 = 0; t0 < N; t0 += kTileItems) {
      uint32_t key[kItems]; int32_t val[kItems]; uint32_t rank[kItems];
      const long long w0 = t0 + (long long)warp * kWarpItems;
#pragma unroll
      for (int k = 0; k < kItems; ++k) {
        const long long i = w0 + k * 32 + lane;
        key[k] = 0; val[k] = -1;
        if (i < N) {
          if (pass == 0) { key[k] = score_to_key(s_in[i]); val[k] = (int32_t)i; }
          else { key[k] = src_k[i]; val[k] = src_v[i]; }
        }
      }
      // this warp's counters, then the rank of every item among the warp's items of its digit
      for (int dgt = lane; dgt < kRadix; dgt += 32) warp_cnt[warp][dgt] = 0;
      __syncwarp();
#pragma unroll
      for (int k = 0; k < kItems; ++k) {
        const bool valid = val[k] >= 0;
        const uint32_t digit = (key[k] >> shift) & 0xffu;
        const uint32_t peers = same_digit_lanes(digit, valid);
        uint32_t before = 0;
        if (valid) before = warp_cnt[warp][digit];
        __syncwarp();
        if (valid && (peers & lt_mask) == 0) warp_cnt[warp][digit] = (uint16_t)(before + __popc(peers));
        __syncwarp();
        rank[k] = before + __popc(peers & lt_mask);
      }
      __syncthreads();
      // per digit: exclusive scan over the warps; then the digit's first slot inside the tile
      // (exclusive scan over the digits) and its first position in the output
      uint32_t run = 0, incl = 0;
      if (tid < kRadix) {
#pragma unroll 8
        for (int wv = 0; wv < kWarps; ++wv) {
          const uint32_t cnt = warp_cnt[wv][tid];
          warp_cnt[wv][tid] = (uint16_t)run;
          run += cnt;
        }
        incl = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += n;
        }
        if (lane == 31) scan_tmp[warp] = incl;
      }
      __syncthreads();
      if (tid < kRadix) {
        uint32_t add = 0;
        for (int wv = 0; wv < warp; ++wv) add += scan_tmp[wv];
        tile_start[tid] = incl - run + add;
        tile_base[tid] = base[tid];
        base[tid] += run;
      }
      __syncthreads();
      // reorder the tile by digit in shared memory ...
#pragma unroll
      for (int k = 0; k < kItems; ++k) {
        if (val[k] >= 0) {
          const uint32_t digit = (key[k] >> shift) & 0xffu;
          const uint32_t slot = tile_start[digit] + warp_cnt[warp][digit] + rank[k];
          stage_k[slot] = key[k];
          stage_v[slot] = val[k];
        }
      }
      __syncthreads();
      // ... and write it out: neighbouring threads hold neighbours of the same digit, so the
      // stores of a warp fall into a few contiguous runs
      const int n_tile = (int)min((long long)kTileItems, N - t0);
#pragma unroll
      for (int k = 0; k < kItems; ++k) {
        const int slot = k * kSortThreads + tid;
        if (slot < n_tile) {
          const uint32_t kk = stage_k[slot];
          const uint32_t digit = (kk >> shift) & 0xffu;
          const uint32_t pos = tile_base[digit] + ((uint32_t)slot - tile_start[digit]);
          dst_k[pos] = kk;
          dst_v[pos] = stage_v[slot];
        }
      }
      __syncthreads();      // the stage and the per-tile tables are reused by the next tile
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
