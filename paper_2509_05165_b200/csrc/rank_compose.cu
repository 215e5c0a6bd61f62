// Per-head ranking (Eq. 17), sorted scores (Eq. 18) and composite scores (Eq. 19).
//
// Every (layer, sequence, KV head) is one segment of N (score, position) pairs that must come
// out in descending score order with equal scores in ascending position.  Scores are mapped to
// 32-bit keys whose ascending order is the wanted order, and all segments are sorted together by
// a stable least-significant-digit radix sort (8-bit digits, 4 passes) over tiles of 4096
// elements.  A pass is two kernels: one counts the digit of every tile, the other gives every
// tile its own CTA, which derives the tile's output ranges from the counts of its segment,
// ranks its elements, reorders them by digit in shared memory and writes them out in runs.
// Tiles are independent inside a pass, so the whole GPU is busy whatever the number of
// segments; the passes ping-pong between two scratch buffers that stay in L2.  The last pass
// writes the positions straight into idx and leaves the sorted keys for the composite kernel,
// which turns them back into scores and reduces over the heads.
#include "kvc_internal.cuh"

namespace kvc {
namespace {

constexpr int kSortThreads = 512;
constexpr int kWarps = kSortThreads / 32;
constexpr int kRadix = 256;
constexpr int kItems = 8;                               // elements per thread
constexpr int kTileItems = kSortThreads * kItems;       // 4096 elements per tile
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

// Source and destination of a pass.  0: scores -> A;  1: A -> B;  2: B -> A;  3: A -> (keys_b, idx).
struct PassIo {
  const uint32_t* src_k; const int32_t* src_v;
  uint32_t* dst_k; int32_t* dst_v;
};
__device__ __forceinline__ PassIo pass_io(const SortBuffers& buf, int32_t* idx_out, int pass, long long seg_off) {
  PassIo io;
  io.src_k = ((pass == 2) ? buf.keys_b : buf.keys_a) + seg_off;
  io.src_v = ((pass == 2) ? buf.vals_b : buf.vals_a) + seg_off;
  io.dst_k = ((pass == 0 || pass == 2) ? buf.keys_a : buf.keys_b) + seg_off;
  io.dst_v = ((pass == 0 || pass == 2) ? buf.vals_a : (pass == 3 ? idx_out : buf.vals_b)) + seg_off;
  return io;
}

// counts[seg][tile][digit]: how many elements of the tile have that digit in this pass.
__global__ void __launch_bounds__(kSortThreads, 4)
sort_count_kernel(const float* __restrict__ scores, SortBuffers buf, int32_t* idx_out,
                  uint32_t* __restrict__ counts, long long N, int tiles, int pass) {
  __shared__ uint32_t hist[kRadix];
  grid_dependency_wait();
  const long long seg = blockIdx.x / tiles;
  const int tile = (int)(blockIdx.x - seg * tiles);
  const PassIo io = pass_io(buf, idx_out, pass, seg * N);
  const float* s_in = scores + seg * N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const int shift = 8 * pass;
  for (int i = tid; i < kRadix; i += kSortThreads) hist[i] = 0;
  __syncthreads();
  // counting does not care about the order inside the tile: where the segment allows 16-byte
  // loads, a thread takes 8 consecutive elements with two of them
  const long long w0 = (long long)tile * kTileItems + (long long)warp * kWarpItems;
  const uint32_t* base = pass == 0 ? reinterpret_cast<const uint32_t*>(s_in) : io.src_k;
  const bool wide = (reinterpret_cast<uintptr_t>(base) & 15u) == 0 && w0 + kWarpItems <= N;
  uint32_t keys[kItems];
  if (wide) {
    const uint4* src = reinterpret_cast<const uint4*>(base) + (w0 >> 2) + lane * 2;
    const uint4 a = src[0], b = src[1];
    keys[0] = a.x; keys[1] = a.y; keys[2] = a.z; keys[3] = a.w;
    keys[4] = b.x; keys[5] = b.y; keys[6] = b.z; keys[7] = b.w;
    if (pass == 0) {
#pragma unroll
      for (int k = 0; k < kItems; ++k) keys[k] = score_to_key(__uint_as_float(keys[k]));
    }
  }
#pragma unroll
  for (int k = 0; k < kItems; ++k) {
    const long long i = w0 + k * 32 + lane;
    const bool valid = wide || i < N;
    uint32_t key = 0;
    if (wide) key = keys[k];
    else if (valid) key = (pass == 0) ? score_to_key(s_in[i]) : io.src_k[i];
    const uint32_t digit = (key >> shift) & 0xffu;
    if (pass < 3) {
      // the low digits are spread over their 256 bins: plain shared-memory atomics hardly collide
      if (valid) atomicAdd(&hist[digit], 1u);
    } else {
      // the top digit (sign and high exponent bits) takes a handful of values: add up per warp first
      const uint32_t peers = same_digit_lanes(digit, valid);
      if (valid && (peers & lt_mask) == 0) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
    }
  }
  __syncthreads();
  for (int i = tid; i < kRadix; i += kSortThreads) counts[((long long)seg * tiles + tile) * kRadix + i] = hist[i];
}

// One tile of one pass: stable scatter.  Inside a tile the order is (warp, item, lane), which
// is the order of the positions.
__global__ void __launch_bounds__(kSortThreads, 2)
sort_scatter_kernel(const float* __restrict__ scores, SortBuffers buf, int32_t* idx_out,
                    const uint32_t* __restrict__ counts, long long N, int tiles, int pass) {
  __shared__ uint32_t tile_base[kRadix];          // first output position of every digit for this tile
  __shared__ uint32_t tile_start[kRadix];         // first slot of every digit inside the reordered tile
  __shared__ uint16_t warp_cnt[kWarps][kRadix];   // count, then exclusive offset, per (warp, digit)
  __shared__ uint32_t scan_tmp[2][kRadix / 32];
  __shared__ uint32_t stage_k[kTileItems];        // the tile, reordered by digit, before it goes out
  __shared__ int32_t stage_v[kTileItems];

  grid_dependency_wait();
  const long long seg = blockIdx.x / tiles;
  const int tile = (int)(blockIdx.x - seg * tiles);
  const PassIo io = pass_io(buf, idx_out, pass, seg * N);
  const float* s_in = scores + seg * N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const int shift = 8 * pass;
  const long long t0 = (long long)tile * kTileItems;

  // ---- the tile's elements (issued first: the loads are in flight during the prologue)
  uint32_t key[kItems]; int32_t val[kItems]; uint32_t rank[kItems];
  {
    const long long w0 = t0 + (long long)warp * kWarpItems;
#pragma unroll
    for (int k = 0; k < kItems; ++k) {
      const long long i = w0 + k * 32 + lane;
      key[k] = 0; val[k] = -1;
      if (i < N) {
        if (pass == 0) { key[k] = score_to_key(s_in[i]); val[k] = (int32_t)i; }
        else { key[k] = io.src_k[i]; val[k] = io.src_v[i]; }
      }
    }
  }

  // ---- where the tile's digits go: (elements of smaller digits in the whole segment) +
  //      (elements of the same digit in earlier tiles); and where they sit inside the tile
  uint32_t total = 0, before = 0, mine = 0, incl_t = 0, incl_m = 0;
  if (tid < kRadix) {
    const uint32_t* c = counts + (long long)seg * tiles * kRadix + tid;
    for (int t = 0; t < tiles; ++t) {
      const uint32_t v = c[(long long)t * kRadix];
      total += v;
      if (t < tile) before += v;
      if (t == tile) mine = v;
    }
    incl_t = total; incl_m = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t a = __shfl_up_sync(0xffffffffu, incl_t, o);
      const uint32_t b2 = __shfl_up_sync(0xffffffffu, incl_m, o);
      if (lane >= o) { incl_t += a; incl_m += b2; }
    }
    if (lane == 31) { scan_tmp[0][warp] = incl_t; scan_tmp[1][warp] = incl_m; }
  }
  // this warp's counters, then the rank of every element among the warp's elements of its digit
  for (int dgt = lane; dgt < kRadix; dgt += 32) warp_cnt[warp][dgt] = 0;
  __syncwarp();
#pragma unroll
  for (int k = 0; k < kItems; ++k) {
    const bool valid = val[k] >= 0;
    const uint32_t digit = (key[k] >> shift) & 0xffu;
    const uint32_t peers = same_digit_lanes(digit, valid);
    uint32_t seen = 0;
    if (valid) seen = warp_cnt[warp][digit];
    __syncwarp();
    if (valid && (peers & lt_mask) == 0) warp_cnt[warp][digit] = (uint16_t)(seen + __popc(peers));
    __syncwarp();
    rank[k] = seen + __popc(peers & lt_mask);
  }
  __syncthreads();
  if (tid < kRadix) {
    uint32_t add_t = 0, add_m = 0;
    for (int wv = 0; wv < warp; ++wv) { add_t += scan_tmp[0][wv]; add_m += scan_tmp[1][wv]; }
    tile_base[tid] = incl_t - total + add_t + before;
    tile_start[tid] = incl_m - mine + add_m;
    // per digit: exclusive scan over the warps
    uint32_t run = 0;
#pragma unroll
    for (int wv = 0; wv < kWarps; ++wv) {
      const uint32_t cnt = warp_cnt[wv][tid];
      warp_cnt[wv][tid] = (uint16_t)run;
      run += cnt;
    }
  }
  __syncthreads();
  // ---- reorder the tile by digit in shared memory ...
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
  // ---- ... and write it out: neighbouring threads hold neighbours of the same digit, so the
  //      stores of a warp fall into a few contiguous runs
  const int n_tile = (int)min((long long)kTileItems, N - t0);
#pragma unroll
  for (int k = 0; k < kItems; ++k) {
    const int slot = k * kSortThreads + tid;
    if (slot < n_tile) {
      const uint32_t kk = stage_k[slot];
      const uint32_t digit = (kk >> shift) & 0xffu;
      const uint32_t pos = tile_base[digit] + ((uint32_t)slot - tile_start[digit]);
      io.dst_k[pos] = kk;
      io.dst_v[pos] = stage_v[slot];
    }
  }
}

// Eq. 19 over the sorted keys: composite[lb, k] = agg_head_h score(keys[lb, h, k]).
// Mean: heads added in ascending order in fp32, one division at the end.
__global__ void compose_kernel(const uint32_t* __restrict__ keys, float* __restrict__ composite,
                               int Hkv, long long N, long long total, int agg_head) {
  grid_dependency_wait();
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

// Eq. 18 as fp32: the sorted keys turned back into scores.
__global__ void sorted_scores_kernel(const uint32_t* __restrict__ keys, float* __restrict__ sorted, long long total) {
  grid_dependency_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) sorted[i] = key_to_score(keys[i]);
}

}  // namespace

static int sort_tiles(const Problem& P) { return (int)((P.N + kTileItems - 1) / kTileItems); }

size_t compose_workspace_bytes(const Problem& P) {
  const size_t items = (size_t)P.L * P.Bt * P.Hkv * P.N;
  const size_t segments = (size_t)P.L * P.Bt * P.Hkv;
  return 4 * align_up(items * 4) + align_up(segments * sort_tiles(P) * kRadix * sizeof(uint32_t));
}

kvc_status launch_sorted_scores(const Problem& P, const void* ws, float* sorted, cudaStream_t st) {
  const size_t items = (size_t)P.L * P.Bt * P.Hkv * P.N;
  const uint32_t* keys_b = reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(ws) + 2 * align_up(items * 4));
  KVC_CUDA(launch_dependent(sorted_scores_kernel, dim3((unsigned)((items + 255) / 256)), dim3(256), 0, st,
                            keys_b, sorted, (long long)items));
  KVC_LAUNCH_CHECK("sorted_scores_kernel");
  return KVC_OK;
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
  uint32_t* counts = reinterpret_cast<uint32_t*>(w + 4 * region);
  const long long segments = (long long)P.L * P.Bt * P.Hkv;
  const int tiles = sort_tiles(P);
  const long long blocks = segments * tiles;
  if (blocks >= (1LL << 31)) {
    set_error("compose: too many sort tiles");
    return KVC_ERR_UNSUPPORTED;
  }
  for (int pass = 0; pass < 4; ++pass) {
    KVC_CUDA(launch_dependent(sort_count_kernel, dim3((unsigned)blocks), dim3(kSortThreads), 0, st,
                              scores, buf, idx, counts, P.N, tiles, pass));
    KVC_LAUNCH_CHECK("sort_count_kernel");
    KVC_CUDA(launch_dependent(sort_scatter_kernel, dim3((unsigned)blocks), dim3(kSortThreads), 0, st,
                              scores, buf, idx, counts, P.N, tiles, pass));
    KVC_LAUNCH_CHECK("sort_scatter_kernel");
  }
  if (composite == nullptr) return KVC_OK;      // ranking only (the unstructured variant has no Eq. 19)
  const long long total = (long long)P.L * P.Bt * P.N;
  KVC_CUDA(launch_dependent(compose_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st,
                            buf.keys_b, composite, P.Hkv, P.N, total, P.agg_head));
  KVC_LAUNCH_CHECK("compose_kernel");
  return KVC_OK;
}

}  // namespace kvc
