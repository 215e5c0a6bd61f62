// Per-head ranking (Eq. 17), sorted scores (Eq. 18) and composite scores (Eq. 19).
//
// Every (layer, sequence, KV head) is one segment of N (score, position) pairs that must come
// out in descending score order with equal scores in ascending position.  Scores are mapped to
// 32-bit keys whose ascending order is the wanted order.  A segment of up to 32768 elements is
// sorted by one CTA inside its SM's shared memory (a stable least-significant-digit radix sort
// with 4-bit digits, thread-private counters, the permutation updated in place): one launch.  A
// longer segment is cut into such chunks, which are then merged pairwise (merge path), one launch
// per level.
//
// The positions go straight into idx and the sorted keys are left for the composite kernel, which turns them back into scores and reduces over the heads.
#include "kvc_internal.cuh"

#include <mutex>
#include <type_traits>

namespace kvc {
namespace {

// ---------------------------------------------------------------------------------------------
// Segments of at most kSegMaxN elements: one CTA sorts one whole segment inside its SM.
//
// A stable least-significant-digit sort with 4-bit digits.  The keys are read from global memory
// once and stay in shared memory, by position; what moves between the passes is a permutation of
// 16-bit positions, in place.  Thread t owns the places [t * ipt, (t + 1) * ipt) of the current
// order.  A pass:
//   count    every thread walks its places in order: position -> byte of the key -> digit, and a
//            counter of its own per digit (shared memory, one bank per lane): the value it finds
//            is the element's rank among the thread's elements of that digit.  No work crosses
//            lanes, so nothing depends on how the digits are distributed.
//   scan     exclusive prefix over (digit, thread), digits ascending: the first place of every
//            thread's elements of every digit.
//   scatter  position -> place = first place + rank.  Every thread read all of its places
//            before the scan, so the permutation is overwritten in place.
// (thread, place inside the thread) is the order itself, so every pass is stable, and with the
// identity as the first order equal keys stay in ascending position.  A digit that all keys of
// the segment share orders nothing and its pass is left out (scores in [2^-31, 2) share the
// top one).  After the last pass positions and keys go out through the permutation, coalesced.
// Global traffic: scores read once, idx and sorted keys written once; one launch.
constexpr int kSegMaxN = 32768;
constexpr int kSegMaxIpt = 32;                 // places per thread
constexpr int kSegBatch = 4;                   // key lookups in flight per thread
constexpr int kMaxDevices = 64;

__device__ __forceinline__ uint32_t lds_u8(uint32_t a) { uint32_t v; asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a) : "memory"); return v; }
__device__ __forceinline__ uint32_t lds_u16(uint32_t a) { uint32_t v; asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(a) : "memory"); return v; }
__device__ __forceinline__ uint32_t lds_u32(uint32_t a) { uint32_t v; asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory"); return v; }
__device__ __forceinline__ uint4 lds_v4(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void sts_u16(uint32_t a, uint32_t v) { asm volatile("st.shared.u16 [%0], %1;" :: "r"(a), "h"((unsigned short)v) : "memory"); }
__device__ __forceinline__ void sts_u32(uint32_t a, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" :: "r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ void sts_v4(uint32_t a, uint4 v) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" :: "r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Shared-memory map of a segment of N elements sorted by T threads (byte offsets).
struct SegLayout {
  int n_pad;            // N rounded up to 32: key_slot and place_slot permute inside aligned blocks of 32
  int lg;               // log2 of the places per thread
  uint32_t keys;        // uint32[n_pad]: the keys, by position
  uint32_t perm;        // uint16[n_pad]: the key slot (key_slot of the position) at every place
  uint32_t cnt;         // uint16[8][T][2]: thread t's counter of digit d in row d & 7, half d >> 3
  uint32_t wtot;        // uint32[32]: the scan's warp totals;  uint32: bits that differ between keys
  uint32_t total;
};
__host__ __device__ inline SegLayout seg_layout(long long N, int T) {
  SegLayout s;
  s.n_pad = (int)((N + 31) / 32 * 32);
  s.lg = 0;
  while (((long long)T << s.lg) < N) ++s.lg;
  s.keys = 0;
  s.perm = 4u * s.n_pad;
  s.cnt = s.perm + 2u * s.n_pad;
  s.wtot = s.cnt + 8u * T * 4u;
  s.total = s.wtot + 256u;
  return s;
}

// Where things sit, to keep the banks apart.  Key of position i: word i ^ ((i >> 5) & 31): the
// threads of a warp start 32 places apart, which in the first pass are 32 positions apart.
// Place j: halfword j ^ (((j >> 6) & 3) << 3): a warp reads 32 stretches of 64 bytes, 16 at a time.
__device__ __forceinline__ uint32_t key_slot(uint32_t i) { return i ^ ((i >> 5) & 31u); }
__device__ __forceinline__ uint32_t place_slot(uint32_t j) { return j ^ (((j >> 6) & 3u) << 3); }

// score_to_key without the branch.
__device__ __forceinline__ uint32_t seg_key(float f) {
  uint32_t b = __float_as_uint(f);
  b = (b == 0x80000000u) ? 0u : b;
  const uint32_t m = (uint32_t)((int32_t)b >> 31) | 0x80000000u;
  return ~(b ^ m);
}

// Every group of 4 consecutive keys of the segment goes to use(i, k0, k1, k2, k3, n): i = position
// of the first (a multiple of 4), n = how many of the 4 exist.  With 16-byte aligned scores all of
// a thread's loads are issued before the first use.
template <int T, typename F>
__device__ __forceinline__ void seg_for_keys(const float* s_in, int N, int tid, F use) {
  constexpr int kGroups = kSegMaxIpt / 4;
  const bool wide = (reinterpret_cast<uintptr_t>(s_in) & 15u) == 0 && N >= 4;
  if (wide) {
    const int last = (N & ~3) - 4;                           // first position of the last whole group
    float4 v[kGroups];
#pragma unroll
    for (int g = 0; g < kGroups; ++g) v[g] = *reinterpret_cast<const float4*>(s_in + min((g * T + tid) * 4, last));
#pragma unroll
    for (int g = 0; g < kGroups; ++g) {
      const int i = (g * T + tid) * 4;
      if (i + 4 <= N) use(i, seg_key(v[g].x), seg_key(v[g].y), seg_key(v[g].z), seg_key(v[g].w), 4);
    }
    if (tid == 0 && (N & 3)) {
      const int i = N & ~3;
      use(i, seg_key(s_in[i]), seg_key(i + 1 < N ? s_in[i + 1] : 0.f), seg_key(i + 2 < N ? s_in[i + 2] : 0.f), seg_key(0.f), N - i);
    }
  } else {
    for (int i = tid * 4; i < N; i += T * 4)
      use(i, seg_key(s_in[i]), seg_key(i + 1 < N ? s_in[i + 1] : 0.f), seg_key(i + 2 < N ? s_in[i + 2] : 0.f),
          seg_key(i + 3 < N ? s_in[i + 3] : 0.f), min(4, N - i));
  }
}

template <int T>
__global__ void __launch_bounds__(T, T == 1024 ? 1 : 4)
segment_sort_kernel(const float* __restrict__ scores, uint32_t* __restrict__ keys_out,
                    int32_t* __restrict__ idx_out, long long seg_len, int chunks) {
  // CTA x sorts chunk x % chunks of segment x / chunks: the positions from chunk * kSegMaxN on (a segment of
  // up to kSegMaxN elements is one chunk; the chunks of a longer one are merged afterwards)
  const long long seg = blockIdx.x / (unsigned)chunks;
  const int chunk = (int)(blockIdx.x - seg * chunks);
  const long long first = seg * seg_len + (long long)chunk * kSegMaxN;      // of this chunk, in all three arrays
  const int N = (int)min((long long)kSegMaxN, seg_len - (long long)chunk * kSegMaxN);
  constexpr int kRowShift = (T == 1024) ? 12 : 10;          // log2 of a row of counters in bytes
  static_assert(T == 1024 || T == 256, "row shift");
  constexpr int kScanWarps = T / 64;                        // the scan runs on the first T / 2 threads
  extern __shared__ __align__(16) unsigned char seg_smem[];
  const SegLayout lay = seg_layout(N, T);
  const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(seg_smem);
  const uint32_t keys = sbase + lay.keys, perm = sbase + lay.perm, cnt = sbase + lay.cnt, wtot = sbase + lay.wtot;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int lg = lay.lg, ipt = 1 << lg;
  const int j0 = tid << lg;
  const int nv = max(0, min(ipt, N - j0));                   // my places: j0 .. j0 + nv - 1
  const bool full = __all_sync(0xffffffffu, nv == kSegMaxIpt);   // the warp's decision
  // My counter of digit d: + ((d & 7) << kRowShift) + ((d >> 3) << 1).  Inside a warp's 32 columns, groups
  // of 4 are permuted by the warp number so that the scan's 16-byte reads of neighbouring columns spread
  // over the banks; a lane keeps a bank of its own.
  const uint32_t cbase = cnt + (uint32_t)(tid ^ (((tid >> 5) & 3) << 2)) * 4u;

  grid_dependency_wait();
  const float* s_in = scores + first;

  // ---- the keys, once; the identity as the first order; which bits differ anywhere in the segment
  uint32_t diff = 0;
  {
    const uint32_t ref = seg_key(s_in[0]);
    if (tid == 0) sts_u32(wtot + 128, 0u);
    seg_for_keys<T>(s_in, N, tid, [&](int i, uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3, int n) {
      const uint32_t sw = ((uint32_t)i >> 5) & 31u;          // the four stay inside their 16 bytes; the table is padded
      sts_u32(keys + (((uint32_t)i) ^ sw) * 4u, k0);
      sts_u32(keys + (((uint32_t)i + 1u) ^ sw) * 4u, k1);
      sts_u32(keys + (((uint32_t)i + 2u) ^ sw) * 4u, k2);
      sts_u32(keys + (((uint32_t)i + 3u) ^ sw) * 4u, k3);
      diff |= k0 ^ ref;
      if (n > 1) diff |= k1 ^ ref;
      if (n > 2) diff |= k2 ^ ref;
      if (n > 3) diff |= k3 ^ ref;
    });
    // (the permutation holds key slots, not positions: a lookup needs no translation)
    if (lg >= 3) {
#pragma unroll
      for (int q = 0; q < kSegMaxIpt / 8; ++q) {
        if (q * 8 < nv) {
          const uint32_t j = (uint32_t)(j0 + q * 8);
          // j is a multiple of 8: the eight slots are (j ^ m's high bits) | (e ^ m's low 3 bits), e = 0..7
          const uint32_t m = (j >> 5) & 31u;
          const uint32_t bb = (j ^ (m & 24u)) * 0x10001u, mm = (m & 7u) * 0x10001u;
          sts_v4(perm + place_slot(j) * 2u, make_uint4(bb | (0x10000u ^ mm), bb | (0x30002u ^ mm),
                                                         bb | (0x50004u ^ mm), bb | (0x70006u ^ mm)));
        }
      }
    } else {
      for (int k = 0; k < nv; ++k) sts_u16(perm + place_slot((uint32_t)(j0 + k)) * 2u, key_slot((uint32_t)(j0 + k)));
    }
    diff = __reduce_or_sync(0xffffffffu, diff);
    __syncthreads();
    if (lane == 0 && diff != 0) atomicOr(reinterpret_cast<uint32_t*>(seg_smem + lay.wtot + 128), diff);
    __syncthreads();
    diff = lds_u32(wtot + 128);
  }

#pragma unroll 1
  for (int B = 0; B < 4; ++B) {
    const uint32_t kb = keys + (uint32_t)B;                  // byte B of the key in slot s: kb + 4 s
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (((diff >> (8 * B + 4 * h)) & 15u) == 0) continue;  // a digit every key shares orders nothing
      // with an element as  key slot | byte << 16 | rank << 24,  its digit d sits at bit 16 + 4 h
      constexpr uint32_t kRowMask = 7u << kRowShift;
      const int sh_row = 16 + 4 * h - kRowShift, sh_half = 18 + 4 * h;

      // ---- count (threads whose 32 places all exist take the copy without the per-place tests)
#pragma unroll
      for (int d = 0; d < 8; ++d) sts_u32(cbase + ((uint32_t)d << kRowShift), 0u);
      uint32_t packed[kSegMaxIpt];
      auto count = [&](auto full_tag) {
        constexpr bool kFull = decltype(full_tag)::value;
        if (kFull || lg >= 3) {
#pragma unroll
          for (int q = 0; q < kSegMaxIpt / 8; ++q) {
            if (kFull || q * 8 < nv) {
              const uint4 w = lds_v4(perm + place_slot((uint32_t)(j0 + q * 8)) * 2u);
              packed[q * 8 + 0] = w.x & 0xffffu; packed[q * 8 + 1] = w.x >> 16;
              packed[q * 8 + 2] = w.y & 0xffffu; packed[q * 8 + 3] = w.y >> 16;
              packed[q * 8 + 4] = w.z & 0xffffu; packed[q * 8 + 5] = w.z >> 16;
              packed[q * 8 + 6] = w.w & 0xffffu; packed[q * 8 + 7] = w.w >> 16;
            }
          }
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k) if (k < nv) packed[k] = lds_u16(perm + place_slot((uint32_t)(j0 + k)) * 2u);
        }
#pragma unroll
        for (int k0 = 0; k0 < kSegMaxIpt; k0 += kSegBatch) {
          uint32_t b[kSegBatch];
#pragma unroll
          for (int k = 0; k < kSegBatch; ++k) if (kFull || k0 + k < nv) b[k] = lds_u8(kb + packed[k0 + k] * 4u);
#pragma unroll
          for (int k = 0; k < kSegBatch; ++k) {
            if (kFull || k0 + k < nv) {
              const uint32_t pk = packed[k0 + k] | (b[k] << 16);
              const uint32_t a = cbase + (((pk >> sh_row) & kRowMask) | ((pk >> sh_half) & 2u));
              const uint32_t seen = lds_u16(a);
              sts_u16(a, seen + 1u);
              packed[k0 + k] = pk + (seen << 24);
            }
          }
        }
      };
      if (full) count(std::true_type{}); else count(std::false_type{});
      __syncthreads();

      // ---- scan.  Thread s < T / 2 owns 16 neighbouring threads' counters of the digits in its row: the low
      //      halves (digit = row) precede all high halves (digit = row + 8) in the order of the places.
      {
        const uint32_t mine = cnt + (uint32_t)tid * 64u;
        const uint32_t rot = (((uint32_t)tid >> 1) & 3u) << 4;                     // the permutation of cbase, seen from here
        uint32_t lo_sum = 0, hi_sum = 0, lo_incl = 0, hi_incl = 0;
        if (tid < T / 2) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 w = lds_v4(mine + ((q * 16) ^ rot));
            lo_sum += (w.x & 0xffffu) + (w.y & 0xffffu) + (w.z & 0xffffu) + (w.w & 0xffffu);
            hi_sum += (w.x >> 16) + (w.y >> 16) + (w.z >> 16) + (w.w >> 16);
          }
          lo_incl = lo_sum; hi_incl = hi_sum;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const uint32_t x = __shfl_up_sync(0xffffffffu, lo_incl, o);
            const uint32_t y = __shfl_up_sync(0xffffffffu, hi_incl, o);
            if (lane >= o) { lo_incl += x; hi_incl += y; }
          }
          if (lane == 31) { sts_u32(wtot + warp * 4, lo_incl); sts_u32(wtot + (kScanWarps + warp) * 4, hi_incl); }
        }
        __syncthreads();
        if (tid < T / 2) {
          const uint32_t x = lane < 2 * kScanWarps ? lds_u32(wtot + lane * 4) : 0u;
          uint32_t e = x;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, e, o);
            if (lane >= o) e += y;
          }
          e -= x;                                                                  // exclusive over the warp totals
          uint32_t lo = __shfl_sync(0xffffffffu, e, warp) + lo_incl - lo_sum;
          uint32_t hi = __shfl_sync(0xffffffffu, e, kScanWarps + warp) + hi_incl - hi_sum;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t a = mine + ((q * 16) ^ rot);
            const uint4 w = lds_v4(a);
            uint4 o4;
            o4.x = lo | (hi << 16); lo += w.x & 0xffffu; hi += w.x >> 16;
            o4.y = lo | (hi << 16); lo += w.y & 0xffffu; hi += w.y >> 16;
            o4.z = lo | (hi << 16); lo += w.z & 0xffffu; hi += w.z >> 16;
            o4.w = lo | (hi << 16); lo += w.w & 0xffffu; hi += w.w >> 16;
            sts_v4(a, o4);
          }
        }
      }
      __syncthreads();

      // ---- scatter (in place: every place was read before the scan)
      auto scatter = [&](auto full_tag) {
        constexpr bool kFull = decltype(full_tag)::value;
#pragma unroll
        for (int k = 0; k < kSegMaxIpt; ++k) {
          if (kFull || k < nv) {
            const uint32_t pk = packed[k];
            const uint32_t off = lds_u16(cbase + (((pk >> sh_row) & kRowMask) | ((pk >> sh_half) & 2u)));
            sts_u16(perm + place_slot(off + (pk >> 24)) * 2u, pk);
          }
        }
      };
      if (full) scatter(std::true_type{}); else scatter(std::false_type{});
      __syncthreads();
    }
  }

  // ---- out: the positions (a slot's position is key_slot of it: the map is its own inverse), and the keys
  uint32_t* k_out = keys_out + first;
  int32_t* i_out = idx_out + first;
  const int pos0 = chunk * kSegMaxN;
  for (int j = tid; j < N; j += T) {
    const uint32_t q = lds_u16(perm + place_slot((uint32_t)j) * 2u);
    i_out[j] = pos0 + (int32_t)key_slot(q);
    k_out[j] = lds_u32(keys + q * 4u);
  }
}

// ---------------------------------------------------------------------------------------------
// Segments longer than kSegMaxN: their chunks come sorted from segment_sort_kernel and are merged
// pairwise, level by level (runs of kSegMaxN << level elements).  A CTA produces kMergeTile
// consecutive outputs of one pair of runs A, B: it finds where the tile's first and last output
// split between A and B (the merge path: a binary search over one diagonal each), brings the two
// stretches into shared memory, and every thread merges kMergeItems consecutive outputs from its
// own diagonal.  Equal keys are taken from A first: A holds the smaller positions and both runs
// are stable, so the merged run is in (key, position) order as well.
constexpr int kMergeThreads = 512;
constexpr int kMergeItems = 8;
constexpr int kMergeTile = kMergeThreads * kMergeItems;       // 4096; divides kSegMaxN

// Number of elements taken from A among the first `diag` outputs of merging A (na) and B (nb).
__device__ __forceinline__ int merge_path(int diag, int na, int nb, const uint32_t* a, const uint32_t* b) {
  int lo = max(0, diag - nb), hi = min(diag, na);
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    // A[mid] is among the first diag outputs iff it does not come after B[diag - 1 - mid]
    if (a[mid] <= b[diag - 1 - mid]) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// The same by one warp over global memory, 32 probes per round (a round trip per round, not per probe).
__device__ __forceinline__ int merge_path_warp(int diag, int na, int nb, const uint32_t* __restrict__ a,
                                               const uint32_t* __restrict__ b) {
  const int lane = threadIdx.x & 31;
  int lo = max(0, diag - nb), hi = min(diag, na);          // the answer lies in [lo, hi]
  while (hi > lo) {
    const int step = (hi - lo + 31) / 32;
    const int i = lo + (lane + 1) * step - 1;              // this lane's probe
    bool before = false;                                   // "A[i] is among the first diag outputs": true for a prefix of the probes
    if (i < hi) before = a[i] <= b[diag - 1 - i];
    const int n_before = __popc(__ballot_sync(0xffffffffu, before));
    const int new_lo = n_before == 0 ? lo : min(hi, lo + n_before * step);
    const int new_hi = n_before == 32 ? hi : min(hi, lo + (n_before + 1) * step - 1);
    lo = new_lo;
    hi = new_hi;
  }
  return lo;
}

__global__ void __launch_bounds__(kMergeThreads)
merge_runs_kernel(const uint32_t* __restrict__ keys_in, const int32_t* __restrict__ vals_in,
                  uint32_t* __restrict__ keys_out, int32_t* __restrict__ vals_out, long long seg_len, long long run,
                  int tiles_per_seg) {
  __shared__ uint32_t s_key[kMergeTile];
  __shared__ int32_t s_val[kMergeTile];
  __shared__ int s_split[2];
  grid_dependency_wait();
  const long long seg = blockIdx.x / (unsigned)tiles_per_seg;
  const long long t0 = (long long)(blockIdx.x - seg * tiles_per_seg) * kMergeTile;    // first output, inside the segment
  const long long pair0 = t0 / (2 * run) * (2 * run);                                  // where this tile's pair of runs starts
  const int na = (int)min(run, seg_len - pair0);
  const int nb = (int)max(0LL, min(run, seg_len - pair0 - run));
  const long long base = seg * seg_len + pair0;
  const uint32_t* ka = keys_in + base;
  const uint32_t* kb = ka + na;
  const int d0 = (int)(t0 - pair0);
  const int d1 = min(d0 + kMergeTile, na + nb);
  const int tid = threadIdx.x;
  if (tid < 64) {                                          // warp 0: the tile's first output; warp 1: one past its last
    const int split = merge_path_warp(tid < 32 ? d0 : d1, na, nb, ka, kb);
    if ((tid & 31) == 0) s_split[tid >> 5] = split;
  }
  __syncthreads();
  const int a0 = s_split[0], a1 = s_split[1];
  const int b0 = d0 - a0, b1 = d1 - a1;
  const int ca = a1 - a0, cb = b1 - b0;                   // this tile's elements of A, then of B, in shared memory
  for (int i = tid; i < ca + cb; i += kMergeThreads) {
    const long long src = base + (i < ca ? (long long)a0 + i : (long long)na + b0 + (i - ca));
    s_key[i] = keys_in[src];
    s_val[i] = vals_in[src];
  }
  __syncthreads();
  const int n_out = d1 - d0;
  const int my0 = min(tid * kMergeItems, n_out);
  int ia = merge_path(my0, ca, cb, s_key, s_key + ca);
  int ib = my0 - ia;
  uint32_t ok[kMergeItems]; int32_t ov[kMergeItems];
#pragma unroll
  for (int k = 0; k < kMergeItems; ++k) {
    const bool has_a = ia < ca, has_b = ib < cb;
    const uint32_t xa = has_a ? s_key[ia] : 0xffffffffu, xb = has_b ? s_key[ca + ib] : 0xffffffffu;
    const bool take_a = has_a && (!has_b || xa <= xb);
    ok[k] = take_a ? xa : xb;
    ov[k] = take_a ? s_val[ia] : (has_b ? s_val[ca + ib] : 0);
    if (take_a) ++ia; else ++ib;
  }
  __syncthreads();                                         // everyone has read its inputs: the buffers take the outputs
#pragma unroll
  for (int k = 0; k < kMergeItems; ++k) {
    if (my0 + k < n_out) { s_key[my0 + k] = ok[k]; s_val[my0 + k] = ov[k]; }
  }
  __syncthreads();
  const long long dst = base + d0;
  for (int i = tid; i < n_out; i += kMergeThreads) {
    keys_out[dst + i] = s_key[i];
    vals_out[dst + i] = s_val[i];
  }
}

// Eq. 19 over the sorted keys: composite[lb, k] = agg_head_h score(keys[lb, h, k]).
// Mean: heads added in ascending order in fp32, one division at the end.
// blockIdx.y = (layer, sequence), blockIdx.x over the ranks.  The heads' keys are fetched eight at a
// time before they are added, so that a thread waits for memory once, not once per head.
__global__ void compose_kernel(const uint32_t* __restrict__ keys, float* __restrict__ composite,
                               int Hkv, long long N, int agg_head) {
  grid_dependency_wait();
  const long long kk = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (kk >= N) return;
  const long long lb = blockIdx.y;
  const uint32_t* p = keys + lb * Hkv * N + kk;
  float acc = 0.f;
  for (int h0 = 0; h0 < Hkv; h0 += 8) {
    uint32_t v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = h0 + j < Hkv ? p[(long long)(h0 + j) * N] : 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (h0 + j < Hkv) {
        const float a = key_to_score(v[j]);
        if (h0 + j == 0) acc = a;
        else acc = (agg_head == KVC_AGG_MAX) ? fmaxf(acc, a) : __fadd_rn(acc, a);
      }
    }
  }
  if (agg_head == KVC_AGG_MEAN) acc = __fdiv_rn(acc, (float)Hkv);
  composite[lb * N + kk] = acc;
}

// Eq. 18 as fp32: the sorted keys turned back into scores.
__global__ void sorted_scores_kernel(const uint32_t* __restrict__ keys, float* __restrict__ sorted, long long total) {
  grid_dependency_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) sorted[i] = key_to_score(keys[i]);
}

}  // namespace

// Can a segment of N elements be sorted inside one SM here?  Sets the shared-memory attribute once
// per device (it is per device), under a lock.  *threads = the CTA size to launch.
static kvc_status segment_sort_prepare(long long N, int* threads) {
  if (N > kSegMaxN) return KVC_ERR_UNSUPPORTED;
  static std::mutex mu;
  static int optin[kMaxDevices];           // 0: not looked at, else the device's opt-in bytes (or -1)
  int dev = 0;
  KVC_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return KVC_ERR_UNSUPPORTED;
  const int T = N > 8192 ? 1024 : 256;
  const size_t need = seg_layout(N, T).total;
  std::lock_guard<std::mutex> lock(mu);
  if (optin[dev] == 0) {
    int bytes = 0;
    KVC_CUDA(cudaDeviceGetAttribute(&bytes, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    KVC_CUDA(cudaFuncSetAttribute(segment_sort_kernel<1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    KVC_CUDA(cudaFuncSetAttribute(segment_sort_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    optin[dev] = bytes > 0 ? bytes : -1;
  }
  if (optin[dev] < 0 || need > (size_t)optin[dev]) return KVC_ERR_UNSUPPORTED;
  *threads = T;
  return KVC_OK;
}

// Scratch of the ranking: the sorted keys [L, Bt, Hkv, N] and, for segments of several chunks, one more
// buffer of keys and one of positions for the merge levels to alternate with (keys, idx).
struct SortRegions {
  size_t keys_a, vals_a, keys_b, total;
};
static SortRegions sort_regions(const Problem& P) {
  const size_t region = align_up((size_t)P.L * P.Bt * P.Hkv * P.N * 4);
  SortRegions r;
  if (P.N <= kSegMaxN) { r.keys_a = r.vals_a = 0; r.keys_b = 0; r.total = region; }
  else { r.keys_a = 0; r.vals_a = region; r.keys_b = 2 * region; r.total = 3 * region; }
  return r;
}

size_t compose_workspace_bytes(const Problem& P) { return sort_regions(P).total; }

kvc_status launch_sorted_scores(const Problem& P, const void* ws, float* sorted, cudaStream_t st) {
  const size_t items = (size_t)P.L * P.Bt * P.Hkv * P.N;
  const uint32_t* keys_b = reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(ws) + sort_regions(P).keys_b);
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
  char* w = reinterpret_cast<char*>(ws);
  const SortRegions reg = sort_regions(P);
  uint32_t* const keys_a = reinterpret_cast<uint32_t*>(w + reg.keys_a);
  int32_t* const vals_a = reinterpret_cast<int32_t*>(w + reg.vals_a);
  uint32_t* const keys_b = reinterpret_cast<uint32_t*>(w + reg.keys_b);
  const long long segments = (long long)P.L * P.Bt * P.Hkv;
  int seg_threads = 0;
  const long long chunk_len = P.N < kSegMaxN ? P.N : (long long)kSegMaxN;
  const kvc_status seg_state = segment_sort_prepare(chunk_len, &seg_threads);
  if (seg_state != KVC_OK && seg_state != KVC_ERR_UNSUPPORTED) return seg_state;
  if (seg_state != KVC_OK) {
    set_error("compose: this device cannot give a CTA the %zu bytes of shared memory the ranking needs",
              (size_t)seg_layout(chunk_len, chunk_len > 8192 ? 1024 : 256).total);
    return KVC_ERR_UNSUPPORTED;
  }
  {
    // Chunks of up to kSegMaxN elements are sorted inside one SM each: a whole segment in one launch, or,
    // for longer segments, its chunks, which are then merged pairwise, level by level.  The levels
    // alternate between (keys_a, vals_a) and (keys_b, idx); the last one has to end in the latter.
    const long long chunks = (P.N + kSegMaxN - 1) / kSegMaxN;
    int levels = 0;
    while ((1LL << levels) < chunks) ++levels;
    const long long merge_tiles = (P.N + kMergeTile - 1) / kMergeTile;
    if (segments * chunks >= (1LL << 31) || segments * merge_tiles >= (1LL << 31)) {
      set_error("compose: too many segments");
      return KVC_ERR_UNSUPPORTED;
    }
    bool in_b = (levels % 2) == 0;                 // where the sorted chunks go
    uint32_t* k_cur = in_b ? keys_b : keys_a;
    int32_t* v_cur = in_b ? idx : vals_a;
    const size_t smem = seg_layout(chunk_len, seg_threads).total;
    const unsigned grid = (unsigned)(segments * chunks);
    if (seg_threads == 1024) {
      KVC_CUDA(launch_dependent(segment_sort_kernel<1024>, dim3(grid), dim3(1024), smem, st,
                                scores, k_cur, v_cur, P.N, (int)chunks));
    } else {
      KVC_CUDA(launch_dependent(segment_sort_kernel<256>, dim3(grid), dim3(256), smem, st,
                                scores, k_cur, v_cur, P.N, (int)chunks));
    }
    KVC_LAUNCH_CHECK("segment_sort_kernel");
    for (int level = 0; level < levels; ++level) {
      in_b = !in_b;
      uint32_t* k_nxt = in_b ? keys_b : keys_a;
      int32_t* v_nxt = in_b ? idx : vals_a;
      KVC_CUDA(launch_dependent(merge_runs_kernel, dim3((unsigned)(segments * merge_tiles)), dim3(kMergeThreads), 0, st,
                                (const uint32_t*)k_cur, (const int32_t*)v_cur, k_nxt, v_nxt, P.N,
                                (long long)kSegMaxN << level, (int)merge_tiles));
      KVC_LAUNCH_CHECK("merge_runs_kernel");
      k_cur = k_nxt;
      v_cur = v_nxt;
    }
  }
  if (composite == nullptr) return KVC_OK;      // ranking only (the unstructured variant has no Eq. 19)
  KVC_CUDA(launch_dependent(compose_kernel, dim3((unsigned)((P.N + 255) / 256), (unsigned)(P.L * P.Bt)), dim3(256), 0, st,
                            keys_b, composite, P.Hkv, P.N, P.agg_head));
  KVC_LAUNCH_CHECK("compose_kernel");
  return KVC_OK;
}

}  // namespace kvc
