// Compaction of the retained rows (Eqs. 23-24):
//   K'[l][h, k, :] = K[l][h, idx[l, h, k], :]  for k < N_l, and the same for V.
//
// Pure data movement: every output row is one contiguous head_dim-wide row of the cache.  A row
// is moved by row_bytes / 16 lanes with one 16-byte load and one 16-byte store each; a warp
// carries 32 / lanes_per_row rows of K and of V per step; parallelism comes from many resident
// CTAs rather than from several rows per thread.
// The per-layer counts and offsets are read on the device, so no host synchronisation is needed
// between allocation and compaction.
#include "kvc_internal.cuh"

namespace kvc {
namespace {

constexpr int kGatherThreads = 256;
constexpr int kUnroll = 1;            // rows per thread and step: more of them in flight was slower (measured 1 to 8)

struct GatherParams {
  int L, Bt, Hkv;
  long long N, budget;
  long long kvs0, kvs1, kvs2;  // in units of 16 bytes
  int lanes_per_row;           // row_bytes / 16
  int lanes_shift;             // log2(lanes_per_row)
  long long rows_per_seq;      // budget * Hkv (per layer) or the budget in entries (per head)
};

__device__ inline uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ inline void st_stream(uint4* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
               :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// kPerHead = false: n_keep / offsets per layer, a layer's block is [Hkv, N_l, d] (Eqs. 23-24).
// kPerHead = true:  n_keep / offsets per (layer, head), a head's block is [n, d] (App. A.2).
template <bool kPerHead>
__global__ void __launch_bounds__(kGatherThreads)
gather_kernel(GatherParams P, LayerPtrs kp, LayerPtrs vp, const int32_t* __restrict__ idx,
              const int32_t* __restrict__ n_keep, const long long* __restrict__ offsets,
              uint4* __restrict__ k_out, uint4* __restrict__ v_out) {
  extern __shared__ long long s_off[];              // the sequence's offsets: R + 1 entries
  grid_dependency_wait();
  const int b = blockIdx.y;
  const int R = kPerHead ? P.L * P.Hkv : P.L;
  for (int i = threadIdx.x; i <= R; i += kGatherThreads) s_off[i] = offsets[(long long)b * (R + 1) + i];
  __syncthreads();

  const int lpr = P.lanes_per_row;
  const int sub = threadIdx.x & (lpr - 1);                       // which 16-byte piece of the row
  const long long rows_per_step = (long long)gridDim.x * (kGatherThreads >> P.lanes_shift);
  long long row = (long long)blockIdx.x * (kGatherThreads >> P.lanes_shift) + (threadIdx.x >> P.lanes_shift);

  for (; row < P.rows_per_seq; row += rows_per_step * kUnroll) {
    uint4 kv[kUnroll], vv[kUnroll];
    long long dst[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const long long r = row + u * rows_per_step;
      dst[u] = -1;
      if (r < P.rows_per_seq) {
        // block: the last one whose first output row is <= r
        const long long mult = kPerHead ? 1 : P.Hkv;
        int lo = 0, hi = R;               // invariant: s_off[lo] * mult <= r < s_off[hi] * mult
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (s_off[mid] * mult <= r) lo = mid; else hi = mid;
        }
        int l, h;
        long long kk;
        if (kPerHead) {
          l = lo / P.Hkv; h = lo - l * P.Hkv;
          kk = r - s_off[lo];
        } else {
          l = lo;
          const long long nl = n_keep[(long long)b * P.L + l];
          const long long local = r - s_off[l] * P.Hkv;          // in [0, Hkv * nl)
          h = (int)(local / nl);
          kk = local - (long long)h * nl;
        }
        const long long c = idx[(((long long)l * P.Bt + b) * P.Hkv + h) * P.N + kk];
        const long long src = b * P.kvs0 + h * P.kvs1 + c * P.kvs2 + sub;
        kv[u] = ld_stream(reinterpret_cast<const uint4*>(kp.p[l]) + src);
        vv[u] = ld_stream(reinterpret_cast<const uint4*>(vp.p[l]) + src);
        dst[u] = ((long long)b * P.rows_per_seq + r) * lpr + sub;
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      if (dst[u] >= 0) {
        st_stream(k_out + dst[u], kv[u]);
        st_stream(v_out + dst[u], vv[u]);
      }
    }
  }
}

}  // namespace

kvc_status launch_gather(const Problem& P, const LayerPtrs& k, const LayerPtrs& v, const int32_t* idx,
                         const int32_t* n_keep, const long long* offsets, long long budget, bool per_head,
                         void* k_out, void* v_out, cudaStream_t st) {
  if (budget == 0) return KVC_OK;
  GatherParams gp;
  gp.L = P.L; gp.Bt = P.Bt; gp.Hkv = P.Hkv; gp.N = P.N; gp.budget = budget;
  const int row_bytes = P.d * P.elem_bytes;
  const int per16 = 16 / P.elem_bytes;
  gp.kvs0 = P.kvs[0] / per16; gp.kvs1 = P.kvs[1] / per16; gp.kvs2 = P.kvs[2] / per16;
  gp.lanes_per_row = row_bytes / 16;
  gp.lanes_shift = 0;
  while ((1 << gp.lanes_shift) < gp.lanes_per_row) ++gp.lanes_shift;
  gp.rows_per_seq = per_head ? budget : budget * P.Hkv;
  const long long rows_per_block = kGatherThreads / gp.lanes_per_row;
  long long blocks = (gp.rows_per_seq + rows_per_block * kUnroll - 1) / (rows_per_block * kUnroll);
  int dev = 0, sms = 0;
  KVC_CUDA(cudaGetDevice(&dev));
  KVC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const long long cap = (long long)sms * 128;   // measured best among 8 to 256 CTAs per SM's worth of grid
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const int R = per_head ? P.L * P.Hkv : P.L;
  const size_t smem = (size_t)(R + 1) * sizeof(long long);
  if (per_head) {
    KVC_CUDA(launch_dependent(gather_kernel<true>, dim3((unsigned)blocks, P.Bt), dim3(kGatherThreads), smem, st,
                              gp, k, v, idx, n_keep, offsets, reinterpret_cast<uint4*>(k_out),
                              reinterpret_cast<uint4*>(v_out)));
  } else {
    KVC_CUDA(launch_dependent(gather_kernel<false>, dim3((unsigned)blocks, P.Bt), dim3(kGatherThreads), smem, st,
                              gp, k, v, idx, n_keep, offsets, reinterpret_cast<uint4*>(k_out),
                              reinterpret_cast<uint4*>(v_out)));
  }
  KVC_LAUNCH_CHECK("gather_kernel");
  return KVC_OK;
}

}  // namespace kvc
