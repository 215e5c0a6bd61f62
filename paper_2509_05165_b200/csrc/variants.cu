// Kernels of the options beyond the default pipeline: the value norms of the v-norm variant
// (App. A.1.3) and the position order of the kept tokens.
#include "kvc_internal.cuh"

namespace kvc {
namespace {

// One warp per value row: lanes take 16-byte pieces, squares are added in fp32, then over the warp.
template <typename T>
__global__ void __launch_bounds__(256)
value_norm_kernel(LayerPtrs vp, float* __restrict__ vnorm, int L, int Bt, int Hkv, int d, long long N,
                  long long vs0, long long vs1, long long vs2) {
  grid_dependency_wait();
  const int lane = threadIdx.x & 31;
  const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
  const long long rows = (long long)L * Bt * Hkv * N;
  constexpr int kPer16 = 16 / (int)sizeof(T);
  for (long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < rows; r += warps) {
    const long long c = r % N;
    long long t = r / N;
    const int h = (int)(t % Hkv); t /= Hkv;
    const int b = (int)(t % Bt);
    const int l = (int)(t / Bt);
    const T* row = reinterpret_cast<const T*>(vp.p[l]) + b * vs0 + h * vs1 + c * vs2;
    float acc = 0.f;
    for (int piece = lane; piece * kPer16 < d; piece += 32) {
      const uint4 w = __ldg(reinterpret_cast<const uint4*>(row) + piece);
      const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (sizeof(T) == 2) {
          // a bf16 is the upper half of the fp32 with the same value
          const float lo = __uint_as_float(ws[i] << 16), hi = __uint_as_float(ws[i] & 0xffff0000u);
          acc = fmaf(lo, lo, acc);
          acc = fmaf(hi, hi, acc);
        } else {
          const float x = __uint_as_float(ws[i]);
          acc = fmaf(x, x, acc);
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) vnorm[r] = sqrtf(acc);
  }
}

// One CTA per (layer, sequence, head): marks the kept positions in a bitmap (global scratch, one
// bit per token), then writes the marked positions back in ascending order.
constexpr int kOrderThreads = 512;

__global__ void __launch_bounds__(kOrderThreads)
order_kept_kernel(int32_t* __restrict__ idx, const int32_t* __restrict__ n_keep, uint32_t* __restrict__ bitmap,
                  int L, int Bt, int Hkv, long long N, int per_head) {
  __shared__ uint32_t warp_tot[kOrderThreads / 32];
  __shared__ uint32_t carry;
  grid_dependency_wait();
  const long long seg = blockIdx.x;                   // (l * Bt + b) * Hkv + h
  const int h = (int)(seg % Hkv);
  const int b = (int)((seg / Hkv) % Bt);
  const int l = (int)(seg / ((long long)Hkv * Bt));
  const long long n = per_head ? n_keep[((long long)b * L + l) * Hkv + h] : n_keep[(long long)b * L + l];
  int32_t* row = idx + seg * N;
  const long long words = (N + 31) / 32;
  uint32_t* bits = bitmap + seg * words;
  for (long long i = threadIdx.x; i < words; i += kOrderThreads) bits[i] = 0u;
  __syncthreads();
  for (long long k = threadIdx.x; k < n; k += kOrderThreads) {
    const int32_t c = row[k];
    atomicOr(&bits[c >> 5], 1u << (c & 31));
  }
  if (threadIdx.x == 0) carry = 0u;
  __syncthreads();
  // every thread takes one bitmap word per round; exclusive prefix of the popcounts over the CTA
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (long long w0 = 0; w0 < words; w0 += kOrderThreads) {
    const long long wi = w0 + threadIdx.x;
    uint32_t word = wi < words ? bits[wi] : 0u;
    const uint32_t cnt = __popc(word);
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    uint32_t before = carry;
    for (int wv = 0; wv < warp; ++wv) before += warp_tot[wv];
    uint32_t pos = before + incl - cnt;
    while (word) {
      const int bit = __ffs(word) - 1;
      word &= word - 1;
      row[pos++] = (int32_t)(wi * 32 + bit);
    }
    __syncthreads();
    if (threadIdx.x == kOrderThreads - 1) carry = before + incl;
    __syncthreads();
  }
}

// Head-sharded scoring: the local part of Eq. 16's sum over the KV heads, and the mean added back.
__global__ void head_sum_kernel(const float* __restrict__ s, float* __restrict__ head_sum, int Hkv, long long N,
                                long long total) {
  grid_dependency_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const long long lb = i / N, c = i - lb * N;
  const float* base = s + lb * Hkv * N + c;
  float sum = 0.f;
  for (int h = 0; h < Hkv; ++h) sum += base[(long long)h * N];
  head_sum[i] = sum;
}

__global__ void add_head_mean_kernel(float* __restrict__ s, const float* __restrict__ head_sum, int Hkv, float inv_total,
                                     long long N, long long total) {
  grid_dependency_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const long long lb = i / N, c = i - lb * N;
  float* base = s + lb * Hkv * N + c;
  const float mean = head_sum[i] * inv_total;
  for (int h = 0; h < Hkv; ++h) base[(long long)h * N] += mean;
}

__global__ void scale_kernel(float* __restrict__ x, long long n, float f) {
  grid_dependency_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) x[i] *= f;
}

}  // namespace

kvc_status launch_head_sum(const Problem& P, const float* scores, float* head_sum, cudaStream_t st) {
  const long long total = (long long)P.L * P.Bt * P.N;
  KVC_CUDA(launch_dependent(head_sum_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, scores, head_sum,
                            P.Hkv, P.N, total));
  KVC_LAUNCH_CHECK("head_sum_kernel");
  return KVC_OK;
}

kvc_status launch_add_head_mean(const Problem& P, float* scores, const float* head_sum, int heads_total,
                                cudaStream_t st) {
  const long long total = (long long)P.L * P.Bt * P.N;
  KVC_CUDA(launch_dependent(add_head_mean_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, scores,
                            head_sum, P.Hkv, 1.0f / (float)heads_total, P.N, total));
  KVC_LAUNCH_CHECK("add_head_mean_kernel");
  return KVC_OK;
}

kvc_status launch_scale(float* x, long long n, float f, cudaStream_t st) {
  if (n <= 0) return KVC_OK;
  KVC_CUDA(launch_dependent(scale_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, x, n, f));
  KVC_LAUNCH_CHECK("scale_kernel");
  return KVC_OK;
}

kvc_status launch_value_norm(const Problem& P, const LayerPtrs& v, float* vnorm, cudaStream_t st) {
  const long long rows = (long long)P.L * P.Bt * P.Hkv * P.N;
  long long blocks = (rows + 7) / 8;
  int dev = 0, sms = 0;
  KVC_CUDA(cudaGetDevice(&dev));
  KVC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const long long cap = (long long)sms * 32;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  if (P.dtype == KVC_BF16) {
    KVC_CUDA(launch_dependent(value_norm_kernel<__nv_bfloat16>, dim3((unsigned)blocks), dim3(256), 0, st, v, vnorm,
                              P.L, P.Bt, P.Hkv, P.d, P.N, P.kvs[0], P.kvs[1], P.kvs[2]));
  } else {
    KVC_CUDA(launch_dependent(value_norm_kernel<float>, dim3((unsigned)blocks), dim3(256), 0, st, v, vnorm,
                              P.L, P.Bt, P.Hkv, P.d, P.N, P.kvs[0], P.kvs[1], P.kvs[2]));
  }
  KVC_LAUNCH_CHECK("value_norm_kernel");
  return KVC_OK;
}

size_t order_kept_workspace_bytes(const Problem& P) {
  return align_up((size_t)P.L * P.Bt * P.Hkv * (size_t)((P.N + 31) / 32) * sizeof(uint32_t));
}

kvc_status launch_order_kept(const Problem& P, int32_t* idx, const int32_t* n_keep, bool per_head,
                             void* ws, size_t ws_bytes, cudaStream_t st) {
  if (ws_bytes < order_kept_workspace_bytes(P)) {
    set_error("order_kept: workspace too small");
    return KVC_ERR_WORKSPACE;
  }
  const long long segs = (long long)P.L * P.Bt * P.Hkv;
  KVC_CUDA(launch_dependent(order_kept_kernel, dim3((unsigned)segs), dim3(kOrderThreads), 0, st, idx, n_keep,
                            reinterpret_cast<uint32_t*>(ws), P.L, P.Bt, P.Hkv, P.N, per_head ? 1 : 0));
  KVC_LAUNCH_CHECK("order_kept_kernel");
  return KVC_OK;
}

}  // namespace kvc
