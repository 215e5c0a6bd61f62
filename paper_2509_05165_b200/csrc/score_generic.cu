// Token-importance scoring on the CUDA cores (Eqs. 3, 14-16).
//
// This is the shape-agnostic path: fp32 or bf16 inputs, head_dim 64 or 128, any window length,
// any GQA map.  It makes two sweeps over K.  Sweep 1 produces, for every query row, the
// log-sum-exp of its logits over the visible keys (per-chunk partials, then a combine kernel).
// Sweep 2 recomputes the logits and emits exp(s - lse) -- the softmax weight of Eq. 3 -- reduced
// over the window rows (Eq. 14) and over the query heads of the KV head (Eq. 15).  A last kernel
// adds the mean over KV heads (Eq. 16).  Logits are kept in the log2 domain so that every
// exponential is a single ex2.
#include <math.h>

#include "kvc_internal.cuh"

namespace kvc {
namespace {

constexpr int kThreads = 128;     // one token per thread
constexpr int kRowTile = 32;      // query rows staged in shared memory at a time
constexpr int kChunkIters = 8;    // sweep-1 chunk = kChunkIters * kThreads tokens
constexpr float kLog2e = 1.4426950408889634f;

struct ScoreParams {
  int L, Bt, Hq, Hkv, w;
  long long N, q_pos0;
  long long qs0, qs1, qs2, kvs0, kvs1, kvs2;
  float scale_log2e;
  int agg_task, agg_group;
  int nchunks;
};

struct KvOfQ {
  int16_t kv[kMaxQHeads];
};

template <typename T>
__device__ inline void load_row(const T* __restrict__ src, float* dst, int D);

template <>
__device__ inline void load_row<float>(const float* __restrict__ src, float* dst, int D) {
  const float4* s4 = reinterpret_cast<const float4*>(src);
#pragma unroll
  for (int i = 0; i < 64; ++i) {
    if (i * 4 < D) {
      float4 v = __ldg(s4 + i);
      dst[i * 4 + 0] = v.x; dst[i * 4 + 1] = v.y; dst[i * 4 + 2] = v.z; dst[i * 4 + 3] = v.w;
    }
  }
}

template <>
__device__ inline void load_row<__nv_bfloat16>(const __nv_bfloat16* __restrict__ src, float* dst, int D) {
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    if (i * 8 < D) {
      uint4 v = __ldg(s4 + i);
      uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        dst[i * 8 + 2 * e + 0] = __uint_as_float(u[e] << 16);          // bf16 -> fp32 is exact
        dst[i * 8 + 2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u);
      }
    }
  }
}

__device__ inline float to_float(float x) { return x; }
__device__ inline float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// Stage rows [r0, r0 + rt) of one query head into shared memory as fp32.
template <typename T, int D>
__device__ inline void stage_q(const T* __restrict__ qhead, long long row_stride, int r0, int rt,
                               float* Qs) {
  for (int i = threadIdx.x; i < rt * D; i += kThreads) {
    int r = i / D, t = i - r * D;
    Qs[i] = to_float(qhead[(long long)(r0 + r) * row_stride + t]);
  }
}

template <int D>
__device__ inline float dot_row(const float* __restrict__ Qrow, const float* kr) {
  const float4* q4 = reinterpret_cast<const float4*>(Qrow);
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
  for (int i = 0; i < D / 4; ++i) {
    float4 qv = q4[i];  // same address for the whole warp: a broadcast
    a0 = fmaf(qv.x, kr[4 * i + 0], a0);
    a1 = fmaf(qv.y, kr[4 * i + 1], a1);
    a2 = fmaf(qv.z, kr[4 * i + 2], a2);
    a3 = fmaf(qv.w, kr[4 * i + 3], a3);
  }
  return (a0 + a1) + (a2 + a3);
}

__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sweep 1: per (layer, sequence, query head, token chunk) the running (max, sum-exp) of every
// window row over the chunk's visible keys, in the log2 domain.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
score_stats_kernel(ScoreParams P, KvOfQ map, LayerPtrs qp, LayerPtrs kp, float2* __restrict__ partial) {
  __shared__ __align__(16) float Qs[kRowTile * D];
  __shared__ float sm_m[kRowTile][kThreads / 32];
  __shared__ float sm_l[kRowTile][kThreads / 32];

  const int chunk = blockIdx.x, j = blockIdx.y, lb = blockIdx.z;
  const int l = lb / P.Bt, b = lb - l * P.Bt;
  const int h = map.kv[j];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const T* kbase = reinterpret_cast<const T*>(kp.p[l]) + b * P.kvs0 + h * P.kvs1;
  const T* qbase = reinterpret_cast<const T*>(qp.p[l]) + b * P.qs0 + j * P.qs1;
  const long long c_begin = (long long)chunk * (kChunkIters * kThreads);

  for (int r0 = 0; r0 < P.w; r0 += kRowTile) {
    const int rt = min(kRowTile, P.w - r0);
    __syncthreads();
    stage_q<T, D>(qbase, P.qs2, r0, rt, Qs);
    for (int i = threadIdx.x; i < kRowTile * (kThreads / 32); i += kThreads) {
      (&sm_m[0][0])[i] = -INFINITY;
      (&sm_l[0][0])[i] = 0.f;
    }
    __syncthreads();
    for (int it = 0; it < kChunkIters; ++it) {
      const long long c = c_begin + (long long)it * kThreads + threadIdx.x;
      if (c_begin + (long long)it * kThreads >= P.N) break;  // uniform for the block
      const bool valid = c < P.N;
      float kr[D];
      if (valid) {
        load_row<T>(kbase + c * P.kvs2, kr, D);
      } else {
#pragma unroll
        for (int i = 0; i < D; ++i) kr[i] = 0.f;
      }
      for (int r = 0; r < rt; ++r) {
        float s = dot_row<D>(Qs + r * D, kr) * P.scale_log2e;
        const bool vis = valid && (c <= P.q_pos0 + r0 + r);
        s = vis ? s : -INFINITY;
        const float m_w = warp_max(s);
        const float m_old = sm_m[r][warp];
        const float m_new = fmaxf(m_old, m_w);
        const float e = (m_new == -INFINITY) ? 0.f : exp2f(s - m_new);
        const float l_w = warp_sum(e);
        __syncwarp();
        if (lane == 0 && m_new > -INFINITY) {
          sm_l[r][warp] = sm_l[r][warp] * exp2f(m_old - m_new) + l_w;
          sm_m[r][warp] = m_new;
        }
        __syncwarp();
      }
    }
    __syncthreads();
    if (threadIdx.x < rt) {
      const int r = threadIdx.x;
      float M = -INFINITY;
#pragma unroll
      for (int wv = 0; wv < kThreads / 32; ++wv) M = fmaxf(M, sm_m[r][wv]);
      float Lsum = 0.f;
      if (M > -INFINITY) {
#pragma unroll
        for (int wv = 0; wv < kThreads / 32; ++wv) Lsum += sm_l[r][wv] * exp2f(sm_m[r][wv] - M);
      }
      const long long row = ((long long)lb * P.Hq + j) * P.w + r0 + r;
      partial[row * P.nchunks + chunk] = make_float2(M, Lsum);
    }
  }
}

// Combine the chunk partials of one query row into lse2 = log2(sum_c 2^{s2_c}).
__global__ void score_lse_kernel(const float2* __restrict__ partial, float* __restrict__ lse2,
                                 long long rows, int nchunks) {
  const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  const float2* p = partial + row * nchunks;
  float M = -INFINITY;
  for (int i = 0; i < nchunks; ++i) M = fmaxf(M, p[i].x);
  float Lsum = 0.f;
  for (int i = 0; i < nchunks; ++i)
    if (p[i].x > -INFINITY) Lsum += p[i].y * exp2f(p[i].x - M);
  lse2[row] = M + log2f(Lsum);
}

// Sweep 2: S_group[l, b, h, c] (Eqs. 14-15) from the logits and the rows' log-sum-exp.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
score_emit_kernel(ScoreParams P, GroupMap gm, LayerPtrs qp, LayerPtrs kp,
                  const float* __restrict__ lse2, float* __restrict__ s_group) {
  __shared__ __align__(16) float Qs[kRowTile * D];
  __shared__ float Ls[kRowTile];

  const int h = blockIdx.y, lb = blockIdx.z;
  const int l = lb / P.Bt, b = lb - l * P.Bt;
  const long long c = (long long)blockIdx.x * kThreads + threadIdx.x;
  const bool valid = c < P.N;
  const T* kbase = reinterpret_cast<const T*>(kp.p[l]) + b * P.kvs0 + h * P.kvs1;

  float kr[D];
  if (valid) {
    load_row<T>(kbase + c * P.kvs2, kr, D);
  } else {
#pragma unroll
    for (int i = 0; i < D; ++i) kr[i] = 0.f;
  }

  const int members = gm.begin[h + 1] - gm.begin[h];
  float gacc = (P.agg_group == KVC_AGG_MAX) ? -INFINITY : 0.f;
  for (int mi = 0; mi < members; ++mi) {
    const int j = gm.qh[gm.begin[h] + mi];
    const T* qbase = reinterpret_cast<const T*>(qp.p[l]) + b * P.qs0 + j * P.qs1;
    const float* lrow = lse2 + ((long long)lb * P.Hq + j) * P.w;
    float tacc = (P.agg_task == KVC_AGG_MAX) ? -INFINITY : 0.f;
    for (int r0 = 0; r0 < P.w; r0 += kRowTile) {
      const int rt = min(kRowTile, P.w - r0);
      __syncthreads();
      stage_q<T, D>(qbase, P.qs2, r0, rt, Qs);
      if (threadIdx.x < rt) Ls[threadIdx.x] = lrow[r0 + threadIdx.x];
      __syncthreads();
      for (int r = 0; r < rt; ++r) {
        const float s = dot_row<D>(Qs + r * D, kr) * P.scale_log2e;
        const bool vis = valid && (c <= P.q_pos0 + r0 + r);
        const float t = vis ? s - Ls[r] : -INFINITY;     // log2 of the attention weight
        if (P.agg_task == KVC_AGG_MAX) tacc = fmaxf(tacc, t);
        else tacc += exp2f(t);
      }
    }
    const float s_task = (P.agg_task == KVC_AGG_MAX) ? exp2f(tacc) : tacc / (float)P.w;
    if (P.agg_group == KVC_AGG_MAX) gacc = fmaxf(gacc, s_task);
    else gacc += s_task;
  }
  if (P.agg_group == KVC_AGG_MEAN) gacc /= (float)members;
  if (valid) s_group[((long long)lb * P.Hkv + h) * P.N + c] = gacc;
}

// Eq. 16: S[h, c] = S_group[h, c] + (1/Hkv) sum_i S_group[i, c], in place.  With row tiles, first
// Eq. 15 from the tiles' partial aggregates (sum or max over the tile's query heads), in tile order.
// With vnorm (App. A.1.3), the group aggregate is multiplied by the token's value norm before Eq. 16.
// With tiles_per_head > 1 (windows longer than 128 rows) a row tile holds one query head's partial
// Eq. 14 -- the maximum or the sum of the attention weights over the tile's rows -- and Eq. 14 is
// completed over the head's tiles (the sum divided by w) before Eq. 15, heads in ascending order.
__global__ void score_augment_kernel(float* __restrict__ s, const float* __restrict__ parts, int row_tiles,
                                     int tiles_per_head, int agg_task, int w, const float* __restrict__ vnorm, int G,
                                     int agg_group, int augment, int Hkv, long long N, long long total) {
  grid_dependency_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const long long lb = i / N, c = i - lb * N;
  float* base = s + lb * Hkv * N + c;
  if (row_tiles > 1 || vnorm != nullptr) {
    const long long tile_stride = (total / N) * Hkv * N;          // one [L*Bt*Hkv][N] block per row tile
    const float* pbase = parts + lb * Hkv * N + c;
    for (int h = 0; h < Hkv; ++h) {
      float acc;
      if (row_tiles > 1 && tiles_per_head > 1) {
        acc = (agg_group == KVC_AGG_MAX) ? -INFINITY : 0.f;
        for (int j = 0; j < row_tiles / tiles_per_head; ++j) {       // the query heads of the group
          float ht = pbase[(long long)(j * tiles_per_head) * tile_stride + (long long)h * N];
          for (int t = 1; t < tiles_per_head; ++t) {
            const float v = pbase[(long long)(j * tiles_per_head + t) * tile_stride + (long long)h * N];
            ht = (agg_task == KVC_AGG_MAX) ? fmaxf(ht, v) : ht + v;
          }
          if (agg_task == KVC_AGG_MEAN) ht = ht / (float)w;
          acc = (agg_group == KVC_AGG_MAX) ? fmaxf(acc, ht) : acc + ht;
        }
        if (agg_group == KVC_AGG_MEAN) acc = acc / (float)G;
      } else if (row_tiles > 1) {
        acc = pbase[(long long)h * N];
        for (int t = 1; t < row_tiles; ++t) {
          const float v = pbase[(long long)t * tile_stride + (long long)h * N];
          acc = (agg_group == KVC_AGG_MAX) ? fmaxf(acc, v) : acc + v;
        }
        if (agg_group == KVC_AGG_MEAN) acc = acc / (float)G;
      } else {
        acc = base[(long long)h * N];
      }
      if (vnorm != nullptr) acc *= vnorm[lb * Hkv * N + (long long)h * N + c];
      base[(long long)h * N] = acc;
    }
  }
  if (!augment) return;
  if (Hkv <= 8) {
    // all heads' values at once: the thread waits for memory once (added in ascending head order all the same)
    float v[8];
#pragma unroll
    for (int h = 0; h < 8; ++h) v[h] = h < Hkv ? base[(long long)h * N] : 0.f;
    float sum = 0.f;
#pragma unroll
    for (int h = 0; h < 8; ++h) if (h < Hkv) sum += v[h];
    const float mean = sum / (float)Hkv;
#pragma unroll
    for (int h = 0; h < 8; ++h) if (h < Hkv) base[(long long)h * N] = v[h] + mean;
    return;
  }
  float sum = 0.f;
  for (int h = 0; h < Hkv; ++h) sum += base[(long long)h * N];
  const float mean = sum / (float)Hkv;
  for (int h = 0; h < Hkv; ++h) base[(long long)h * N] += mean;
}

template <typename T, int D>
kvc_status run(const Problem& P, const GroupMap& gm, const LayerPtrs& q, const LayerPtrs& k,
               float* scores, float2* partial, float* lse2, int nchunks, cudaStream_t st) {
  ScoreParams sp;
  sp.L = P.L; sp.Bt = P.Bt; sp.Hq = P.Hq; sp.Hkv = P.Hkv; sp.w = P.w;
  sp.N = P.N; sp.q_pos0 = P.q_pos0;
  sp.qs0 = P.qs[0]; sp.qs1 = P.qs[1]; sp.qs2 = P.qs[2];
  sp.kvs0 = P.kvs[0]; sp.kvs1 = P.kvs[1]; sp.kvs2 = P.kvs[2];
  sp.scale_log2e = P.scale * kLog2e;
  sp.agg_task = P.agg_task; sp.agg_group = P.agg_group;
  sp.nchunks = nchunks;
  KvOfQ map;
  for (int h = 0; h < P.Hkv; ++h)
    for (int i = gm.begin[h]; i < gm.begin[h + 1]; ++i) map.kv[gm.qh[i]] = (int16_t)h;

  const long long rows = (long long)P.L * P.Bt * P.Hq * P.w;
  score_stats_kernel<T, D><<<dim3(nchunks, P.Hq, P.L * P.Bt), kThreads, 0, st>>>(sp, map, q, k, partial);
  KVC_LAUNCH_CHECK("score_stats_kernel");
  score_lse_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(partial, lse2, rows, nchunks);
  KVC_LAUNCH_CHECK("score_lse_kernel");
  score_emit_kernel<T, D><<<dim3((unsigned)((P.N + kThreads - 1) / kThreads), P.Hkv, P.L * P.Bt),
                            kThreads, 0, st>>>(sp, gm, q, k, lse2, scores);
  KVC_LAUNCH_CHECK("score_emit_kernel");
  return KVC_OK;
}

}  // namespace

static int generic_nchunks(const Problem& P) {
  const long long per = (long long)kChunkIters * kThreads;
  return (int)((P.N + per - 1) / per);
}

size_t score_generic_workspace_bytes(const Problem& P) {
  const size_t rows = (size_t)P.L * P.Bt * P.Hq * P.w;
  return align_up(rows * generic_nchunks(P) * sizeof(float2)) + align_up(rows * sizeof(float));
}

kvc_status launch_score_augment(const Problem& P, float* scores, const float* parts, int row_tiles,
                                int tiles_per_head, const float* vnorm, cudaStream_t st) {
  if (!P.augment && row_tiles <= 1 && vnorm == nullptr) return KVC_OK;
  const long long total = (long long)P.L * P.Bt * P.N;
  KVC_CUDA(launch_dependent(score_augment_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st,
                            scores, parts, row_tiles, tiles_per_head, P.agg_task, P.w, vnorm, P.max_group, P.agg_group,
                            P.augment, P.Hkv, P.N, total));
  KVC_LAUNCH_CHECK("score_augment_kernel");
  return KVC_OK;
}

kvc_status launch_score_generic(const Problem& P, const GroupMap& gm, const LayerPtrs& q,
                                const LayerPtrs& k, float* scores, const float* vnorm, void* ws,
                                size_t ws_bytes, cudaStream_t st) {
  if (ws_bytes < score_generic_workspace_bytes(P)) {
    set_error("score: workspace too small");
    return KVC_ERR_WORKSPACE;
  }
  const size_t rows = (size_t)P.L * P.Bt * P.Hq * P.w;
  const int nchunks = generic_nchunks(P);
  float2* partial = reinterpret_cast<float2*>(ws);
  float* lse2 = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) +
                                         align_up(rows * nchunks * sizeof(float2)));
  kvc_status s;
  if (P.dtype == KVC_BF16) {
    if (P.d == 64) s = run<__nv_bfloat16, 64>(P, gm, q, k, scores, partial, lse2, nchunks, st);
    else s = run<__nv_bfloat16, 128>(P, gm, q, k, scores, partial, lse2, nchunks, st);
  } else {
    if (P.d == 64) s = run<float, 64>(P, gm, q, k, scores, partial, lse2, nchunks, st);
    else s = run<float, 128>(P, gm, q, k, scores, partial, lse2, nchunks, st);
  }
  if (s != KVC_OK) return s;
  return launch_score_augment(P, scores, nullptr, 1, 1, vnorm, st);
}

}  // namespace kvc
