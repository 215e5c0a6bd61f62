// Internal declarations shared by the kvc translation units (not part of the public ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvc.h"

namespace kvc {

constexpr int kMaxQHeads = 256;
constexpr int kMaxKvHeads = 128;

// Resolved problem: the public descriptor with defaults filled in and the GQA map expanded.
struct Problem {
  int L, Bt, Hq, Hkv, d, w;
  long long N, q_pos0;
  int dtype;  // kvc_dtype
  float scale;
  int agg_task, agg_group, agg_head, augment;
  long long qs[3], kvs[3];        // element strides (batch, head, row/token)
  int elem_bytes;                 // 2 or 4
  int max_group;                  // largest number of query heads sharing one KV head
  bool contiguous_groups;         // q_to_kv[j] == j / G
  int value_norm, min_keep, keep_position_order;   // the options of kvc_desc
};

constexpr int kMaxSelectRows = 2048;   // rows (layers, or layer-head pairs) of one sequence's selection pool

// Query heads grouped by KV head: members of KV head h are qh[begin[h] .. begin[h+1]).
struct GroupMap {
  int16_t begin[kMaxKvHeads + 1];
  int16_t qh[kMaxQHeads];
};

// Per-layer device pointers, passed by value to kernels.
struct LayerPtrs {
  const void* p[KVC_MAX_LAYERS];
};

void set_error(const char* fmt, ...);
kvc_status check_cuda(cudaError_t e, const char* what);
void count_launch(int n = 1);

#define KVC_CUDA(call)                                        \
  do {                                                        \
    kvc_status _s = ::kvc::check_cuda((call), #call);         \
    if (_s != KVC_OK) return _s;                              \
  } while (0)

#define KVC_LAUNCH_CHECK(name)                                \
  do {                                                        \
    ::kvc::count_launch();                                    \
    kvc_status _s = ::kvc::check_cuda(cudaGetLastError(), name); \
    if (_s != KVC_OK) return _s;                              \
  } while (0)

// Programmatic dependent launch: the kernel may be scheduled while the kernel before it in the
// stream is still draining, which hides its launch latency.  Every kernel launched this way
// calls grid_dependency_wait() before it touches global memory: the call returns once the
// preceding kernel has completed and its writes are visible (and so, transitively, all earlier
// work in the stream).
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args) {
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// Host-side validation shared by the entry points that live outside kvc_api.cu.
kvc_status resolve_desc(const kvc_desc* d, Problem* P);
kvc_status require_budget(const Problem& P, long long budget);
kvc_status require_device();

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// ---- score ------------------------------------------------------------------------------------
// Scratch bytes the scoring step needs.
size_t score_workspace_bytes(const Problem& P);
// Eqs. 3, 14-16: writes scores [L, Bt, Hkv, N].
// vnorm: nullptr, or ||v|| per (layer, sequence, KV head, token), laid out like scores (App. A.1.3).
kvc_status launch_score(const Problem& P, const GroupMap& gm, const LayerPtrs& q, const LayerPtrs& k,
                        float* scores, const float* vnorm, int* device_status, void* ws, size_t ws_bytes,
                        cudaStream_t st);
// The two implementations behind it: CUDA cores (any supported shape) and tcgen05 (bf16,
// contiguous GQA groups, window of at most 128 rows).
size_t score_generic_workspace_bytes(const Problem& P);
kvc_status launch_score_generic(const Problem& P, const GroupMap& gm, const LayerPtrs& q,
                                const LayerPtrs& k, float* scores, const float* vnorm, void* ws,
                                size_t ws_bytes, cudaStream_t st);
// Eq. 16 in place; before it, with `row_tiles` > 1, the group aggregate (Eq. 15) of every KV head
// from its row tiles' partial aggregates `parts` [row_tiles][L*Bt*Hkv][N], in tile order.
// With vnorm, the group aggregate is multiplied by the token's value norm before Eq. 16.  With
// tiles_per_head > 1 (windows longer than 128 rows) every row tile holds a query head's partial
// Eq. 14, and Eq. 14 is completed over a head's tiles before Eq. 15.
kvc_status launch_score_augment(const Problem& P, float* scores, const float* parts, int row_tiles,
                                int tiles_per_head, const float* vnorm, cudaStream_t st);
bool score_sm100_shape_ok(const Problem& P);
bool score_sm100_supported(const Problem& P);
size_t score_sm100_workspace_bytes(const Problem& P);
kvc_status launch_score_sm100(const Problem& P, const LayerPtrs& q, const LayerPtrs& k, float* scores,
                              int* device_status, void* ws, size_t ws_bytes, cudaStream_t st,
                              const float** parts_out, int* row_tiles_out, int* tiles_per_head_out);

// ---- rank + compose ---------------------------------------------------------------------------
size_t compose_workspace_bytes(const Problem& P);
// Eqs. 17-19: idx [L, Bt, Hkv, N], composite [L, Bt, N].
kvc_status launch_compose(const Problem& P, const float* scores, int32_t* idx, float* composite,
                          void* ws, size_t ws_bytes, cudaStream_t st);

// Eq. 18 as fp32: the sorted scores of every head, from the keys the ranking leaves in the workspace
// of launch_compose (which must have run on the same workspace).
kvc_status launch_sorted_scores(const Problem& P, const void* ws, float* sorted, cudaStream_t st);

// ---- allocate ---------------------------------------------------------------------------------
size_t allocate_workspace_bytes(const Problem& P);
// Eqs. 20-22: n_keep [Bt, L], offsets [Bt, L + 1], with the per-layer minimum `min_keep`.
// heads_per_row = 1: the pool's rows are the layers, composite [L, Bt, N].  heads_per_row = Hkv (the
// unstructured variant, App. A.2): the rows are the (layer, head) pairs, composite = the heads'
// sorted scores [L, Bt, Hkv, N], n_keep [Bt, L * Hkv], offsets [Bt, L * Hkv + 1].
// How the budget's threshold is found: on the sorted rows by one CTA per sequence (pools of up to 128
// rows; uses no workspace), or by the histogram passes of a radix select over the workspace.
enum class SelectPath { kAuto, kHistograms, kSortedRows };
kvc_status launch_allocate(const Problem& P, const float* composite, long long budget, int heads_per_row,
                           long long min_keep, int32_t* n_keep, long long* offsets, void* ws,
                           size_t ws_bytes, cudaStream_t st, SelectPath path = SelectPath::kAuto);
// Test hooks: path 0 = automatic, 1 = histograms, 2 = sorted rows where they apply; max_rounds < 0 = default.
void set_select_hooks(int path, int max_rounds);

// ---- gather -----------------------------------------------------------------------------------
// Eqs. 23-24.
// per_head: n_keep / offsets are per (layer, head) and `budget` counts entries (App. A.2).
kvc_status launch_gather(const Problem& P, const LayerPtrs& k, const LayerPtrs& v, const int32_t* idx,
                         const int32_t* n_keep, const long long* offsets, long long budget, bool per_head,
                         void* k_out, void* v_out, cudaStream_t st);

// ---- variants ---------------------------------------------------------------------------------
// ||v||_2 of every value row in fp32: vnorm [L, Bt, Hkv, N] (App. A.1.3).
kvc_status launch_value_norm(const Problem& P, const LayerPtrs& v, float* vnorm, cudaStream_t st);
// Head-sharded scoring (see kvc.h).
kvc_status launch_head_sum(const Problem& P, const float* scores, float* head_sum, cudaStream_t st);
kvc_status launch_add_head_mean(const Problem& P, float* scores, const float* head_sum, int heads_total, cudaStream_t st);
kvc_status launch_scale(float* x, long long n, float f, cudaStream_t st);
// The first n_keep entries of every idx row in ascending position, in place.  n_keep per layer
// [Bt, L] or, per_head, per (layer, head) [Bt, L * Hkv].
size_t order_kept_workspace_bytes(const Problem& P);
kvc_status launch_order_kept(const Problem& P, int32_t* idx, const int32_t* n_keep, bool per_head,
                             void* ws, size_t ws_bytes, cudaStream_t st);

// Order-preserving map from an fp32 score to an unsigned key whose ASCENDING order is the
// score's DESCENDING order; -0 is folded onto +0 so that equal scores get equal keys.
__host__ __device__ inline uint32_t score_to_key(float s) {
#ifdef __CUDA_ARCH__
  uint32_t b = __float_as_uint(s);
#else
  union { float f; uint32_t u; } cv; cv.f = s; uint32_t b = cv.u;
#endif
  if (b == 0x80000000u) b = 0u;
  uint32_t asc = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return ~asc;
}

__host__ __device__ inline float key_to_score(uint32_t key) {
  uint32_t asc = ~key;
  uint32_t b = (asc & 0x80000000u) ? (asc & 0x7fffffffu) : ~asc;
#ifdef __CUDA_ARCH__
  return __uint_as_float(b);
#else
  union { float f; uint32_t u; } cv; cv.u = b; return cv.f;
#endif
}

}  // namespace kvc
