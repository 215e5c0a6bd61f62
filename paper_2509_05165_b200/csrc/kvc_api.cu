// C-ABI entry points: argument validation, workspace carving and stream-ordered launches.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include "kvc_internal.cuh"

namespace kvc {

static thread_local char g_err[512] = "";
static thread_local long long g_launches = 0;

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

kvc_status check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return KVC_OK;
  set_error("CUDA error in %s: %s", what, cudaGetErrorString(e));
  return KVC_ERR_CUDA;
}

void count_launch(int n) { g_launches += n; }

// Scratch of the scoring kernels; kvc_score keeps its device status word right behind it.
static size_t score_scratch_bytes(const Problem& P) {
  size_t a = score_generic_workspace_bytes(P);
  if (score_sm100_shape_ok(P)) {          // (by the shape alone: the size must not depend on the machine)
    const size_t b = score_sm100_workspace_bytes(P);
    if (b > a) a = b;
  }
  return align_up(a);
}

// [scratch][status word, 256 B][value norms, with the v-norm option]
size_t score_workspace_bytes(const Problem& P) {
  size_t n = score_scratch_bytes(P) + 256;
  if (P.value_norm) n += align_up((size_t)P.L * P.Bt * P.Hkv * P.N * sizeof(float));
  return n;
}

kvc_status launch_score(const Problem& P, const GroupMap& gm, const LayerPtrs& q, const LayerPtrs& k,
                        float* scores, const float* vnorm, int* device_status, void* ws, size_t ws_bytes,
                        cudaStream_t st) {
  if (score_sm100_supported(P)) {
    const float* parts = nullptr;
    int row_tiles = 1, tiles_per_head = 1;
    const kvc_status s = launch_score_sm100(P, q, k, scores, device_status, ws, ws_bytes, st, &parts, &row_tiles,
                                            &tiles_per_head);
    if (s == KVC_OK) return launch_score_augment(P, scores, parts, row_tiles, tiles_per_head, vnorm, st);
    if (s != KVC_ERR_UNSUPPORTED) return s;      // a real failure; UNSUPPORTED = strides TMA cannot take
  }
  return launch_score_generic(P, gm, q, k, scores, vnorm, ws, ws_bytes, st);
}

// Scoring as the entry points run it: status word and value norms carved from the score workspace.
static kvc_status run_score(const Problem& P, const GroupMap& gm, const LayerPtrs& q, const LayerPtrs& k,
                            const LayerPtrs* v, float* scores, int* device_status, void* ws, cudaStream_t st) {
  char* w = reinterpret_cast<char*>(ws);
  const size_t scratch = score_scratch_bytes(P);
  float* vnorm = nullptr;
  if (P.value_norm) {
    vnorm = reinterpret_cast<float*>(w + scratch + 256);
    const kvc_status s = launch_value_norm(P, *v, vnorm, st);
    if (s != KVC_OK) return s;
  }
  return launch_score(P, gm, q, k, scores, vnorm, device_status, ws, scratch, st);
}

namespace {

#define KVC_REQUIRE(cond, code, ...)   \
  do {                                 \
    if (!(cond)) {                     \
      set_error(__VA_ARGS__);          \
      return code;                     \
    }                                  \
  } while (0)

kvc_status resolve(const kvc_desc* d, Problem* P, GroupMap* gm) {
  KVC_REQUIRE(d != nullptr, KVC_ERR_INVALID_ARG, "desc is NULL");
  KVC_REQUIRE(d->n_layers >= 1, KVC_ERR_INVALID_ARG, "n_layers must be >= 1");
  KVC_REQUIRE(d->n_layers <= KVC_MAX_LAYERS, KVC_ERR_UNSUPPORTED, "n_layers > %d", KVC_MAX_LAYERS);
  KVC_REQUIRE(d->batch >= 1, KVC_ERR_INVALID_ARG, "batch must be >= 1");
  KVC_REQUIRE((long long)d->n_layers * d->batch <= 65535, KVC_ERR_UNSUPPORTED, "n_layers * batch > 65535");
  KVC_REQUIRE(d->n_q_heads >= 1 && d->n_kv_heads >= 1, KVC_ERR_INVALID_ARG, "head counts must be >= 1");
  KVC_REQUIRE(d->n_q_heads <= kMaxQHeads && d->n_kv_heads <= kMaxKvHeads, KVC_ERR_UNSUPPORTED,
              "more than %d query heads or %d KV heads", kMaxQHeads, kMaxKvHeads);
  KVC_REQUIRE(d->head_dim == 64 || d->head_dim == 128, KVC_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  KVC_REQUIRE(d->window >= 1, KVC_ERR_INVALID_ARG, "window must be >= 1");
  KVC_REQUIRE(d->window <= 65536, KVC_ERR_UNSUPPORTED, "window > 65536");
  KVC_REQUIRE(d->n_ctx >= 1, KVC_ERR_INVALID_ARG, "n_ctx must be >= 1");
  KVC_REQUIRE(d->n_ctx < (1LL << 31), KVC_ERR_UNSUPPORTED, "n_ctx must be < 2^31");
  KVC_REQUIRE(d->q_pos0 >= 0, KVC_ERR_INVALID_ARG, "q_pos0 must be >= 0");
  KVC_REQUIRE(d->dtype == KVC_F32 || d->dtype == KVC_BF16, KVC_ERR_INVALID_ARG, "unknown dtype");
  KVC_REQUIRE(d->agg_task == KVC_AGG_MAX || d->agg_task == KVC_AGG_MEAN, KVC_ERR_INVALID_ARG, "bad agg_task");
  KVC_REQUIRE(d->agg_group == KVC_AGG_MAX || d->agg_group == KVC_AGG_MEAN, KVC_ERR_INVALID_ARG, "bad agg_group");
  KVC_REQUIRE(d->agg_head == KVC_AGG_MAX || d->agg_head == KVC_AGG_MEAN, KVC_ERR_INVALID_ARG, "bad agg_head");
  KVC_REQUIRE(!(d->scale != d->scale) && !isinf(d->scale), KVC_ERR_INVALID_ARG, "scale is not finite");
  KVC_REQUIRE(d->value_norm == 0 || d->value_norm == 1, KVC_ERR_INVALID_ARG, "value_norm must be 0 or 1");
  KVC_REQUIRE(d->keep_position_order == 0 || d->keep_position_order == 1, KVC_ERR_INVALID_ARG,
              "keep_position_order must be 0 or 1");
  KVC_REQUIRE(d->min_keep_per_layer >= 0 && d->min_keep_per_layer <= d->n_ctx, KVC_ERR_INVALID_ARG,
              "min_keep_per_layer must lie in [0, n_ctx]");
  KVC_REQUIRE(d->reserved_ == 0, KVC_ERR_INVALID_ARG, "reserved_ must be 0");

  P->L = d->n_layers; P->Bt = d->batch; P->Hq = d->n_q_heads; P->Hkv = d->n_kv_heads;
  P->d = d->head_dim; P->w = d->window; P->N = d->n_ctx; P->q_pos0 = d->q_pos0;
  P->dtype = d->dtype; P->elem_bytes = (d->dtype == KVC_BF16) ? 2 : 4;
  P->scale = (d->scale > 0.f) ? d->scale : 1.0f / sqrtf((float)d->head_dim);
  P->agg_task = d->agg_task; P->agg_group = d->agg_group; P->agg_head = d->agg_head;
  P->augment = d->augment_head_mean ? 1 : 0;
  P->value_norm = d->value_norm; P->min_keep = d->min_keep_per_layer; P->keep_position_order = d->keep_position_order;

  if (d->q_stride[0] == 0) {
    P->qs[2] = P->d; P->qs[1] = (long long)P->w * P->d; P->qs[0] = P->qs[1] * P->Hq;
  } else {
    for (int i = 0; i < 3; ++i) P->qs[i] = d->q_stride[i];
  }
  if (d->kv_stride[0] == 0) {
    P->kvs[2] = P->d; P->kvs[1] = P->N * P->d; P->kvs[0] = P->kvs[1] * P->Hkv;
  } else {
    for (int i = 0; i < 3; ++i) P->kvs[i] = d->kv_stride[i];
  }
  const int per16 = 16 / P->elem_bytes;
  for (int i = 0; i < 3; ++i) {
    KVC_REQUIRE(P->qs[i] >= (i == 2 ? P->d : 0) && P->qs[i] % per16 == 0, KVC_ERR_INVALID_ARG,
                "q_stride[%d] must be a non-negative multiple of 16 bytes (rows >= head_dim apart)", i);
    KVC_REQUIRE(P->kvs[i] >= (i == 2 ? P->d : 0) && P->kvs[i] % per16 == 0, KVC_ERR_INVALID_ARG,
                "kv_stride[%d] must be a non-negative multiple of 16 bytes (rows >= head_dim apart)", i);
  }

  // GQA map (Sec. 3.2.2: the reshape Hq -> Hkv x G before Eq. 15)
  int count[kMaxKvHeads];
  for (int h = 0; h < P->Hkv; ++h) count[h] = 0;
  int kv_of[kMaxQHeads];
  P->contiguous_groups = true;
  if (d->q_to_kv == nullptr) {
    KVC_REQUIRE(P->Hq % P->Hkv == 0, KVC_ERR_INVALID_ARG, "n_q_heads must be a multiple of n_kv_heads");
    const int G = P->Hq / P->Hkv;
    for (int j = 0; j < P->Hq; ++j) kv_of[j] = j / G;
  } else {
    for (int j = 0; j < P->Hq; ++j) {
      kv_of[j] = d->q_to_kv[j];
      KVC_REQUIRE(kv_of[j] >= 0 && kv_of[j] < P->Hkv, KVC_ERR_INVALID_ARG, "q_to_kv[%d] out of range", j);
    }
  }
  for (int j = 0; j < P->Hq; ++j) count[kv_of[j]]++;
  gm->begin[0] = 0;
  P->max_group = 0;
  for (int h = 0; h < P->Hkv; ++h) {
    KVC_REQUIRE(count[h] > 0, KVC_ERR_INVALID_ARG, "KV head %d has no query head", h);
    gm->begin[h + 1] = (int16_t)(gm->begin[h] + count[h]);
    if (count[h] > P->max_group) P->max_group = count[h];
  }
  int fill[kMaxKvHeads];
  for (int h = 0; h < P->Hkv; ++h) fill[h] = gm->begin[h];
  for (int j = 0; j < P->Hq; ++j) gm->qh[fill[kv_of[j]]++] = (int16_t)j;
  if (P->Hq % P->Hkv != 0) P->contiguous_groups = false;
  else {
    const int G = P->Hq / P->Hkv;
    for (int j = 0; j < P->Hq; ++j) if (kv_of[j] != j / G) P->contiguous_groups = false;
  }
  return KVC_OK;
}

kvc_status check_ptrs(const void* const* arr, int L, const char* name, LayerPtrs* out) {
  KVC_REQUIRE(arr != nullptr, KVC_ERR_INVALID_ARG, "%s pointer array is NULL", name);
  for (int l = 0; l < L; ++l) {
    KVC_REQUIRE(arr[l] != nullptr, KVC_ERR_INVALID_ARG, "%s[%d] is NULL", name, l);
    KVC_REQUIRE((reinterpret_cast<uintptr_t>(arr[l]) & 15u) == 0, KVC_ERR_INVALID_ARG,
                "%s[%d] is not 16-byte aligned", name, l);
    out->p[l] = arr[l];
  }
  return KVC_OK;
}

kvc_status check_ws(const void* ws, size_t have, size_t need) {
  if (need == 0) return KVC_OK;
  KVC_REQUIRE(ws != nullptr, KVC_ERR_WORKSPACE, "workspace is NULL (%zu bytes needed)", need);
  KVC_REQUIRE((reinterpret_cast<uintptr_t>(ws) & 255u) == 0, KVC_ERR_WORKSPACE, "workspace is not 256-byte aligned");
  KVC_REQUIRE(have >= need, KVC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", have, need);
  return KVC_OK;
}

kvc_status check_budget(const Problem& P, long long budget) {
  KVC_REQUIRE(budget >= 0 && budget <= (long long)P.L * P.N, KVC_ERR_INVALID_ARG,
              "budget %lld outside [0, L * N = %lld]", budget, (long long)P.L * P.N);
  return KVC_OK;
}

kvc_status check_device() {
  static thread_local int checked_dev = -1;
  int dev = 0;
  KVC_CUDA(cudaGetDevice(&dev));
  if (dev == checked_dev) return KVC_OK;
  int major = 0;
  KVC_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  KVC_REQUIRE(major == 10, KVC_ERR_UNSUPPORTED, "device %d has compute capability %d.x; 10.x (B200) required", dev, major);
  checked_dev = dev;
  return KVC_OK;
}

struct CompressLayout {
  size_t scores, idx, composite, stage, alloc, total;   // byte offsets; stage is shared by score and compose
};

CompressLayout compress_layout(const Problem& P) {
  CompressLayout c;
  const size_t items = (size_t)P.L * P.Bt * P.Hkv * P.N;
  size_t off = 0;
  c.scores = off; off += align_up(items * 4);
  c.idx = off; off += align_up(items * 4);
  c.composite = off; off += align_up((size_t)P.L * P.Bt * P.N * 4);
  c.stage = off;
  // (the bitmap of kvc_order_kept also lives here: the sort buffers are dead by then)
  size_t a = score_workspace_bytes(P);
  const size_t b = compose_workspace_bytes(P), o = order_kept_workspace_bytes(P);
  if (b > a) a = b;
  if (o > a) a = o;
  off += align_up(a);
  c.alloc = off; off += align_up(allocate_workspace_bytes(P));
  c.total = off;
  return c;
}

}  // namespace

kvc_status resolve_desc(const kvc_desc* d, Problem* P) {
  GroupMap gm;
  return resolve(d, P, &gm);
}
kvc_status require_budget(const Problem& P, long long budget) { return check_budget(P, budget); }
kvc_status require_device() { return check_device(); }

}  // namespace kvc

using namespace kvc;

extern "C" {

void kvc_desc_init(kvc_desc* d, int32_t n_layers, int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                   int32_t head_dim, int64_t n_ctx, int32_t window, int32_t dtype) {
  if (!d) return;
  memset(d, 0, sizeof(*d));
  d->n_layers = n_layers; d->batch = batch; d->n_q_heads = n_q_heads; d->n_kv_heads = n_kv_heads;
  d->head_dim = head_dim; d->window = window; d->n_ctx = n_ctx;
  d->q_pos0 = n_ctx - window > 0 ? n_ctx - window : 0;
  d->dtype = dtype; d->scale = 0.f;
  d->agg_task = KVC_AGG_MAX; d->agg_group = KVC_AGG_MEAN; d->agg_head = KVC_AGG_MEAN;
  d->augment_head_mean = 1; d->q_to_kv = nullptr;
}

int64_t kvc_budget_from_ratio(const kvc_desc* d, double r_target) {
  if (!d || d->n_layers < 1 || d->n_ctx < 1 || !(r_target >= 0.0 && r_target <= 1.0)) {
    set_error("kvc_budget_from_ratio: bad descriptor or ratio");
    return -1;
  }
  const double total = (double)d->n_layers * (double)d->n_ctx;
  const double x = (1.0 - r_target) * total;
  double b = floor(x + fabs(x) * 1e-12 + 1e-9);
  if (b < 0) b = 0;
  if (b > total) b = total;
  return (int64_t)b;
}

kvc_status kvc_workspace_size(const kvc_desc* d, int64_t budget, size_t* bytes) {
  Problem P; GroupMap gm;
  kvc_status s = resolve(d, &P, &gm);
  if (s != KVC_OK) return s;
  KVC_REQUIRE(bytes != nullptr, KVC_ERR_INVALID_ARG, "bytes is NULL");
  if ((s = check_budget(P, budget)) != KVC_OK) return s;
  *bytes = compress_layout(P).total;
  return KVC_OK;
}

kvc_status kvc_score(const kvc_desc* d, const void* const* q, const void* const* k, float* scores,
                     void* ws, size_t ws_bytes, void* stream) {
  Problem P; GroupMap gm; LayerPtrs qp, kp;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  if ((s = check_ptrs(q, P.L, "q", &qp)) != KVC_OK) return s;
  if ((s = check_ptrs(k, P.L, "k", &kp)) != KVC_OK) return s;
  KVC_REQUIRE(scores != nullptr, KVC_ERR_INVALID_ARG, "scores is NULL");
  KVC_REQUIRE(!P.value_norm, KVC_ERR_INVALID_ARG, "desc->value_norm is set: kvc_score has no V, use kvc_score_weighted");
  if ((s = check_ws(ws, ws_bytes, score_workspace_bytes(P))) != KVC_OK) return s;
  if ((s = check_device()) != KVC_OK) return s;
  // conditions detected on the device are reported in a word behind the scratch (kvc_score_status_offset)
  int* status = reinterpret_cast<int*>(reinterpret_cast<char*>(ws) + score_scratch_bytes(P));
  KVC_CUDA(cudaMemsetAsync(status, 0, sizeof(int), (cudaStream_t)stream));
  return run_score(P, gm, qp, kp, nullptr, scores, status, ws, (cudaStream_t)stream);
}

kvc_status kvc_score_weighted(const kvc_desc* d, const void* const* q, const void* const* k,
                              const void* const* v, float* scores, void* ws, size_t ws_bytes, void* stream) {
  Problem P; GroupMap gm; LayerPtrs qp, kp, vp;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  P.value_norm = 1;                               // (the descriptor's flag is ignored here)
  if ((s = check_ptrs(q, P.L, "q", &qp)) != KVC_OK) return s;
  if ((s = check_ptrs(k, P.L, "k", &kp)) != KVC_OK) return s;
  if ((s = check_ptrs(v, P.L, "v", &vp)) != KVC_OK) return s;
  KVC_REQUIRE(scores != nullptr, KVC_ERR_INVALID_ARG, "scores is NULL");
  if ((s = check_ws(ws, ws_bytes, score_workspace_bytes(P))) != KVC_OK) return s;
  if ((s = check_device()) != KVC_OK) return s;
  int* status = reinterpret_cast<int*>(reinterpret_cast<char*>(ws) + score_scratch_bytes(P));
  KVC_CUDA(cudaMemsetAsync(status, 0, sizeof(int), (cudaStream_t)stream));
  return run_score(P, gm, qp, kp, &vp, scores, status, ws, (cudaStream_t)stream);
}

int32_t kvc_score_uses_tensor_cores(const kvc_desc* d) {
  Problem P; GroupMap gm;
  const kvc_status s = resolve(d, &P, &gm);
  if (s != KVC_OK) return (int32_t)s;
  return score_sm100_shape_ok(P) ? 1 : 0;
}

kvc_status kvc_score_status_offset(const kvc_desc* d, size_t* offset) {
  Problem P; GroupMap gm;
  const kvc_status s = resolve(d, &P, &gm);
  if (s != KVC_OK) return s;
  KVC_REQUIRE(offset != nullptr, KVC_ERR_INVALID_ARG, "offset is NULL");
  *offset = score_scratch_bytes(P);
  return KVC_OK;
}

kvc_status kvc_compose(const kvc_desc* d, const float* scores, int32_t* idx, float* composite,
                       void* ws, size_t ws_bytes, void* stream) {
  Problem P; GroupMap gm;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  KVC_REQUIRE(scores && idx && composite, KVC_ERR_INVALID_ARG, "scores, idx or composite is NULL");
  if ((s = check_ws(ws, ws_bytes, compose_workspace_bytes(P))) != KVC_OK) return s;
  if ((s = check_device()) != KVC_OK) return s;
  return launch_compose(P, scores, idx, composite, ws, ws_bytes, (cudaStream_t)stream);
}

kvc_status kvc_allocate(const kvc_desc* d, const float* composite, int64_t budget, int32_t* n_keep,
                        int64_t* offsets, void* ws, size_t ws_bytes, void* stream) {
  Problem P; GroupMap gm;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  KVC_REQUIRE(composite && n_keep && offsets, KVC_ERR_INVALID_ARG, "composite, n_keep or offsets is NULL");
  if ((s = check_budget(P, budget)) != KVC_OK) return s;
  if ((s = check_ws(ws, ws_bytes, allocate_workspace_bytes(P))) != KVC_OK) return s;
  if ((s = check_device()) != KVC_OK) return s;
  return launch_allocate(P, composite, budget, 1, P.min_keep, n_keep, reinterpret_cast<long long*>(offsets), ws,
                         ws_bytes, (cudaStream_t)stream);
}

kvc_status kvc_order_kept(const kvc_desc* d, int32_t* idx, const int32_t* n_keep, void* ws, size_t ws_bytes,
                          void* stream) {
  Problem P; GroupMap gm;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  KVC_REQUIRE(idx && n_keep, KVC_ERR_INVALID_ARG, "idx or n_keep is NULL");
  if ((s = check_ws(ws, ws_bytes, order_kept_workspace_bytes(P))) != KVC_OK) return s;
  if ((s = check_device()) != KVC_OK) return s;
  return launch_order_kept(P, idx, n_keep, false, ws, ws_bytes, (cudaStream_t)stream);
}

kvc_status kvc_gather(const kvc_desc* d, const void* const* k, const void* const* v, const int32_t* idx,
                      const int32_t* n_keep, const int64_t* offsets, int64_t budget, void* k_out,
                      void* v_out, void* stream) {
  Problem P; GroupMap gm; LayerPtrs kp, vp;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  if ((s = check_ptrs(k, P.L, "k", &kp)) != KVC_OK) return s;
  if ((s = check_ptrs(v, P.L, "v", &vp)) != KVC_OK) return s;
  KVC_REQUIRE(idx && n_keep && offsets, KVC_ERR_INVALID_ARG, "idx, n_keep or offsets is NULL");
  if ((s = check_budget(P, budget)) != KVC_OK) return s;
  if (budget > 0) {
    KVC_REQUIRE(k_out && v_out, KVC_ERR_INVALID_ARG, "k_out or v_out is NULL");
    KVC_REQUIRE(((reinterpret_cast<uintptr_t>(k_out) | reinterpret_cast<uintptr_t>(v_out)) & 15u) == 0,
                KVC_ERR_INVALID_ARG, "k_out / v_out must be 16-byte aligned");
  }
  if ((s = check_device()) != KVC_OK) return s;
  return launch_gather(P, kp, vp, idx, n_keep, reinterpret_cast<const long long*>(offsets), budget, false,
                       k_out, v_out, (cudaStream_t)stream);
}

kvc_status kvc_compress(const kvc_desc* d, const void* const* q, const void* const* k,
                        const void* const* v, int64_t budget, void* k_out, void* v_out,
                        int32_t* n_keep, int64_t* offsets, int32_t* idx_out, float* scores_out,
                        float* composite_out, int32_t* device_status, void* ws, size_t ws_bytes,
                        void* stream) {
  Problem P; GroupMap gm; LayerPtrs qp, kp, vp;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  if ((s = check_ptrs(q, P.L, "q", &qp)) != KVC_OK) return s;
  if ((s = check_ptrs(k, P.L, "k", &kp)) != KVC_OK) return s;
  if ((s = check_ptrs(v, P.L, "v", &vp)) != KVC_OK) return s;
  KVC_REQUIRE(n_keep && offsets, KVC_ERR_INVALID_ARG, "n_keep or offsets is NULL");
  if ((s = check_budget(P, budget)) != KVC_OK) return s;
  if (budget > 0) {
    KVC_REQUIRE(k_out && v_out, KVC_ERR_INVALID_ARG, "k_out or v_out is NULL");
    KVC_REQUIRE(((reinterpret_cast<uintptr_t>(k_out) | reinterpret_cast<uintptr_t>(v_out)) & 15u) == 0,
                KVC_ERR_INVALID_ARG, "k_out / v_out must be 16-byte aligned");
  }
  const CompressLayout lay = compress_layout(P);
  if ((s = check_ws(ws, ws_bytes, lay.total)) != KVC_OK) return s;
  if ((s = check_device()) != KVC_OK) return s;

  cudaStream_t st = (cudaStream_t)stream;
  char* w = reinterpret_cast<char*>(ws);
  float* scores = scores_out ? scores_out : reinterpret_cast<float*>(w + lay.scores);
  int32_t* idx = idx_out ? idx_out : reinterpret_cast<int32_t*>(w + lay.idx);
  float* composite = composite_out ? composite_out : reinterpret_cast<float*>(w + lay.composite);
  const size_t stage_bytes = lay.alloc - lay.stage;

  if (device_status) KVC_CUDA(cudaMemsetAsync(device_status, 0, sizeof(int32_t), st));
  if ((s = run_score(P, gm, qp, kp, &vp, scores, device_status, w + lay.stage, st)) != KVC_OK) return s;
  if ((s = launch_compose(P, scores, idx, composite, w + lay.stage, stage_bytes, st)) != KVC_OK) return s;
  if ((s = launch_allocate(P, composite, budget, 1, P.min_keep, n_keep, reinterpret_cast<long long*>(offsets),
                           w + lay.alloc, lay.total - lay.alloc, st)) != KVC_OK) return s;
  if (P.keep_position_order &&
      (s = launch_order_kept(P, idx, n_keep, false, w + lay.stage, stage_bytes, st)) != KVC_OK) return s;
  return launch_gather(P, kp, vp, idx, n_keep, reinterpret_cast<const long long*>(offsets), budget, false,
                       k_out, v_out, st);
}

// ---- the unstructured variant (App. A.2) ----------------------------------------------------------

static kvc_status check_entries(const Problem& P, long long budget_entries) {
  KVC_REQUIRE(budget_entries >= 0 && budget_entries <= (long long)P.L * P.Hkv * P.N, KVC_ERR_INVALID_ARG,
              "budget_entries %lld outside [0, L * Hkv * N = %lld]", budget_entries, (long long)P.L * P.Hkv * P.N);
  KVC_REQUIRE(P.L * P.Hkv <= kMaxSelectRows, KVC_ERR_UNSUPPORTED, "L * Hkv = %d exceeds %d", P.L * P.Hkv,
              kMaxSelectRows);
  return KVC_OK;
}

// Ranking, the heads' sorted scores (into `sorted`), and the global selection over (layer, head).
static kvc_status run_select_unstructured(const Problem& P, const float* scores, long long budget_entries,
                                          int32_t* idx, int32_t* n_keep, long long* offsets, float* sorted,
                                          char* w, const CompressLayout& lay, cudaStream_t st) {
  kvc_status s;
  const size_t stage_bytes = lay.alloc - lay.stage;
  if ((s = launch_compose(P, scores, idx, nullptr, w + lay.stage, stage_bytes, st)) != KVC_OK) return s;
  if ((s = launch_sorted_scores(P, w + lay.stage, sorted, st)) != KVC_OK) return s;
  return launch_allocate(P, sorted, budget_entries, P.Hkv, 0, n_keep, offsets, w + lay.alloc, lay.total - lay.alloc, st);
}

kvc_status kvc_select_unstructured(const kvc_desc* d, const float* scores, int64_t budget_entries, int32_t* idx,
                                   int32_t* n_keep, int64_t* offsets, void* ws, size_t ws_bytes, void* stream) {
  Problem P; GroupMap gm;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  KVC_REQUIRE(scores && idx && n_keep && offsets, KVC_ERR_INVALID_ARG, "scores, idx, n_keep or offsets is NULL");
  if ((s = check_entries(P, budget_entries)) != KVC_OK) return s;
  const CompressLayout lay = compress_layout(P);
  if ((s = check_ws(ws, ws_bytes, lay.total)) != KVC_OK) return s;
  if ((s = check_device()) != KVC_OK) return s;
  char* w = reinterpret_cast<char*>(ws);
  // the caller's scores are not in the workspace, so its score region is free for the sorted scores
  return run_select_unstructured(P, scores, budget_entries, idx, n_keep, reinterpret_cast<long long*>(offsets),
                                 reinterpret_cast<float*>(w + lay.scores), w, lay, (cudaStream_t)stream);
}

kvc_status kvc_gather_unstructured(const kvc_desc* d, const void* const* k, const void* const* v,
                                   const int32_t* idx, const int32_t* n_keep, const int64_t* offsets,
                                   int64_t budget_entries, void* k_out, void* v_out, void* stream) {
  Problem P; GroupMap gm; LayerPtrs kp, vp;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  if ((s = check_ptrs(k, P.L, "k", &kp)) != KVC_OK) return s;
  if ((s = check_ptrs(v, P.L, "v", &vp)) != KVC_OK) return s;
  KVC_REQUIRE(idx && n_keep && offsets, KVC_ERR_INVALID_ARG, "idx, n_keep or offsets is NULL");
  if ((s = check_entries(P, budget_entries)) != KVC_OK) return s;
  if (budget_entries > 0) {
    KVC_REQUIRE(k_out && v_out, KVC_ERR_INVALID_ARG, "k_out or v_out is NULL");
    KVC_REQUIRE(((reinterpret_cast<uintptr_t>(k_out) | reinterpret_cast<uintptr_t>(v_out)) & 15u) == 0,
                KVC_ERR_INVALID_ARG, "k_out / v_out must be 16-byte aligned");
  }
  if ((s = check_device()) != KVC_OK) return s;
  return launch_gather(P, kp, vp, idx, n_keep, reinterpret_cast<const long long*>(offsets), budget_entries, true,
                       k_out, v_out, (cudaStream_t)stream);
}

kvc_status kvc_compress_unstructured(const kvc_desc* d, const void* const* q, const void* const* k,
                                     const void* const* v, int64_t budget_entries, void* k_out, void* v_out,
                                     int32_t* n_keep, int64_t* offsets, int32_t* idx_out, float* scores_out,
                                     int32_t* device_status, void* ws, size_t ws_bytes, void* stream) {
  Problem P; GroupMap gm; LayerPtrs qp, kp, vp;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  if ((s = check_ptrs(q, P.L, "q", &qp)) != KVC_OK) return s;
  if ((s = check_ptrs(k, P.L, "k", &kp)) != KVC_OK) return s;
  if ((s = check_ptrs(v, P.L, "v", &vp)) != KVC_OK) return s;
  KVC_REQUIRE(n_keep && offsets, KVC_ERR_INVALID_ARG, "n_keep or offsets is NULL");
  if ((s = check_entries(P, budget_entries)) != KVC_OK) return s;
  if (budget_entries > 0) {
    KVC_REQUIRE(k_out && v_out, KVC_ERR_INVALID_ARG, "k_out or v_out is NULL");
    KVC_REQUIRE(((reinterpret_cast<uintptr_t>(k_out) | reinterpret_cast<uintptr_t>(v_out)) & 15u) == 0,
                KVC_ERR_INVALID_ARG, "k_out / v_out must be 16-byte aligned");
  }
  const CompressLayout lay = compress_layout(P);
  if ((s = check_ws(ws, ws_bytes, lay.total)) != KVC_OK) return s;
  if ((s = check_device()) != KVC_OK) return s;

  cudaStream_t st = (cudaStream_t)stream;
  char* w = reinterpret_cast<char*>(ws);
  float* scores = scores_out ? scores_out : reinterpret_cast<float*>(w + lay.scores);
  int32_t* idx = idx_out ? idx_out : reinterpret_cast<int32_t*>(w + lay.idx);
  // the sorted scores: the workspace's score region if the scores themselves go to the caller,
  // else the composite-score region and what follows it cannot hold them -- they take the place of
  // the scores, which nobody reads after the ranking
  float* sorted = reinterpret_cast<float*>(w + lay.scores);
  const size_t stage_bytes = lay.alloc - lay.stage;

  if (device_status) KVC_CUDA(cudaMemsetAsync(device_status, 0, sizeof(int32_t), st));
  if ((s = run_score(P, gm, qp, kp, &vp, scores, device_status, w + lay.stage, st)) != KVC_OK) return s;
  if ((s = run_select_unstructured(P, scores, budget_entries, idx, n_keep, reinterpret_cast<long long*>(offsets),
                                   sorted, w, lay, st)) != KVC_OK) return s;
  if (P.keep_position_order &&
      (s = launch_order_kept(P, idx, n_keep, true, w + lay.stage, stage_bytes, st)) != KVC_OK) return s;
  return launch_gather(P, kp, vp, idx, n_keep, reinterpret_cast<const long long*>(offsets), budget_entries, true,
                       k_out, v_out, st);
}

kvc_status kvc_head_sum(const kvc_desc* d, const float* scores, float* head_sum, void* stream) {
  Problem P; GroupMap gm;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  KVC_REQUIRE(scores && head_sum, KVC_ERR_INVALID_ARG, "scores or head_sum is NULL");
  if ((s = check_device()) != KVC_OK) return s;
  return launch_head_sum(P, scores, head_sum, (cudaStream_t)stream);
}

kvc_status kvc_add_head_mean(const kvc_desc* d, float* scores, const float* head_sum, int32_t n_kv_heads_total,
                             void* stream) {
  Problem P; GroupMap gm;
  kvc_status s;
  if ((s = resolve(d, &P, &gm)) != KVC_OK) return s;
  KVC_REQUIRE(scores && head_sum, KVC_ERR_INVALID_ARG, "scores or head_sum is NULL");
  KVC_REQUIRE(n_kv_heads_total >= P.Hkv, KVC_ERR_INVALID_ARG, "n_kv_heads_total is smaller than the local head count");
  if ((s = check_device()) != KVC_OK) return s;
  return launch_add_head_mean(P, scores, head_sum, n_kv_heads_total, (cudaStream_t)stream);
}

kvc_status kvc_scale(float* x, int64_t n, float factor, void* stream) {
  KVC_REQUIRE(x != nullptr && n >= 0, KVC_ERR_INVALID_ARG, "x is NULL or n < 0");
  kvc_status s;
  if ((s = check_device()) != KVC_OK) return s;
  return launch_scale(x, n, factor, (cudaStream_t)stream);
}

const char* kvc_last_error(void) { return g_err; }

int64_t kvc_launch_count(int32_t reset) {
  const long long n = g_launches;
  if (reset) g_launches = 0;
  return n;
}

int32_t kvc_version(void) { return 100; }

}  // extern "C"
