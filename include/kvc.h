/*
 * kvc -- the KVCompose compression pass over a prefilled KV cache, for NVIDIA B200 (sm_100a).
 *
 * Given, for every layer, the cached keys/values K, V in R^{Hkv x N x d} (Sec. 3.1 of the paper)
 * and the post-RoPE queries of a scoring window (the "task tokens" of Sec. 3.2.2), the pass
 *   (1) scores every cached token per layer and KV head          -- kvc_score    (Eqs. 3, 14-16)
 *   (2) sorts the tokens of every head by score, aligns the rank-k token of each head into the
 *       k-th composite token and gives it a composite score      -- kvc_compose  (Eqs. 17-19)
 *   (3) splits one global budget of token slots over the layers  -- kvc_allocate (Eqs. 20-22)
 *   (4) copies the retained K/V rows into a dense cache that is uniform across the heads of a
 *       layer                                                    -- kvc_gather   (Eqs. 23-24)
 * kvc_compress runs (1)-(4) back to back on one stream without a host synchronisation.
 *
 * General conventions
 *   - Plain C ABI.  Every data pointer is a DEVICE pointer owned by the caller unless it is
 *     marked "host".  The library allocates no device memory and frees none: scratch space comes
 *     from the caller's workspace (kvc_workspace_size bytes, 256-byte aligned).
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = the default stream);
 *     calls return without synchronising.  The return value reports errors the host can see
 *     (bad arguments, a failed launch); kvc_last_error() then holds a message.
 *   - Inputs are never modified.  Indices are 0-based.  Sequences of a batch are independent:
 *     each has its own pool and its own budget (the paper has no batch dimension).
 *   - Finite inputs are a precondition; NaN/Inf in Q or K give unspecified scores.
 *   - All entry points need a CUDA device of compute capability 10.0; there is no CPU path.
 */
#ifndef KVC_H_
#define KVC_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define KVC_API __attribute__((visibility("default")))
#else
#define KVC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  KVC_OK = 0,
  KVC_ERR_INVALID_ARG = -1, /* NULL pointer, inconsistent sizes, misaligned buffer, bad budget */
  KVC_ERR_UNSUPPORTED = -2, /* shape outside what the kernels handle (see kvc_desc) */
  KVC_ERR_WORKSPACE = -3,   /* workspace missing, misaligned or smaller than kvc_workspace_size */
  KVC_ERR_CUDA = -4,        /* a CUDA runtime call failed; message in kvc_last_error() */
  KVC_ERR_TIMEOUT = -5      /* device_status only: a bounded device-side wait gave up */
} kvc_status;

typedef enum { KVC_F32 = 0, KVC_BF16 = 1 } kvc_dtype;

/* Aggregation operator of Eqs. 14, 15, 19: max-pooling or average-pooling. */
typedef enum { KVC_AGG_MAX = 0, KVC_AGG_MEAN = 1 } kvc_agg;

#define KVC_MAX_LAYERS 128
#define KVC_STATIC_MAX_BATCH 64 /* largest batch kvc_allocate_static accepts */

/*
 * Problem description (Sec. 3.1: L layers, K, V in R^{Hkv x N x d}; Sec. 2.2: G = Hq / Hkv).
 *
 * Layouts, per layer l (one device pointer per layer):
 *   Q^(l)  [batch, n_q_heads,  window, head_dim]   element strides q_stride  = (batch, head, row)
 *   K^(l), V^(l) [batch, n_kv_heads, n_ctx, head_dim]  element strides kv_stride = (batch, head, token)
 * The last dimension is contiguous; every row must start on a 16-byte boundary.  A stride of 0
 * in slot 0 of either array means "dense" and all three are filled in from the shape.
 */
typedef struct {
  int32_t n_layers;   /* L, 1..KVC_MAX_LAYERS; L * batch <= 65535 */
  int32_t batch;      /* independent sequences, >= 1 */
  int32_t n_q_heads;  /* Hq */
  int32_t n_kv_heads; /* Hkv */
  int32_t head_dim;   /* d: 64 or 128 */
  int32_t window;     /* w = M: scoring-query rows per query head (Sec. 3.2.2), >= 1 */
  int64_t n_ctx;      /* N cached tokens per sequence, 1 <= N < 2^31 */
  int64_t q_pos0;     /* absolute position of window row 0.  Row m attends to key c iff
                         c <= q_pos0 + m (the model's causal mask).  N - w scores the last w
                         context tokens against the context; any value >= N disables masking
                         (task tokens that follow the context).  Must be >= 0. */
  int32_t dtype;      /* kvc_dtype of Q, K, V and of the compressed K', V' */
  float scale;        /* logit scale; <= 0 selects 1/sqrt(head_dim) (Eq. 3) */
  int32_t agg_task;   /* Eq. 14, over the window rows.   Paper default: KVC_AGG_MAX  */
  int32_t agg_group;  /* Eq. 15, over the G query heads. Paper default: KVC_AGG_MEAN */
  int32_t agg_head;   /* Eq. 19, over the KV heads.      Paper default: KVC_AGG_MEAN */
  int32_t augment_head_mean; /* Eq. 16: add the mean over KV heads to every head's score (default 1) */
  const int32_t* q_to_kv;    /* HOST pointer, n_q_heads entries: KV head of each query head;
                                NULL = j / G with G = Hq / Hkv (Sec. 3.2.2, the reshape before
                                Eq. 15; then Hq % Hkv must be 0).  Every KV head needs >= 1 member. */
  int64_t q_stride[3];
  int64_t kv_stride[3];
  /* Options beyond the paper's default pipeline; kvc_desc_init sets all of them to 0. */
  int32_t value_norm;          /* 1: the v-norm variant of App. A.1.3 -- every attention weight A[m, c] is
                                  multiplied by the Euclidean norm of token c's value row (in the KV head the
                                  query head reads) before Eq. 14.  Used by kvc_compress and
                                  kvc_compress_unstructured (which have V); kvc_score refuses it, use
                                  kvc_score_weighted. */
  int32_t min_keep_per_layer;  /* per-layer minimum m for Eq. 22 (the paper has none: a layer may get no
                                  slot): every layer first keeps its m best composite tokens, the other
                                  budget - L * m slots are handed out as in Eqs. 20-22 among the rest.
                                  0 <= m <= N and L * m <= budget.  Used by kvc_allocate, kvc_compress. */
  int32_t keep_position_order; /* 1: the rows of a head in K', V' come in ascending original position
                                  instead of descending score (the kept set is the same).  Used by
                                  kvc_compress and kvc_compress_unstructured; staged callers apply
                                  kvc_order_kept to idx before kvc_gather. */
  int32_t reserved_;           /* must be 0 */
} kvc_desc;

/* Fill *desc with the paper's defaults for the given shape (dense strides, q_pos0 = N - w,
 * scale 1/sqrt(d), max / mean / mean, head-mean on, contiguous GQA groups). */
KVC_API void kvc_desc_init(kvc_desc* desc, int32_t n_layers, int32_t batch, int32_t n_q_heads,
                   int32_t n_kv_heads, int32_t head_dim, int64_t n_ctx, int32_t window,
                   int32_t dtype);

/* B_total = floor((1 - r_target) * L * N), per sequence (Eq. 21).  The product is evaluated in
 * double and nudged up by a relative 1e-12 before the floor so that decimal ratios such as 0.8
 * behave as in exact arithmetic.  Returns -1 on a bad descriptor or r_target outside [0, 1]. */
KVC_API int64_t kvc_budget_from_ratio(const kvc_desc* desc, double r_target);

/* Bytes of scratch any entry point below may need for this problem (with the options set in desc)
 * and budget (host call). */
KVC_API kvc_status kvc_workspace_size(const kvc_desc* desc, int64_t budget, size_t* bytes);

/*
 * Token importance (Sec. 3.2.2).  For layer l, sequence b, query head j, window row m:
 *   A[m, c] = softmax over the visible keys c of  scale * <q[j, m], k[kv(j), c]>      (Eq. 3)
 *   S_task[j, c]  = agg_task over m of A[m, c]   (a masked entry counts as 0)          (Eq. 14)
 *   S_group[h, c] = agg_group over the query heads of KV head h                        (Eq. 15)
 *   S[h, c] = S_group[h, c] + mean over the KV heads i of S_group[i, c]                (Eq. 16)
 * q, k: HOST arrays of n_layers device pointers.  scores: [L, batch, Hkv, N] fp32, dense.
 * bf16 inputs are multiplied exactly and accumulated in fp32; the attention tensor A is
 * never written to memory.
 *
 * Conditions that only the device can detect (KVC_ERR_TIMEOUT, see kvc_compress) are reported in
 * an int32 inside the workspace, at the byte offset kvc_score_status_offset() returns: 0 after a
 * good run.  Read it once the stream has finished the call; the scores are meaningless otherwise.
 */
KVC_API kvc_status kvc_score(const kvc_desc* desc, const void* const* q, const void* const* k,
                     float* scores, void* workspace, size_t workspace_bytes, void* stream);

/* Byte offset, inside the workspace handed to kvc_score, of the int32 device status word that call
 * writes (host call; depends on the problem only). */
KVC_API kvc_status kvc_score_status_offset(const kvc_desc* desc, size_t* offset);

/* 1 if kvc_score / kvc_compress score this problem with the tensor-core kernel (bf16, contiguous GQA
 * groups q_to_kv[j] = j / G, at most 112 layers), 0 if they take the CUDA-core kernels (fp32, explicit
 * group maps, anything else) -- same results, an order of magnitude slower --, negative on a bad
 * descriptor.  Host call.  Strides that a tensor map cannot express (found when the maps are encoded)
 * also send a call to the CUDA-core kernels. */
KVC_API int32_t kvc_score_uses_tensor_cores(const kvc_desc* desc);

/*
 * kvc_score with value-norm weighting (App. A.1.3 "Effect of Value Norms on Token Scores", the
 * v-norm variant): A^(w)[m, c] = A[m, c] * ||v[kv(j), c]||_2 takes the place of A in Eqs. 14-16.
 * v: HOST array of n_layers device pointers, laid out like k.  The norm of a row is taken in fp32
 * over its head_dim entries.  Because the weight depends on (KV head, token) only and the pooling
 * operators are positively homogeneous, the weighting is applied to the group aggregate of Eq. 15.
 * Everything else as kvc_score (same workspace, same status word); desc->value_norm is ignored.
 */
KVC_API kvc_status kvc_score_weighted(const kvc_desc* desc, const void* const* q, const void* const* k,
                              const void* const* v, float* scores, void* workspace,
                              size_t workspace_bytes, void* stream);

/*
 * Ranking and composite tokens (Sec. 3.3).  For every (l, b, h):
 *   idx[l, b, h, :] = positions 0..N-1 sorted by score, descending; equal scores keep the
 *                     smaller position first                                            (Eq. 17)
 *   composite token k of layer l = { idx[l, b, h, k] : h }  (column k of idx, no copy)
 *   composite[l, b, k] = agg_head over h of scores[l, b, h, idx[l, b, h, k]]       (Eqs. 18-19)
 * The mean is evaluated in fp32 as ((S'_0 + S'_1) + ...) / Hkv, heads in ascending order.
 * idx: [L, batch, Hkv, N] int32.  composite: [L, batch, N] fp32, non-increasing in k.
 * Scores must be non-negative and finite (what kvc_score produces).
 */
KVC_API kvc_status kvc_compose(const kvc_desc* desc, const float* scores, int32_t* idx, float* composite,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * Layer-adaptive budget (Sec. 3.3, Eqs. 20-22).  Per sequence b, all composite[l, b, k] form one
 * pool; the `budget` largest are kept, ties resolved by the total order (score descending,
 * layer ascending, k ascending); n_keep[b, l] = how many of them lie in layer l.
 *   n_keep:  [batch, L] int32,  sum over l == budget exactly, 0 <= n_keep <= N
 *   offsets: [batch, L + 1] int64, exclusive prefix sum of n_keep (offsets[b, L] == budget)
 * composite must be non-increasing in k within a layer (what kvc_compose produces) and
 * non-negative.  0 <= budget <= L * N.  workspace: kvc_workspace_size bytes (the selection over
 * pools of more than 128 rows keeps its histograms there; smaller pools are selected by one
 * kernel on the sorted rows and leave it untouched).
 */
KVC_API kvc_status kvc_allocate(const kvc_desc* desc, const float* composite, int64_t budget,
                        int32_t* n_keep, int64_t* offsets, void* workspace,
                        size_t workspace_bytes, void* stream);

/*
 * Output order option (the paper keeps idx[:N_l], i.e. descending score, Eq. 23): rewrites, in
 * place, the first n_keep[b, l] entries of every idx[l, b, h, :] in ascending position; the rest
 * of each row is left as it is.  A later kvc_gather then writes each head's rows of K', V' in
 * their original order.  n_keep: [batch, L] (device).  Scratch: kvc_workspace_size bytes.
 */
KVC_API kvc_status kvc_order_kept(const kvc_desc* desc, int32_t* idx, const int32_t* n_keep,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * kvc_allocate without a workspace argument (the paper has no counterpart to this entry point; it
 * is kvc_allocate, same inputs, same outputs, same result).
 *
 * It is meant for callers that may not allocate device memory and so cannot supply a workspace:
 * an inference server that plans all of its device memory at start-up and forbids cudaMalloc
 * afterwards (the call synchronises the device and can fail once memory is fragmented), or a
 * plug-in that is handed the host application's tensors but no allocator.  The scratch of the
 * selection lives instead in a fixed array inside the library image: 256 KiB of device memory on
 * every GPU that loads the library, held until the process exits.  The call itself calls no
 * allocator, on the device or through any library.  One thing to plan for: with CUDA's lazy module
 * loading the array is reserved on a device when the library's code is first used there, which can
 * be this entry point's first call on that device -- so make that first call during start-up.
 *
 *   - desc->batch must be <= KVC_STATIC_MAX_BATCH; a larger batch returns KVC_ERR_UNSUPPORTED
 *     and launches nothing.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps what the last call left in it; each
 *     call clears the part it uses, in stream order, before its first kernel.  Two calls whose
 *     work overlaps on the GPU (different streams, no dependency between them) race on it: order
 *     them, or use kvc_allocate with separate workspaces.
 */
KVC_API kvc_status kvc_allocate_static(const kvc_desc* desc, const float* composite, int64_t budget,
                               int32_t* n_keep, int64_t* offsets, void* stream);

/*
 * Compaction (Eqs. 23-24): K'[l][h, k, :] = K[l][h, idx[l, h, k], :] for k < n_keep[l]; V alike.
 * k_out, v_out: [batch, budget * Hkv * d] elements of the cache dtype.  Within sequence b, layer l
 * starts at element offsets[b, l] * Hkv * d and is a dense [Hkv, n_keep[b, l], d] tensor, rows in
 * descending score order.  Rows are copied bit for bit.  n_keep / offsets are read on the device
 * (no host synchronisation); the output size is known beforehand because sum_l n_keep == budget.
 */
KVC_API kvc_status kvc_gather(const kvc_desc* desc, const void* const* k, const void* const* v,
                      const int32_t* idx, const int32_t* n_keep, const int64_t* offsets,
                      int64_t budget, void* k_out, void* v_out, void* stream);

/*
 * The whole pass, stream-ordered.  idx_out [L, batch, Hkv, N], scores_out [L, batch, Hkv, N] and
 * composite_out [L, batch, N] may be NULL (the workspace then holds them).  device_status, if
 * not NULL, receives KVC_OK or a negative kvc_status detected on the device.
 *
 * The bf16 scoring kernel (kvc_score and kvc_compress) is one persistent grid of a CTA per SM
 * whose CTAs exchange the softmax statistics through global memory, so all of them have to be
 * resident at the same time.  Give it the GPU to itself: while other work holds SMs (another
 * stream's kernels, a second kvc_score / kvc_compress in flight, an MPS share smaller than the
 * device) its CTAs may wait for CTAs that cannot start.  Such a wait is bounded (2 s): the kernel
 * then stops, the status word is KVC_ERR_TIMEOUT, the outputs of the call are meaningless, and
 * the context stays usable.  Calls on one stream, or ordered by events, never overlap.
 */
KVC_API kvc_status kvc_compress(const kvc_desc* desc, const void* const* q, const void* const* k,
                        const void* const* v, int64_t budget, void* k_out, void* v_out,
                        int32_t* n_keep, int64_t* offsets, int32_t* idx_out, float* scores_out,
                        float* composite_out, int32_t* device_status, void* workspace,
                        size_t workspace_bytes, void* stream);

/*
 * The unstructured variant (App. A.2 "Discussion on unstructured eviction methods"): the
 * aggregation over the heads (Eq. 19) is left out and every head keeps its own tokens.  Per
 * sequence, all entries scores[l, b, h, c] form one pool; the `budget_entries` best are kept (ties:
 * layer, head, position ascending -- the structured budget of Eq. 21 corresponds to
 * budget_entries = B_total * Hkv); n_keep[b, l, h] = how many of them lie in head h of layer l,
 * which are the first n_keep[b, l, h] entries of idx[l, b, h, :].
 *
 * kvc_select_unstructured: ranking (Eq. 17) and the global selection.
 *   idx:     [L, batch, Hkv, N] int32            n_keep: [batch, L, Hkv] int32
 *   offsets: [batch, L * Hkv + 1] int64, exclusive prefix sum of n_keep over (l, h)
 * kvc_gather_unstructured: k_out, v_out [batch, budget_entries * d]; head (l, h) of sequence b
 *   starts at element offsets[b, l * Hkv + h] * d and is a dense [n_keep[b, l, h], d] tensor (a
 *   ragged cache: heads of a layer differ in length).
 * kvc_compress_unstructured: score (with desc->value_norm if set) + select + (position order if
 *   set) + gather, stream-ordered.  L * Hkv <= 2048.  0 <= budget_entries <= L * Hkv * N.
 */
KVC_API kvc_status kvc_select_unstructured(const kvc_desc* desc, const float* scores, int64_t budget_entries,
                                   int32_t* idx, int32_t* n_keep, int64_t* offsets, void* workspace,
                                   size_t workspace_bytes, void* stream);
KVC_API kvc_status kvc_gather_unstructured(const kvc_desc* desc, const void* const* k, const void* const* v,
                                   const int32_t* idx, const int32_t* n_keep, const int64_t* offsets,
                                   int64_t budget_entries, void* k_out, void* v_out, void* stream);
KVC_API kvc_status kvc_compress_unstructured(const kvc_desc* desc, const void* const* q, const void* const* k,
                                     const void* const* v, int64_t budget_entries, void* k_out,
                                     void* v_out, int32_t* n_keep, int64_t* offsets, int32_t* idx_out,
                                     float* scores_out, int32_t* device_status, void* workspace,
                                     size_t workspace_bytes, void* stream);

/*
 * Support for sharding ONE sequence's KV heads over several GPUs (tensor-parallel serving).  Scoring
 * and ranking are per head and stay local; two steps need the other ranks' heads: the head-mean term
 * of Eq. 16 and the aggregation over heads of Eq. 19.  With desc describing the LOCAL heads (and
 * augment_head_mean = 0 for kvc_score, so that it returns the group aggregates of Eq. 15):
 *   kvc_head_sum:      head_sum[l, b, c] = sum over the local KV heads of scores[l, b, h, c]
 *                      -- the caller all-reduces (sum) head_sum over the ranks --
 *   kvc_add_head_mean: scores[l, b, h, c] += head_sum[l, b, c] / n_kv_heads_total            (Eq. 16)
 *   kvc_compose on the local heads gives the local mean (or max) of Eq. 19; the caller all-reduces it
 *   (sum, then kvc_scale by 1 / ranks for equal shards; max for KVC_AGG_MAX); kvc_allocate then runs
 *   replicated on identical inputs and kvc_gather on the local heads.
 * The paper has no multi-GPU formulation; the sums are the same terms in another order, so scores and
 * composite scores agree with the single-GPU pass to fp32 rounding, not bit for bit.
 * scores: [L, batch, Hkv_local, N]; head_sum: [L, batch, N]; x: n floats.  No workspace needed.
 */
KVC_API kvc_status kvc_head_sum(const kvc_desc* desc, const float* scores, float* head_sum, void* stream);
KVC_API kvc_status kvc_add_head_mean(const kvc_desc* desc, float* scores, const float* head_sum,
                             int32_t n_kv_heads_total, void* stream);
KVC_API kvc_status kvc_scale(float* x, int64_t n, float factor, void* stream);

/* Message of the last error returned on this thread (static storage; never NULL). */
KVC_API const char* kvc_last_error(void);

/* Number of kernels the library has launched on this thread since the last call with reset != 0
 * (a host-side counter for benchmarks; it does not touch the device). */
KVC_API int64_t kvc_launch_count(int32_t reset);

/* Test hook, not for production use: sets the bound of the scoring kernel's device-side waits
 * (nanoseconds; <= 0 restores the default of 2 s) and names one work unit of that kernel -- (layer,
 * sequence, KV head, row tile) numbered in that order -- whose softmax statistics are withheld, so
 * that the waits for them run into the bound and the call ends with KVC_ERR_TIMEOUT in its status
 * word (-1: none).  Process-wide; takes effect at the next launch. */
KVC_API void kvc_debug_score_hooks(int64_t wait_limit_ns, int32_t withhold_unit);

/* Test hook, not for production use: how kvc_allocate (and the allocation inside kvc_compress and
 * kvc_select_unstructured) finds the threshold of Eqs. 20-22.  path 0: the library chooses (pools of up
 * to 128 rows: one kernel that narrows windows on the sorted rows; larger pools: the histogram passes of
 * a radix select); 1: always the histogram passes; 2: the sorted-rows kernel wherever the pool has few
 * enough rows.  max_rounds bounds the narrowing rounds of that kernel before it falls back to a
 * bisection over the key range (< 0: the default of 40; 0: bisect at once).  Both ways give identical
 * results.  Process-wide; takes effect at the next call.  kvc_allocate_static is not affected. */
KVC_API void kvc_debug_select_hooks(int32_t path, int32_t max_rounds);

/* Library version as major * 10000 + minor * 100 + patch. */
KVC_API int32_t kvc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KVC_H_ */
