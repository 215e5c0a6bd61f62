// Token-importance scoring on the Blackwell tensor cores (Eqs. 3, 14, 15), bf16 inputs.
//
// One persistent kernel, one CTA per SM.  K is streamed from HBM exactly once:
//
//   pass 1 (statistics)  tile = 128 tokens.  D[query row, token] = Q K^T on tcgen05 with the
//                        accumulator in TMEM; every query row keeps a running (max, sum-exp) in
//                        registers (rows sit on TMEM lanes, so the row reduction is in-thread).
//   exchange             the partial (max, sum) of the CTAs that shared a (layer, sequence, KV
//                        head) unit are combined by whichever CTA finishes the unit last, which
//                        publishes the rows' log-sum-exp and raises the unit's flag.
//   pass 2 (emit)        runs a fixed number of work items behind pass 1, so its K tiles are still
//                        in L2.  D[token, query row] = K Q^T (operands swapped: tokens on TMEM
//                        lanes), so the max over the window rows (Eq. 14) and the mean/max over the
//                        query heads of the group (Eq. 15) are in-thread and the score store is
//                        coalesced.  max_m exp(s_m - lse_m) is evaluated as exp(max_m(s_m - lse_m)):
//                        one exponential per query head, not per row.
//
// Both passes are interleaved in one static, globally ordered work list that every CTA walks
// with the same stride; an item of pass 2 only ever waits for items of pass 1 that lie a full
// round earlier in that order, so the walk cannot deadlock while all CTAs are resident.  Every
// wait (mbarrier or flag) is bounded; on expiry the kernel records KVC_ERR_TIMEOUT and drains.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 4-7 and 8-11 =
// two epilogue warpgroups (each takes every other tile and owns two of the four TMEM buffers).
#include <cuda.h>

#include "kvc_internal.cuh"

namespace kvc {
namespace {

constexpr int kTile = 128;            // tokens per tile = MMA M = MMA N
constexpr int kFastThreads = 384;
constexpr int kEpiWarp0 = 4;
constexpr int kRows = 128;            // query rows per unit handled by one MMA (R <= 128)
constexpr float kLog2eF = 1.4426950408889634f;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s: far beyond any healthy wait

constexpr int kMaxFastLayers = 112;   // 2 tensor maps per layer must fit the 32 KB kernel-parameter space

struct FastParams {
  CUtensorMap k_maps[kMaxFastLayers];   // K^(l) as (d, N, Hkv, Bt), box 64 x 128 x 1 x 1, 128-byte swizzle
  CUtensorMap q_maps[kMaxFastLayers];   // Q^(l) as (d, w, Hq, Bt), box 64 x w x G x 1
  float2* partial;             // [U][NS][2][128]
  float* lse2;                 // [U][128]
  int* counter;                // [U]
  int* flag;                   // [U]
  int* status;                 // device status word (may be null)
  float* scores;               // [U][N]
  int L, Bt, Hkv, G, R;
  long long N, q_pos0;
  int U, C, NT, RUN, LAG, NS;  // units, items per unit, tiles per unit, run length, lag, partial slots
  long long E;                 // number of list entries = U * C + LAG
  float sl2e;                  // scale * log2(e)
  int agg_group;
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the abort word is set or the time limit expires (and sets it).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_word) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 1023u) == 0) {
      if (*abort_word) return false;
      if (globaltimer_ns() - t0 > kWaitLimitNs) { *abort_word = 1; return false; }
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void named_bar(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 B apart,
// 8-row groups 1024 B apart; `addr` may be advanced by 32 B per 16-element K step.
__device__ __forceinline__ uint64_t umma_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);        // start address
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset
  d |= (uint64_t)1 << 46;                          // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = N = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTile >> 3) << 17) |
                            ((uint32_t)(kTile >> 4) << 24);

// ------------------------------------------------------------------------------------------------
// Work list
// ------------------------------------------------------------------------------------------------
struct Entry {
  bool has1, has2;
  int u1, ch1, u2, ch2;
};
__device__ __forceinline__ Entry decode(const FastParams& P, long long e) {
  Entry t;
  const long long n1 = (long long)P.U * P.C;
  t.has1 = e < n1;
  t.u1 = t.has1 ? (int)(e / P.C) : -1;
  t.ch1 = t.has1 ? (int)(e - (long long)t.u1 * P.C) : 0;
  const long long p = e - P.LAG;
  t.has2 = p >= 0 && p < n1;
  t.u2 = t.has2 ? (int)(p / P.C) : -1;
  t.ch2 = t.has2 ? (int)(p - (long long)t.u2 * P.C) : 0;
  return t;
}
// Next list entry of this CTA after e (runs of RUN consecutive entries, stride gridDim.x runs).
__device__ __forceinline__ long long next_entry(const FastParams& P, long long e) {
  const long long r = e / P.RUN;
  const int k = (int)(e - r * P.RUN);
  if (k + 1 < P.RUN && e + 1 < P.E) return e + 1;
  const long long e2 = (r + gridDim.x) * P.RUN;
  return e2 < P.E ? e2 : -1;
}
__device__ __forceinline__ void unit_coords(const FastParams& P, int u, int* l, int* b, int* h) {
  *h = u % P.Hkv;
  const int lb = u / P.Hkv;
  *b = lb % P.Bt;
  *l = lb / P.Bt;
}

template <int D>
struct SmemLayout {
  static constexpr int kHalves = D / 64;
  static constexpr int kTileBytes = kTile * D * 2;
  static constexpr int kStages = (D == 128) ? 4 : 8;
  static constexpr int kQ = 0;                                 // two Q buffers
  static constexpr int kK = 2 * kTileBytes;                    // K stage ring
  static constexpr int kMisc = kK + kStages * kTileBytes;
  // misc: barriers then small arrays
  static constexpr int kBarFull = kMisc;                       // kStages x 8
  static constexpr int kBarEmpty = kBarFull + 8 * kStages;
  static constexpr int kBarTFull = kBarEmpty + 8 * kStages;    // 4 x 8
  static constexpr int kBarTEmpty = kBarTFull + 32;
  static constexpr int kBarQFull = kBarTEmpty + 32;            // 2 x 8
  static constexpr int kBarQFree = kBarQFull + 16;
  static constexpr int kTmemSlot = kBarQFree + 16;             // 4 B (+ padding)
  static constexpr int kAbort = kTmemSlot + 8;                 // 4 B
  static constexpr int kBcast = kAbort + 8;                    // 2 x 4 B
  static constexpr int kLse = kBcast + 16;                     // 2 x 128 floats
  static constexpr int kTotal = kLse + 2 * kRows * 4;
  static constexpr int kDynamic = kTotal + 1024;               // slack for 1024-byte alignment
};

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
template <int D, int W, bool kTaskMean>
__global__ void __launch_bounds__(kFastThreads, 1)
score_sm100_kernel(const __grid_constant__ FastParams P) {
  using SL = SmemLayout<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_word = reinterpret_cast<volatile int*>(smem + SL::kAbort);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SL::kTmemSlot);

  auto bar_full = [&](int s) { return sbase + SL::kBarFull + 8 * s; };
  auto bar_empty = [&](int s) { return sbase + SL::kBarEmpty + 8 * s; };
  auto bar_tfull = [&](int b) { return sbase + SL::kBarTFull + 8 * b; };
  auto bar_tempty = [&](int b) { return sbase + SL::kBarTEmpty + 8 * b; };
  auto bar_qfull = [&](int q) { return sbase + SL::kBarQFull + 8 * q; };
  auto bar_qfree = [&](int q) { return sbase + SL::kBarQFree + 8 * q; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < SL::kStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
    for (int b = 0; b < 4; ++b) { mbar_init(bar_tfull(b), 1); mbar_init(bar_tempty(b), 4); }
    for (int q = 0; q < 2; ++q) { mbar_init(bar_qfull(q), 1); mbar_init(bar_qfree(q), 1); }
    *abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const uint32_t q_bytes = (uint32_t)P.R * D * 2;

  if (warp == 0) {
    // ============================== TMA producer ==============================================
    if (lane == 0) {
      long long n = 0;                 // tiles issued so far
      int cur_u[2] = {-1, -1};
      uint32_t qfree_phase[2] = {0, 0};
      bool ok = true;
      for (long long e = (long long)blockIdx.x * P.RUN; e >= 0 && e < P.E && ok; e = next_entry(P, e)) {
        const Entry t = decode(P, e);
        for (int part = 0; part < 2 && ok; ++part) {
          if (!(part == 0 ? t.has1 : t.has2)) continue;
          const int u = part == 0 ? t.u1 : t.u2;
          const int ch = part == 0 ? t.ch1 : t.ch2;
          int l, b, h;
          unit_coords(P, u, &l, &b, &h);
          if (u != cur_u[part]) {
            if (cur_u[part] >= 0) {           // the MMAs that read the old Q must have completed
              ok = mbar_wait(bar_qfree(part), qfree_phase[part], abort_word);
              qfree_phase[part] ^= 1;
              if (!ok) break;
            }
            mbar_expect_tx(bar_qfull(part), q_bytes);
            for (int hf = 0; hf < SL::kHalves; ++hf)
              tma_load_4d(sbase + SL::kQ + part * SL::kTileBytes + hf * (kTile * 128), P.q_maps + l,
                          bar_qfull(part), hf * 64, 0, h * P.G, b);
            cur_u[part] = u;
          }
          for (int tt = 0; tt < 2; ++tt) {
            const int tile = 2 * ch + tt;
            if (tile >= P.NT) break;
            const int s = (int)(n % SL::kStages);
            const uint32_t ph = (uint32_t)((n / SL::kStages) & 1);
            if (n >= SL::kStages) {
              ok = mbar_wait(bar_empty(s), ph ^ 1, abort_word);
              if (!ok) break;
            }
            mbar_expect_tx(bar_full(s), SL::kTileBytes);
            for (int hf = 0; hf < SL::kHalves; ++hf)
              tma_load_4d(sbase + SL::kK + s * SL::kTileBytes + hf * (kTile * 128), P.k_maps + l, bar_full(s),
                          hf * 64, tile * kTile, h, b);
            ++n;
          }
        }
      }
      // drain: every issued copy must have landed before the CTA's shared memory is released
      const long long first = n > SL::kStages ? n - SL::kStages : 0;
      for (long long i = first; i < n; ++i)
        mbar_wait(bar_full((int)(i % SL::kStages)), (uint32_t)((i / SL::kStages) & 1), abort_word);
    }
  } else if (warp == 1) {
    // ============================== MMA issuer =================================================
    if (lane == 0) {
      long long n = 0;
      long long nw[2] = {0, 0};        // tiles issued per warpgroup
      int cur_u[2] = {-1, -1};
      uint32_t qfull_phase[2] = {0, 0};
      bool ok = true;
      for (long long e = (long long)blockIdx.x * P.RUN; e >= 0 && e < P.E && ok; e = next_entry(P, e)) {
        const Entry t = decode(P, e);
        const long long e_next = next_entry(P, e);
        Entry tn;
        tn.has1 = tn.has2 = false; tn.u1 = tn.u2 = -1; tn.ch1 = tn.ch2 = 0;
        if (e_next >= 0) tn = decode(P, e_next);
        for (int part = 0; part < 2 && ok; ++part) {
          if (!(part == 0 ? t.has1 : t.has2)) continue;
          const int u = part == 0 ? t.u1 : t.u2;
          const int ch = part == 0 ? t.ch1 : t.ch2;
          if (u != cur_u[part]) {
            ok = mbar_wait(bar_qfull(part), qfull_phase[part], abort_word);
            qfull_phase[part] ^= 1;
            if (!ok) break;
            cur_u[part] = u;
          }
          const uint32_t q_addr = sbase + SL::kQ + part * SL::kTileBytes;
          for (int tt = 0; tt < 2; ++tt) {
            const int tile = 2 * ch + tt;
            if (tile >= P.NT) break;
            const int s = (int)(n % SL::kStages);
            const int buf = tt * 2 + (int)(nw[tt] & 1);
            ok = mbar_wait(bar_full(s), (uint32_t)((n / SL::kStages) & 1), abort_word);
            if (ok && nw[tt] >= 2) ok = mbar_wait(bar_tempty(buf), (uint32_t)(((nw[tt] >> 1) & 1) ^ 1), abort_word);
            if (!ok) break;
            tc_fence_after();
            const uint32_t k_addr = sbase + SL::kK + s * SL::kTileBytes;
            const uint32_t d_tmem = tmem_base + (uint32_t)buf * kTile;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t off = (uint32_t)(kk >> 2) * (kTile * 128) + (uint32_t)(kk & 3) * 32;
              const uint64_t dq = umma_desc(q_addr + off), dk = umma_desc(k_addr + off);
              // pass 1: rows = query rows (A = Q), columns = tokens (B = K); pass 2: swapped
              if (part == 0) tc_mma_bf16(d_tmem, dq, dk, kIdesc, kk > 0);
              else tc_mma_bf16(d_tmem, dk, dq, kIdesc, kk > 0);
            }
            tc_commit(bar_empty(s));      // the K stage may be refilled once these MMAs are done
            tc_commit(bar_tfull(buf));    // ... and the accumulator is then complete
            ++n; ++nw[tt];
          }
          // release the Q buffer as soon as the last MMA that reads it has been issued
          const int u_next = part == 0 ? (tn.has1 ? tn.u1 : -1) : (tn.has2 ? tn.u2 : -1);
          const bool more = e_next >= 0 && (part == 0 ? tn.has1 : tn.has2);
          if (ok && more && u_next != u) tc_commit(bar_qfree(part));
        }
      }
    }
  } else if (warp >= kEpiWarp0) {
    // ============================== epilogue warpgroups ========================================
    const int wg = (warp - kEpiWarp0) >> 2;          // 0 or 1: takes tile 2*ch + wg of every item
    const int quarter = warp & 3;                    // TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;             // TMEM lane = query row (pass 1) or token (pass 2)
    const int wtid = threadIdx.x - (kEpiWarp0 + 4 * wg) * 32;   // 0..127 within the warpgroup
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    int* bcast = reinterpret_cast<int*>(smem + SL::kBcast) + wg;
    float* lse_s = reinterpret_cast<float*>(smem + SL::kLse) + wg * kRows;
    const int bar_id = 1 + wg;

    long long nwg = 0;               // tiles consumed by this warpgroup
    int acc_u = -1;                  // unit whose statistics are being accumulated
    long long acc_run = 0;
    float m_run = -INFINITY, l_run = 0.f;
    int lse_u = -1;
    bool ok = true;

    // flush the running statistics of (acc_u, acc_run) and, if this was the unit's last part,
    // reduce all parts to the rows' log-sum-exp and raise the unit's flag
    auto flush = [&]() {
      const int u = acc_u;
      const long long r_first = ((long long)u * P.C) / P.RUN;
      const long long r_last = ((long long)(u + 1) * P.C - 1) / P.RUN;
      const int slot = (int)(acc_run - r_first);
      P.partial[(((long long)u * P.NS + slot) * 2 + wg) * kRows + wtid] = make_float2(m_run, l_run);
      __threadfence();
      named_bar(bar_id, 128);
      if (wtid == 0) {
        const int expected = 2 * (int)(r_last - r_first + 1);
        const int old = atomicAdd(P.counter + u, 1);
        *bcast = (old == expected - 1) ? 1 : 0;
      }
      named_bar(bar_id, 128);
      if (*bcast) {
        __threadfence();
        const int nparts = 2 * (int)(r_last - r_first + 1);
        const float2* p = P.partial + ((long long)u * P.NS * 2) * kRows + wtid;
        float M = -INFINITY, Ls = 0.f;
        for (int i = 0; i < nparts; ++i) {
          const float2 v = __ldcg(p + (long long)i * kRows);
          const float Mn = fmaxf(M, v.x);
          if (Mn > -INFINITY) Ls = Ls * ex2(M - Mn) + v.y * ex2(v.x - Mn);
          M = Mn;
        }
        P.lse2[(long long)u * kRows + wtid] = M + log2f(Ls);
        __threadfence();
        named_bar(bar_id, 128);
        if (wtid == 0) st_release(P.flag + u, 1);
      }
      named_bar(bar_id, 128);
      acc_u = -1;
      m_run = -INFINITY; l_run = 0.f;
    };

    for (long long e = (long long)blockIdx.x * P.RUN; e >= 0 && e < P.E; e = next_entry(P, e)) {
      const Entry t = decode(P, e);
      const long long run = e / P.RUN;
      // ---------------- pass 1: statistics ----------------
      if (t.has1) {
        if (acc_u >= 0 && (acc_u != t.u1 || acc_run != run)) flush();
        if (acc_u < 0) { acc_u = t.u1; acc_run = run; }
        const int tile = 2 * t.ch1 + wg;
        if (tile < P.NT) {
          const int buf = wg * 2 + (int)(nwg & 1);
          if (ok) ok = mbar_wait(bar_tfull(buf), (uint32_t)((nwg >> 1) & 1), abort_word);
          tc_fence_after();
          const long long c0 = (long long)tile * kTile;
          const long long last_vis = min(P.N - 1, P.q_pos0 + (row % W));   // last visible key of this row
          const bool full_tile = (c0 + kTile - 1 <= min(P.N - 1, P.q_pos0)); // no masking anywhere in the tile
#pragma unroll 1
          for (int j = 0; j < kTile / 32; ++j) {
            float v[32];
            tc_ld32(lane_addr + (uint32_t)buf * kTile + j * 32, v);
            if (ok) {
              if (!full_tile) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (c0 + j * 32 + i > last_vis) v[i] = -INFINITY;
              }
              float x0 = v[0], x1 = v[1], x2 = v[2], x3 = v[3];
#pragma unroll
              for (int i = 4; i < 32; i += 4) {
                x0 = fmaxf(x0, v[i + 0]); x1 = fmaxf(x1, v[i + 1]);
                x2 = fmaxf(x2, v[i + 2]); x3 = fmaxf(x3, v[i + 3]);
              }
              const float cmax = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
              const float m_new = fmaxf(m_run, cmax * P.sl2e);
              if (m_new > -INFINITY) {
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                  a0 += ex2(fmaf(v[i + 0], P.sl2e, -m_new));
                  a1 += ex2(fmaf(v[i + 1], P.sl2e, -m_new));
                  a2 += ex2(fmaf(v[i + 2], P.sl2e, -m_new));
                  a3 += ex2(fmaf(v[i + 3], P.sl2e, -m_new));
                }
                l_run = l_run * ex2(m_run - m_new) + ((a0 + a1) + (a2 + a3));
                m_run = m_new;
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tempty(buf));
          ++nwg;
        }
      }
      // flush at the end of a run (the next entry of this CTA lies in another run) or of pass 1
      if (acc_u >= 0) {
        const long long e_next = next_entry(P, e);
        const bool run_ends = e_next < 0 || e_next / P.RUN != run || !(e_next < (long long)P.U * P.C);
        if (run_ends) flush();
      }
      // ---------------- pass 2: emit ----------------
      if (t.has2) {
        if (lse_u != t.u2) {
          if (wtid == 0 && ok) {
            const unsigned long long t0 = globaltimer_ns();
            uint32_t spins = 0;
            while (ld_acquire(P.flag + t.u2) == 0) {
              __nanosleep(64);
              if ((++spins & 255u) == 0) {
                if (*abort_word) break;
                if (globaltimer_ns() - t0 > kWaitLimitNs) { *abort_word = 1; break; }
              }
            }
          }
          named_bar(bar_id, 128);
          lse_s[wtid] = __ldcg(P.lse2 + (long long)t.u2 * kRows + wtid);
          named_bar(bar_id, 128);
          lse_u = t.u2;
          if (*abort_word) ok = false;
        }
        const int tile = 2 * t.ch2 + wg;
        if (tile < P.NT) {
          const int buf = wg * 2 + (int)(nwg & 1);
          if (ok) ok = mbar_wait(bar_tfull(buf), (uint32_t)((nwg >> 1) & 1), abort_word);
          tc_fence_after();
          const long long c = (long long)tile * kTile + row;          // this thread's token
          const bool full_tile = ((long long)tile * kTile + kTile - 1 <= P.q_pos0);
          const long long m_min = c - P.q_pos0;                       // rows m >= m_min see token c
          float gacc = (P.agg_group == KVC_AGG_MAX) ? -INFINITY : 0.f;
          float hacc = kTaskMean ? 0.f : -INFINITY;
#pragma unroll 1
          for (int j = 0; j < kTile / 32; ++j) {
            if (j * 32 >= P.R) break;
            float v[32];
            tc_ld32(lane_addr + (uint32_t)buf * kTile + j * 32, v);
            const float4* l4 = reinterpret_cast<const float4*>(lse_s + j * 32);
#pragma unroll
            for (int i4 = 0; i4 < 8; ++i4) {
              const float4 lv = l4[i4];
              const float lsv[4] = {lv.x, lv.y, lv.z, lv.w};
#pragma unroll
              for (int ii = 0; ii < 4; ++ii) {
                const int i = i4 * 4 + ii;
                const int col = j * 32 + i;
                float x = fmaf(v[i], P.sl2e, -lsv[ii]);               // log2 of the attention weight
                if (!full_tile && (col % W) < m_min) x = -INFINITY;
                if (kTaskMean) hacc += ex2(x); else hacc = fmaxf(hacc, x);
                if ((col + 1) % W == 0) {                              // a query head is complete
                  if (col < P.R) {
                    const float s_task = kTaskMean ? hacc * (1.0f / W) : ex2(hacc);
                    gacc = (P.agg_group == KVC_AGG_MAX) ? fmaxf(gacc, s_task) : gacc + s_task;
                  }
                  hacc = kTaskMean ? 0.f : -INFINITY;
                }
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tempty(buf));
          ++nwg;
          if (P.agg_group == KVC_AGG_MEAN) gacc = gacc / (float)P.G;
          if (ok && c < P.N) P.scores[(long long)t.u2 * P.N + c] = gacc;
        }
      }
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_word && P.status) atomicCAS(P.status, 0, (int)KVC_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool encode_map(CUtensorMap* m, const void* base, const long long dims[4], const long long strides_bytes[3],
                const unsigned box[4]) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gd[4]; cuuint64_t gs[3]; cuuint32_t bx[4]; cuuint32_t es[4] = {1, 1, 1, 1};
  for (int i = 0; i < 4; ++i) { gd[i] = (cuuint64_t)dims[i]; bx[i] = box[i]; }
  for (int i = 0; i < 3; ++i) gs[i] = (cuuint64_t)strides_bytes[i];
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), gd, gs, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct FastPlan {
  int U, C, NT, RUN, LAG, NS, grid;
  size_t off_partial, off_lse, off_counter, off_total;
};

bool make_plan(const Problem& P, FastPlan* pl) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return false;
  pl->U = P.L * P.Bt * P.Hkv;
  pl->NT = (int)((P.N + kTile - 1) / kTile);
  pl->C = (pl->NT + 1) / 2;
  pl->RUN = 4;
  pl->grid = sms;
  // pass 2 trails pass 1 by one full round of the grid plus one unit
  pl->LAG = ((pl->grid * pl->RUN + pl->C + pl->RUN - 1) / pl->RUN) * pl->RUN;
  pl->NS = (pl->C + pl->RUN - 1) / pl->RUN + 1;
  size_t off = 0;
  pl->off_partial = off; off += align_up((size_t)pl->U * pl->NS * 2 * kRows * sizeof(float2));
  pl->off_lse = off; off += align_up((size_t)pl->U * kRows * sizeof(float));
  pl->off_counter = off; off += align_up((size_t)pl->U * 2 * sizeof(int));
  pl->off_total = off;
  return true;
}

template <int D, int W, bool M>
kvc_status launch_t(const FastParams& fp, int grid, cudaStream_t st) {
  using SL = SmemLayout<D>;
  static bool attr_set = false;
  if (!attr_set) {
    KVC_CUDA(cudaFuncSetAttribute(score_sm100_kernel<D, W, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kDynamic));
    attr_set = true;
  }
  score_sm100_kernel<D, W, M><<<grid, kFastThreads, SL::kDynamic, st>>>(fp);
  KVC_LAUNCH_CHECK("score_sm100_kernel");
  return KVC_OK;
}

template <int D, bool M>
kvc_status launch_w(int W, const FastParams& fp, int grid, cudaStream_t st) {
  switch (W) {
    case 8: return launch_t<D, 8, M>(fp, grid, st);
    case 16: return launch_t<D, 16, M>(fp, grid, st);
    case 32: return launch_t<D, 32, M>(fp, grid, st);
    case 64: return launch_t<D, 64, M>(fp, grid, st);
    default: return launch_t<D, 128, M>(fp, grid, st);
  }
}

}  // namespace

bool score_sm100_supported(const Problem& P) {
  if (P.dtype != KVC_BF16 || !P.contiguous_groups) return false;
  if (P.w != 8 && P.w != 16 && P.w != 32 && P.w != 64 && P.w != 128) return false;
  const int G = P.Hq / P.Hkv;
  if ((long long)G * P.w > kRows) return false;
  if (P.L > kMaxFastLayers || (long long)P.L * P.Bt * P.Hkv > (1 << 24)) return false;
  if (P.N >= (1LL << 30)) return false;
  return encode_fn() != nullptr;
}

size_t score_sm100_workspace_bytes(const Problem& P) {
  FastPlan pl;
  if (!make_plan(P, &pl)) {
    // no device yet (host-only size query): assume the largest SM count this library targets
    pl.U = P.L * P.Bt * P.Hkv;
    pl.NT = (int)((P.N + kTile - 1) / kTile);
    pl.C = (pl.NT + 1) / 2;
    pl.RUN = 4;
    pl.NS = (pl.C + pl.RUN - 1) / pl.RUN + 1;
    return align_up((size_t)pl.U * pl.NS * 2 * kRows * sizeof(float2)) +
           align_up((size_t)pl.U * kRows * sizeof(float)) + align_up((size_t)pl.U * 2 * sizeof(int));
  }
  return pl.off_total;
}

// Returns KVC_ERR_UNSUPPORTED (without setting an error) when the tensor maps cannot be encoded
// for these strides; the caller then uses the CUDA-core path.
kvc_status launch_score_sm100(const Problem& P, const LayerPtrs& q, const LayerPtrs& k, float* scores,
                              int* device_status, void* ws, size_t ws_bytes, cudaStream_t st) {
  FastPlan pl;
  if (!make_plan(P, &pl)) return KVC_ERR_UNSUPPORTED;
  if (ws_bytes < pl.off_total) { set_error("score: workspace too small"); return KVC_ERR_WORKSPACE; }
  const int G = P.Hq / P.Hkv;
  static thread_local FastParams fp;
  for (int l = 0; l < P.L; ++l) {
    const long long kd[4] = {P.d, P.N, P.Hkv, P.Bt};
    const long long ks[3] = {P.kvs[2] * 2, P.kvs[1] * 2, P.kvs[0] * 2};
    const unsigned kb[4] = {64, (unsigned)kTile, 1, 1};
    const long long qd[4] = {P.d, P.w, P.Hq, P.Bt};
    const long long qs[3] = {P.qs[2] * 2, P.qs[1] * 2, P.qs[0] * 2};
    const unsigned qb[4] = {64, (unsigned)P.w, (unsigned)G, 1};
    if (!encode_map(&fp.k_maps[l], k.p[l], kd, ks, kb)) return KVC_ERR_UNSUPPORTED;
    if (!encode_map(&fp.q_maps[l], q.p[l], qd, qs, qb)) return KVC_ERR_UNSUPPORTED;
  }
  char* w = reinterpret_cast<char*>(ws);
  KVC_CUDA(cudaMemsetAsync(w + pl.off_counter, 0, (size_t)pl.U * 2 * sizeof(int), st));

  fp.partial = reinterpret_cast<float2*>(w + pl.off_partial);
  fp.lse2 = reinterpret_cast<float*>(w + pl.off_lse);
  fp.counter = reinterpret_cast<int*>(w + pl.off_counter);
  fp.flag = fp.counter + pl.U;
  fp.status = device_status;
  fp.scores = scores;
  fp.L = P.L; fp.Bt = P.Bt; fp.Hkv = P.Hkv; fp.G = G; fp.R = G * P.w;
  fp.N = P.N; fp.q_pos0 = P.q_pos0;
  fp.U = pl.U; fp.C = pl.C; fp.NT = pl.NT; fp.RUN = pl.RUN; fp.LAG = pl.LAG; fp.NS = pl.NS;
  fp.E = (long long)pl.U * pl.C + pl.LAG;
  fp.sl2e = P.scale * kLog2eF;
  fp.agg_group = P.agg_group;
  const bool mean = P.agg_task == KVC_AGG_MEAN;
  if (P.d == 128) return mean ? launch_w<128, true>(P.w, fp, pl.grid, st) : launch_w<128, false>(P.w, fp, pl.grid, st);
  return mean ? launch_w<64, true>(P.w, fp, pl.grid, st) : launch_w<64, false>(P.w, fp, pl.grid, st);
}

}  // namespace kvc
