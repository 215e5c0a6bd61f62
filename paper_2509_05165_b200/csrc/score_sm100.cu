// Token-importance scoring on the Blackwell tensor cores (Eqs. 3, 14, 15), bf16 inputs.
//
// One persistent kernel, one CTA per SM.  K is streamed from HBM exactly once:
//
//   pass 1 (statistics)  tile = 128 tokens.  D[query row, token] = Q K^T on tcgen05 with the
//                        accumulator in TMEM.  Query rows sit on TMEM lanes, so the softmax
//                        denominator of a row (Eq. 3) is an in-thread sum: every row keeps a
//                        reference exponent and a running sum of 2^(logit - reference).
//   exchange             a run of RT consecutive tiles of one (layer, sequence, KV head) unit
//                        yields one (reference, sum) per row.  The short way: every row has a
//                        fixed reference (its logit against token 0, from a small kernel that
//                        runs first) and one 64-bit word; the run's sum is rescaled to that
//                        reference, converted to fixed point (2^-20) and added, together with an
//                        arrival count in the top byte, with one integer reduction.  Integer
//                        addition makes the total independent of the order of arrival, and sum
//                        and count travel in one word, so a reader of the sum needs no fence: the
//                        word is complete when its count equals the unit's runs.  That is two round
//                        trips to L2 between the last pass-1 tile of a unit and its first pass-2
//                        tile.  The long way, for a run's sum that does not fit the fixed-point
//                        range (a token about 14 nats above token 0): the run writes its
//                        (reference, sum) of that row to global memory, marks itself in the row's
//                        bitmap of such runs, and only then counts itself into the word, with
//                        release semantics (the runs that fit add relaxed and write nothing
//                        else); a pass-2 thread whose word shows such runs acquires the complete
//                        word and folds their records, in run order (the same order for every
//                        reader), into the fixed-point sum of the others.
//   pass 2 (emit)        the same CTA revisits its tiles a fixed number of runs later, when their
//                        K rows are still in L2.  D[token, query row] = K Q^T (operands swapped:
//                        tokens on TMEM lanes), so the max over the window rows (Eq. 14) and the
//                        mean/max over the query heads of the group (Eq. 15) are in-thread and
//                        the score store is coalesced.  max_m exp(s_m - lse_m) is evaluated as
//                        exp(max_m(s_m - lse_m)): one exponential per query head, not per row.
//
// A unit is a (layer, sequence, KV head, row tile): the G x w window rows of a KV head are cut
// into row tiles of at most 128 rows (whole query heads), so that any GQA group / window size
// with w <= 128 runs here (w = 8, 16, 32, 64, 128 as compile-time specialisations, any other
// length through one variant that reads it at run time); with more than one row tile the
// pass-2 results are partial group aggregates that the Eq. 16 kernel combines in a fixed order.
//
// Every CTA walks one static sequence that alternates a pass-1 tile with a pass-2 tile; the
// pass-2 stream trails the pass-1 stream by `shift` tiles (two runs where a unit has no more
// runs than there are CTAs: 38 MB of K at 148 CTAs, which L2 still holds).  A pass-2 tile only
// ever waits for pass-1 tiles that lie earlier in every CTA's sequence, so the walk cannot
// deadlock while all CTAs are resident (the host checks that they can be).  Every wait
// (mbarrier or global word) is bounded; on expiry the kernel records
// KVC_ERR_TIMEOUT, stops computing and drains.
//
// Warp roles (512 threads): warp 0 = TMA producer (K ring, Q ring, L2 prefetch); warp 1 = MMA
// issuer of pass 1 and TMEM owner; warp 2 = MMA issuer of pass 2 (two issuers: issuing the eight
// MMAs of a tile takes a thread about 420 clocks, a commit about 50 and every barrier wait
// about 100 even when it succeeds at once, which together is more than the 512 tensor clocks of
// the tile, and the tensor pipe would idle meanwhile); warp 3 has no role; warps 4-7 =
// pass-2 epilogue; warps 8-15 = pass-1 epilogue (two groups of four warps, each takes one half
// of every tile's columns).
#include <cuda.h>

#include <atomic>
#include <mutex>

#include "kvc_internal.cuh"

#ifndef KVC_SCORE_RUN_TILES
#define KVC_SCORE_RUN_TILES 4      // tiles per run
#endif
#ifndef KVC_SCORE_LAG_TILES
#define KVC_SCORE_LAG_TILES 0      // tiles of slack beyond the runs a unit's statistics have to wait for
#endif
#ifndef KVC_SCORE_PREFETCH
#define KVC_SCORE_PREFETCH 2       // pass-1 tiles prefetched into L2 ahead of their load
#endif

namespace kvc {
namespace {

constexpr int kTile = 128;            // tokens per tile = MMA M = MMA N
constexpr int kFastThreads = 512;
constexpr int kRows = 128;            // query rows per unit handled by one MMA (R <= 128)
constexpr int kMinRunTiles = KVC_SCORE_RUN_TILES;   // runs are longer only where a unit would otherwise have more than 255
constexpr int kQSlots = 3;
constexpr int kPrefetch = KVC_SCORE_PREFETCH;
constexpr float kLog2eF = 1.4426950408889634f;
constexpr float kRescaleLimit = 1.8446744e19f;               // 2^64: a chunk sum beyond it restarts with a new reference
constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;   // 2 s: far beyond any healthy wait

constexpr int kMaxFastLayers = 112;   // 2 tensor maps per layer must fit the 32 KB kernel-parameter space

struct FastParams {
  CUtensorMap k_maps[kMaxFastLayers];   // K^(l) as (64, N, d / 64, Hkv, Bt), box 64 x 128 x d / 64 x 1 x 1, 128-byte swizzle:
                                        // a tile arrives as d / 64 blocks of 128 rows of 128 bytes with one copy
  CUtensorMap q_maps[kMaxFastLayers];   // Q^(l) as (d, w, Hq, Bt), box 64 x w x G x 1
  float2* partial;             // [U][RPU][128]: (ref, sum) of a row over one run, written only where the sum
                               // does not fit the row's word
  unsigned long long* ovf;     // [U][128][4], preset to 0: per row, the runs (bit j) that wrote such a record
  unsigned long long* acc;     // [U][128], preset to 0: per row  arrivals << 56 | overflows << 48 | sum in units
                               // of 2^-20 of 2^(logit - ref[row]), added to by every run of the unit
  const float* ref;            // [U][128]: the row's reference exponent (its scaled logit against token 0)
  int* status;                 // device status word (may be null)
  float* scores;               // [L*Bt*Hkv][N], or with QT > 1 the partial aggregates [QT][L*Bt*Hkv][N]
  int L, Bt, Hkv, G;
  int HPT, QT, w;              // query heads per row tile, row tiles per KV head, window rows per query head
  int CH;                      // row tiles per query head: 1, or ceil(w / 128) for windows longer than 128 rows
                               // (then HPT = 1 and row tile q holds rows (q % CH) * 128 .. of query head q / CH)
  long long N, q_pos0;
  int U, NT, RPU, grid;        // units, tiles per unit, runs per unit, CTAs
  int RT;                      // tiles per run
  int step_u, step_j;          // grid = step_u * RPU + step_j: how a CTA's next run moves (unit, run in unit)
  int step_l, step_b, step_h, step_q;  // step_u = ((step_l * Bt + step_b) * Hkv + step_h) * QT + step_q
  unsigned int total_runs;     // U * RPU
  int shift;                   // tiles by which the pass-2 stream trails the pass-1 stream
  float sl2e;                  // scale * log2(e)
  int agg_group;
  unsigned long long wait_limit_ns;   // bound of every device-side wait
  int withhold_unit;           // test hook: the statistics of this unit are never sent (-1: none), so that
                               // the waits for them run into their bound
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
// Per-CTA control block in shared memory.
struct Ctl {
  int abort;                       // set by the first wait of this CTA that gives up
  int pad;
  unsigned long long limit_ns;     // bound of every wait
  const int* grid_status;          // the device status word (may be null): non-zero once any CTA gave up
};
// Called from the slow part of every wait loop: has this CTA, or any other, given up, or has this
// wait lasted longer than the bound?  (Then it marks the CTA as aborted.)
__device__ __noinline__ bool give_up(volatile Ctl* ctl, unsigned long long t0) {
  if (ctl->abort) return true;
  const int* gs = ctl->grid_status;
  if (gs != nullptr && *reinterpret_cast<const volatile int*>(gs) != 0) { ctl->abort = 1; return true; }
  if (globaltimer_ns() - t0 > ctl->limit_ns) { ctl->abort = 1; return true; }
  return false;
}
// Bounded wait.  Returns false when the CTA has given up (see give_up).  The retry loop is kept
// out of line: the kernel's hot loops have to stay small enough for the instruction cache.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile Ctl* ctl) {
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 1023u) == 0 && give_up(ctl, t0)) return false;
  }
  return true;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile Ctl* ctl) {
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, ctl);
}
// The same for a copy or an MMA that has been issued and therefore completes whatever the rest
// of the grid does: only the time bound ends this wait early, not the abort flag.
__device__ __noinline__ bool mbar_wait_issued(uint32_t bar, uint32_t parity, volatile Ctl* ctl) {
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 1023u) == 0 && globaltimer_ns() - t0 > ctl->limit_ns) { ctl->abort = 1; return false; }
  }
  return true;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3, unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4, unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_prefetch_5d(const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4) {
  asm volatile("cp.async.bulk.prefetch.tensor.5d.L2.global.tile [%0, {%1, %2, %3, %4, %5}];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
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
// 32 consecutive accumulator columns of this thread's TMEM lane; the caller waits for the load.
__device__ __forceinline__ void tc_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
// Wait for a TMEM load, tied to the registers it filled: the compiler may not use them before it.
__device__ __forceinline__ void tc_wait_ld(uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.wait::ld.sync.aligned;"
      : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
        "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
        "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
        "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
      :: "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Two fp32 lanes in one 64-bit register (Blackwell packed fp32 arithmetic).
__device__ __forceinline__ unsigned long long pack2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ unsigned long long pack2u(uint32_t a, uint32_t b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long p, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(p));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ void named_bar(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// (release: what this thread wrote before -- the run's record of the row -- is visible to whoever
// acquires a value of the word that includes this addition)
__device__ __forceinline__ void red_add_release_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void red_add_relaxed_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void red_or_relaxed_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.relaxed.gpu.global.or.b64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
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

// (reference, sum) pairs of the same row: fold (m, l) into (M, Ls).  Exponents are base 2.
__device__ __forceinline__ void combine(float& M, float& Ls, float m, float l) {
  const float Mn = fmaxf(M, m);
  if (Mn > -INFINITY) Ls = Ls * ex2(M - Mn) + l * ex2(m - Mn);
  M = Mn;
}

// ------------------------------------------------------------------------------------------------
// The static per-CTA sequence.  Stream position idx -> (run ordinal, tile); a run is RT
// consecutive tiles of one unit, runs are dealt to the CTAs round-robin.
// ------------------------------------------------------------------------------------------------
// Walks one stream of this CTA: position -> (run, tile).  Run k of the CTA is the global run
// blockIdx.x + k * grid; the cursor moves from run to run by additions only (the per-run
// increments come from the host), because a division would queue behind the exponentials in the
// special-function pipe.
struct Cursor {
  int t;            // position inside the run, 0 .. RT-1
  int u, j;         // unit, run inside the unit
  int l, b, h, q;   // the unit's layer, sequence, KV head, row tile
  __device__ __forceinline__ void init(const FastParams& P) {
    t = 0;
    u = (int)(blockIdx.x / (unsigned int)P.RPU);
    j = (int)(blockIdx.x - (unsigned int)u * (unsigned int)P.RPU);
    const int uh = u / P.QT;
    q = u - uh * P.QT;
    const int lb = uh / P.Hkv;
    h = uh - lb * P.Hkv;
    l = lb / P.Bt;
    b = lb - l * P.Bt;
  }
  // window rows of this unit's row tile (whole query heads; the last tile of a KV head may be short)
  // (kLong: the instantiation that also handles windows longer than 128 rows, CH > 1; everywhere else
  // that case is compiled out of the hot loops)
  template <bool kLong>
  __device__ __forceinline__ int rows(const FastParams& P) const {
    return (!kLong || P.CH == 1) ? min(P.HPT, P.G - q * P.HPT) * P.w : min(kRows, P.w - (q % P.CH) * kRows);
  }
  // first window row of this row tile inside its query head, and the tile's first query head in the group
  template <bool kLong>
  __device__ __forceinline__ int row0(const FastParams& P) const { return (!kLong || P.CH == 1) ? 0 : (q % P.CH) * kRows; }
  template <bool kLong>
  __device__ __forceinline__ int head0(const FastParams& P) const { return (!kLong || P.CH == 1) ? q * P.HPT : q / P.CH; }
  // index of the (layer, sequence, KV head)
  __device__ __forceinline__ int kv_unit(const FastParams& P) const { return (l * P.Bt + b) * P.Hkv + h; }
  __device__ __forceinline__ int tile(const FastParams& P) const { return j * P.RT + t; }
  __device__ __forceinline__ bool valid(const FastParams& P) const { return tile(P) < P.NT; }
  // last valid tile of its run
  __device__ __forceinline__ bool last(const FastParams& P) const { return t == P.RT - 1 || tile(P) + 1 >= P.NT; }
  __device__ __forceinline__ void next_run(const FastParams& P) {
    j += P.step_j;
    int c = 0;
    if (j >= P.RPU) { j -= P.RPU; c = 1; }
    u += P.step_u + c;
    q += P.step_q + c; c = 0;
    if (q >= P.QT) { q -= P.QT; c = 1; }
    h += P.step_h + c; c = 0;
    if (h >= P.Hkv) { h -= P.Hkv; c = 1; }
    b += P.step_b + c; c = 0;
    if (b >= P.Bt) { b -= P.Bt; c = 1; }
    l += P.step_l + c;
  }
  __device__ __forceinline__ void advance(const FastParams& P) {
    if (++t == P.RT) { t = 0; next_run(P); }
  }
};

// A ring position with its mbarrier phase bit.
struct Ring {
  int i, phase;
  __device__ __forceinline__ void next(int n) { if (++i == n) { i = 0; phase ^= 1; } }
};

template <int D>
struct SmemLayout {
  static constexpr int kHalves = D / 64;
  static constexpr int kTileBytes = kTile * D * 2;
  static constexpr int kStages = (D == 128) ? 4 : 8;
  static constexpr int kQ = 0;                                 // Q ring
  static constexpr int kK = kQSlots * kTileBytes;              // K stage ring
  static constexpr int kMisc = kK + kStages * kTileBytes;
  static constexpr int kBarKFull = kMisc;                      // kStages x 8
  static constexpr int kBarKEmpty = kBarKFull + 8 * kStages;
  static constexpr int kBarTFull = kBarKEmpty + 8 * kStages;   // 4 x 8
  static constexpr int kBarTEmpty = kBarTFull + 32;
  static constexpr int kBarQFull = kBarTEmpty + 32;            // kQSlots x 8
  static constexpr int kBarQFree = kBarQFull + 8 * kQSlots;
  static constexpr int kBarMmaDone = kBarQFree + 8 * kQSlots;  // 2 x 8
  static constexpr int kTmemSlot = kBarMmaDone + 16;           // 4 B (+ padding)
  static constexpr int kCtl = kTmemSlot + 8;                   // Ctl, 24 B
  static constexpr int kNegLse = (kCtl + 24 + 15) / 16 * 16;   // 128 floats, read as 16-byte vectors:
                                                               // -log-sum-exp of the pass-2 unit
  static constexpr int kStats = kNegLse + kRows * 4;           // 128 rows x float2: the upper half's statistics
  static constexpr int kTotal = kStats + kRows * 8;
  static_assert(kCtl % 8 == 0 && kNegLse % 16 == 0 && kStats % 8 == 0 && kTotal <= 232448, "shared-memory layout");
};

// The pushed statistics of one row (see FastParams::acc).
constexpr int kAccFracBits = 20;                              // the sum counts units of 2^-20
constexpr float kAccLimitLog2 = 20.f;                         // a run's contribution must stay below 2^20
constexpr unsigned long long kAccArrival = 1ull << 56, kAccOverflow = 1ull << 48;
constexpr unsigned long long kAccSumMask = kAccOverflow - 1;

// Bounded poll of a row's pushed statistics until all `runs` runs of the unit have arrived.
__device__ __noinline__ unsigned long long poll_acc_slow(const unsigned long long* src, unsigned int runs,
                                                         volatile Ctl* ctl) {
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  unsigned long long v;
  while ((unsigned int)((v = ld_relaxed_u64(src)) >> 56) != runs) {
    __nanosleep(100);
    if ((++spins & 255u) == 0 && give_up(ctl, t0)) break;
  }
  return v;
}

// ------------------------------------------------------------------------------------------------
// Cold paths, out of line: tiles that touch the causal boundary or the end of the context, and
// the aggregator variants other than the paper's defaults.
// ------------------------------------------------------------------------------------------------

// Pass 1, 64 columns (tokens c_first ..) of this thread's query row, with masking: the row's
// (reference, sum) follows the running maximum.  Reads the accumulator itself.
__device__ __noinline__ void p1_masked_half(uint32_t taddr, long long c_first, long long row_vis, float sl2e,
                                            float* mref_io, float* lsum_io) {
  float mref = *mref_io, lsum = *lsum_io;
#pragma unroll 1
  for (int part = 0; part < 2; ++part) {
    uint32_t r[32];
    tc_ld32_nowait(taddr + part * 32, r);
    tc_wait_ld(r);
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      v[i] = __uint_as_float(r[i]);
      if (c_first + part * 32 + i > row_vis) v[i] = -INFINITY;
    }
    float x0 = v[0], x1 = v[1];
#pragma unroll
    for (int i = 2; i < 32; i += 2) { x0 = max3(x0, v[i], v[i + 1]); }
    const float m_new = fmaxf(mref, fmaxf(x0, x1) * sl2e);
    if (m_new > -INFINITY) {
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
      for (int i = 0; i < 32; i += 4) {
        a0 += ex2(fmaf(v[i + 0], sl2e, -m_new));
        a1 += ex2(fmaf(v[i + 1], sl2e, -m_new));
        a2 += ex2(fmaf(v[i + 2], sl2e, -m_new));
        a3 += ex2(fmaf(v[i + 3], sl2e, -m_new));
      }
      lsum = lsum * ex2(mref - m_new) + ((a0 + a1) + (a2 + a3));
      mref = m_new;
    }
  }
  *mref_io = mref;
  *lsum_io = lsum;
}

// Pass 2, one token (this thread's TMEM lane) against all query rows, any aggregator, with
// masking.  Returns the group aggregate before the division of the mean.  W is the window length
// where it is one of the specialised powers of two, 0 where it is only known at run time (`w`).
template <int W, bool kTaskMean>
__device__ __noinline__ float p2_generic_tile(uint32_t taddr, const float* neg_lse, int n_chunks, int R, float sl2e,
                                              bool full, long long m_min, int agg_group, int w) {
  float gacc = (agg_group == KVC_AGG_MAX) ? -INFINITY : 0.f;
  float hacc = kTaskMean ? 0.f : -INFINITY;
  int m = 0;                                                             // row inside its query head (W == 0)
#pragma unroll 1
  for (int j = 0; j < n_chunks; ++j) {
    uint32_t r[32];
    tc_ld32_nowait(taddr + j * 32, r);
    tc_wait_ld(r);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int col = j * 32 + i;
      float xi = fmaf(__uint_as_float(r[i]), sl2e, neg_lse[col]);       // log2 of the attention weight
      bool head_done;
      if (W > 0) {
        constexpr int Wd = W > 0 ? W : 1;
        if (!full && (col % Wd) < m_min) xi = -INFINITY;
        head_done = (col + 1) % Wd == 0;
      } else {
        if (!full && m < m_min) xi = -INFINITY;
        head_done = ++m == w;
        if (head_done) m = 0;
      }
      if (kTaskMean) hacc += ex2(xi); else hacc = fmaxf(hacc, xi);
      if (head_done) {                                                   // a query head is complete
        if (col < R) {
          const float s_task = kTaskMean ? hacc / (float)w : ex2(hacc);
          gacc = (agg_group == KVC_AGG_MAX) ? fmaxf(gacc, s_task) : gacc + s_task;
        }
        hacc = kTaskMean ? 0.f : -INFINITY;
      }
    }
  }
  return gacc;
}

// Pass 2, one token against the R rows of one query head that this row tile holds (windows longer
// than 128 rows), with masking: rows below m_min do not see the token.  Returns the tile's part of
// Eq. 14 for the token: the largest attention weight, or the sum of the weights, over these rows.
template <bool kTaskMean>
__device__ __noinline__ float p2_long_tile(uint32_t taddr, const float* neg_lse, int n_chunks, int R, float sl2e,
                                           bool full, long long m_min) {
  float hacc = kTaskMean ? 0.f : -INFINITY;
#pragma unroll 1
  for (int j = 0; j < n_chunks; ++j) {
    uint32_t r[32];
    tc_ld32_nowait(taddr + j * 32, r);
    tc_wait_ld(r);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int col = j * 32 + i;
      float xi = fmaf(__uint_as_float(r[i]), sl2e, neg_lse[col]);       // log2 of the attention weight
      if (col >= R || (!full && col < m_min)) xi = -INFINITY;
      if (kTaskMean) hacc += ex2(xi); else hacc = fmaxf(hacc, xi);
    }
  }
  return kTaskMean ? hacc : ex2(hacc);
}

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
template <int D, int W, bool kTaskMean>
__global__ void __launch_bounds__(kFastThreads, 1)
score_sm100_kernel(const __grid_constant__ FastParams P) {
  using SL = SmemLayout<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile Ctl* ctl = reinterpret_cast<volatile Ctl*>(smem + SL::kCtl);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SL::kTmemSlot);

  auto bar_kfull = [&](int s) { return sbase + SL::kBarKFull + 8 * s; };
  auto bar_kempty = [&](int s) { return sbase + SL::kBarKEmpty + 8 * s; };
  auto bar_tfull = [&](int b) { return sbase + SL::kBarTFull + 8 * b; };
  auto bar_tempty = [&](int b) { return sbase + SL::kBarTEmpty + 8 * b; };
  auto bar_qfull = [&](int q) { return sbase + SL::kBarQFull + 8 * q; };
  auto bar_qfree = [&](int q) { return sbase + SL::kBarQFree + 8 * q; };
  auto bar_mma_done = [&](int p) { return sbase + SL::kBarMmaDone + 8 * p; };

  const bool aligned = (sbase & 1023u) == 0;     // the swizzled tiles need a 1024-byte aligned base
  if (threadIdx.x == 0) {
    for (int s = 0; s < SL::kStages; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_kempty(s), 2); }
    // the accumulators of pass 1 are read by eight warps (two column halves), those of pass 2 by four
    for (int b = 0; b < 4; ++b) { mbar_init(bar_tfull(b), 1); mbar_init(bar_tempty(b), b < 2 ? 8 : 4); }
    for (int q = 0; q < kQSlots; ++q) { mbar_init(bar_qfull(q), 1); mbar_init(bar_qfree(q), 2); }
    mbar_init(bar_mma_done(0), 1); mbar_init(bar_mma_done(1), 1);
    ctl->abort = 0;
    ctl->limit_ns = P.wait_limit_ns;
    ctl->grid_status = P.status;
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
  grid_dependency_wait();      // everything above overlapped the end of the kernel before this one

  // this CTA's share of the runs and the length of its sequence
  // (the host keeps all of these below 2^31)
  int my_runs = (P.total_runs > blockIdx.x) ? (int)((P.total_runs - blockIdx.x + P.grid - 1) / P.grid) : 0;
  if (!aligned) {
    if (threadIdx.x == 0 && P.status) atomicCAS(P.status, 0, (int)KVC_ERR_CUDA);
    my_runs = 0;               // nothing is computed; the teardown below still frees the TMEM columns
  }
  const int my_tiles = my_runs * P.RT;                  // stream length (some positions hold no tile)
  const int n_steps = my_tiles > 0 ? my_tiles + P.shift : 0;
  constexpr bool kLong = (W == 0);   // only the run-time window variant has windows longer than 128 rows
  // the whole box arrives (rows outside the tensor as zeros)
  const uint32_t q_bytes = (uint32_t)((!kLong || P.CH == 1) ? P.HPT * P.w : kRows) * D * 2;
  const long long vis_all = min(P.N - 1, P.q_pos0);          // tokens up to here are seen by every row

  // (The order of the roles in the code is not neutral: their hot loops share the instruction caches,
  // and this order measured fastest.)
  if (warp >= 8) {
    // ============================== pass-1 epilogue ============================================
    const int half = (warp - 8) >> 2;                 // which 64 columns (tokens) of every tile
    const int quarter = warp & 3;                     // TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;              // TMEM lane = query row
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float2* stage = reinterpret_cast<float2*>(smem + SL::kStats) + row;
    const int row_m = row % (W > 0 ? W : P.w);        // the row inside its query head (windows of up to 128 rows)
    const unsigned long long scale2 = pack2(P.sl2e, P.sl2e);

    int n1 = 0;
    float mref = -INFINITY, lsum = 0.f;               // sum over the run so far of 2^(logit - mref)
    float row_ref = 0.f;                              // the row's reference exponent for the pushed sum
    bool ok = true;

    // 32 unmasked logits against the row's current reference: no maximum, packed arithmetic.
    // Any logit of the row will do as a reference; if a chunk's sum leaves the range of fp32
    // the reference is moved up by 64 and the chunk is summed again.
    auto fast_chunk = [&](const uint32_t (&r)[32]) {
      if (mref == -INFINITY) mref = __uint_as_float(r[0]) * P.sl2e;
#pragma unroll 1
      for (int attempt = 0; attempt < 8; ++attempt) {
        const unsigned long long neg_ref = pack2(-mref, -mref);
        unsigned long long acc0 = 0ull, acc1 = 0ull;      // +0.0f twice
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const unsigned long long y0 = fma2(pack2u(r[i], r[i + 1]), scale2, neg_ref);
          const unsigned long long y1 = fma2(pack2u(r[i + 2], r[i + 3]), scale2, neg_ref);
          float a, b, c, d;
          unpack2(y0, a, b);
          unpack2(y1, c, d);
          acc0 = add2(acc0, pack2(ex2(a), ex2(b)));
          acc1 = add2(acc1, pack2(ex2(c), ex2(d)));
        }
        float s0, s1, s2, s3;
        unpack2(acc0, s0, s1);
        unpack2(acc1, s2, s3);
        const float sum = (s0 + s1) + (s2 + s3);
        if (sum < kRescaleLimit) { lsum += sum; break; }   // (false for inf / NaN as well)
        mref += 64.f;
        lsum *= 5.421010862427522e-20f;                    // 2^-64
      }
    };

    Cursor c;
    c.init(P);
    for (int idx = 0; idx < my_tiles; ++idx, c.advance(P)) {
      if (!c.valid(P)) continue;
      const int tile = c.tile(P);
      const bool run_ends = c.last(P);
      const bool row_used = row < c.template rows<kLong>(P);
      if (c.t == 0 && half == 0) row_ref = __ldg(P.ref + (long long)c.u * kRows + row);   // used at the run's end
      const int buf = n1 & 1;
      // (the TMEM loads below are warp-wide instructions: the decision has to be the warp's)
      ok = __all_sync(0xffffffffu, ok && mbar_wait(bar_tfull(buf), (uint32_t)((n1 >> 1) & 1), ctl));
      ++n1;
      if (ok) {
        tc_fence_after();
        const long long c0 = (long long)tile * kTile + half * 64;
        const bool full = (long long)tile * kTile + kTile - 1 <= vis_all;       // no masking anywhere in the tile
        const uint32_t taddr = lane_addr + (uint32_t)buf * kTile + half * 64;
        if (full) {
          uint32_t ra[32], rb[32];
          tc_ld32_nowait(taddr, ra);
          tc_ld32_nowait(taddr + 32, rb);
          tc_wait_ld(ra);
          tc_wait_ld(rb);
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tempty(buf));    // the accumulator is in registers now
          if (row_used) { fast_chunk(ra); fast_chunk(rb); }
        } else {
          float m2 = mref, l2 = lsum;                     // (the whole warp takes part in the TMEM loads)
          const long long row_vis = min(P.N - 1, P.q_pos0 + ((!kLong || P.CH == 1) ? row_m : c.template row0<kLong>(P) + row));   // last key this row sees
          p1_masked_half(taddr, c0, row_vis, P.sl2e, &m2, &l2);
          if (row_used) { mref = m2; lsum = l2; }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tempty(buf));
        }
      }
      if (run_ends) {
        // the two halves of every row meet through shared memory; the lower half's warps send the
        // run's sum of every row
        if (half == 1) *stage = make_float2(row_used ? mref : -INFINITY, row_used ? lsum : 0.f);
        named_bar(3, 256);
        const float2 other = *stage;
        named_bar(3, 256);                                // the stage may be written again
        if (half == 0 && ok && c.u != P.withhold_unit) {
          float M = row_used ? mref : -INFINITY, Ls = row_used ? lsum : 0.f;
          combine(M, Ls, other.x, other.y);
          // the short way: add the run's sum, rescaled to the row's fixed reference, to the row's
          // 64-bit word (integer addition: the total does not depend on the order)
          unsigned long long* word = P.acc + (long long)c.u * kRows + row;
          const float lv = lg2(Ls) + (M - row_ref);                     // log2 of the contribution
          if (!(Ls > 0.f)) {
            red_add_relaxed_u64(word, kAccArrival);
          } else if (lv < kAccLimitLog2) {
            red_add_relaxed_u64(word, kAccArrival + __float2ull_rn(ex2(lv + (float)kAccFracBits)));
          } else {
            // it does not fit: the run's record and its bit in the row's bitmap, then the arrival with
            // release semantics, so that both are visible to whoever acquires the complete word
            P.partial[((long long)c.u * P.RPU + c.j) * kRows + row] = make_float2(M, Ls);
            red_or_relaxed_u64(P.ovf + ((long long)c.u * kRows + row) * 4 + (c.j >> 6), 1ull << (c.j & 63));
            red_add_release_u64(word, kAccArrival + kAccOverflow);
          }
        }
        mref = -INFINITY; lsum = 0.f;
      }
    }
  } else if (warp >= 4 && warp < 8) {
    // ============================== pass-2 epilogue ============================================
    const int quarter = warp & 3;
    const int trow = quarter * 32 + lane;             // TMEM lane = token inside the tile; also 0..127 in the group
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float* neg_lse = reinterpret_cast<float*>(smem + SL::kNegLse);
    const unsigned long long scale2 = pack2(P.sl2e, P.sl2e);
    int n2 = 0;
    bool ok = true;
    // per-tile work is kept to a minimum here: this group's instruction stream is what the kernel waits for
    const bool gmax = P.agg_group == KVC_AGG_MAX;
    const float inv_g = (P.QT == 1 && !gmax) ? 1.f / (float)P.G : 1.f;   // one row tile: the mean of Eq. 15 is finished here
    const int vis_all_i = (int)vis_all;                // (N < 2^30)
    const int n_ctx = (int)P.N;
    int rows_u = 0, n_chunks = 0;                      // of the current run's unit
    float* score_row = nullptr;                        // where that unit's scores (or partial aggregates) go

    Cursor cu;
    cu.init(P);
    unsigned long long early_word = 0ull;             // a coming run's pushed word and reference, fetched ahead
    float early_ref = 0.f;
    int early_u = -1;                                 // ... and the unit they belong to
    if (my_tiles > 0) {
      early_word = ld_relaxed_u64(P.acc + (long long)cu.u * kRows + trow);
      early_ref = __ldg(P.ref + (long long)cu.u * kRows + trow);
      early_u = cu.u;
    }
    for (int idx = 0; idx < my_tiles; ++idx, cu.advance(P)) {
      if (!cu.valid(P)) continue;
      const int tok0 = cu.tile(P) * kTile;             // first token of the tile
      if (cu.t == 0) {
        rows_u = cu.template rows<kLong>(P);
        n_chunks = (rows_u + 31) / 32;
        score_row = P.scores + ((long long)cu.q * ((long long)P.L * P.Bt * P.Hkv) + cu.kv_unit(P)) * P.N;
        // a new run: its unit's log-sum-exp.  The short way: the row's pushed word, complete once
        // every run of the unit has arrived (fetched a tile or two ago; polled if it was not
        // complete then).  If a run's sum did not fit, the runs' records decide.
        float lse = 0.f;
        if (ok && trow < rows_u) {
          bool pushed = false;
          {
            if (early_u != cu.u) { early_word = 0ull; early_ref = __ldg(P.ref + (long long)cu.u * kRows + trow); }
            unsigned long long word = early_word;
            if ((unsigned int)(word >> 56) != (unsigned int)P.RPU)
              word = poll_acc_slow(P.acc + (long long)cu.u * kRows + trow, (unsigned int)P.RPU, ctl);
            const unsigned long long sum = word & kAccSumMask;
            if (((word >> 48) & 0xffull) == 0 && sum != 0) {
              lse = early_ref + lg2((float)sum) - (float)kAccFracBits;
              pushed = true;
            }
          }
          if (!pushed) {
            // the long way: all runs have arrived (the count in the word); those whose sum did not fit
            // wrote a record and set their bit before their release.  Fold them, in run order (the same
            // order for every reader), into the fixed-point sum of the others.
            asm volatile("fence.acq_rel.gpu;" ::: "memory");
            const unsigned long long word = ld_relaxed_u64(P.acc + (long long)cu.u * kRows + trow);
            const unsigned long long sum = word & kAccSumMask;
            float M = -INFINITY, Ls = 0.f;
            if (sum != 0) { M = early_ref; Ls = (float)sum * 9.5367431640625e-07f; }       // 2^-20
            const float2* rec = P.partial + (long long)cu.u * P.RPU * kRows + trow;
            const unsigned long long* bits_of = P.ovf + ((long long)cu.u * kRows + trow) * 4;
#pragma unroll 1
            for (int wi = 0; wi < 4; ++wi) {
              unsigned long long bits = __ldcg(bits_of + wi);
              while (bits) {
                const int j = wi * 64 + __ffsll((long long)bits) - 1;
                bits &= bits - 1;
                const float2 v = __ldcg(rec + (long long)j * kRows);
                combine(M, Ls, v.x, v.y);
              }
            }
            lse = M + log2f(Ls);
          }
        }
        early_u = -1;
        named_bar(1, 128);                             // everyone is done with the previous unit's values
        neg_lse[trow] = (trow < rows_u) ? -lse : 0.f;
        named_bar(1, 128);
        ok = !__any_sync(0xffffffffu, ctl->abort != 0) && ok;
      }
      if (early_u < 0 && cu.t >= P.RT - 2 && idx + (P.RT - cu.t) < my_tiles) {
        // the next run's word and reference: in flight while the rest of this run is computed
        Cursor nx = cu;
        nx.next_run(P);
        early_word = ld_relaxed_u64(P.acc + (long long)nx.u * kRows + trow);
        early_ref = __ldg(P.ref + (long long)nx.u * kRows + trow);
        early_u = nx.u;
      }
      const int buf = 2 + (n2 & 1);
      const uint32_t tmem_col = (uint32_t)buf * kTile;
      // (the TMEM loads below are warp-wide instructions: the decision has to be the warp's)
      ok = __all_sync(0xffffffffu, ok && mbar_wait(bar_tfull(buf), (uint32_t)((n2 >> 1) & 1), ctl));
      ++n2;
      if (!ok) continue;
      tc_fence_after();
      const int c = tok0 + trow;                                     // this thread's token
      const bool full = tok0 + kTile - 1 <= vis_all_i;
      float gacc;
      if (!kTaskMean && W >= 32 && full) {
        // the paper's default (max over the window) on a tile no mask touches: every 32-column
        // chunk belongs to one query head
        gacc = gmax ? -INFINITY : 0.f;
        float hacc = -INFINITY;
        uint32_t r[32];
        tc_ld32_nowait(lane_addr + tmem_col, r);
        auto chunk = [&](const int j, const bool last) {
          // the rows' -log-sum-exp for this chunk, fetched while the accumulator load is in flight
          ulonglong2 nl[8];
          {
            const ulonglong2* l2 = reinterpret_cast<const ulonglong2*>(neg_lse + j * 32);
#pragma unroll
            for (int i = 0; i < 8; ++i) nl[i] = l2[i];
          }
          tc_wait_ld(r);
          float x[32];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const unsigned long long y0 = fma2(pack2u(r[4 * i], r[4 * i + 1]), scale2, nl[i].x);
            const unsigned long long y1 = fma2(pack2u(r[4 * i + 2], r[4 * i + 3]), scale2, nl[i].y);
            unpack2(y0, x[4 * i], x[4 * i + 1]);                     // log2 of the attention weights
            unpack2(y1, x[4 * i + 2], x[4 * i + 3]);
          }
          if (!last) {
            tc_ld32_nowait(lane_addr + tmem_col + (j + 1) * 32, r);
          } else {
            tc_fence_before();                                        // the accumulator has been read
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty(buf));
          }
          float a = x[0], b = x[1];
#pragma unroll
          for (int i = 2; i < 30; i += 4) { a = max3(a, x[i], x[i + 1]); b = max3(b, x[i + 2], x[i + 3]); }
          hacc = max3(hacc, a, b);
          hacc = max3(hacc, x[30], x[31]);
          if (((j + 1) * 32) % (W > 0 ? W : 1) == 0) {
            const float s_task = ex2(hacc);
            gacc = gmax ? fmaxf(gacc, s_task) : gacc + s_task;
            hacc = -INFINITY;
          }
        };
#pragma unroll 1
        for (int j = 0; j < n_chunks; ++j) chunk(j, j + 1 == n_chunks);
      } else if (W == 0 && P.CH > 1) {
        // a window longer than 128 rows: the tile holds rows row0 .. of one query head and yields
        // that head's partial Eq. 14 (the maximum, or the sum, over these rows)
        gacc = p2_long_tile<kTaskMean>(lane_addr + tmem_col, neg_lse, n_chunks, rows_u, P.sl2e, full,
                                       (long long)c - P.q_pos0 - cu.template row0<kLong>(P));
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty(buf));
      } else {
        gacc = p2_generic_tile<W, kTaskMean>(lane_addr + tmem_col, neg_lse, n_chunks, rows_u, P.sl2e, full,
                                             (long long)c - P.q_pos0, P.agg_group, P.w);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty(buf));
      }
      // one row tile: the group aggregate itself; several: this tile's part of it
      if (c < n_ctx) score_row[c] = gacc * inv_g;
    }
  } else if (warp == 1 || warp == 2) {
    // ============================== MMA issuers ================================================
    // Both walk the whole sequence (the rings are shared and filled in sequence order) and each
    // issues the tiles of its own pass.  Each also waits for the fills that belong to the other
    // pass and acknowledges them: a parity wait is only meaningful for the phase that follows the
    // last one seen, so neither thread may skip a phase of a ring barrier, and the producer must
    // not refill a slot before both have seen its fill (the "empty" barriers count two arrivals:
    // the user's commit and the other thread's acknowledgement).
    if (lane == 0) {
      const int mine = warp - 1;       // the pass this thread issues
      Ring kr = {0, 0}, qr = {0, 0};
      Ring tb = {0, 0};                // accumulator buffer of this pass (two per pass)
      int nt = 0;                      // tiles issued (saturating at 2)
      int cur_slot = 0;
      bool ok = true;
      Cursor cur[2];
      cur[0].init(P); cur[1].init(P);
      for (int i = 0; i < n_steps && ok; ++i) {
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
          const int idx = pass == 0 ? i : i - P.shift;
          if (!ok || idx < 0 || idx >= my_tiles) continue;
          Cursor& c = cur[pass];
          if (c.valid(P)) {
            if (c.t == 0) {
              ok = mbar_wait(bar_qfull(qr.i), (uint32_t)qr.phase, ctl);
              if (pass == mine) cur_slot = qr.i;
              else if (ok) mbar_arrive(bar_qfree(qr.i));
            }
            if (ok) ok = mbar_wait(bar_kfull(kr.i), (uint32_t)kr.phase, ctl);
            if (ok && pass != mine) mbar_arrive(bar_kempty(kr.i));
            if (pass == mine) {
              const int buf = pass * 2 + tb.i;
              if (ok && nt >= 2) ok = mbar_wait(bar_tempty(buf), (uint32_t)(tb.phase ^ 1), ctl);
              if (ok) {
                tc_fence_after();
                const uint64_t dq0 = umma_desc(sbase + SL::kQ + cur_slot * SL::kTileBytes);
                const uint64_t dk0 = umma_desc(sbase + SL::kK + kr.i * SL::kTileBytes);
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * kTile;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                  // the start-address field counts 16-byte units: 64-element half, then 32 B per K step
                  const uint64_t off = (uint64_t)(((kk >> 2) * (kTile * 128) + (kk & 3) * 32) >> 4);
                  // pass 1: rows = query rows (A = Q), columns = tokens (B = K); pass 2: swapped
                  if (pass == 0) tc_mma_bf16(d_tmem, dq0 + off, dk0 + off, kIdesc, kk > 0);
                  else tc_mma_bf16(d_tmem, dk0 + off, dq0 + off, kIdesc, kk > 0);
                }
                tc_commit(bar_kempty(kr.i));   // the K stage may be refilled once these MMAs are done
                tc_commit(bar_tfull(buf));     // ... and the accumulator is then complete
                if (c.last(P)) tc_commit(bar_qfree(cur_slot));
                tb.next(2);
                if (nt < 2) ++nt;
              }
            }
            if (c.t == 0) qr.next(kQSlots);
            kr.next(SL::kStages);
          }
          c.advance(P);
        }
      }
      // no MMA may be in flight when the TMEM columns and the shared memory are given back
      if (nt > 0) {
        tc_commit(bar_mma_done(mine));
        mbar_wait_issued(bar_mma_done(mine), 0u, ctl);
      }
    }
  } else if (warp == 0) {
    // ============================== TMA producer ==============================================
    if (lane == 0) {
      unsigned long long pol_stream, pol_keep;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
      Ring kr = {0, 0}, qr = {0, 0};   // next K stage / Q slot to fill; phase = parity of the fill count / ring size
      int nk = 0, qc = 0;              // K tiles / Q tiles issued (saturating small counts are all that is needed)
      bool ok = true;
      Cursor cur[2], ahead;            // the two streams, and the pass-1 stream kPrefetch tiles ahead
      cur[0].init(P); cur[1].init(P); ahead.init(P);
      int ahead_pos = 0;
      auto prefetch_next = [&]() {
        if (ahead_pos >= my_tiles) return;
        if (ahead.valid(P)) {
          tma_prefetch_5d(P.k_maps + ahead.l, 0, ahead.tile(P) * kTile, 0, ahead.h, ahead.b);
        }
        ahead.advance(P);
        ++ahead_pos;
      };
      for (int i = 0; i < kPrefetch; ++i) prefetch_next();
      for (int i = 0; i < n_steps && ok; ++i) {
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
          const int idx = pass == 0 ? i : i - P.shift;
          if (!ok || idx < 0 || idx >= my_tiles) continue;
          Cursor& c = cur[pass];
          if (c.valid(P)) {
            if (c.t == 0) {                                    // a new run: its Q goes into the next ring slot
              if (qc >= kQSlots) ok = mbar_wait(bar_qfree(qr.i), (uint32_t)(qr.phase ^ 1), ctl);
              if (ok) {
                mbar_expect_tx(bar_qfull(qr.i), q_bytes);
                for (int hf = 0; hf < SL::kHalves; ++hf)
                  tma_load_4d(sbase + SL::kQ + qr.i * SL::kTileBytes + hf * (kTile * 128), P.q_maps + c.l,
                              bar_qfull(qr.i), hf * 64, c.template row0<kLong>(P), c.h * P.G + c.template head0<kLong>(P), c.b, pol_keep);
                qr.next(kQSlots);
                if (qc < kQSlots) ++qc;
              }
            }
            if (ok && nk >= SL::kStages) ok = mbar_wait(bar_kempty(kr.i), (uint32_t)(kr.phase ^ 1), ctl);
            if (ok) {
              mbar_expect_tx(bar_kfull(kr.i), SL::kTileBytes);
              // pass 1 leaves the rows in L2 for pass 2; pass 2 is their last use
              // (one copy for the whole tile: the 64-element halves of the rows are a dimension of the map)
              tma_load_5d(sbase + SL::kK + kr.i * SL::kTileBytes, P.k_maps + c.l, bar_kfull(kr.i), 0, c.tile(P) * kTile, 0,
                          c.h, c.b, pass == 0 ? pol_keep : pol_stream);
              kr.next(SL::kStages);
              if (nk < SL::kStages) ++nk;
            }
          }
          c.advance(P);
          if (pass == 0) prefetch_next();
        }
      }
      // drain: every issued copy must have landed before the CTA's shared memory is released
      // (an issued copy always completes, so these waits do not take the abort shortcut).
      // The last fill of stage i is complete once its full barrier has left the phase of that fill.
      for (int n = 0; n < nk; ++n) {
        // walk the ring backwards from the slot before kr
        int i2 = kr.i - 1 - n, ph = kr.phase;
        if (i2 < 0) { i2 += SL::kStages; ph ^= 1; }
        mbar_wait_issued(bar_kfull(i2), (uint32_t)ph, ctl);
      }
      for (int n = 0; n < qc; ++n) {
        int i2 = qr.i - 1 - n, ph = qr.phase;
        if (i2 < 0) { i2 += kQSlots; ph ^= 1; }
        mbar_wait_issued(bar_qfull(i2), (uint32_t)ph, ctl);
      }
    }
  }
  // (warp 3 has no role)

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && ctl->abort && P.status) atomicCAS(P.status, 0, (int)KVC_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// The rows' reference exponents: the scaled logit (base 2) of every window row against token 0 of
// its KV head, which every row sees.  Only a common scale for the pushed sums: a row's sum of
// 2^(logit - ref) is then at least about 1, so fixed point with 20 fractional bits keeps it.
// ------------------------------------------------------------------------------------------------
struct RefParams {
  int Bt, Hkv, G, HPT, QT, CH, w, d;
  unsigned long long* acc;     // [U][128]: cleared here
  unsigned long long* ovf;     // [U][128][4]: cleared here
  long long qs0, qs1, qs2, kvs0, kvs1;
  float sl2e;
};

__global__ void __launch_bounds__(kRows)
score_ref_kernel(RefParams P, LayerPtrs qp, LayerPtrs kp, float* __restrict__ ref) {
  grid_dependency_wait();
  const int u = blockIdx.x, row = threadIdx.x;
  // the unit's exchange state: empty words
  P.acc[(long long)u * kRows + row] = 0ull;
  {
    ulonglong2* o = reinterpret_cast<ulonglong2*>(P.ovf + ((long long)u * kRows + row) * 4);
    o[0] = make_ulonglong2(0ull, 0ull);
    o[1] = make_ulonglong2(0ull, 0ull);
  }
  const int uh = u / P.QT, qt = u - uh * P.QT;
  const int lb = uh / P.Hkv, h = uh - lb * P.Hkv;
  const int l = lb / P.Bt, b = lb - l * P.Bt;
  const int rows_u = P.CH == 1 ? min(P.HPT, P.G - qt * P.HPT) * P.w : min(kRows, P.w - (qt % P.CH) * kRows);
  float r = 0.f;
  if (row < rows_u) {
    const int j = P.CH == 1 ? h * P.G + qt * P.HPT + row / P.w : h * P.G + qt / P.CH;
    const int m = P.CH == 1 ? row % P.w : (qt % P.CH) * kRows + row;
    const __nv_bfloat16* qv = reinterpret_cast<const __nv_bfloat16*>(qp.p[l]) + b * P.qs0 + j * P.qs1 + m * P.qs2;
    const __nv_bfloat16* kv = reinterpret_cast<const __nv_bfloat16*>(kp.p[l]) + b * P.kvs0 + h * P.kvs1;
    // 16-byte pieces (rows are 16-byte aligned), all in flight at once; products added in order
    const uint4* q4 = reinterpret_cast<const uint4*>(qv);
    const uint4* k4 = reinterpret_cast<const uint4*>(kv);
    float acc = 0.f;
#pragma unroll 4
    for (int t = 0; t < P.d / 8; ++t) {
      const uint4 a = __ldg(q4 + t), b2 = __ldg(k4 + t);
      const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b2.x, b2.y, b2.z, b2.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        // a bf16 is the upper half of the fp32 with the same value
        acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
        acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
      }
    }
    r = acc * P.sl2e;
  }
  ref[(long long)u * kRows + row] = r;
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

bool encode_map(CUtensorMap* m, const void* base, int rank, const long long* dims, const long long* strides_bytes,
                const unsigned* box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gd[5]; cuuint64_t gs[4]; cuuint32_t bx[5]; cuuint32_t es[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < rank; ++i) { gd[i] = (cuuint64_t)dims[i]; bx[i] = box[i]; }
  for (int i = 0; i < rank - 1; ++i) gs[i] = (cuuint64_t)strides_bytes[i];
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct FastPlan {
  int U, NT, RPU, grid, RT;
  int HPT, QT, CH;             // query heads per row tile, row tiles per KV head, row tiles per query head
  long long total_runs, shift;
  size_t off_partial, off_parts, off_acc, off_ovf, off_ref, off_total;
};

// sms <= 0: no device yet (host-only size query) -- the workspace does not depend on it
void make_plan(const Problem& P, int sms, FastPlan* pl) {
  const int G = P.Hq / P.Hkv;
  if (P.w <= kRows) {
    pl->HPT = kRows / P.w < G ? kRows / P.w : G;
    pl->CH = 1;
    pl->QT = (G + pl->HPT - 1) / pl->HPT;
  } else {                      // a window longer than one accumulator: several row tiles per query head
    pl->HPT = 1;
    pl->CH = (P.w + kRows - 1) / kRows;
    pl->QT = G * pl->CH;
  }
  pl->U = P.L * P.Bt * P.Hkv * pl->QT;
  pl->NT = (int)((P.N + kTile - 1) / kTile);
  pl->RT = kMinRunTiles;
  if ((pl->NT + pl->RT - 1) / pl->RT > 255) pl->RT = (pl->NT + 254) / 255;   // the arrivals of a unit are counted in 8 bits
  pl->RPU = (pl->NT + pl->RT - 1) / pl->RT;
  pl->total_runs = (long long)pl->U * pl->RPU;
  pl->grid = sms > 0 ? (int)(pl->total_runs < sms ? pl->total_runs : sms) : 1;
  // pass 2 of a run starts once every CTA has been through the rest of the run's unit, at most
  // ceil(RPU / grid) runs later, and through one run more, which covers the exchange (the pushed
  // sums take two round trips to L2); the K rows of that many tiles are still in L2 then
  const long long lag_runs = (pl->RPU + pl->grid - 1) / pl->grid + 1;
  pl->shift = lag_runs * pl->RT + KVC_SCORE_LAG_TILES;
  size_t off = 0;
  pl->off_partial = off; off += align_up((size_t)pl->total_runs * kRows * sizeof(float2));
  pl->off_acc = off; off += align_up((size_t)pl->U * kRows * sizeof(unsigned long long));
  pl->off_ovf = off; off += align_up((size_t)pl->U * kRows * 4 * sizeof(unsigned long long));
  pl->off_ref = off; off += align_up((size_t)pl->U * kRows * sizeof(float));
  pl->off_parts = off;         // partial group aggregates [QT][L*Bt*Hkv][N], only with several row tiles
  if (pl->QT > 1) off += align_up((size_t)pl->U * P.N * sizeof(float));
  pl->off_total = off;
}

int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

// Test hooks (kvc_debug_score_hooks): the bound of the device-side waits and a unit whose
// statistics are withheld.
std::atomic<unsigned long long> g_wait_limit_ns{kDefaultWaitLimitNs};
std::atomic<int> g_withhold_unit{-1};

constexpr int kMaxDevices = 64;
std::mutex g_launch_mutex;

// The kernel's CTAs wait for one another, so all of them have to be resident at once: one per
// SM with the opt-in amount of shared memory.  Checked once per device and instantiation (the
// attribute is per device); KVC_ERR_UNSUPPORTED sends the caller to the CUDA-core path.
template <int D, int W, bool M>
kvc_status prepare_t(int grid) {
  using SL = SmemLayout<D>;
  static signed char state[kMaxDevices];      // 0: not looked at, 1: fits, -1: does not
  int dev = 0;
  KVC_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return KVC_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_launch_mutex);
  if (state[dev] == 0) {
    KVC_CUDA(cudaFuncSetAttribute(score_sm100_kernel<D, W, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kTotal));
    int per_sm = 0, sms = 0;
    KVC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, score_sm100_kernel<D, W, M>, kFastThreads,
                                                           (size_t)SL::kTotal));
    KVC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    state[dev] = (per_sm >= 1 && sms >= 1) ? 1 : -1;
  }
  (void)grid;                                 // grid <= SM count by construction (make_plan)
  return state[dev] == 1 ? KVC_OK : KVC_ERR_UNSUPPORTED;
}

template <int D, int W, bool M>
kvc_status launch_t(const FastParams& fp, int grid, cudaStream_t st) {
  using SL = SmemLayout<D>;
  const kvc_status s = prepare_t<D, W, M>(grid);
  if (s != KVC_OK) return s;
  KVC_CUDA(launch_dependent(score_sm100_kernel<D, W, M>, dim3(grid), dim3(kFastThreads), (size_t)SL::kTotal, st, fp));
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
    case 128: return launch_t<D, 128, M>(fp, grid, st);
    default: return launch_t<D, 0, M>(fp, grid, st);      // any other window length: known at run time only
  }
}

}  // namespace

// The descriptor alone: is this a shape the tensor-core kernel handles?
bool score_sm100_shape_ok(const Problem& P) {
  if (P.dtype != KVC_BF16 || !P.contiguous_groups) return false;
  if (P.w < 1) return false;
  if (P.L > kMaxFastLayers) return false;
  if (P.N >= (1LL << 30)) return false;
  FastPlan pl;
  make_plan(P, 0, &pl);
  if ((long long)P.L * P.Bt * P.Hkv * pl.QT > (1 << 24)) return false;
  if ((pl.total_runs + 4096) * pl.RT + pl.shift >= (1LL << 31)) return false;   // 32-bit sequence indices
  return true;
}

// ... and can its tensor maps be encoded here (a driver with the encoder is present)?
bool score_sm100_supported(const Problem& P) { return score_sm100_shape_ok(P) && encode_fn() != nullptr; }

size_t score_sm100_workspace_bytes(const Problem& P) {
  FastPlan pl;
  make_plan(P, 0, &pl);
  return pl.off_total;
}

// Returns KVC_ERR_UNSUPPORTED (without setting an error) when the tensor maps cannot be encoded
// for these strides; the caller then uses the CUDA-core path.
kvc_status launch_score_sm100(const Problem& P, const LayerPtrs& q, const LayerPtrs& k, float* scores,
                              int* device_status, void* ws, size_t ws_bytes, cudaStream_t st,
                              const float** parts_out, int* row_tiles_out, int* tiles_per_head_out) {
  const int sms = sm_count();
  if (sms < 1) return KVC_ERR_UNSUPPORTED;
  FastPlan pl;
  make_plan(P, sms, &pl);
  if (ws_bytes < pl.off_total) { set_error("score: workspace too small"); return KVC_ERR_WORKSPACE; }
  const int G = P.Hq / P.Hkv;
  static thread_local FastParams fp;
  for (int l = 0; l < P.L; ++l) {
    const long long kd[5] = {64, P.N, P.d / 64, P.Hkv, P.Bt};
    const long long ks[4] = {P.kvs[2] * 2, 128, P.kvs[1] * 2, P.kvs[0] * 2};
    const unsigned kb[5] = {64, (unsigned)kTile, (unsigned)(P.d / 64), 1, 1};
    const long long qd[4] = {P.d, P.w, P.Hq, P.Bt};
    const long long qs[3] = {P.qs[2] * 2, P.qs[1] * 2, P.qs[0] * 2};
    const unsigned qb[4] = {64, (unsigned)(pl.CH == 1 ? P.w : kRows), (unsigned)pl.HPT, 1};
    if (!encode_map(&fp.k_maps[l], k.p[l], 5, kd, ks, kb)) return KVC_ERR_UNSUPPORTED;
    if (!encode_map(&fp.q_maps[l], q.p[l], 4, qd, qs, qb)) return KVC_ERR_UNSUPPORTED;
  }
  char* w = reinterpret_cast<char*>(ws);

  fp.partial = reinterpret_cast<float2*>(w + pl.off_partial);
  fp.acc = reinterpret_cast<unsigned long long*>(w + pl.off_acc);
  fp.ovf = reinterpret_cast<unsigned long long*>(w + pl.off_ovf);
  float* ref = reinterpret_cast<float*>(w + pl.off_ref);
  fp.ref = ref;
  {
    RefParams rp;
    rp.acc = fp.acc;
    rp.ovf = fp.ovf;
    rp.Bt = P.Bt; rp.Hkv = P.Hkv; rp.G = G; rp.HPT = pl.HPT; rp.QT = pl.QT; rp.CH = pl.CH; rp.w = P.w; rp.d = P.d;
    rp.qs0 = P.qs[0]; rp.qs1 = P.qs[1]; rp.qs2 = P.qs[2]; rp.kvs0 = P.kvs[0]; rp.kvs1 = P.kvs[1];
    rp.sl2e = P.scale * kLog2eF;
    KVC_CUDA(launch_dependent(score_ref_kernel, dim3(pl.U), dim3(kRows), 0, st, rp, q, k, ref));
    KVC_LAUNCH_CHECK("score_ref_kernel");
  }
  fp.status = device_status;
  float* parts = pl.QT > 1 ? reinterpret_cast<float*>(w + pl.off_parts) : nullptr;
  fp.scores = pl.QT > 1 ? parts : scores;
  *parts_out = parts;
  *row_tiles_out = pl.QT;
  *tiles_per_head_out = pl.CH;
  fp.L = P.L; fp.Bt = P.Bt; fp.Hkv = P.Hkv; fp.G = G;
  fp.HPT = pl.HPT; fp.QT = pl.QT; fp.CH = pl.CH; fp.w = P.w;
  fp.N = P.N; fp.q_pos0 = P.q_pos0;
  fp.U = pl.U; fp.NT = pl.NT; fp.RPU = pl.RPU; fp.RT = pl.RT; fp.grid = pl.grid;
  fp.total_runs = (unsigned int)pl.total_runs; fp.shift = (int)pl.shift;
  fp.step_u = pl.grid / pl.RPU; fp.step_j = pl.grid % pl.RPU;
  fp.step_q = fp.step_u % pl.QT;
  fp.step_h = (fp.step_u / pl.QT) % P.Hkv;
  fp.step_b = (fp.step_u / pl.QT / P.Hkv) % P.Bt;
  fp.step_l = fp.step_u / pl.QT / P.Hkv / P.Bt;
  fp.sl2e = P.scale * kLog2eF;
  fp.agg_group = P.agg_group;
  fp.wait_limit_ns = g_wait_limit_ns.load();
  fp.withhold_unit = g_withhold_unit.load();
  const bool mean = P.agg_task == KVC_AGG_MEAN;
  if (P.d == 128) return mean ? launch_w<128, true>(P.w, fp, pl.grid, st) : launch_w<128, false>(P.w, fp, pl.grid, st);
  return mean ? launch_w<64, true>(P.w, fp, pl.grid, st) : launch_w<64, false>(P.w, fp, pl.grid, st);
}

}  // namespace kvc


// Test hook: the bound of the scoring kernel's device-side waits (<= 0: the default of 2 s) and a
// unit (layer, sequence, KV head, row tile in that order) whose statistics are never sent, so
// that the waits for them expire (-1: none).  Process-wide; takes effect at the next launch.
extern "C" __attribute__((visibility("default"))) void kvc_debug_score_hooks(int64_t wait_limit_ns,
                                                                             int32_t withhold_unit) {
  kvc::g_wait_limit_ns.store(wait_limit_ns > 0 ? (unsigned long long)wait_limit_ns : kvc::kDefaultWaitLimitNs);
  kvc::g_withhold_unit.store(withhold_unit);
}
