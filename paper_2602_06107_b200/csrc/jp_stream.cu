// Row-streaming kernels: each valid row of the actor and policy logits is read
// from HBM once; the pass yields both log-sum-exps (online reference exponent /
// rescaled sum), the sampled token's logits and the two top-k lists (Section 4.4.1:
// V_k is the union of top-k(p_inf) and top-k(p_new)), each candidate carrying both
// logits.  A second kernel sums the exact normaliser Z over the vocabulary
// (Eq. obrs_dist).
//
// Shape of the stream kernel (one persistent CTA per SM, one row pair at a time):
//
//   producer warp   one lane issues 1-D bulk async copies (global -> shared,
//                   completion counted on an mbarrier) of the next tile of both
//                   rows into a ring of shared-memory stages;
//   consumer warps  two groups that take alternate tiles of a row: wait for a stage,
//                   pull their 16-byte vectors into registers pass by pass (a pass
//                   is two vectors per tensor), add the terms to the online sums of
//                   both rows, compare the maximum of each pass with the row's running
//                   threshold tau, and free the stage once arithmetic has consumed the
//                   tile.  A pass at or above tau (a fraction of a percent) is appended
//                   to the row's candidate buffer: one atomic and one store;
//   top-k warps     eight of them, one per (row slot, tensor).  Before a row starts its
//                   warp reads a sample (the first vectors) of the row and publishes
//                   the k-th best vector maximum of the sample as the first tau: the
//                   k-th best of any subset is a lower bound of the row's k-th best
//                   logit.  While the row streams it counts the candidates into a
//                   histogram as they appear and raises tau to the highest bin with at
//                   least k of them at or above it (k different passes hold k different
//                   entries).  When the row is done it drops the candidates that tau
//                   has overtaken, reads the vectors of the others back, sorts their
//                   entries at or above tau into the list (bitonic sort / merge across
//                   the lanes), finishes the log-sum-exp, gathers the sampled token's
//                   logit and writes the row's record.  Candidates beyond the buffer
//                   go to a spill area in the workspace; a row with more than that
//                   holds too is read again by its warp (exact, slow, adversarial).
//
// Rows cycle through four "slots" (histogram, candidates, partial sums, barriers),
// so the consumers never wait for the top-k warps unless those fall three rows
// behind.  The total order of the top-k is (logit desc, index asc), one 64-bit key;
// the result does not depend on the order in which candidates arrive or on when tau
// was raised.
//
// Every mbarrier is waited on phase by phase by the same warps, each keeping its
// own phase bits: a parity wait cannot tell a phase not yet reached from one that
// is done, so a waiter that skipped phases could run ahead of the data.
//
// Every wait is bounded: a wait that runs out raises the CTA's abort flag, the
// status word gets JP_ERR_TIMEOUT and every warp leaves its loop.
#include <type_traits>

#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {

constexpr int NC = 16;                    // consumer warps
constexpr int NG = 2;                     // consumer groups: a row's tiles go to them in turn, starting with first_group(row)
constexpr int WPT = NC / NG;              // warps that share one tile
constexpr int VPL = 4;                    // 16-byte vectors per lane per tensor per tile
constexpr int TV = WPT * 32 * VPL;        // vectors per tensor per tile
constexpr int HV = 2;                     // vectors per tensor a lane holds at a time
static_assert(VPL % HV == 0, "a tile is taken in passes of HV vectors");
static_assert(NG == 2, "tiles go to consumer groups by parity; the producer keeps two phase masks");
static_assert(NC % NG == 0, "consumer groups must divide the warps");
constexpr int NSLOT = 4;                  // rows in flight between the consumers and the top-k warps
constexpr int SCAP = 288;                 // keys a top-k warp buffers before it sorts them into the list
constexpr int NB = 256;                   // histogram bins
constexpr int TP = TV / HV;               // passes per tensor per tile
constexpr int SAMPLE = 32 * 32;            // vectors of a row its top-k warp looks at before the row starts
constexpr int NTOPK = NSLOT * 2;          // top-k warps: (slot, tensor)
constexpr int NWARPS = 1 + NC + NTOPK;
constexpr int NTHREADS = NWARPS * 32;
constexpr long long kSpinLimit = 4000000000ll;   // clock cycles a wait may last (about 2 s)
constexpr uint32_t kTauPollNs = 200u;     // how long a top-k warp sleeps between two looks at its row's candidates

// NSTAGES: depth of the ring.  NCAND: candidate passes a row may collect before it
// falls back to a re-scan.  The kernel for k <= 64 takes 5 stages and 1024 candidates;
// for k <= 128 (about k (1 + ln(passes / k)) candidates per row) 4 stages and 2048.
// NT: tensors a stage holds.  With one tensor streamed (the sparse-actor forward) the ring has
// twice the stages of half the size: the same bytes in flight as with two tensors.
template <int NSTAGES, int NCAND, int NT>
struct __align__(128) StreamSmemT {
  static constexpr int STAGES = NSTAGES;
  static constexpr int TENSORS = NT;
  static constexpr int CAP = NCAND;
  static_assert(NG < NSTAGES, "every consumer group needs a stage of its own and one must be in flight");
  static_assert(SAMPLE <= NCAND, "the sample's vector maxima are parked in the candidate buffer");
  uint4 ring[STAGES][NT][TV];             // [stage][tensor][vector]
  unsigned long long skeys[NSLOT][2][SCAP];  // [slot][tensor] keys waiting to be sorted into the list
  uint32_t cand[NSLOT][2][CAP];           // [slot][tensor] candidate passes: high bits of the maximum's order bits | pass id; 0 = not written yet
  uint32_t hist[NSLOT][2][NB];            // [slot][tensor] candidate passes per bin of their maximum (kept by the top-k warp)
  unsigned long long full[NG][STAGES];    // [consumer group] producer -> that group: the tile's bytes have landed.  One set per
                                          // group, so that every waiter sees every phase of its barriers in turn: a group that
                                          // skipped the other group's phases could take an unfinished earlier phase for its own
  unsigned long long empty[STAGES];       // consumers -> producer: the stage may be refilled
  unsigned long long slot_ready[NSLOT];   // top-k warps -> consumers: the slot is set up for its next row
  unsigned long long row_done[NSLOT];     // consumers -> top-k warps: the row has been streamed
  float tau[NSLOT][2];                    // running threshold (only rises while a row streams)
  uint32_t ncand[NSLOT][2];               // candidate passes appended so far (may pass CAP: then the row is re-scanned)
  float part_mL[NSLOT][2][NC];
  float part_s[NSLOT][2][NC];
  uint32_t g0[NSLOT];                     // group that takes tile 0 of the slot's row
  int abort;
};

template <int KPL, bool SINGLE = false>
using StreamSmemFor = StreamSmemT<(KPL == 4 ? 4 : 5) * (SINGLE ? 2 : 1), (KPL == 4 ? 2048 : 1024), (SINGLE ? 1 : 2)>;
static_assert(sizeof(StreamSmemFor<1>) <= 232448 && sizeof(StreamSmemFor<4>) <= 232448 &&
                  sizeof(StreamSmemFor<1, true>) <= 232448 && sizeof(StreamSmemFor<4, true>) <= 232448,
              "the CTA's shared memory exceeds the 227 KB an sm_100 CTA can have");

// ---- mbarrier / bulk-copy wrappers ----------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Arrival that cannot be issued before `dep` has been computed: the value is an input
// of the statement, though the instruction does not use it.
__device__ __forceinline__ void mbar_arrive_after(unsigned long long* bar, uint32_t dep) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];  // after %1" ::"r"(smem_u32(bar)), "r"(dep) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Same, but the thread may stay suspended for up to `ns` nanoseconds before it answers.
__device__ __forceinline__ bool mbar_try_wait_for(unsigned long long* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}
// Bounded wait; false = gave up (or another warp did).  The first poll is inline;
// the loop is out of line (the streaming code stays small).  The clock is read once
// in 64 polls, each of which may itself suspend the thread for a while.
__device__ __noinline__ bool mbar_wait_slow(unsigned long long* bar, uint32_t parity, volatile int* abort,
                                            long long limit = kSpinLimit) {
  long long t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait_for(bar, parity, 2000u)) return true;
    if ((i & 63u) == 0u) {
      if (*abort) return false;
      const long long now = clock64();
      if (i == 0u) t0 = now;
      else if (now - t0 > limit) { *abort = 1; return false; }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, volatile int* abort) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort);
}
// The copy carries an L2 policy: the streamed tiles are marked "evict first", so that
// they do not push out the few lines that are read twice (a row's sample, read by its
// top-k warp shortly before the row streams).
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, unsigned long long* bar,
                                         unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ float lds_volatile_f32(const float* p) {
  float v;
  asm volatile("ld.volatile.shared.f32 %0, [%1];" : "=f"(v) : "r"(smem_u32(p)) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t lds_volatile_u32(const void* p) {
  uint32_t v;
  asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
  return v;
}
__device__ __forceinline__ void sts_volatile_f32(float* p, float v) {
  asm volatile("st.volatile.shared.f32 [%0], %1;" ::"r"(smem_u32(p)), "f"(v) : "memory");
}
__device__ __forceinline__ uint4 lds_volatile_v4(const void* p) {
  uint4 v;
  asm volatile("ld.volatile.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(smem_u32(p))
               : "memory");
  return v;
}

// ---- packed fp32x2 arithmetic (two lanes of one 64-bit register pair) ------
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long r, float& lo, float& hi) {
  asm("mov.b64 {%0,%1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ unsigned long long ffma2(unsigned long long a, unsigned long long b,
                                                    unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long fadd2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long fmul2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// 2^d for an integer-valued d <= 0, exact (built from the exponent field).
__device__ __forceinline__ float exp2_int(float d) {
  return d < -126.f ? 0.f : __int_as_float(((int)d + 127) << 23);
}

// (mL, s) pairs: s is a sum relative to 2^mL with mL an integer, so that moving a
// sum to another reference is an exact power-of-two scaling; mL == -inf marks an
// empty pair.
__device__ __forceinline__ void merge_scaled(float& mL, float& s, float mL2, float s2) {
  float M = fmaxf(mL, mL2);
  float a = (mL == JP_NEG_INF) ? 0.f : exp2_int(mL - M);
  float b = (mL2 == JP_NEG_INF) ? 0.f : exp2_int(mL2 - M);
  s = s * a + s2 * b;
  mL = M;
}

// Online softmax state of one thread for one tensor: an integer reference exponent
// mL and two partial sums (packed) of the terms 2^(z log2 e - mL).  The reference is
// set from the first maximum the thread meets and moves again only when a logit
// climbs more than kHeadroom binades above it (`lim` is that limit as a logit;
// -inf = nothing seen yet): terms stay below 2^kHeadroom, far from overflow, and
// anything more than 126 - kHeadroom binades below the row's maximum is below 2^-62
// of the sum.  Tracking the exact running maximum instead made a few lanes of almost
// every pass take the rescaling branch on their own.
constexpr float kHeadroom = 64.f;
struct Online {
  float lim, mL;
  unsigned long long s2;
};

// Makes sure the reference exponent covers a maximum vm: moves it (and the sums,
// by an exact power of two) when vm is beyond the limit.
__device__ __forceinline__ void raise_max(float vm, Online& o) {
  if (vm > o.lim) {
    const float nmL = ceilf(__fmul_rn(vm, kLog2e));
    if (o.lim != JP_NEG_INF) {
      const float f = exp2_int(o.mL - nmL);
      o.s2 = fmul2(o.s2, pack2(f, f));
    }
    o.mL = nmL;
    o.lim = __fmul_rn(nmL + kHeadroom, kLn2);
  }
}

// Adds the terms 2^(z log2 e - mL) of one 16-byte vector to the sums; the reference
// exponent already covers the vector.
template <int DT>
__device__ __forceinline__ void add_terms(const uint4& v, Online& o) {
  const unsigned long long L2 = pack2(kLog2e, kLog2e);
  const unsigned long long nm2 = pack2(-o.mL, -o.mL);
  if (DT == JP_BF16) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      unsigned long long a = ffma2(pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u)), L2, nm2);
      float a0, a1;
      unpack2(a, a0, a1);
      o.s2 = fadd2(o.s2, pack2(ex2_approx(a0), ex2_approx(a1)));
    }
  } else {
    unsigned long long a = ffma2(pack2(__uint_as_float(v.x), __uint_as_float(v.y)), L2, nm2);
    unsigned long long b = ffma2(pack2(__uint_as_float(v.z), __uint_as_float(v.w)), L2, nm2);
    float a0, a1, b0, b1;
    unpack2(a, a0, a1);
    unpack2(b, b0, b1);
    o.s2 = fadd2(o.s2, pack2(ex2_approx(a0), ex2_approx(a1)));
    o.s2 = fadd2(o.s2, pack2(ex2_approx(b0), ex2_approx(b1)));
  }
}

// One 16-byte vector, whose maximum is vm, into the online (max, sum).
template <int DT>
__device__ __forceinline__ void accumulate(const uint4& v, float vm, Online& o) {
  raise_max(vm, o);
  add_terms<DT>(v, o);
}

// Hands a ring stage back to the producer once this warp has consumed its part of the tile.
// The stage may be overwritten (by the copy engine) as soon as the arrival is counted, so
// every shared-memory load of the tile must have returned its value by then.  That is made
// a data dependence rather than a matter of instruction order: the running sums take in
// every loaded word, the vote below takes in the sums of all 32 lanes, and the arrival takes
// the vote's result as an operand.  A load whose value has been consumed has been performed,
// and the arrival (release) / the producer's wait (acquire) order the copy after it.
// (An arrival placed right after the loads was seen to overtake one that was still queued
// behind a burst of shared-memory atomics: the lane then read the next tile's bytes.)
__device__ __forceinline__ void release_stage(unsigned long long* empty_bar, const Online& oa, const Online& op,
                                              int lane) {
  const uint32_t mix = (uint32_t)oa.s2 ^ (uint32_t)(oa.s2 >> 32) ^ (uint32_t)op.s2 ^ (uint32_t)(op.s2 >> 32);
  const uint32_t vote = __ballot_sync(0xffffffffu, mix == 0x7fc00001u);   // any predicate of the sums will do
  if (lane == 0) mbar_arrive_after(empty_bar, vote);
}

// The ragged end of a row (fewer than one 16-byte vector) as a -inf padded vector.
template <int DT>
__device__ __forceinline__ uint4 load_tail_vector(const char* row, int64_t first, int tail) {
  uint4 v = Vec<DT>::neg_inf();
#pragma unroll
  for (int e = 0; e < Vec<DT>::N - 1; ++e)
    if (e < tail) Vec<DT>::set(v, e, Vec<DT>::load_scalar(row, first + e));
  return v;
}

// ---- the sorted list of a top-k warp ---------------------------------------
// 32*KPL keys, sorted descending, position p = lane*KPL + j in register j of a lane.
__device__ __forceinline__ unsigned long long u64max(unsigned long long a, unsigned long long b) { return a > b ? a : b; }
__device__ __forceinline__ unsigned long long u64min(unsigned long long a, unsigned long long b) { return a < b ? a : b; }

// One compare-exchange layer of a bitonic network at distance `stride` (in
// positions).  `asc_of(p)` gives the direction of the block position p is in.
template <int KPL, int STRIDE>
__device__ __forceinline__ void bitonic_layer(unsigned long long (&x)[KPL], int lane, int size, bool all_desc) {
  if (STRIDE < KPL) {
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
      if ((j & STRIDE) == 0) {
        const int p = lane * KPL + j;
        const bool asc = all_desc ? false : ((p & size) == 0);
        const unsigned long long a = x[j], b = x[j | STRIDE];
        const unsigned long long lo = u64min(a, b), hi = u64max(a, b);
        x[j] = asc ? lo : hi;
        x[j | STRIDE] = asc ? hi : lo;
      }
    }
  } else {
    constexpr int LS = STRIDE / KPL;            // lane distance
    const bool lower = (lane & LS) == 0;
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
      const int p = lane * KPL + j;
      const bool asc = all_desc ? false : ((p & size) == 0);
      const unsigned long long o = __shfl_xor_sync(0xffffffffu, x[j], LS);
      x[j] = (lower == asc) ? u64min(x[j], o) : u64max(x[j], o);
    }
  }
}

template <int KPL, int STRIDE>
struct BitonicDown {   // layers STRIDE, STRIDE/2, ..., 1
  static __device__ __forceinline__ void run(unsigned long long (&x)[KPL], int lane, int size, bool all_desc) {
    bitonic_layer<KPL, STRIDE>(x, lane, size, all_desc);
    BitonicDown<KPL, STRIDE / 2>::run(x, lane, size, all_desc);
  }
};
template <int KPL>
struct BitonicDown<KPL, 0> {
  static __device__ __forceinline__ void run(unsigned long long (&)[KPL], int, int, bool) {}
};

template <int KPL, int SIZE>
struct BitonicSort {   // full sort, ascending, of 32*KPL keys
  static __device__ __forceinline__ void run(unsigned long long (&x)[KPL], int lane) {
    BitonicSort<KPL, SIZE / 2>::run(x, lane);
    BitonicDown<KPL, SIZE / 2>::run(x, lane, SIZE, false);
  }
};
template <int KPL>
struct BitonicSort<KPL, 1> {
  static __device__ __forceinline__ void run(unsigned long long (&)[KPL], int) {}
};

// Folds up to 32*KPL keys taken from the end of the staging buffer into the list.
template <int KPL>
__device__ __forceinline__ void merge_staged(unsigned long long (&L)[KPL], const unsigned long long* stg,
                                             int& staged, int lane) {
  constexpr int NL = 32 * KPL;
  const int m = staged < NL ? staged : NL;
  unsigned long long nw[KPL];
#pragma unroll
  for (int j = 0; j < KPL; ++j) {
    const int i = lane * KPL + j;
    nw[j] = i < m ? stg[staged - m + i] : 0ull;
  }
  BitonicSort<KPL, NL>::run(nw, lane);                       // ascending
#pragma unroll
  for (int j = 0; j < KPL; ++j) L[j] = u64max(L[j], nw[j]);    // the NL largest of the union, bitonic
  BitonicDown<KPL, NL / 2>::run(L, lane, NL, true);          // descending
  staged -= m;
}

// Inserts one key into the descending list, dropping the smallest.
template <int KPL>
__device__ __forceinline__ void insert_one(unsigned long long (&L)[KPL], unsigned long long key, int lane) {
  unsigned long long up = __shfl_up_sync(0xffffffffu, L[KPL - 1], 1);
  if (lane == 0) up = ~0ull;
#pragma unroll
  for (int j = KPL - 1; j >= 0; --j) {
    const unsigned long long before = j == 0 ? up : L[j - 1];
    L[j] = L[j] > key ? L[j] : (before > key ? key : before);
  }
}

template <int KPL>
__device__ __forceinline__ unsigned long long kth_key(const unsigned long long (&L)[KPL], int k) {
  unsigned long long v = L[0];
#pragma unroll
  for (int j = 1; j < KPL; ++j)
    if (((k - 1) % KPL) == j) v = L[j];
  return __shfl_sync(0xffffffffu, v, (k - 1) / KPL);
}

// First vector index of pass `id` (= tile * TP + entry); its HV vectors are WPT * 32 apart.
__device__ __forceinline__ uint32_t pass_first_vector(uint32_t id) {
  const uint32_t tile = id / TP, e = id % TP;
  return tile * TV + (e / (WPT * 32)) * HV * (WPT * 32) + e % (WPT * 32);
}

// The highest histogram bin with at least k counted entries at or above it (0 if
// fewer than k were counted, or if the k-th lies in bin 0).  Lane l sums bins
// 8 l .. 8 l + 7, a shuffle suffix scan finds the lane in which the count crosses
// k, and that lane walks its bins from the top.  The histogram may be growing
// while it is read: a count read early is only smaller, and so is the result.
__device__ __forceinline__ int find_tau_bin(const uint32_t* hist, int k, int lane) {
  static_assert(NB == 256, "8 bins per lane");
  uint32_t b[8];
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const uint4 v = lds_volatile_v4(hist + lane * 8 + q * 4);
    b[4 * q] = v.x; b[4 * q + 1] = v.y; b[4 * q + 2] = v.z; b[4 * q + 3] = v.w;
  }
  int mine = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) mine += (int)b[i];
  int suf = mine;                                   // entries in this lane's bins and all higher lanes'
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int o = __shfl_down_sync(0xffffffffu, suf, off);
    if (lane + off < 32) suf += o;
  }
  const uint32_t ge = __ballot_sync(0xffffffffu, suf >= k);
  if (ge == 0u) return 0;
  const int L = 31 - __clz(ge);                     // the highest lane whose suffix reaches k
  int run = suf - mine, bin = 0;
  bool found = false;
#pragma unroll
  for (int i = 7; i >= 0; --i) {
    run += (int)b[i];
    if (!found && run >= k) { bin = i; found = true; }
  }
  return __shfl_sync(0xffffffffu, lane * 8 + bin, L);
}

// Low edge, as a logit, of histogram bin `bin` >= 1 under (base, shift).
__device__ __forceinline__ float bin_edge(uint32_t base, uint32_t shift, int bin) {
  const uint32_t top = 0xffffffffu >> shift;
  const uint32_t code = base + (uint32_t)bin < top ? base + (uint32_t)bin : top;
  return order_bits_f32(code << shift);
}

// What a consumer lane does with a pass whose maximum reached the row's threshold
// (a fraction of a percent of the passes): append it to the row's candidates as the
// high bits of the maximum's order bits over the pass id.  The slot's top-k warp
// counts the candidates into its histogram as they appear.
// Where the candidates of (row slot p, tensor t) of this CTA go when shared memory is full.
__device__ __forceinline__ uint32_t* spill_area(const StreamArgs& A, int p, int t) {
  static_assert(NSLOT == kStreamSlots, "the workspace is laid out for this many row slots");
  return A.spill + (((size_t)blockIdx.x * NSLOT + (size_t)p) * 2 + (size_t)t) * (size_t)kSpillCap;
}
// No room in shared memory: the entry goes to the workspace (out of line: rows with
// that many candidates are rare, and the streaming code stays small).
__device__ __noinline__ void spill_hit(uint32_t* spill, int pt, uint32_t o, uint32_t e) {
  if (o < (uint32_t)kSpillCap) spill[((size_t)blockIdx.x * (NSLOT * 2) + (size_t)pt) * (size_t)kSpillCap + o] = e;
}
template <int CAP>
__device__ __forceinline__ void record_hit(uint32_t* ncand, uint32_t* cand, uint32_t* spill, int pt, uint32_t id,
                                           uint32_t idmask, float m) {
  const uint32_t o = atomicAdd(ncand, 1u);
  const uint32_t e = (f32_order_bits(m) & ~idmask) | id;
  if (o < (uint32_t)CAP) cand[o] = e;
  else spill_hit(spill, pt, o - (uint32_t)CAP, e);
}

__device__ __forceinline__ uint32_t ldg_cg_u32(const uint32_t* p) {   // from L2: another warp of the CTA wrote it
  uint32_t v;
  asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Candidate i of a row: the first `cap` are in shared memory, later ones in the
// workspace (read from L2: a consumer warp of this CTA wrote them).
__device__ __forceinline__ uint32_t cand_load(const uint32_t* cand, const uint32_t* spill, uint32_t cap, uint32_t i) {
  return i < cap ? lds_volatile_u32(cand + i) : ldg_cg_u32(spill + (i - cap));
}

// Top-k warp: counts the candidates [seen, n) that have been written so far into
// the histogram and returns the new `seen`.  A consumer bumps the counter before
// it writes the entry, so an entry may still read 0 (the buffer is zeroed before
// the row starts and no entry of a finite maximum is 0): counting stops there
// unless `all` says that the row is done and everything has been written (only
// then may n reach beyond the shared-memory buffer).
__device__ __forceinline__ uint32_t count_candidates(const uint32_t* cand, const uint32_t* spill, uint32_t cap,
                                                     uint32_t seen, uint32_t n, uint32_t* hist, uint32_t base,
                                                     uint32_t shift, bool all, int lane) {
  while (seen < n) {
    const uint32_t i = seen + (uint32_t)lane;
    const uint32_t e = i < n ? cand_load(cand, spill, cap, i) : 0u;
    const bool there = i < n && (all || e != 0u);
    const uint32_t missing = ~__ballot_sync(0xffffffffu, there);
    const uint32_t run = missing ? (uint32_t)(__ffs(missing) - 1) : 32u;   // leading lanes whose entry is there
    if ((uint32_t)lane < run) {
      const uint32_t c = e >> shift;                       // shift >= id bits: the pass id falls away
      const uint32_t bin = c > base ? (c - base < (uint32_t)(NB - 1) ? c - base : (uint32_t)(NB - 1)) : 0u;
      atomicAdd(&hist[bin], 1u);
    }
    seen += run;
    if (run < 32u) break;
  }
  __syncwarp();
  return seen;
}

// Appends to the key buffer the keys of one vector's entries (one vector per lane)
// that can still be among the k best: at or above the threshold (as order bits) and
// above the list's current k-th key.  Returns the new number of buffered keys.
template <int DT>
__device__ __forceinline__ int stage_entries(const uint4& v, uint32_t vi, bool have, int64_t V, uint32_t tau_ob,
                                             unsigned long long kth, unsigned long long* stg, int staged,
                                             int lane) {
  constexpr int N = Vec<DT>::N;
  const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
  for (int e = 0; e < N; ++e) {
    const uint32_t idx = vi * N + e;
    const uint32_t ob = f32_order_bits(Vec<DT>::get(v, e));
    const unsigned long long key = ((unsigned long long)ob << 32) | (unsigned long long)(uint32_t)(~idx);
    const bool keep = have && (int64_t)idx < V && ob >= tau_ob && key > kth;
    const uint32_t bk = __ballot_sync(0xffffffffu, keep);
    if (keep) stg[staged + __popc(bk & lt)] = key;
    staged += __popc(bk);
  }
  __syncwarp();
  return staged;
}

// Folds every buffered key into the sorted list; returns the list's k-th key.
template <int KPL>
__device__ __forceinline__ unsigned long long merge_all(unsigned long long (&L)[KPL], const unsigned long long* stg,
                                                     int& staged, int k, int lane) {
  constexpr int SORT_MIN = 6 * KPL;       // below this, single inserts are cheaper than a sort + merge
  __syncwarp();
  while (staged >= SORT_MIN) merge_staged<KPL>(L, stg, staged, lane);
  while (staged > 0) {
    insert_one<KPL>(L, stg[staged - 1], lane);
    --staged;
  }
  __syncwarp();
  return kth_key<KPL>(L, k);
}

// Staging for the end of a row, where almost no entry passes: a lane first marks its
// entries at or above the threshold (as a logit), and keys are built only for the
// marked ones, one round per marked entry of the busiest lane; the buffer is folded
// into the list only when the next round might not fit.
template <int DT, int KPL>
__device__ __forceinline__ int stage_above(unsigned long long (&L)[KPL], const uint4& v, uint32_t vi, bool have,
                                           int64_t V, float tau_val, unsigned long long& kth,
                                           unsigned long long* stg, int staged, int k, int lane) {
  constexpr int N = Vec<DT>::N;
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t marks = 0u;
#pragma unroll
  for (int e = 0; e < N; ++e) marks |= (have && Vec<DT>::get(v, e) >= tau_val ? 1u : 0u) << e;
  while (__any_sync(0xffffffffu, marks != 0u)) {
    if (staged > SCAP - 32) kth = merge_all<KPL>(L, stg, staged, k, lane);
    bool keep = false;
    unsigned long long key = 0ull;
    if (marks) {
      const int e = __ffs(marks) - 1;
      marks &= marks - 1u;
      float x = Vec<DT>::get(v, 0);
#pragma unroll
      for (int q = 1; q < N; ++q)
        if (q == e) x = Vec<DT>::get(v, q);
      const uint32_t idx = vi * N + (uint32_t)e;
      key = make_key(x, idx);
      keep = (int64_t)idx < V && key > kth;
    }
    const uint32_t bk = __ballot_sync(0xffffffffu, keep);
    if (keep) stg[staged + __popc(bk & lt)] = key;
    staged += __popc(bk);
  }
  __syncwarp();
  return staged;
}

// Drops the candidates whose maximum is below the row's final threshold; those left
// are packed at the front of the shared-memory buffer.  Returns how many, or -1 if
// they do not fit there (only with spilled candidates and long runs of ties).
__device__ __noinline__ int compact_candidates(uint32_t* cand, const uint32_t* spill, int cap, int n, uint32_t tau_ob,
                                               uint32_t idmask, int lane) {
  int out = 0;
  for (int b = 0; b < n; b += 32) {
    const int i = b + lane;
    const uint32_t c = i < n ? cand_load(cand, spill, (uint32_t)cap, (uint32_t)i) : 0u;
    // the stored high bits with the low ones filled in bound the maximum from above
    const bool keep = i < n && (c | idmask) >= tau_ob;
    const uint32_t bm = __ballot_sync(0xffffffffu, keep);
    __syncwarp();
    if (out + __popc(bm) > cap) return -1;
    if (keep) cand[out + __popc(bm & ((1u << lane) - 1u))] = c;     // out <= b: never ahead of the reads
    out += __popc(bm);
    __syncwarp();
  }
  return out;
}

// Sorts the entries of the candidate passes into the list.  The vectors of a pass
// are read back from memory (they left the ring long ago; a few hundred 16-byte
// reads per row, mostly L2 hits).  `kth` is the list's k-th key so far (0 for an
// empty list); returns the new one.
template <int DT, int KPL>
__device__ __forceinline__ unsigned long long candidates_to_list(unsigned long long (&L)[KPL], const uint32_t* cand,
                                                              int n, uint32_t idmask, const char* row, int64_t nvec,
                                                              int64_t V, float tau_val, unsigned long long kth,
                                                              unsigned long long* stg, int k, int lane) {
  int staged = 0;
  for (int b = 0; b < n; b += 32) {
    const int i = b + lane;
    const uint32_t v0 = i < n ? pass_first_vector(cand[i] & idmask) : 0u;
    uint4 v[HV];
    bool in[HV];
#pragma unroll
    for (int j = 0; j < HV; ++j) {
      const uint32_t vi = v0 + j * (WPT * 32);
      in[j] = i < n && (int64_t)vi < nvec;
      v[j] = in[j] ? ldg_stream((const uint4*)row + vi) : Vec<DT>::neg_inf();
    }
#pragma unroll
    for (int j = 0; j < HV; ++j) {
      staged = stage_above<DT, KPL>(L, v[j], v0 + j * (WPT * 32), in[j], V, tau_val, kth, stg, staged, k, lane);
    }
  }
  return merge_all<KPL>(L, stg, staged, k, lane);
}

// The exact top-k of a whole row read again from memory by one warp: the way out
// for a row whose candidates did not fit the buffer (long runs of ties at the top,
// rows that keep rising, -inf padding above the k-th entry).  Leaves the list in the
// key buffer.
template <int DT, int KPL>
__device__ __noinline__ void scan_row_exact(const char* row, int64_t nvec, int64_t V, unsigned long long* stg, int k,
                                            int lane) {
  unsigned long long L[KPL];
#pragma unroll
  for (int j = 0; j < KPL; ++j) L[j] = 0ull;
  int staged = 0;
  unsigned long long kth = 0ull;
  for (int64_t b = 0; b < nvec; b += 32) {
    const int64_t vi = b + lane;
    const bool in = vi < nvec;
    const uint4 v = in ? ldg_stream((const uint4*)row + vi) : Vec<DT>::neg_inf();
    // skip the 32 vectors at once when none reaches the value of the current k-th key
    const uint32_t ob = f32_order_bits(Vec<DT>::vmax(v));
    if (!__any_sync(0xffffffffu, in && ob >= (uint32_t)(kth >> 32))) continue;
    staged = stage_entries<DT>(v, (uint32_t)vi, in, V, 0u, kth, stg, staged, lane);
    if (staged > SCAP - 32 * Vec<DT>::N) kth = merge_all<KPL>(L, stg, staged, k, lane);
  }
  merge_all<KPL>(L, stg, staged, k, lane);
  // hand the list back through the key buffer (position lane * KPL + j), so that the
  // caller's list can stay in registers
#pragma unroll
  for (int j = 0; j < KPL; ++j) stg[lane * KPL + j] = L[j];
  __syncwarp();
}

// Before a row starts: the k-th best vector maximum of the row's first SAMPLE
// vectors, as the low edge of its histogram bin (-inf if the sample has fewer than
// k vectors), and the bin geometry (base, shift) for the row's candidate histogram.
// The window of NB codes is anchored at the sample's maximum; the shift starts at 16
// (bf16 resolution; more for rows so long that a pass id needs more than 16 bits) and grows until the k-th best falls inside the window, so a
// sample that spans many binades, or zero, gets coarser bins rather than none.
template <int DT>
__device__ __noinline__ float sample_threshold(const char* row, int64_t nvec, int k, uint32_t* hist, float* park,
                                               uint32_t& base, uint32_t& shift, uint32_t min_shift, int lane) {
  const int ns = (int)(nvec < (int64_t)SAMPLE ? nvec : (int64_t)SAMPLE);
  base = 0xffffffffu;                       // nothing above it: every maximum counts in bin 0 = "no threshold"
  shift = min_shift > 16u ? min_shift : 16u;  // a candidate keeps only the order bits above its pass id
  if (ns < k) return JP_NEG_INF;
  // ask L2 for the whole sample first: the loads below go eight at a time
  for (int line = lane; line * 8 < ns; line += 32)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(row + (size_t)line * 128));
  float mx = JP_NEG_INF;
#pragma unroll 1
  for (int c = 0; c < ns; c += 8 * 32) {
    uint4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int vi = c + j * 32 + lane;
      v[j] = vi < ns ? ldg_stream((const uint4*)row + vi) : Vec<DT>::neg_inf();
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int vi = c + j * 32 + lane;
      const float m = Vec<DT>::vmax(v[j]);
      if (vi < ns) park[vi] = m;
      mx = fmaxf(mx, m);
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  const uint32_t ob_max = f32_order_bits(mx);
  __syncwarp();
  float tau0 = JP_NEG_INF;
  for (uint32_t sh = shift; sh < 32u; ++sh) {
    const uint32_t cmax = ob_max >> sh;
    const uint32_t b0 = cmax > (uint32_t)(NB - 1) ? cmax - (uint32_t)(NB - 1) : 0u;
    for (int i = lane; i < NB; i += 32) hist[i] = 0u;
    __syncwarp();
    for (int i = lane; i < ns; i += 32) {
      const uint32_t c = f32_order_bits(park[i]) >> sh;
      // c <= cmax for every number, so the bin is at most NB - 1; a NaN's order bits lie above
      // every number's (the maximum ignores NaNs), hence the clamp
      const uint32_t bin = c > b0 ? c - b0 : 0u;
      atomicAdd(&hist[bin < (uint32_t)(NB - 1) ? bin : (uint32_t)(NB - 1)], 1u);
    }
    __syncwarp();
    const int bin = find_tau_bin(hist, k, lane);
    if (bin > 0) {
      const uint32_t code0 = b0 + (uint32_t)bin;
      tau0 = order_bits_f32(code0 << sh);
      base = code0 - 1u;                                 // the threshold's own code is bin 1; cmax is at most bin NB - 1
      shift = sh;
      break;
    }
    if (b0 == 0u) break;                                 // the window reaches the bottom of the order: no threshold
  }
  __syncwarp();
  if (!(tau0 == tau0)) tau0 = JP_NEG_INF;                // the low edge of -inf's own bin is not a number
  return tau0;
}

// Which consumer group takes tile 0 of a row.  Tiles go to the groups in turn; starting every
// row with the same group would leave that group one tile behind on every row with an odd
// number of tiles.  The choice hangs on the row's index in the batch alone (a hash bit), never on where
// the row sits in the CTA's walk, so that a row's sums are added in the same order in every run.
__device__ __forceinline__ uint32_t first_group(int64_t row) {
  return (uint32_t)(((uint32_t)row * 0x9E3779B1u) >> 16) % (uint32_t)NG;
}

template <class SM>
__device__ __forceinline__ void raise_timeout(SM& sm, Scalars* sc) {
  sm.abort = 1;
  atomicExch(&sc->status, (int)JP_ERR_TIMEOUT);
}

// ---- producer ---------------------------------------------------------------
template <int DT, bool SINGLE, class SM>
__device__ void producer_loop(const StreamArgs& A, SM& sm, int64_t n_rows) {
  constexpr int N = Vec<DT>::N;
  constexpr int STAGES = SM::STAGES;
  const int64_t nvec = A.V / N;
  const int ntiles = nvec > 0 ? (int)((nvec + TV - 1) / TV) : 1;
  const uint32_t last_bytes = (uint32_t)((nvec - (int64_t)(ntiles - 1) * TV) * 16);   // 0 only when nvec == 0
  const int64_t pitch = A.ld * Vec<DT>::ESIZE;
  // This lane is the one latency-critical thread of the CTA: a freed stage waits for it.
  // Stage and phase advance by increments, addresses by additions, and the next row's
  // index is fetched one row ahead.
  const unsigned long long policy = l2_evict_first_policy();
  uint32_t s = 0, ph = 0, armed = 0;
  uint32_t fph0 = 0u, fph1 = 0u, last_grp = 0u, last_ph = 0u;   // per stage: phase bits of full[0], full[1]; group and phase armed last
  bool ok = true;
  int64_t it = blockIdx.x;
  int64_t row = it < n_rows ? A.list[it] : 0;
  while (it < n_rows && ok) {
    const char* ra = (const char*)A.za + row * pitch;
    const char* rp = (const char*)A.zp + row * pitch;
    const int g0 = (int)first_group(A.record_offset + row);
    it += gridDim.x;
    if (it < n_rows) row = A.list[it];
    for (int tile = 0; tile < ntiles; ++tile, ra += TV * 16, rp += TV * 16) {
      if (!mbar_wait(&sm.empty[s], ph ^ 1u, &sm.abort)) { ok = false; break; }
      const uint32_t bytes = tile == ntiles - 1 ? last_bytes : (uint32_t)(TV * 16);
      const int grp = (tile + g0) % NG;
      if (bytes > 0) {
        mbar_arrive_expect_tx(&sm.full[grp][s], SINGLE ? bytes : 2u * bytes);
        if (!SINGLE) bulk_g2s(&sm.ring[s][0][0], ra, bytes, &sm.full[grp][s], policy);
        bulk_g2s(&sm.ring[s][SM::TENSORS - 1][0], rp, bytes, &sm.full[grp][s], policy);
      } else {
        mbar_arrive(&sm.full[grp][s]);
      }
      // remember what was armed last on this stage (for the clean-up after a time-out)
      last_grp = (last_grp & ~(1u << s)) | ((uint32_t)grp << s);
      if (grp) { last_ph = (last_ph & ~(1u << s)) | (((fph1 >> s) & 1u) << s); fph1 ^= 1u << s; }
      else     { last_ph = (last_ph & ~(1u << s)) | (((fph0 >> s) & 1u) << s); fph0 ^= 1u << s; }
      ++armed;
      if (++s == STAGES) { s = 0; ph ^= 1u; }
    }
  }
  if (!ok) {
    // Leave no copy in flight: the stages this lane armed last and nobody consumed
    // complete once their bytes have landed.
    raise_timeout(sm, A.sc);
    const uint32_t n_back = armed < (uint32_t)STAGES ? armed : (uint32_t)STAGES;
    for (uint32_t st = 0; st < n_back; ++st) {          // stages 0 .. n_back-1 are the ones ever armed
      const long long t0 = clock64();
      while (!mbar_try_wait(&sm.full[(last_grp >> st) & 1u][st], (last_ph >> st) & 1u))
        if (clock64() - t0 > kSpinLimit) break;
    }
  }
}

// ---- consumers ----------------------------------------------------------------
template <int DT, bool TOPK, bool UNROLL, bool SINGLE, class SM>
__device__ void consumer_loop(const StreamArgs& A, SM& sm, int64_t n_rows, int cw, int lane) {
  constexpr int N = Vec<DT>::N;
  constexpr int STAGES = SM::STAGES, CAP = SM::CAP;
  const int64_t nvec = A.V / N;
  const int tail = (int)(A.V - nvec * N);
  const uint32_t ntiles = nvec > 0 ? (uint32_t)((nvec + TV - 1) / TV) : 1u;
  const uint32_t idmask = 0xffffffffu >> __clz(ntiles * (uint32_t)TP - 1u);   // covers every pass id of a row
  const int gq = cw / WPT;              // this warp's group: it takes every NG-th tile of a row
  const int wq = cw % WPT;              // its place among the warps that share a tile
  static_assert(HV == 2, "a pass takes its maximum over two vectors");
  const uint32_t nfull = (uint32_t)(nvec / TV);            // tiles of a row that need no bounds checks
  const uint32_t row_step = ntiles % (uint32_t)STAGES;     // how far a row moves the ring position of tile 0
  uint32_t s_row = 0u;                  // stage of tile 0 of the current row
  uint32_t fphase = 0u;                 // per stage: phase bit of this group's full barrier
  int lr = 0;
  for (int64_t it = blockIdx.x; it < n_rows; it += gridDim.x, ++lr) {
    const int p = lr % NSLOT;
    const uint32_t ph = (uint32_t)((lr / NSLOT) & 1);
    // the slot's top-k warps have finished the row that used it before and set it up for this one
    if (!mbar_wait(&sm.slot_ready[p], ph, &sm.abort)) { raise_timeout(sm, A.sc); return; }

    Online oa{JP_NEG_INF, 0.f, 0ull}, op{JP_NEG_INF, 0.f, 0ull};

    // One tile of both rows, taken in passes of HV vectors per tensor (few live
    // registers); the two passes of a full tile are unrolled (UNROLL), the partial tile's are not.  All a consumer does for the top-k is to compare the maximum of
    // every pass with the row's threshold.
    auto consume_tile = [&](uint32_t tile, uint32_t s) -> bool {
      if (!mbar_wait(&sm.full[gq][s], (fphase >> s) & 1u, &sm.abort)) return false;
      fphase ^= 1u << s;
      const uint4* sa = &sm.ring[s][0][wq * 32 + lane];
      const uint4* sp = &sm.ring[s][SM::TENSORS - 1][wq * 32 + lane];
      float ta = 0.f, tp = 0.f;
      if (TOPK) { ta = lds_volatile_f32(&sm.tau[p][0]); tp = lds_volatile_f32(&sm.tau[p][1]); }
      uint32_t id = tile * (uint32_t)TP + (uint32_t)(wq * 32 + lane);
      if (tile < nfull) {
        // a full tile: no bounds checks
#pragma unroll(UNROLL ? VPL / HV : 1)
        for (int h = 0; h < VPL / HV; ++h, sa += HV * WPT * 32, sp += HV * WPT * 32, id += WPT * 32) {
          uint4 va[HV], vp[HV];
#pragma unroll
          for (int j = 0; j < HV; ++j) {
            if (!SINGLE) va[j] = sa[j * WPT * 32];
            vp[j] = sp[j * WPT * 32];
          }
          // one maximum and one check against the reference exponent per tensor per pass
          float ma = JP_NEG_INF;
          if (!SINGLE) { ma = Vec<DT>::vmax2(va[0], va[1]); raise_max(ma, oa); }
          const float mp = Vec<DT>::vmax2(vp[0], vp[1]);
          raise_max(mp, op);
#pragma unroll
          for (int j = 0; j < HV; ++j) {
            if (!SINGLE) add_terms<DT>(va[j], oa);
            add_terms<DT>(vp[j], op);
          }
          if (TOPK) {
            if (!SINGLE && ma >= ta) record_hit<CAP>(&sm.ncand[p][0], sm.cand[p][0], A.spill, 2 * p, id, idmask, ma);
            if (mp >= tp) record_hit<CAP>(&sm.ncand[p][1], sm.cand[p][1], A.spill, 2 * p + 1, id, idmask, mp);
          }
        }
        release_stage(&sm.empty[s], oa, op, lane);
      } else {
        // the row's last, partial tile: bounds checked
        const uint32_t v0 = tile * TV + wq * 32 + lane;
#pragma unroll 1
        for (int h = 0; h < VPL / HV; ++h, id += WPT * 32) {
          float ma = JP_NEG_INF, mp = JP_NEG_INF;
#pragma unroll 1
          for (int j = 0; j < HV; ++j) {
            const int o = (h * HV + j) * WPT * 32;
            uint4 a4 = Vec<DT>::neg_inf(), p4 = Vec<DT>::neg_inf();
            if ((int64_t)(v0 + o) < nvec) { if (!SINGLE) a4 = sa[o]; p4 = sp[o]; }
            const float vm_a = Vec<DT>::vmax(a4), vm_p = Vec<DT>::vmax(p4);
            if (!SINGLE) accumulate<DT>(a4, vm_a, oa);
            accumulate<DT>(p4, vm_p, op);
            ma = fmaxf(ma, vm_a);
            mp = fmaxf(mp, vm_p);
          }
          // a pass with no vector inside the row holds nothing
          if (TOPK && (int64_t)(v0 + h * HV * WPT * 32) < nvec) {
            if (!SINGLE && ma >= ta) record_hit<CAP>(&sm.ncand[p][0], sm.cand[p][0], A.spill, 2 * p, id, idmask, ma);
            if (mp >= tp) record_hit<CAP>(&sm.ncand[p][1], sm.cand[p][1], A.spill, 2 * p + 1, id, idmask, mp);
          }
        }
        release_stage(&sm.empty[s], oa, op, lane);
      }
      return true;
    };
    {
      const uint32_t g0 = sm.g0[p];          // written by the slot's top-k warp before it opened the slot
      const uint32_t first = ((uint32_t)gq + (uint32_t)NG - g0) % (uint32_t)NG;   // this group's first tile of the row
      uint32_t s = s_row + first;
      if (s >= (uint32_t)STAGES) s -= (uint32_t)STAGES;
      for (uint32_t tile = first; tile < ntiles; tile += NG) {
        if (!consume_tile(tile, s)) { raise_timeout(sm, A.sc); return; }
        s += NG;
        if (s >= (uint32_t)STAGES) s -= (uint32_t)STAGES;
      }
      s_row += row_step;
      if (s_row >= (uint32_t)STAGES) s_row -= (uint32_t)STAGES;
    }

    if (tail > 0 && cw == 0 && lane == 0) {     // ragged end of the row: scalar loads
      const int64_t row = A.list[it];
      const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
      const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;
      if (!SINGLE) {
        const uint4 ta = load_tail_vector<DT>(ra, nvec * N, tail);
        accumulate<DT>(ta, Vec<DT>::vmax(ta), oa);
      }
      const uint4 tp = load_tail_vector<DT>(rp, nvec * N, tail);
      accumulate<DT>(tp, Vec<DT>::vmax(tp), op);
    }

    // per-warp (max, sum) pairs, merged in a fixed tree
    float mL_a = oa.mL, mL_p = op.mL, s_a, s_p;
    {
      float s0, s1;
      unpack2(oa.s2, s0, s1); s_a = s0 + s1;
      unpack2(op.s2, s0, s1); s_p = s0 + s1;
    }
    if (oa.lim == JP_NEG_INF) mL_a = JP_NEG_INF;   // a thread that saw nothing must not set the scale
    if (op.lim == JP_NEG_INF) mL_p = JP_NEG_INF;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      merge_scaled(mL_a, s_a, __shfl_xor_sync(0xffffffffu, mL_a, off), __shfl_xor_sync(0xffffffffu, s_a, off));
      merge_scaled(mL_p, s_p, __shfl_xor_sync(0xffffffffu, mL_p, off), __shfl_xor_sync(0xffffffffu, s_p, off));
    }
    if (lane == 0) {
      sm.part_mL[p][0][cw] = mL_a; sm.part_s[p][0][cw] = s_a;
      sm.part_mL[p][1][cw] = mL_p; sm.part_s[p][1][cw] = s_p;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.row_done[p]);
  }
}

// ---- top-k warps ---------------------------------------------------------------
// One warp per (row slot p, tensor t); it owns rows p, p + NSLOT, ... of the CTA.
template <int DT, int KPL, bool SINGLE, class SM>
__device__ void topk_loop(const StreamArgs& A, SM& sm, int64_t n_rows, int t, int p, int lane) {
  constexpr int N = Vec<DT>::N;
  constexpr int CAP = SM::CAP;
  constexpr bool TOPK = KPL > 0;
  constexpr int KL = KPL > 0 ? KPL : 1;
  const int64_t nvec = A.V / N;
  const int tail = (int)(A.V - nvec * N);
  const uint32_t ntiles = nvec > 0 ? (uint32_t)((nvec + TV - 1) / TV) : 1u;
  const uint32_t idbits = 32u - (uint32_t)__clz(ntiles * (uint32_t)TP - 1u);
  const uint32_t idmask = 0xffffffffu >> (32u - idbits);
  const int k = A.k;
  unsigned long long* stg = sm.skeys[p][t];
  uint32_t* hist = sm.hist[p][t];
  uint32_t* cand = sm.cand[p][t];
  int lr = p;
  uint32_t watched = 0u;                     // phases of the watched slot's row_done seen so far
  for (int64_t it = (int64_t)blockIdx.x + (int64_t)p * gridDim.x; it < n_rows;
       it += (int64_t)NSLOT * gridDim.x, lr += NSLOT) {
    const uint32_t ph = (uint32_t)((lr / NSLOT) & 1);
    if (SINGLE && t == 0) {
      // one tensor only (the rollout model is known through its stored record): this warp has no
      // list to build; it keeps the slot's hand-shake going
      if (lane == 0) sm.g0[p] = first_group(A.record_offset + A.list[it]);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.slot_ready[p]);
      if (!mbar_wait(&sm.row_done[p], ph, &sm.abort)) { raise_timeout(sm, A.sc); return; }
      continue;
    }
    if (TOPK && lr >= 2) {
      // Do not look at the row before the consumers are one row away from it (the row two
      // before it is done): the sample then still sits in L2 when the row streams, instead
      // of being read from HBM twice.  The watched barrier is another slot's; its phases
      // are waited for one by one, none skipped.
      const uint32_t need = (uint32_t)(lr - 2) / NSLOT;
      for (; watched <= need; ++watched)
        if (!mbar_wait(&sm.row_done[(p + 2) % NSLOT], watched & 1u, &sm.abort)) { raise_timeout(sm, A.sc); return; }
    }
    const int64_t row = A.list[it];
    const int64_t rrow = A.record_offset + row;
    const char* rmine = (const char*)(t == 0 ? A.za : A.zp) + row * A.ld * Vec<DT>::ESIZE;

    // the sampled token's logit is needed only at the end of the row: fetch it now
    float zx = 0.f;
    if (lane == 0) zx = Vec<DT>::load_scalar(rmine, A.tokens[row]);

    // set the slot up for this row: first threshold from a sample, empty histogram and buffer
    float cur = JP_NEG_INF;
    uint32_t base = 0xffffffffu, shift = 16u;
    if (TOPK) {
      cur = sample_threshold<DT>(rmine, nvec, k, hist, reinterpret_cast<float*>(cand), base, shift, idbits, lane);
      for (int i = lane; i < NB; i += 32) hist[i] = 0u;
      for (int i = lane; i < CAP / 4; i += 32) reinterpret_cast<uint4*>(cand)[i] = make_uint4(0u, 0u, 0u, 0u);
      if (lane == 0) {
        sm.ncand[p][t] = 0u;
        sm.tau[p][t] = cur;
      }
    }
    uint32_t seen = 0u;                       // candidates counted into the histogram so far
    if (t == 0 && lane == 0) sm.g0[p] = first_group(rrow);
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.slot_ready[p]);

    // while the row streams: raise tau to the highest bin with k candidates at or above it
    {
      long long t0 = 0;
      for (uint32_t i = 0; !mbar_try_wait_for(&sm.row_done[p], ph, kTauPollNs); ++i) {
        if (TOPK) {
          const uint32_t nc = lds_volatile_u32(&sm.ncand[p][t]);
          const uint32_t n = nc < (uint32_t)CAP ? nc : (uint32_t)CAP;
          if (n > seen) {
            seen = count_candidates(cand, nullptr, (uint32_t)CAP, seen, n, hist, base, shift, false, lane);
            const int bin = find_tau_bin(hist, k, lane);
            if (bin > 0) {
              const float val = bin_edge(base, shift, bin);
              if (val > cur) {
                cur = val;
                if (lane == 0) sts_volatile_f32(&sm.tau[p][t], cur);
              }
            }
          }
        }
        if ((i & 63u) == 0u) {
          const long long now = clock64();
          if (i == 0u) t0 = now;
          const int give_up = *(volatile int*)&sm.abort || now - t0 > kSpinLimit;
          if (__any_sync(0xffffffffu, give_up)) { raise_timeout(sm, A.sc); return; }
        }
      }
    }

    if (TOPK) {
      const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
      const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;
      unsigned long long L[KL];
#pragma unroll
      for (int j = 0; j < KL; ++j) L[j] = 0ull;
      unsigned long long kth;
      uint32_t tau_ob = 0u;
      const uint32_t total = lds_volatile_u32(&sm.ncand[p][t]);
      int n = -1;
      if (total <= (uint32_t)(CAP + kSpillCap)) {
        // (candidates beyond the shared-memory buffer are in the workspace: rare)
        const uint32_t* spill = spill_area(A, p, t);
        count_candidates(cand, spill, (uint32_t)CAP, seen, total, hist, base, shift, true, lane);
        const int bin = find_tau_bin(hist, k, lane);
        if (bin > 0) {
          const float val = bin_edge(base, shift, bin);
          if (val > cur) cur = val;
        }
        tau_ob = f32_order_bits(cur);
        n = compact_candidates(cand, spill, CAP, (int)total, tau_ob, idmask, lane);
      }
      if (n >= 0) {
        kth = candidates_to_list<DT, KL>(L, cand, n, idmask, rmine, nvec, A.V, cur, 0ull, stg, k, lane);
      } else {
        // more candidates than shared memory and the spill area hold, or than fit after
        // the threshold has thinned them out (rows that keep rising, long runs of ties at
        // the top): read the row again
        tau_ob = 0u;
        scan_row_exact<DT, KL>(rmine, nvec, A.V, stg, k, lane);
#pragma unroll
        for (int j = 0; j < KL; ++j) L[j] = stg[lane * KL + j];
        __syncwarp();
        kth = kth_key<KL>(L, k);
      }
      if (tail > 0) {                 // the ragged end of the row
        uint4 v = Vec<DT>::neg_inf();
        if (lane == 0) v = load_tail_vector<DT>(rmine, nvec * N, tail);
        int staged = stage_entries<DT>(v, (uint32_t)nvec, lane == 0, A.V, tau_ob, kth, stg, 0, lane);
        kth = merge_all<KL>(L, stg, staged, k, lane);
      }
      // the record: this tensor's list, best first, every entry with both logits
#pragma unroll
      for (int j = 0; j < KL; ++j) {
        const int pos = lane * KL + j;
        if (pos < k) {
          const int64_t o = rrow * (2 * k) + (int64_t)t * k + pos;
          const unsigned long long key = L[j];
          if (key != 0ull) {
            const uint32_t idx = key_index(key);
            A.rec.idx[o] = (int32_t)idx;
            A.rec.za[o] = SINGLE ? 0.f : Vec<DT>::load_scalar(ra, idx);
            A.rec.zp[o] = Vec<DT>::load_scalar(rp, idx);
          } else {
            A.rec.idx[o] = -1; A.rec.za[o] = 0.f; A.rec.zp[o] = 0.f;
          }
        }
      }
    }

    if (lane == 0) {
      // log-sum-exp = ln2 (M + log2 S).  S = 2^e f with f in [1,2): logf(f) is good to an
      // ulp of a number below 0.7, and the large part (M + e) ln2 is formed in double, so
      // the published fp32 values are rounded once.
      float M = sm.part_mL[p][t][0];
      for (int w = 1; w < NC; ++w) M = fmaxf(M, sm.part_mL[p][t][w]);
      float S = 0.f;
      for (int w = 0; w < NC; ++w)
        if (sm.part_mL[p][t][w] != JP_NEG_INF) S += sm.part_s[p][t][w] * exp2_int(sm.part_mL[p][t][w] - M);
      int e;
      const float f = 2.f * frexpf(S, &e);                // S = f * 2^(e-1)
      // The exponents were formed with the fp32 constant log2(e), which is short of log2(e) by a
      // factor 1 - 1.335e-8: what was summed is exp(z (1 - eps)), whose log-sum-exp is lse - eps * (lse - H)
      // with H the entropy of the row (at most ln V).  Scaling by 1 + eps leaves eps * H < 2e-7.
      const double lse = (((double)M + (double)(e - 1)) * 0.6931471805599453 + (double)logf(f)) * (1.0 + 1.33497582e-8);
      const float lsef = (float)lse;
      const float lpx = (float)((double)zx - lse);
      const float lo = (float)(lse - (double)lsef);
      if (t == 0) { A.rec.lse_a[rrow] = lsef; A.rec.lse_a_lo[rrow] = lo; A.rec.lq[rrow] = lpx; A.rec.flag[rrow] = kRowValid; }
      else        { A.rec.lse_p[rrow] = lsef; A.rec.lse_p_lo[rrow] = lo; A.rec.lp[rrow] = lpx; }
      if (SINGLE) {
        // log p_inf(a_t) comes from the rollout record, not from a row of logits
        A.rec.lse_a[rrow] = 0.f; A.rec.lse_a_lo[rrow] = 0.f;
        A.rec.lq[rrow] = A.logp_inf[row];
        A.rec.flag[rrow] = kRowValid;
      }
    }
    __syncwarp();
  }
}

template <int DT, int KPL, bool SINGLE>
__global__ void __launch_bounds__(NTHREADS, 1) stream_kernel(StreamArgs A) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  using SM = StreamSmemFor<KPL, SINGLE>;
  constexpr int STAGES = SM::STAGES;
  SM& sm = *reinterpret_cast<SM*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      for (int q = 0; q < NG; ++q) mbar_init(&sm.full[q][s], 1);
      mbar_init(&sm.empty[s], WPT);
    }
    for (int p = 0; p < NSLOT; ++p) {
      mbar_init(&sm.row_done[p], NC);
      mbar_init(&sm.slot_ready[p], 2);
    }
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // The kernel is launched as a programmatic dependent of the row-list kernel: its CTAs are set up
  // (shared memory carved, barriers initialised) while that kernel still runs; nothing it wrote
  // is read before this point.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // whatever follows may be set up; it waits for this grid's end itself
  const int64_t n_rows = A.sc->n_list;

  if (warp == 0) {
    if (lane == 0) producer_loop<DT, SINGLE, SM>(A, sm, n_rows);
  } else if (warp <= NC) {
    // (unrolling a tile's two passes saves 3 % of the instructions; the kernel for the longest
    // lists is faster with them rolled)
    consumer_loop<DT, (KPL > 0), (KPL != 4), SINGLE, SM>(A, sm, n_rows, warp - 1, lane);
  } else {
    const int tw = warp - 1 - NC;
    topk_loop<DT, KPL, SINGLE, SM>(A, sm, n_rows, tw & 1, tw >> 1, lane);
  }
}

// Splits the rows of one call into the list of valid rows the stream kernel walks
// and the masked / out-of-range ones, whose records are cleared here.
__global__ void __launch_bounds__(256) prep_rows_kernel(StreamArgs A) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the stream kernel may start setting up
  const int64_t row = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int lane = threadIdx.x & 31;
  bool valid = false, bad = false;
  if (row < A.T) {
    valid = A.mask == nullptr || A.mask[row] != 0;
    if (valid) {
      const int32_t x = A.tokens[row];
      if (x < 0 || (int64_t)x >= A.V) { valid = false; bad = true; }
    }
    if (!valid) {
      const int64_t rrow = A.record_offset + row;
      A.rec.flag[rrow] = 0;
      A.rec.lse_a[rrow] = 0.f; A.rec.lse_p[rrow] = 0.f;
      A.rec.lse_a_lo[rrow] = 0.f; A.rec.lse_p_lo[rrow] = 0.f;
      A.rec.lq[rrow] = 0.f; A.rec.lp[rrow] = 0.f;
    }
  }
  const uint32_t vm = __ballot_sync(0xffffffffu, valid), bm = __ballot_sync(0xffffffffu, bad);
  int base = 0;
  if (lane == 0 && vm) base = atomicAdd(&A.sc->n_list, __popc(vm));
  base = __shfl_sync(0xffffffffu, base, 0);
  if (valid) A.list[base + __popc(vm & ((1u << lane) - 1u))] = (int32_t)row;
  if (lane == 0 && bm) atomicAdd(&A.sc->n_bad_token, (unsigned long long)__popc(bm));
}

// ---- exact normaliser -----------------------------------------------------------
constexpr int XNT = 256;
constexpr int XNWARP = XNT / 32;
constexpr int XUNROLL = 4;
constexpr int XCTAS_PER_SM = 2;

template <int DT>
__device__ __forceinline__ void load_tile(uint4 (&va)[XUNROLL], uint4 (&vp)[XUNROLL], const char* ra,
                                          const char* rp, int64_t v0, int64_t nvec, int tail, int tid) {
#pragma unroll
  for (int j = 0; j < XUNROLL; ++j) {
    int64_t vi = v0 + (int64_t)j * XNT + tid;
    if (vi < nvec) {
      va[j] = ldg_stream((const uint4*)ra + vi);
      vp[j] = ldg_stream((const uint4*)rp + vi);
    } else if (vi == nvec && tail > 0) {
      va[j] = load_tail_vector<DT>(ra, nvec * Vec<DT>::N, tail);
      vp[j] = load_tail_vector<DT>(rp, nvec * Vec<DT>::N, tail);
    } else {
      va[j] = Vec<DT>::neg_inf();
      vp[j] = Vec<DT>::neg_inf();
    }
  }
}

// One more pass over the rows with the log-sum-exps known.
//   WANT_Z : the exact normaliser Z_t = sum_v min(q_t(v), p_t(v) / lambda) (Eq. obrs_dist;
//            Appendix A, Z_C)
//   WANT_KL: KL(p_t || q_t) = sum_v p_t(v) (zp_v - za_v) - lse_p + lse_a, the divergence
//            between target and rollout distribution that the paper tracks during training
// Exponents are taken relative to integers M near lse log2(e), so that the fused
// multiply-add z log2(e) - M is rounded once and the fractional remainder is a factor
// common to the row, applied in double at the end.  The remainder also carries the share
// of the fp32 constant's shortfall (log2(e) - kLog2e) that matters, taken at z = lse, where
// the terms that dominate the sums lie.
template <int DT, bool WANT_Z, bool WANT_KL>
__global__ void __launch_bounds__(XNT, XCTAS_PER_SM) exact_z_kernel(ExactZArgs A) {
  __shared__ float red[2][XNWARP];
  __shared__ int s_row;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int N = Vec<DT>::N;
  constexpr double kLog2e64 = 1.4426950408889634074;
  const double kLog2eShort = kLog2e64 - (double)kLog2e;      // what the fp32 constant lacks
  const int64_t nvec = A.V / N;
  const int tail = (int)(A.V - nvec * N);
  const int64_t nvt = nvec + (tail > 0 ? 1 : 0);
  const double lambda = WANT_Z ? (double)A.sc->lambda : 1.0;
  const double log2_lambda = log2(lambda);
  for (;;) {
    if (tid == 0) s_row = atomicAdd(&A.sc->row_counter2, 1);
    __syncthreads();
    const int64_t row = s_row;
    __syncthreads();
    if (row >= A.T) break;
    const int64_t rrow = A.record_offset + row;
    if (A.rec.flag[rrow] != kRowValid) {
      if (tid == 0) {
        if (WANT_Z) A.out[rrow] = 0.f;
        if (WANT_KL) A.out_kl[rrow] = 0.f;
      }
      continue;
    }
    const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
    const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;
    const double lse_a = (double)A.rec.lse_a[rrow] + (double)A.rec.lse_a_lo[rrow];
    const double lse_p = (double)A.rec.lse_p[rrow] + (double)A.rec.lse_p_lo[rrow];
    const double ca = lse_a * kLog2e64, cp = lse_p * kLog2e64 + log2_lambda;
    // the clamp keeps M an integer that fp32 holds exactly; rows that far out are non-finite anyway
    const float Ma = (float)rint(fmin(fmax(ca, -16777216.0), 16777216.0));
    const float Mp = (float)rint(fmin(fmax(cp, -16777216.0), 16777216.0));
    const double fq = exp2(((double)Ma - ca) + lse_a * kLog2eShort);     // q = fq 2^(za kLog2e - Ma)
    const double fp = exp2(((double)Mp - cp) + lse_p * kLog2eShort);     // p / lambda = fp 2^(zp kLog2e - Mp)
    const float ratio = (float)(fp / fq);
    float acc = 0.f, kl = 0.f;
    for (int64_t v0 = 0; v0 < nvt; v0 += (int64_t)XNT * XUNROLL) {
      uint4 va[XUNROLL], vp[XUNROLL];
      load_tile<DT>(va, vp, ra, rp, v0, nvec, tail, tid);
#pragma unroll
      for (int j = 0; j < XUNROLL; ++j) {
#pragma unroll
        for (int e = 0; e < N; ++e) {
          const float za = Vec<DT>::get(va[j], e), zp = Vec<DT>::get(vp[j], e);
          const float p = ex2_approx(fmaf(zp, kLog2e, -Mp));
          if (WANT_Z) {
            const float q = ex2_approx(fmaf(za, kLog2e, -Ma));
            acc += fminf(q, p * ratio);
          }
          if (WANT_KL && p > 0.f) kl = fmaf(p, zp - za, kl);
        }
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      acc += __shfl_xor_sync(0xffffffffu, acc, off);
      kl += __shfl_xor_sync(0xffffffffu, kl, off);
    }
    if (lane == 0) { red[0][warp] = acc; red[1][warp] = kl; }
    __syncthreads();
    if (tid == 0) {
      double S = 0.0, K = 0.0;
      for (int w = 0; w < XNWARP; ++w) { S += (double)red[0][w]; K += (double)red[1][w]; }
      if (WANT_Z) A.out[rrow] = (float)(S * fq);
      if (WANT_KL) A.out_kl[rrow] = (float)(K * fp * lambda - lse_p + lse_a);
    }
    __syncthreads();
  }
}

// Self-test of the bounded wait: one CTA whose warps wait, through the same routine as the row
// kernel's roles, on a barrier that nobody ever arrives at, with a limit the caller gives.  The
// wait must run out, raise the CTA's abort flag (which releases the warps still waiting), leave
// JP_ERR_TIMEOUT in the status word and let the kernel end: no trap, no hang, the context stays
// usable.
__global__ void __launch_bounds__(128) wait_selftest_kernel(long long limit_cycles, int32_t* status) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // warp 0 has the caller's limit; the others the kernel's own two seconds: they must be let go by
  // the abort flag, as the row kernel's other roles are
  const bool ok = mbar_wait_slow(&bar, 0u, &abort_flag, (threadIdx.x >> 5) == 0 ? limit_cycles : kSpinLimit);
  if (!ok && (threadIdx.x & 31) == 0) atomicExch(status, (int)JP_ERR_TIMEOUT);
}

cudaError_t launch_wait_selftest(long long limit_cycles, int32_t* status, cudaStream_t s) {
  wait_selftest_kernel<<<1, 128, 0, s>>>(limit_cycles, status);
  return cudaGetLastError();
}

int stream_grid_size(int device) {
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  return sms;
}

template <int DT, int KPL, bool SINGLE>
static cudaError_t launch_stream_variant(const StreamArgs& a, cudaStream_t s, int grid) {
  // per device, and cheap: set on every launch rather than cached per process
  cudaError_t e = cudaFuncSetAttribute(stream_kernel<DT, KPL, SINGLE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)sizeof(StreamSmemFor<KPL, SINGLE>));
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(NTHREADS);
  cfg.dynamicSmemBytes = sizeof(StreamSmemFor<KPL, SINGLE>);
  cfg.stream = s;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may begin while the row-list kernel before it runs
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, stream_kernel<DT, KPL, SINGLE>, a);
}

template <int DT>
static cudaError_t launch_stream_dt(const StreamArgs& a, cudaStream_t s, int grid) {
  const int kpl = a.k <= 0 ? 0 : a.k <= 32 ? 1 : a.k <= 64 ? 2 : 4;
  if (a.za == nullptr) {           // the policy tensor alone (the rollout model comes as a stored record)
    switch (kpl) {
      case 0: return cudaErrorInvalidValue;
      case 1: return launch_stream_variant<DT, 1, true>(a, s, grid);
      case 2: return launch_stream_variant<DT, 2, true>(a, s, grid);
      default: return launch_stream_variant<DT, 4, true>(a, s, grid);
    }
  }
  switch (kpl) {
    case 0: return launch_stream_variant<DT, 0, false>(a, s, grid);
    case 1: return launch_stream_variant<DT, 1, false>(a, s, grid);
    case 2: return launch_stream_variant<DT, 2, false>(a, s, grid);
    default: return launch_stream_variant<DT, 4, false>(a, s, grid);
  }
}

cudaError_t launch_stream(const StreamArgs& a, cudaStream_t s, int sms) {
  if (a.T <= 0) return cudaSuccess;
  prep_rows_kernel<<<(unsigned)((a.T + 255) / 256), 256, 0, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  int grid = (int)(a.T < sms ? a.T : sms);
  if (grid > kStreamMaxCtas) grid = kStreamMaxCtas;      // the spill area is laid out for that many CTAs
  return a.dtype == JP_BF16 ? launch_stream_dt<JP_BF16>(a, s, grid) : launch_stream_dt<JP_F32>(a, s, grid);
}

template <int DT>
static void launch_exact_z_dt(const ExactZArgs& a, int g, cudaStream_t s) {
  if (a.out && a.out_kl) exact_z_kernel<DT, true, true><<<g, XNT, 0, s>>>(a);
  else if (a.out) exact_z_kernel<DT, true, false><<<g, XNT, 0, s>>>(a);
  else exact_z_kernel<DT, false, true><<<g, XNT, 0, s>>>(a);
}

cudaError_t launch_exact_z(const ExactZArgs& a, cudaStream_t s, int sms) {
  if (a.T <= 0 || (!a.out && !a.out_kl)) return cudaSuccess;
  const int grid = sms * XCTAS_PER_SM;
  int g = (int)(a.T < grid ? a.T : grid);
  if (a.dtype == JP_BF16) launch_exact_z_dt<JP_BF16>(a, g, s);
  else launch_exact_z_dt<JP_F32>(a, g, s);
  return cudaGetLastError();
}

}  // namespace jp
