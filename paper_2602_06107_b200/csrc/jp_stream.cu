// Row-streaming kernels: each valid row of the actor and policy logits is read
// from HBM once; the pass yields both log-sum-exps (online max / rescaled sum),
// the sampled token's logits and the two top-k lists (Section 4.4.1: V_k is the
// union of top-k(p_inf) and top-k(p_new)), each candidate carrying both logits.
// A second kernel sums the exact normaliser Z over the vocabulary (Eq. obrs_dist).
//
// Shape of the stream kernel (one persistent CTA per SM, one row pair at a time):
//
//   producer warp   one lane issues 1-D bulk async copies (global -> shared,
//                   completion counted on an mbarrier) of the next tile of both
//                   rows into a ring of STAGES shared-memory stages;
//   consumer warps  two groups that take alternate tiles of a row: wait for a stage,
//                   pull their 16-byte vectors into registers pass by pass, update
//                   the online (max, sum) of both rows and leave the maximum of
//                   every pass (two vectors) in shared memory beside the stage;
//   top-k warps     eight of them, one per (tensor, row slot, tile parity).  Per
//                   tile a warp loads the 512 pass maxima (16 per lane), frees the
//                   stage and counts the passes at or above its running threshold
//                   tau in a histogram over the 16-bit order code of the maximum;
//                   tau is the highest code with at least k passes at or above it
//                   (k different passes hold k different entries, so the k-th best
//                   logit is not below it): nothing is sorted while streaming.  A
//                   pass at or above tau is kept as (pass, maximum).  At the end of
//                   the row the vectors of the kept passes are read back, their
//                   entries at or above tau are sorted into the list (bitonic sort /
//                   merge across the lanes), the two parity warps' lists are merged,
//                   and the warp finishes the log-sum-exp, gathers the sampled
//                   token's logit and writes the row's record.
//
// Rows alternate between two "slots" (histograms, survivors, partial sums,
// barriers), so the consumers start the next row while the top-k warps finish
// the previous one.  The total order of the top-k is (logit desc, index asc), one
// 64-bit key; the result does not depend on the order in which candidates arrive.
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

#ifndef JP_NC
#define JP_NC 16
#endif
#ifndef JP_VPL
#define JP_VPL 4
#endif
#ifndef JP_TOPK_SLEEP_NS
#define JP_TOPK_SLEEP_NS 300
#endif
#ifndef JP_STAGES
#define JP_STAGES 5
#endif
#ifndef JP_NG
#define JP_NG 2
#endif
constexpr int NC = JP_NC;                 // consumer warps
constexpr int NG = JP_NG;                 // consumer groups: group q takes tiles q, q + NG, ...
constexpr int WPT = NC / NG;              // warps that share one tile
constexpr int VPL = JP_VPL;               // 16-byte vectors per lane per tensor per tile
constexpr int TV = WPT * 32 * VPL;        // vectors per tensor per tile
constexpr int HV = 2;                     // vectors per tensor a lane holds at a time
static_assert(JP_VPL % HV == 0, "a tile is taken in passes of HV vectors");
static_assert(JP_NG == 2, "tiles go to consumer groups and top-k warps by parity; the producer keeps two phase masks");
static_assert(NC % NG == 0 && NG < JP_STAGES, "consumer groups must divide the warps and fit the ring");
constexpr int STAGES = JP_STAGES;
constexpr int SCAP = 288;                 // buffered keys per top-k warp (used while sorting survivors into the list)
constexpr int SVCAP = 288;                // candidate passes a top-k warp keeps until the row ends
constexpr int NB = 256;                   // histogram bins: 16-bit order codes below the warp's first tile's maximum
constexpr int TP = TV / HV;               // passes per tensor per tile = pass maxima a top-k warp scans per tile
static_assert(TP == 512, "a top-k lane scans 16 pass maxima per tile (4 x 16 bytes)");
constexpr int NTOPK = 8;                  // top-k warps: (tensor, slot, tile parity)
constexpr int NWARPS = 1 + NC + NTOPK;
constexpr int NTHREADS = NWARPS * 32;
constexpr uint32_t QEMPTY = 0xffffffffu;
constexpr long long kSpinLimit = 4000000000ll;   // clock cycles a wait may last (about 2 s)

struct __align__(128) StreamSmem {
  uint4 ring[STAGES][2][TV];              // [stage][tensor][vector]
  float passmax[STAGES][2][TP];           // [stage][tensor] maximum of each consumer pass (HV vectors) of the tile
  unsigned long long skeys[2][2][2][SCAP];  // [slot][tensor][tile parity] keys waiting to be sorted into the list; the parity-0 warp leaves its finished list here
  uint32_t svpass[2][2][2][SVCAP];        // [slot][tensor][tile parity] candidate passes still alive under tau: tile * TP + entry ...
  float svmax[2][2][2][SVCAP];            // ... and their maxima
  uint32_t hist[2][2][2][NB];             // [slot][tensor][tile parity] passes seen per order code of their maximum
  unsigned long long full[NG][STAGES];    // [consumer group] producer -> that group: the tile's bytes have landed.  One set per
                                          // group, so that every waiter sees every phase of its barriers in turn: a group that
                                          // skipped the other group's phases could take an unfinished earlier phase for its own
  unsigned long long seen[2][2][STAGES];  // [slot][tile parity] consumers -> top-k warps: tile consumed, pass maxima written
  unsigned long long empty[STAGES];       // -> producer: the stage may be refilled
  unsigned long long row_done[2], slot_free[2];
  unsigned long long scan_done[2][2];     // [slot][tensor] parity-0 warp -> parity-1 warp: my part of the row is in shared memory
  unsigned long long final_done[2][2];    // [slot][tensor] parity-1 warp -> parity-0 warp: I have read it
  int xstate[2][2][4];                    // [slot][tensor] parity-0 hand-over: kept vectors, tau code, keys in xkeys
  float part_mL[2][2][NC];
  float part_s[2][2][NC];
  int abort;
};

static_assert(sizeof(StreamSmem) <= 232448, "the CTA's shared memory exceeds the 227 KB an sm_100 CTA can have");

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
// Bounded wait; false = gave up (or another warp did).  The clock is read once in
// 64 polls, each of which may itself suspend the thread for a while.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, volatile int* abort) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait_for(bar, parity, 2000u)) return true;
    if ((i & 63u) == 0u) {
      if (*abort) return false;
      const long long now = clock64();
      if (i == 0u) t0 = now;
      else if (now - t0 > kSpinLimit) { *abort = 1; return false; }
    }
  }
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
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

// Online softmax state of one thread for one tensor: running max m, the integer
// reference exponent mL = ceil(m * log2 e), and two partial sums (packed)
// relative to 2^mL.  Every term is 2^(z log2 e - mL) <= 1.
struct Online {
  float m, mL;
  unsigned long long s2;
};

#ifndef JP_POLY_WORDS
#define JP_POLY_WORDS 0
#endif
// 2^x for two x <= ~0 without the special-function unit, folded into the running
// sums: returns s + 2^x (both lanes).  x is rounded to the nearest integer n with the
// 1.5 * 2^23 trick, 2^(x - n) comes from a degree-5 polynomial on [-0.5, 0.5] (fitted
// for the smallest maximum relative error, 1.7e-7, about that of ex2.approx) and 2^n
// is built in the exponent field.  x is clamped at -125 so that the exponent stays
// valid: terms below 2^-125 count as 2^-125, far below one ulp of any sum that holds
// a term near 1.  A NaN stays a NaN.
__device__ __forceinline__ unsigned long long add_exp2_poly2(unsigned long long s2, unsigned long long x2) {
  float x0, x1;
  unpack2(x2, x0, x1);
  asm("max.NaN.f32 %0, %0, %1;" : "+f"(x0) : "f"(-125.f));
  asm("max.NaN.f32 %0, %0, %1;" : "+f"(x1) : "f"(-125.f));
  x2 = pack2(x0, x1);
  const unsigned long long t2 = fadd2(x2, pack2(12582912.f, 12582912.f));
  const unsigned long long n2 = fadd2(t2, pack2(-12582912.f, -12582912.f));
  const unsigned long long f2 = ffma2(n2, pack2(-1.f, -1.f), x2);
  unsigned long long p2 = ffma2(pack2(1.326462603e-03f, 1.326462603e-03f), f2, pack2(9.671481326e-03f, 9.671481326e-03f));
  p2 = ffma2(p2, f2, pack2(5.550733581e-02f, 5.550733581e-02f));
  p2 = ffma2(p2, f2, pack2(2.402224243e-01f, 2.402224243e-01f));
  p2 = ffma2(p2, f2, pack2(6.931470037e-01f, 6.931470037e-01f));
  p2 = ffma2(p2, f2, pack2(1.f, 1.f));
  float t0, t1;
  unpack2(t2, t0, t1);
  const float sc0 = __int_as_float((__float_as_int(t0) << 23) + 0x3f800000);
  const float sc1 = __int_as_float((__float_as_int(t1) << 23) + 0x3f800000);
  return ffma2(p2, pack2(sc0, sc1), s2);
}

// One 16-byte vector into the online (max, sum).
template <int DT>
__device__ __forceinline__ void accumulate(const uint4& v, float vm, Online& o) {
  if (vm > o.m) {
    const float nmL = ceilf(__fmul_rn(vm, kLog2e));
    if (o.m == JP_NEG_INF) {
      o.s2 = 0ull;
    } else if (nmL != o.mL) {
      const float f = exp2_int(o.mL - nmL);
      o.s2 = fmul2(o.s2, pack2(f, f));
    }
    o.m = vm;
    o.mL = nmL;
  }
#ifdef JP_SCALAR_ACC
  {
    float s0, s1;
    unpack2(o.s2, s0, s1);
    const float nm = -o.mL;
    if (DT == JP_BF16) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        s0 += ex2_approx(fmaf(__uint_as_float(w[i] << 16), kLog2e, nm));
        s1 += ex2_approx(fmaf(__uint_as_float(w[i] & 0xffff0000u), kLog2e, nm));
      }
    } else {
      s0 += ex2_approx(fmaf(__uint_as_float(v.x), kLog2e, nm));
      s1 += ex2_approx(fmaf(__uint_as_float(v.y), kLog2e, nm));
      s0 += ex2_approx(fmaf(__uint_as_float(v.z), kLog2e, nm));
      s1 += ex2_approx(fmaf(__uint_as_float(v.w), kLog2e, nm));
    }
    o.s2 = pack2(s0, s1);
    return;
  }
#endif
  const unsigned long long L2 = pack2(kLog2e, kLog2e);
  const unsigned long long nm2 = pack2(-o.mL, -o.mL);
  if (DT == JP_BF16) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      unsigned long long a = ffma2(pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u)), L2, nm2);
      if (i >= 4 - JP_POLY_WORDS) {
        // a share of the exponentials runs on the FMA pipe: one ex2 per logit would
        // saturate the special-function unit before HBM
        o.s2 = add_exp2_poly2(o.s2, a);
      } else {
        float a0, a1;
        unpack2(a, a0, a1);
        o.s2 = fadd2(o.s2, pack2(ex2_approx(a0), ex2_approx(a1)));
      }
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

// The running threshold of one (row, tensor).  `code` is the highest 16-bit order
// code with at least k of the candidate vectors seen so far having their maximum
// at or above it: k different vectors hold k different entries, so the k-th best
// logit of the row is at or above the low edge of that code's bin.  `cnt` counts
// the vectors at or above it.  `key` is the exact k-th best key of the sorted
// list once candidates have been sorted into it (0 before).
struct Tau {
  uint32_t code;
  int cnt;
  unsigned long long key;
};

__device__ __forceinline__ uint32_t order_code(float v) { return f32_order_bits(v) >> 16; }
// low edge of a code's bin, as a logit
__device__ __forceinline__ float code_value(uint32_t code) { return order_bits_f32(code << 16); }

// v[i] for a run-time i in 0..15 without indexing the register array (a select tree).
__device__ __forceinline__ float select16(const float (&v)[16], int i) {
  float a[8], b[4], c[2];
#pragma unroll
  for (int j = 0; j < 8; ++j) a[j] = (i & 1) ? v[2 * j + 1] : v[2 * j];
#pragma unroll
  for (int j = 0; j < 4; ++j) b[j] = (i & 2) ? a[2 * j + 1] : a[2 * j];
#pragma unroll
  for (int j = 0; j < 2; ++j) c[j] = (i & 4) ? b[2 * j + 1] : b[2 * j];
  return (i & 8) ? c[1] : c[0];
}

// First vector index of pass `id` (= tile * TP + entry) and the step to its next vector.
__device__ __forceinline__ uint32_t pass_first_vector(uint32_t id) {
  const uint32_t tile = id / TP, e = id % TP;
  return tile * TV + (e / (WPT * 32)) * HV * (WPT * 32) + e % (WPT * 32);
}

// Can the pass with maximum order bits `ob` still hold one of the k best?
__device__ __forceinline__ bool pass_alive(uint32_t ob, uint32_t id, int n_per_vec, const Tau& tau) {
  if ((ob >> 16) < tau.code) return false;
  if (tau.key == 0ull) return true;
  // its best possible entry: the maximum at the first index of the pass's first vector
  const uint32_t idx = pass_first_vector(id) * (uint32_t)n_per_vec;
  return (((unsigned long long)ob << 32) | (unsigned long long)(uint32_t)(~idx)) > tau.key;
}

// The highest histogram bin with at least k counted passes at or above it (0 if
// fewer than k passes were counted).  Lane l sums bins 8 l .. 8 l + 7, a shuffle
// suffix scan finds the lane in which the count crosses k, and that lane walks its
// bins from the top.
__device__ __forceinline__ int find_tau_bin(const uint32_t* hist, int k, int lane) {
  static_assert(NB == 256, "8 bins per lane");
  const uint4* h4 = reinterpret_cast<const uint4*>(hist) + lane * 2;
  uint32_t b[8];
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const uint4 v = h4[q];
    b[4 * q] = v.x; b[4 * q + 1] = v.y; b[4 * q + 2] = v.z; b[4 * q + 3] = v.w;
  }
  int mine = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) mine += (int)b[i];
  int suf = mine;                                   // passes in this lane's bins and all higher lanes'
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

// Drops the kept candidate passes that tau has ruled out since they were kept.
__device__ __noinline__ int compact_survivors(uint32_t* svp, float* svm, int nsv, Tau tau, int n_per_vec, int lane) {
  int out = 0;
  for (int b = 0; b < nsv; b += 32) {
    const int i = b + lane;
    uint32_t id = 0u;
    float m = 0.f;
    bool keep = false;
    if (i < nsv) {
      id = svp[i];
      m = svm[i];
      keep = pass_alive(f32_order_bits(m), id, n_per_vec, tau);
    }
    const uint32_t bm = __ballot_sync(0xffffffffu, keep);
    __syncwarp();
    if (keep) {
      const int o = out + __popc(bm & ((1u << lane) - 1u));
      svp[o] = id;
      svm[o] = m;
    }
    out += __popc(bm);
    __syncwarp();
  }
  return out;
}

// Appends to the key buffer the keys of one vector's entries (one vector per lane)
// that can still be among the k best.  Returns the new number of buffered keys.
template <int DT>
__device__ __forceinline__ int stage_entries(const uint4& v, uint32_t vi, bool have, int64_t V, const Tau& tau,
                                             unsigned long long* stg, int staged, int lane) {
  constexpr int N = Vec<DT>::N;
  const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
  for (int e = 0; e < N; ++e) {
    const uint32_t idx = vi * N + e;
    const uint32_t ob = f32_order_bits(Vec<DT>::get(v, e));
    const unsigned long long key = ((unsigned long long)ob << 32) | (unsigned long long)(uint32_t)(~idx);
    const bool keep = have && (int64_t)idx < V && (ob >> 16) >= tau.code && key > tau.key;
    const uint32_t bk = __ballot_sync(0xffffffffu, keep);
    if (keep) stg[staged + __popc(bk & lt)] = key;
    staged += __popc(bk);
  }
  __syncwarp();
  return staged;
}

// Folds every buffered key into the sorted list; returns the list's k-th key.
template <int KPL>
__device__ __noinline__ unsigned long long merge_all(unsigned long long (&L)[KPL], const unsigned long long* stg,
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

// Sorts the entries of every kept pass into the list (exact from here on: tau.key
// becomes the list's k-th key) and empties the survivor buffer.  The vectors of a
// pass are read back from memory (they left the ring long ago; a few hundred
// 16-byte reads per row, mostly L2 hits).
template <int DT, int KPL>
__device__ __noinline__ void survivors_to_list(unsigned long long (&L)[KPL], const uint32_t* svp, int& nsv,
                                               const char* row, int64_t nvec, int64_t V, Tau& tau,
                                               unsigned long long* stg, int k, int lane) {
  int staged = 0;
  for (int b = 0; b < nsv; b += 32) {
    const int i = b + lane;
    const uint32_t v0 = i < nsv ? pass_first_vector(svp[i]) : 0u;
    uint4 v[HV];
    bool in[HV];
#pragma unroll
    for (int j = 0; j < HV; ++j) {
      const uint32_t vi = v0 + j * (WPT * 32);
      in[j] = i < nsv && (int64_t)vi < nvec;
      v[j] = in[j] ? ldg_stream((const uint4*)row + vi) : Vec<DT>::neg_inf();
    }
#pragma unroll
    for (int j = 0; j < HV; ++j) {
      staged = stage_entries<DT>(v[j], v0 + j * (WPT * 32), in[j], V, tau, stg, staged, lane);
      if (staged > SCAP - 32 * Vec<DT>::N) tau.key = merge_all<KPL>(L, stg, staged, k, lane);
    }
  }
  tau.key = merge_all<KPL>(L, stg, staged, k, lane);
  nsv = 0;
}

__device__ __forceinline__ void raise_timeout(StreamSmem& sm, Scalars* sc) {
  sm.abort = 1;
  atomicExch(&sc->status, (int)JP_ERR_TIMEOUT);
}

// ---- producer ---------------------------------------------------------------
template <int DT>
__device__ void producer_loop(const StreamArgs& A, StreamSmem& sm, int64_t n_rows) {
  constexpr int N = Vec<DT>::N;
  const int64_t nvec = A.V / N;
  const int ntiles = nvec > 0 ? (int)((nvec + TV - 1) / TV) : 1;
  const uint32_t last_bytes = (uint32_t)((nvec - (int64_t)(ntiles - 1) * TV) * 16);   // 0 only when nvec == 0
  const int64_t pitch = A.ld * Vec<DT>::ESIZE;
  // This lane is the one latency-critical thread of the CTA: a freed stage waits for it.
  // Stage and phase advance by increments, addresses by additions, and the next row's
  // index is fetched one row ahead.
  uint32_t s = 0, ph = 0, armed = 0;
  uint32_t fph0 = 0u, fph1 = 0u, last_grp = 0u, last_ph = 0u;   // per stage: phase bits of full[0], full[1]; group and phase armed last
  bool ok = true;
  int64_t it = blockIdx.x;
  int64_t row = it < n_rows ? A.list[it] : 0;
  while (it < n_rows && ok) {
    const char* ra = (const char*)A.za + row * pitch;
    const char* rp = (const char*)A.zp + row * pitch;
    it += gridDim.x;
    if (it < n_rows) row = A.list[it];
    for (int tile = 0; tile < ntiles; ++tile, ra += TV * 16, rp += TV * 16) {
      if (!mbar_wait(&sm.empty[s], ph ^ 1u, &sm.abort)) { ok = false; break; }
      const uint32_t bytes = tile == ntiles - 1 ? last_bytes : (uint32_t)(TV * 16);
      const int grp = tile % NG;
      if (bytes > 0) {
        mbar_arrive_expect_tx(&sm.full[grp][s], 2u * bytes);
        bulk_g2s(&sm.ring[s][0][0], ra, bytes, &sm.full[grp][s]);
        bulk_g2s(&sm.ring[s][1][0], rp, bytes, &sm.full[grp][s]);
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
template <int DT, bool TOPK>
__device__ void consumer_loop(const StreamArgs& A, StreamSmem& sm, int64_t n_rows, int cw, int lane) {
  constexpr int N = Vec<DT>::N;
  const int64_t nvec = A.V / N;
  const int tail = (int)(A.V - nvec * N);
  const uint32_t ntiles = nvec > 0 ? (uint32_t)((nvec + TV - 1) / TV) : 1u;
  const int gq = cw / WPT;              // this warp's group: it takes tiles gq, gq + NG, ...
  const int wq = cw % WPT;              // its place among the warps that share a tile
  uint32_t g0 = 0;                      // ring position of the current row's tile 0
  uint32_t fphase = 0u;                 // per stage: phase bit of this group's full barrier
  int lr = 0;
  for (int64_t it = blockIdx.x; it < n_rows; it += gridDim.x, ++lr, g0 += ntiles) {
    const int p = lr & 1;
    const uint32_t ph = (uint32_t)((lr >> 1) & 1);
    // the slot's partial sums are free once both of its top-k warps have finished
    // the row that used it before
    if (!mbar_wait(&sm.slot_free[p], ph ^ 1u, &sm.abort)) { raise_timeout(sm, A.sc); return; }

    Online oa{JP_NEG_INF, 0.f, 0ull}, op{JP_NEG_INF, 0.f, 0ull};

    // One tile of both rows, taken in passes of HV vectors per tensor: a short loop
    // body keeps the streaming code small for the instruction caches and the live
    // registers few.  The only thing a consumer does for the top-k is to leave the
    // maximum of every pass in shared memory; the top-k warps scan those.
    auto consume_tile = [&](uint32_t tile) -> bool {
      const uint32_t g = g0 + tile;
      const uint32_t s = g % STAGES;
      if (!mbar_wait(&sm.full[gq][s], (fphase >> s) & 1u, &sm.abort)) return false;
      fphase ^= 1u << s;
      const uint4* sa = &sm.ring[s][0][wq * 32 + lane];
      const uint4* sp = &sm.ring[s][1][wq * 32 + lane];
      float* pma = &sm.passmax[s][0][wq * 32 + lane];
      float* pmp = &sm.passmax[s][1][wq * 32 + lane];
      if ((int64_t)(tile + 1) * TV <= nvec) {
        // a full tile: no bounds checks
#pragma unroll 1
        for (int h = 0; h < VPL / HV; ++h, sa += HV * WPT * 32, sp += HV * WPT * 32, pma += WPT * 32, pmp += WPT * 32) {
          uint4 va[HV], vp[HV];
#pragma unroll
          for (int j = 0; j < HV; ++j) { va[j] = sa[j * WPT * 32]; vp[j] = sp[j * WPT * 32]; }
          if (!TOPK && h == VPL / HV - 1) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[s]);   // the last vectors are in registers: stage free
          }
          float ma = JP_NEG_INF, mp = JP_NEG_INF;
#pragma unroll
          for (int j = 0; j < HV; ++j) {
            const float vm_a = Vec<DT>::vmax(va[j]), vm_p = Vec<DT>::vmax(vp[j]);
            accumulate<DT>(va[j], vm_a, oa);
            accumulate<DT>(vp[j], vm_p, op);
            ma = fmaxf(ma, vm_a);
            mp = fmaxf(mp, vm_p);
          }
          if (TOPK) { *pma = ma; *pmp = mp; }
        }
      } else {
        // the row's last, partial tile: bounds checked
        const uint32_t v0 = tile * TV + wq * 32 + lane;
#pragma unroll 1
        for (int h = 0; h < VPL / HV; ++h, pma += WPT * 32, pmp += WPT * 32) {
          float ma = JP_NEG_INF, mp = JP_NEG_INF;
#pragma unroll 1
          for (int j = 0; j < HV; ++j) {
            const int o = (h * HV + j) * WPT * 32;
            uint4 a4 = Vec<DT>::neg_inf(), p4 = Vec<DT>::neg_inf();
            if ((int64_t)(v0 + o) < nvec) { a4 = sa[o]; p4 = sp[o]; }
            const float vm_a = Vec<DT>::vmax(a4), vm_p = Vec<DT>::vmax(p4);
            accumulate<DT>(a4, vm_a, oa);
            accumulate<DT>(p4, vm_p, op);
            ma = fmaxf(ma, vm_a);
            mp = fmaxf(mp, vm_p);
          }
          if (TOPK) { *pma = ma; *pmp = mp; }
        }
        if (!TOPK) {
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.empty[s]);
        }
      }
      if (TOPK) {
        // the top-k warps of this row's slot take it from here; they free the stage
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.seen[p][tile & 1u][s]);
      }
      return true;
    };
    for (uint32_t tile = gq; tile < ntiles; tile += NG)
      if (!consume_tile(tile)) { raise_timeout(sm, A.sc); return; }

    if (tail > 0 && cw == 0 && lane == 0) {     // ragged end of the row: scalar loads
      const int64_t row = A.list[it];
      const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
      const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;
      const uint4 ta = load_tail_vector<DT>(ra, nvec * N, tail);
      const uint4 tp = load_tail_vector<DT>(rp, nvec * N, tail);
      accumulate<DT>(ta, Vec<DT>::vmax(ta), oa);
      accumulate<DT>(tp, Vec<DT>::vmax(tp), op);
    }

    // per-warp (max, sum) pairs, merged in a fixed tree
    float mL_a = oa.mL, mL_p = op.mL, s_a, s_p;
    {
      float s0, s1;
      unpack2(oa.s2, s0, s1); s_a = s0 + s1;
      unpack2(op.s2, s0, s1); s_p = s0 + s1;
    }
    if (oa.m == JP_NEG_INF) mL_a = JP_NEG_INF;   // a thread that saw nothing must not set the scale
    if (op.m == JP_NEG_INF) mL_p = JP_NEG_INF;
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
// One warp per (tensor t, row slot p).  For every tile of its row it waits until
// the consumers are through with the stage, scans the 512 pass maxima they left
// (16 per lane), counts in the histogram those at or above the running threshold
// and copies the vectors behind them that are still alive from the stage into the
// survivor buffer; then it frees the stage.  The threshold is the low edge of the
// highest histogram bin with k counted passes at or above it: k different passes
// hold k different entries of the row, so the k-th best logit is not below it.
template <int DT, int KPL>
__device__ void topk_loop(const StreamArgs& A, StreamSmem& sm, int64_t n_rows, int t, int p, int par, int lane) {
  constexpr int N = Vec<DT>::N;
  constexpr bool TOPK = KPL > 0;
  constexpr int KL = KPL > 0 ? KPL : 1;
  const int64_t nvec = A.V / N;
  const int tail = (int)(A.V - nvec * N);
  const uint32_t ntiles = nvec > 0 ? (uint32_t)((nvec + TV - 1) / TV) : 1u;
  const int k = A.k;
  unsigned long long* stg = sm.skeys[p][t][par];
  uint32_t* hist = sm.hist[p][t][par];
  uint32_t* svp = sm.svpass[p][t][par];
  float* svm = sm.svmax[p][t][par];
  // The tiles of a row are shared out by parity between two warps, each with a
  // histogram, a threshold and a survivor buffer of its own (the k-th best pass of
  // half the tiles is still a lower bound of the row's k-th best logit).  The
  // parity-0 warp hands its survivors over in shared memory at the end of the row;
  // the parity-1 warp sorts both sets into the list and writes the record.
  // A (slot, parity) `seen` barrier completes once per tile of that slot's rows with
  // that parity, and this warp waits for every one of them in turn, so one phase bit
  // per stage is enough.  (A barrier shared by warps that skip phases would not do: a
  // parity wait cannot tell "not yet reached" from "done".)
  uint32_t seen_phase = 0u;
  int lr = p;
  for (int64_t it = (int64_t)blockIdx.x + (int64_t)p * gridDim.x; it < n_rows; it += 2ll * gridDim.x, lr += 2) {
    const uint32_t ph = (uint32_t)((lr >> 1) & 1);
    const uint32_t g0 = (uint32_t)lr * ntiles;        // ring position of this row's tile 0
    const int64_t row = A.list[it];
    const int64_t rrow = A.record_offset + row;
    const char* rmine = (const char*)(t == 0 ? A.za : A.zp) + row * A.ld * Vec<DT>::ESIZE;
    unsigned long long L[KL];
#pragma unroll
    for (int j = 0; j < KL; ++j) L[j] = 0ull;
    Tau tau{0u, 0, 0ull};
    uint32_t base = 0u;
    float tau_val = JP_NEG_INF;
    int nsv = 0;                                      // candidate vectors kept so far

    // the sampled token's logit is needed only at the end of the row: fetch it now
    float zx = 0.f;
    if (lane == 0) zx = Vec<DT>::load_scalar(rmine, A.tokens[row]);

    if (TOPK) {
      // the parity-1 warp must have read what this warp handed over two rows ago
      if (par == 0 && !mbar_wait(&sm.final_done[p][t], ph ^ 1u, &sm.abort)) { raise_timeout(sm, A.sc); return; }
      for (uint32_t tile = (uint32_t)par; tile < ntiles; tile += 2) {
        const uint32_t g = g0 + tile;
        const uint32_t s = g % STAGES;
        if (!mbar_wait(&sm.seen[p][par][s], (seen_phase >> s) & 1u, &sm.abort)) { raise_timeout(sm, A.sc); return; }
        seen_phase ^= 1u << s;
        const float* pm = sm.passmax[s][t];
        // this lane's 16 pass maxima: entries q * 128 + lane * 4 + c
        float v[16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 f = reinterpret_cast<const float4*>(pm)[q * 32 + lane];
          v[4 * q] = f.x; v[4 * q + 1] = f.y; v[4 * q + 2] = f.z; v[4 * q + 3] = f.w;
        }
        // everything this warp needs of the tile is in registers: the stage (logits and
        // pass maxima) may be refilled once the other tensor's warp says the same
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[s]);
        uint32_t hit = 0u;
        if (tile == (uint32_t)par) {
          // this warp's first tile of a new row: the histogram covers the NB order codes below this tile's maximum
          // (everything lower shares bin 0, which stands for "no threshold"); every pass
          // of the tile is counted, then the threshold is read off the histogram
          float mx = v[0];
#pragma unroll
          for (int i = 1; i < 16; ++i) mx = fmaxf(mx, v[i]);
          uint32_t top = __reduce_max_sync(0xffffffffu, order_code(mx));
          base = top > (uint32_t)(NB - 1) ? top - (uint32_t)(NB - 1) : 0u;
          for (int i = lane; i < NB; i += 32) hist[i] = 0u;
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint32_t code = order_code(v[i]);
            atomicAdd(&hist[code > base ? code - base : 0u], 1u);
          }
          __syncwarp();
          const int bin = find_tau_bin(hist, k, lane);
          tau.code = bin > 0 ? base + (uint32_t)bin : 0u;
          tau_val = bin > 0 ? code_value(tau.code) : JP_NEG_INF;
#pragma unroll
          for (int i = 0; i < 16; ++i) hit |= (v[i] >= tau_val ? 1u : 0u) << i;
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) hit |= (v[i] >= tau_val ? 1u : 0u) << i;
          if (__any_sync(0xffffffffu, hit != 0u)) {
            // count the passes at or above the threshold (those are all there are: it only rises)
            uint32_t hcount = hit;
            while (__any_sync(0xffffffffu, hcount != 0u)) {
              if (hcount) {
                const int i = __ffs(hcount) - 1;
                hcount &= hcount - 1u;
                const uint32_t code = order_code(select16(v, i));
                const uint32_t bin = code > base ? code - base : 0u;
                atomicAdd(&hist[bin < (uint32_t)(NB - 1) ? bin : (uint32_t)(NB - 1)], 1u);
              }
            }
            __syncwarp();
            const int bin = find_tau_bin(hist, k, lane);
            tau.code = bin > 0 ? base + (uint32_t)bin : 0u;
            tau_val = bin > 0 ? code_value(tau.code) : JP_NEG_INF;
          }
        }
        // keep the passes behind the hits that can still hold one of the k best: only
        // their place and their maximum; their vectors are read back when the row ends
        while (__any_sync(0xffffffffu, hit != 0u)) {
          const bool have = hit != 0u;
          uint32_t id = 0u;
          float m = JP_NEG_INF;
          if (have) {
            const int i = __ffs(hit) - 1;
            hit &= hit - 1u;
            const int e = (i >> 2) * 128 + lane * 4 + (i & 3);
            id = tile * TP + (uint32_t)e;
            m = select16(v, i);
          }
          const bool in = have && pass_alive(f32_order_bits(m), id, N, tau);
          const uint32_t bm = __ballot_sync(0xffffffffu, in);
          if (in) {
            const int o = nsv + __popc(bm & ((1u << lane) - 1u));
            svp[o] = id;
            svm[o] = m;
          }
          nsv += __popc(bm);
          __syncwarp();
          if (nsv > SVCAP - 32) {
            // the buffer is filling up: drop what the threshold has ruled out; if ties keep
            // it full, sort the kept entries into the list and go on with the exact k-th key
            nsv = compact_survivors(svp, svm, nsv, tau, N, lane);
            if (nsv > SVCAP / 2) {
              survivors_to_list<DT, KL>(L, svp, nsv, rmine, nvec, A.V, tau, stg, k, lane);
            }
          }
        }
      }
    }

    if (par == 0) {
      // this half of the row: sort the survivors into the list and leave the list in
      // this warp's key buffer for the parity-1 warp
      if (TOPK) {
        nsv = compact_survivors(svp, svm, nsv, tau, N, lane);
        survivors_to_list<DT, KL>(L, svp, nsv, rmine, nvec, A.V, tau, stg, k, lane);
#pragma unroll
        for (int j = 0; j < KL; ++j) stg[lane * KL + j] = L[j];
        if (lane == 0) { sm.xstate[p][t][0] = 0; sm.xstate[p][t][1] = (int)tau.code; sm.xstate[p][t][2] = 32 * KL; }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.scan_done[p][t]);
      }
      continue;
    }

    // the consumers' per-warp (max, sum) pairs of this row
    if (!mbar_wait(&sm.row_done[p], ph, &sm.abort)) { raise_timeout(sm, A.sc); return; }

    if (TOPK) {
      const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
      const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;
      // this warp's half of the row into its list ...
      nsv = compact_survivors(svp, svm, nsv, tau, N, lane);
      survivors_to_list<DT, KL>(L, svp, nsv, rmine, nvec, A.V, tau, stg, k, lane);
      // ... then the other half's list
      if (!mbar_wait(&sm.scan_done[p][t], ph, &sm.abort)) { raise_timeout(sm, A.sc); return; }
      const int nk0 = sm.xstate[p][t][2];
      if (tail > 0) {                 // the ragged end of the row
        uint4 v = Vec<DT>::neg_inf();
        if (lane == 0) v = load_tail_vector<DT>(rmine, nvec * N, tail);
        int staged = stage_entries<DT>(v, (uint32_t)nvec, lane == 0, A.V, tau, stg, 0, lane);
        tau.key = merge_all<KL>(L, stg, staged, k, lane);
      }
      if (nk0 > 0) {
        int staged = 0;
        for (int b = 0; b < nk0; b += 32) {
          const unsigned long long key = sm.skeys[p][t][0][b + lane];
          const bool keep = key > tau.key;
          const uint32_t m = __ballot_sync(0xffffffffu, keep);
          if (keep) stg[staged + __popc(m & ((1u << lane) - 1u))] = key;
          staged += __popc(m);
        }
        tau.key = merge_all<KL>(L, stg, staged, k, lane);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.final_done[p][t]);     // the parity-0 warp may reuse its buffers
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
            A.rec.za[o] = Vec<DT>::load_scalar(ra, idx);
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
      const double lse = ((double)M + (double)(e - 1)) * 0.6931471805599453 + (double)logf(f);
      const float lsef = (float)lse;
      const float lpx = (float)((double)zx - lse);
      if (t == 0) { A.rec.lse_a[rrow] = lsef; A.rec.lq[rrow] = lpx; A.rec.flag[rrow] = 1; }
      else        { A.rec.lse_p[rrow] = lsef; A.rec.lp[rrow] = lpx; }
      if (!isfinite(lsef)) atomicAdd(&A.sc->n_nonfinite, 1ull);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.slot_free[p]);
  }
}

template <int DT, int KPL>
__global__ void __launch_bounds__(NTHREADS, 1) stream_kernel(StreamArgs A) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  StreamSmem& sm = *reinterpret_cast<StreamSmem*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      for (int q = 0; q < NG; ++q) mbar_init(&sm.full[q][s], 1);
      for (int q = 0; q < 4; ++q) mbar_init(&sm.seen[q >> 1][q & 1][s], WPT);
      mbar_init(&sm.empty[s], KPL > 0 ? 2 : WPT);     // with top-k the two top-k warps of the row free the stage
    }
    for (int p = 0; p < 2; ++p) {
      mbar_init(&sm.row_done[p], NC);
      mbar_init(&sm.slot_free[p], 2);
      for (int t = 0; t < 2; ++t) { mbar_init(&sm.scan_done[p][t], 1); mbar_init(&sm.final_done[p][t], 1); }
    }
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int64_t n_rows = A.sc->n_list;

  if (warp == 0) {
    if (lane == 0) producer_loop<DT>(A, sm, n_rows);
  } else if (warp <= NC) {
    consumer_loop<DT, (KPL > 0)>(A, sm, n_rows, warp - 1, lane);
  } else {
    const int tw = warp - 1 - NC;
    // without top-k there is nothing to share out: the parity-0 warps leave
    if (KPL > 0 || (tw >> 2) == 1) topk_loop<DT, KPL>(A, sm, n_rows, tw & 1, (tw >> 1) & 1, tw >> 2, lane);
  }
}

// Splits the rows of one call into the list of valid rows the stream kernel walks
// and the masked / out-of-range ones, whose records are cleared here.
__global__ void __launch_bounds__(256) prep_rows_kernel(StreamArgs A) {
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

// Exact normaliser: Z_t = sum_v min(q_t(v), p_t(v)/lambda), one more pass over the
// row with the log-sum-exps known (Eq. obrs_dist; Appendix A, Z_C).
template <int DT>
__global__ void __launch_bounds__(XNT, XCTAS_PER_SM) exact_z_kernel(ExactZArgs A) {
  __shared__ float red[XNWARP];
  __shared__ int s_row;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int N = Vec<DT>::N;
  const int64_t nvec = A.V / N;
  const int tail = (int)(A.V - nvec * N);
  const int64_t nvt = nvec + (tail > 0 ? 1 : 0);
  const float log2_lambda = log2f(A.sc->lambda);
  for (;;) {
    if (tid == 0) s_row = atomicAdd(&A.sc->row_counter2, 1);
    __syncthreads();
    const int64_t row = s_row;
    __syncthreads();
    if (row >= A.T) break;
    const int64_t rrow = A.record_offset + row;
    if (!A.rec.flag[rrow]) {
      if (tid == 0) A.out[rrow] = 0.f;
      continue;
    }
    const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
    const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;
    const float ca = A.rec.lse_a[rrow] * kLog2e;
    const float cp = A.rec.lse_p[rrow] * kLog2e + log2_lambda;
    float acc = 0.f;
    for (int64_t v0 = 0; v0 < nvt; v0 += (int64_t)XNT * XUNROLL) {
      uint4 va[XUNROLL], vp[XUNROLL];
      load_tile<DT>(va, vp, ra, rp, v0, nvec, tail, tid);
#pragma unroll
      for (int j = 0; j < XUNROLL; ++j) {
#pragma unroll
        for (int e = 0; e < N; ++e) {
          float q = ex2_approx(fmaf(Vec<DT>::get(va[j], e), kLog2e, -ca));
          float p = ex2_approx(fmaf(Vec<DT>::get(vp[j], e), kLog2e, -cp));
          acc += fminf(q, p);
        }
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) red[warp] = acc;
    __syncthreads();
    if (tid == 0) {
      double S = 0.0;
      for (int w = 0; w < XNWARP; ++w) S += (double)red[w];
      A.out[rrow] = (float)S;
    }
    __syncthreads();
  }
}

int stream_grid_size(int device) {
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  return sms;
}

template <int DT, int KPL>
static cudaError_t launch_stream_variant(const StreamArgs& a, cudaStream_t s, int grid) {
  // per device, and cheap: set on every launch rather than cached per process
  cudaError_t e = cudaFuncSetAttribute(stream_kernel<DT, KPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)sizeof(StreamSmem));
  if (e != cudaSuccess) return e;
  stream_kernel<DT, KPL><<<grid, NTHREADS, sizeof(StreamSmem), s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_stream(const StreamArgs& a, cudaStream_t s, int sms) {
  if (a.T <= 0) return cudaSuccess;
  prep_rows_kernel<<<(unsigned)((a.T + 255) / 256), 256, 0, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int grid = (int)(a.T < sms ? a.T : sms);
  const int kpl = a.k <= 0 ? 0 : a.k <= 32 ? 1 : a.k <= 64 ? 2 : 4;
  if (a.dtype == JP_BF16) {
    switch (kpl) {
      case 0: return launch_stream_variant<JP_BF16, 0>(a, s, grid);
      case 1: return launch_stream_variant<JP_BF16, 1>(a, s, grid);
      case 2: return launch_stream_variant<JP_BF16, 2>(a, s, grid);
      default: return launch_stream_variant<JP_BF16, 4>(a, s, grid);
    }
  }
  switch (kpl) {
    case 0: return launch_stream_variant<JP_F32, 0>(a, s, grid);
    case 1: return launch_stream_variant<JP_F32, 1>(a, s, grid);
    case 2: return launch_stream_variant<JP_F32, 2>(a, s, grid);
    default: return launch_stream_variant<JP_F32, 4>(a, s, grid);
  }
}

cudaError_t launch_exact_z(const ExactZArgs& a, cudaStream_t s, int sms) {
  if (a.T <= 0) return cudaSuccess;
  const int grid = sms * XCTAS_PER_SM;
  int g = (int)(a.T < grid ? a.T : grid);
  if (a.dtype == JP_BF16) exact_z_kernel<JP_BF16><<<g, XNT, 0, s>>>(a);
  else exact_z_kernel<JP_F32><<<g, XNT, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace jp
