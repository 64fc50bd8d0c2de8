// The row pass fused into the output layer (Section 4.4: the [tokens, vocabulary] logit tensor
// is the memory bottleneck of the method; here it never exists).  One model's logits
//   z[t, v] = sum_h hidden[t, h] * weight[v, h]          (bf16 operands, fp32 accumulation)
// are produced tile by tile on the tensor cores and consumed straight from the accumulator:
// per row the log-sum-exp, the sampled token's logit and the k best entries under the order
// (logit desc, index asc).  Nothing of size T x V is written.
//
// Shape of the kernel (one CTA per SM, 192 threads; with more than 128 rows the CTAs work in pairs,
// see LmSmemT):
//   warp 0      one lane issues the TMA loads (cp.async.bulk.tensor.2d, 128-byte swizzle; every
//               byte is fetched by exactly one CTA) of the next K-slab of both operands into a ring of shared-memory
//               stages; completion is counted on an mbarrier per stage;
//   warp 1      allocates tensor memory; one lane issues tcgen05.mma (M = 128 rows, N = 256
//               columns, K = 16 per instruction, cta_group::1) into one of two accumulators of
//               256 fp32 columns each, frees a stage with tcgen05.commit when its MMAs have read
//               it, and hands a finished accumulator to the epilogue the same way;
//   warps 2..5  the epilogue: thread i of the warp that owns lane quarter q reads row 32 q + i of
//               the accumulator with tcgen05.ld (32 columns at a time) and folds it into the row's
//               running (max, sum) and its top-k list, while the tensor cores fill the other
//               accumulator with the next tile.
// A CTA owns 128 rows and a contiguous range of 256-column vocabulary tiles; the ranges of one
// row block are spread over the SMs (the grid is rows/128 x splits) and a second small kernel
// merges the splits' partial results: lse = log sum_j exp(lse_j), the token's logit from the
// split that holds it, the k best of the splits' k best.
//
// Every wait is bounded; a wait that runs out raises an error flag that the host reports, the
// roles leave their loops and tensor memory is freed before the CTA exits.
#include <cuda.h>

#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {
namespace {

constexpr int LM_BM = 128;                 // rows per CTA (= TMEM lanes)
constexpr int LM_BN = 256;                 // vocabulary columns per accumulator
constexpr int LM_BK = 64;                  // K per stage: 64 bf16 = one 128-byte swizzle row
constexpr int LM_UMMA_K = 16;              // K per tcgen05.mma of kind::f16
constexpr int LM_THREADS = 192;
constexpr uint32_t LM_A_BYTES = LM_BM * LM_BK * 2;     // 16 KB
constexpr uint32_t LM_B_BYTES = LM_BN * LM_BK * 2;     // 32 KB
constexpr uint32_t LM_TMEM_COLS = 512;     // two accumulators of 256 columns
constexpr long long kLmSpin = 4000000000ll;

// PAIR: two CTAs of a cluster work as one (tcgen05 cta_group::2): the pair owns 256 rows, each CTA
// loads its own 128 rows of `hidden` and HALF of the 256 `weight` rows of a tile (16 KB instead of
// 32 KB per stage), one thread of the even CTA issues MMAs of M = 256 that read both CTAs' shared
// memory and fill both CTAs' tensor memory.  Per SM the operand traffic of a tile falls by a
// third, and six stages fit where four did.
// KMAX: the longest list a row keeps (32 or 64); the longer lists take the place of one stage.
template <bool PAIR, int KMAX>
struct __align__(1024) LmSmemT {
  static constexpr int STAGES = (PAIR ? 6 : 4) - (KMAX > 32 ? 1 : 0);
  static constexpr uint32_t B_BYTES = PAIR ? LM_B_BYTES / 2 : LM_B_BYTES;
  unsigned char a[STAGES][LM_A_BYTES];     // [stage] 128 rows x 128 B, swizzled by the copy engine
  unsigned char b[STAGES][B_BYTES];        // [stage] 256 (PAIR: 128) rows x 128 B
  unsigned long long list[KMAX][LM_BM];    // per row: the k best so far as (order bits, ~column) keys, unsorted
                                           // (row fastest: no bank conflicts); 0 = empty place
  unsigned long long full[STAGES], empty[STAGES];
  unsigned long long acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort;
};
static_assert(sizeof(LmSmemT<false, 32>) <= 231424 && sizeof(LmSmemT<true, 32>) <= 231424 &&
                  sizeof(LmSmemT<false, 64>) <= 231424 && sizeof(LmSmemT<true, 64>) <= 231424,
              "beyond the 227 KB a CTA can have");

struct LmArgs {
  const int32_t* tokens;
  const uint8_t* mask;
  int64_t T, H, V;
  int32_t k, splits, tiles_per_split, n_tiles;
  // per (split, row) partial results
  float* part_m;       // running maximum, in units of log2
  double* part_s;      // sum of 2^(z log2 e - m)
  float* part_zx;      // the sampled token's logit (NaN if another split holds it)
  float* part_val;     // [split][T][k]
  int32_t* part_idx;
  int32_t* status;     // device status word
};

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(unsigned long long* b, uint32_t n) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(b)), "r"(n) : "memory");
}
__device__ __forceinline__ void bar_arrive(unsigned long long* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(b)) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(unsigned long long* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try(unsigned long long* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 1000;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(s32(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false = gave up (or another role did).
__device__ __noinline__ bool bar_wait(unsigned long long* b, uint32_t parity, volatile int* abort) {
  long long t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (bar_try(b, parity)) return true;
    if ((i & 63u) == 0u) {
      if (*abort) return false;
      const long long now = clock64();
      if (i == 0u) t0 = now;
      else if (now - t0 > kLmSpin) { *abort = 1; return false; }
    }
  }
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          s32(dst)),
      "l"(map), "r"(x), "r"(y), "r"(s32(bar))
      : "memory");
}
// Shared-memory matrix descriptor of a K-major operand tile whose rows are 128 bytes and which
// the copy engine wrote with the 128-byte swizzle: start address / 16, leading offset unused
// (1), 1024 bytes between groups of 8 rows, descriptor version 1, layout 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(const void* p) {
  uint64_t d = 0;
  d |= (uint64_t)((s32(p) & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor of kind::f16: fp32 accumulator, bf16 x bf16, both K-major, N = 256, M = 128.
constexpr uint32_t kLmIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(LM_BN >> 3) << 17) |
                              ((uint32_t)(LM_BM >> 4) << 24);
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(kLmIdesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(bar)) : "memory");
}
// The same instructions for a pair of CTAs.  The copy's completion is counted on the barrier of
// the pair's even CTA (bit 24 of a shared::cluster address is the CTA's rank in the pair).
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          s32(dst)),
      "l"(map), "r"(x), "r"(y), "r"(s32(bar) & 0xFEFFFFFFu)
      : "memory");
}
constexpr uint32_t kLmIdescPair = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(LM_BN >> 3) << 17) |
                                  ((uint32_t)((2 * LM_BM) >> 4) << 24);       // M = 256 over the pair
__device__ __forceinline__ void umma_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(kLmIdescPair), "r"(accumulate)
      : "memory");
}
// Arrival, once the MMAs issued so far are done, on the same barrier in both CTAs of the pair.
__device__ __forceinline__ void umma_commit_pair(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                   s32(bar)),
               "h"((unsigned short)3)
               : "memory");
}
// Arrival on the barrier at the same place in the shared memory of CTA `rank` of the cluster.
__device__ __forceinline__ void bar_arrive_remote(unsigned long long* bar, uint32_t rank) {
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
      "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}" ::"r"(s32(bar)),
      "r"(rank)
      : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(addr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}


// The row's k best so far are kept unsorted, as 64-bit keys under which a larger key is a better
// entry (higher logit; equal logits: lower column), with the place of the worst of them known.  A
// new entry that beats the worst overwrites that place, and one scan of the k keys (independent
// loads, four at a time: no chain of dependent shared-memory accesses as in a sorted insert) finds
// the next worst.  Returns its value (-inf while places are empty).
template <class SM>
__device__ __noinline__ float list_replace_worst(SM& sm, int row, int k, unsigned long long key, int& worst) {
  sm.list[worst][row] = key;
  unsigned long long wk = ~0ull;
  int w = 0;
  int j = 0;
  for (; j + 4 <= k; j += 4) {
    const unsigned long long k0 = sm.list[j][row], k1 = sm.list[j + 1][row], k2 = sm.list[j + 2][row],
                             k3 = sm.list[j + 3][row];
    if (k0 < wk) { wk = k0; w = j; }
    if (k1 < wk) { wk = k1; w = j + 1; }
    if (k2 < wk) { wk = k2; w = j + 2; }
    if (k3 < wk) { wk = k3; w = j + 3; }
  }
  for (; j < k; ++j) {
    const unsigned long long kj = sm.list[j][row];
    if (kj < wk) { wk = kj; w = j; }
  }
  worst = w;
  return wk == 0ull ? JP_NEG_INF : key_value(wk);
}

// Orders the row's k keys best first at the end of the CTA's range.
template <class SM>
__device__ __forceinline__ void list_sort(SM& sm, int row, int k) {
  for (int a = 0; a < k - 1; ++a) {
    unsigned long long bk = sm.list[a][row];
    int b = a;
    for (int j = a + 1; j < k; ++j) {
      const unsigned long long x = sm.list[j][row];
      if (x > bk) { bk = x; b = j; }
    }
    if (b != a) {
      sm.list[b][row] = sm.list[a][row];
      sm.list[a][row] = bk;
    }
  }
}

template <bool PAIR, int KMAX>
__global__ void __launch_bounds__(LM_THREADS, 1) lmhead_kernel(const __grid_constant__ CUtensorMap map_a,
                                                               const __grid_constant__ CUtensorMap map_b, LmArgs A) {
  extern __shared__ unsigned char lm_raw[];
  using SM = LmSmemT<PAIR, KMAX>;
  constexpr int LM_STAGES = SM::STAGES;
  SM& sm = *reinterpret_cast<SM*>(((uintptr_t)lm_raw + 1023) & ~(uintptr_t)1023);
  // in a pair the even CTA leads: it issues the MMAs and owns the barriers the copies are counted on
  uint32_t rank = 0;
  if (PAIR) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const bool leader = rank == 0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int m_block = blockIdx.x, split = blockIdx.y;
  const int tile0 = split * A.tiles_per_split;
  const int tile1 = min(tile0 + A.tiles_per_split, A.n_tiles);
  const int n_my = tile1 > tile0 ? tile1 - tile0 : 0;
  const int ksteps = (int)((A.H + LM_BK - 1) / LM_BK);

  if (tid == 0) {
    for (int s = 0; s < LM_STAGES; ++s) { bar_init(&sm.full[s], 1); bar_init(&sm.empty[s], 1); }
    for (int b = 0; b < 2; ++b) { bar_init(&sm.acc_full[b], 1); bar_init(&sm.acc_empty[b], PAIR ? 8 : 4); }
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    // tensor memory: all 512 columns (this CTA has the SM to itself: its shared memory fills it)
    if (PAIR) {                                              // the same warp of both CTAs, the same place for the address
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm.tmem_base)),
                   "r"(LM_TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm.tmem_base)),
                   "r"(LM_TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
  }
  __syncthreads();
  if (PAIR) cluster_sync_all();                              // the partner's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)&sm.tmem_base;

  if (warp == 0) {
    // ---- producer: K-slabs of both operands, tile after tile -------------------------------
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      bool ok = true;
      uint32_t armed = 0;
      for (int t = 0; t < n_my && ok; ++t) {
        const int col0 = (tile0 + t) * LM_BN;
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!bar_wait(&sm.empty[s], ph ^ 1u, &sm.abort)) { ok = false; break; }
          // coordinates: x = first K element (a multiple of 64: 128 bytes), y = first row
          if (PAIR) {
            // both CTAs' bytes are counted on the leader's barrier, which the leader arms for all four copies
            if (leader) bar_expect_tx(&sm.full[s], 2u * (LM_A_BYTES + SM::B_BYTES));
            tma_load_2d_pair(sm.a[s], &map_a, ks * LM_BK, m_block * LM_BM, &sm.full[s]);
            tma_load_2d_pair(sm.b[s], &map_b, ks * LM_BK, col0 + (int)rank * (LM_BN / 2), &sm.full[s]);
          } else {
            bar_expect_tx(&sm.full[s], LM_A_BYTES + SM::B_BYTES);
            tma_load_2d(sm.a[s], &map_a, ks * LM_BK, m_block * LM_BM, &sm.full[s]);
            tma_load_2d(sm.b[s], &map_b, ks * LM_BK, col0, &sm.full[s]);
          }
          ++armed;
          if (++s == LM_STAGES) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) atomicExch(A.status, (int)JP_ERR_TIMEOUT);
      if (!ok && leader) {
        // leave no copy in flight: wait (bounded) for what was armed last on every stage
        const uint32_t n_back = armed < (uint32_t)LM_STAGES ? armed : (uint32_t)LM_STAGES;
        for (uint32_t i = 1; i <= n_back; ++i) {
          const uint32_t idx = armed - i;                       // the i-th last armed slab
          const uint32_t st = idx % LM_STAGES, par = (idx / LM_STAGES) & 1u;
          const long long t0 = clock64();
          while (!bar_try(&sm.full[st], par))
            if (clock64() - t0 > kLmSpin) break;
        }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer (in a pair: the leader's) -------------------------------------------------
    if (lane == 0 && leader) {
      uint32_t s = 0, ph = 0;
      bool ok = true;
      for (int t = 0; t < n_my && ok; ++t) {
        const uint32_t buf = (uint32_t)t & 1u, use = (uint32_t)t >> 1;
        // the epilogue has drained this accumulator (first use of each: free from the start)
        if (!bar_wait(&sm.acc_empty[buf], (use & 1u) ^ 1u, &sm.abort)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d = tmem + buf * LM_BN;
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!bar_wait(&sm.full[s], ph, &sm.abort)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = smem_desc(sm.a[s]), db = smem_desc(sm.b[s]);
#pragma unroll
          for (int kk = 0; kk < LM_BK / LM_UMMA_K; ++kk) {
            // 16 bf16 = 32 bytes further along K inside the 128-byte swizzle row: start address + 2
            if (PAIR) umma_pair(d, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), (ks | kk) != 0 ? 1u : 0u);
            else umma(d, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), (ks | kk) != 0 ? 1u : 0u);
          }
          // the stage is free (in both CTAs of a pair) once these MMAs have read it
          if (PAIR) umma_commit_pair(&sm.empty[s]); else umma_commit(&sm.empty[s]);
          if (++s == LM_STAGES) { s = 0; ph ^= 1u; }
        }
        if (ok) {                                             // the accumulator is complete (in both CTAs)
          if (PAIR) umma_commit_pair(&sm.acc_full[buf]); else umma_commit(&sm.acc_full[buf]);
        }
      }
      if (!ok) atomicExch(A.status, (int)JP_ERR_TIMEOUT);
    }
  } else {
    // ---- epilogue ----------------------------------------------------------------------------
    const int q = warp & 3;                                   // the TMEM lane quarter this warp may read
    const int row = q * 32 + lane;                            // row of the CTA's block = TMEM lane
    const int64_t grow = (int64_t)m_block * LM_BM + row;
    const bool live = grow < A.T && (A.mask == nullptr || A.mask[grow] != 0);
    const int k = A.k;
    int32_t tok = -1;
    if (grow < A.T) tok = A.tokens[grow];
    for (int j = 0; j < k; ++j) sm.list[j][row] = 0ull;
    float tau = JP_NEG_INF;                                   // the row's k-th best value so far ...
    int worst = 0;                                            // ... and where it sits in the row's list
    float m_run = JP_NEG_INF;                                 // running maximum of z log2(e)
    double s_run = 0.0;                                       // sum of 2^(z log2 e - m_run)
    float zx = __int_as_float(0x7fc00000);
    bool ok = true;
    for (int t = 0; t < n_my && ok; ++t) {
      const uint32_t buf = (uint32_t)t & 1u, use = (uint32_t)t >> 1;
      if (!bar_wait(&sm.acc_full[buf], use & 1u, &sm.abort)) { ok = false; break; }
      tc_fence_after();
      const int col_tile = (tile0 + t) * LM_BN;
      const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + buf * LM_BN;
#pragma unroll 1
      for (int c = 0; c < LM_BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(taddr + (uint32_t)(c * 32), r);
        const int col0 = col_tile + c * 32;
        if ((int64_t)col0 >= A.V) continue;                  // beyond the vocabulary: zero fill of the copy engine
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        if ((int64_t)col0 + 32 > A.V) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if ((int64_t)(col0 + j) >= A.V) v[j] = JP_NEG_INF;
        }
        float cm = v[0];
#pragma unroll
        for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
        if (live && cm > tau) {
          // which of the 32 beat the threshold; then one list update per set bit (a lane loops as
          // often as it has hits, not once per position at which any lane of the warp has one)
          uint32_t hm = 0u;
#pragma unroll
          for (int j = 0; j < 32; ++j) hm |= (v[j] > tau ? 1u : 0u) << j;
          while (hm) {
            const int j = __ffs(hm) - 1;
            hm &= hm - 1u;
            float x = v[0];
#pragma unroll
            for (int i = 1; i < 32; ++i)
              if (i == j) x = v[i];
            if (x > tau) tau = list_replace_worst(sm, row, k, make_key(x, (uint32_t)(col0 + j)), worst);
          }
        }
        if (tok >= col0 && tok < col0 + 32) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (tok == col0 + j) zx = v[j];
        }
        const float ym = cm * kLog2e;
        if (ym > m_run) {
          s_run = m_run == JP_NEG_INF ? 0.0 : s_run * (double)ex2_approx(m_run - ym);
          m_run = ym;
        }
        float cs = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) cs += ex2_approx(fmaf(v[j], kLog2e, -m_run));
        s_run += (double)cs;
      }
      // this warp has read its quarter of the accumulator: one arrival per warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) bar_arrive_remote(&sm.acc_empty[buf], 0u);  // the leader's barrier counts both CTAs' epilogue warps
        else bar_arrive(&sm.acc_empty[buf]);
      }
    }
    if (!ok && lane == 0) atomicExch(A.status, (int)JP_ERR_TIMEOUT);
    if (grow < A.T) {
      list_sort(sm, row, k);
      const int64_t o = (int64_t)split * A.T + grow;
      A.part_m[o] = m_run;
      A.part_s[o] = s_run;
      A.part_zx[o] = zx;
      for (int j = 0; j < k; ++j) {
        const unsigned long long key = sm.list[j][row];
        A.part_val[o * k + j] = key ? key_value(key) : 0.f;
        A.part_idx[o * k + j] = key ? (int32_t)key_index(key) : -1;
      }
    }
  }
  // ---- common exit: tensor memory goes back ----------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();                              // neither CTA leaves while the other may still use its memory
  if (warp == 1) {
    tc_fence_after();
    if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(LM_TMEM_COLS) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(LM_TMEM_COLS) : "memory");
  }
}


// One warp per row: the splits' partial results into the row's log-sum-exp, the sampled token's
// log-probability and the k best entries.  Lane j walks split j's list (sorted, and the splits'
// column ranges ascend with j), so every round the best head under (logit desc, index asc) wins.
__global__ void __launch_bounds__(128) lmhead_merge_kernel(LmArgs A, float* out_lse, float* out_logp,
                                                           int32_t* out_idx, float* out_val) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
  if (r >= A.T) return;
  const int k = A.k, S = A.splits;
  const int32_t tok = A.tokens[r];
  const bool valid = (A.mask == nullptr || A.mask[r] != 0) && tok >= 0 && (int64_t)tok < A.V;
  if (!valid) {
    if (lane == 0) { out_lse[r] = 0.f; out_logp[r] = 0.f; }
    for (int j = lane; j < k; j += 32) { out_idx[r * k + j] = -1; out_val[r * k + j] = 0.f; }
    return;
  }
  const int64_t o = (int64_t)lane * A.T + r;
  float m = lane < S ? A.part_m[o] : JP_NEG_INF;
  float M = m;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
  double s = (lane < S && m != JP_NEG_INF) ? A.part_s[o] * exp2((double)m - (double)M) : 0.0;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  float zx = lane < S ? A.part_zx[o] : __int_as_float(0x7fc00000);
  const uint32_t has = __ballot_sync(0xffffffffu, zx == zx);
  zx = __shfl_sync(0xffffffffu, zx, has ? __ffs(has) - 1 : 0);
  // the exponents were formed with the fp32 constant log2(e), short of log2(e) by a factor
  // 1 - 1.335e-8: scaling the result back leaves an error below 1.335e-8 x the row's entropy
  const double lse = ((double)M + log2(s)) * 0.6931471805599453 * (1.0 + 1.33497582e-8);
  if (lane == 0) {
    out_lse[r] = (float)lse;
    out_logp[r] = (float)((double)zx - lse);
  }
  int head = 0;                                              // next unread entry of this lane's split
  for (int j = 0; j < k; ++j) {
    unsigned long long key = 0ull;
    float v = 0.f;
    if (lane < S && head < k) {
      const int32_t idx = A.part_idx[o * k + head];
      v = A.part_val[o * k + head];
      if (idx >= 0) key = make_key(v, (uint32_t)idx);
    }
    unsigned long long best = key;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, off);
      best = other > best ? other : best;
    }
    const uint32_t win = __ballot_sync(0xffffffffu, key == best && key != 0ull);
    if (win == 0u) {                                         // fewer than k entries in all
      if (lane == 0) { out_idx[r * k + j] = -1; out_val[r * k + j] = 0.f; }
      continue;
    }
    const int w = __ffs(win) - 1;
    if (lane == w) {
      out_idx[r * k + j] = (int32_t)key_index(key);
      out_val[r * k + j] = v;
      ++head;
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows, ld] bf16 row-major, viewed as a 2-D tensor (inner dimension H) and fetched in boxes of
// 64 x box_rows elements with the 128-byte swizzle; out-of-range elements read as zero.
bool make_map(EncodeTiledFn enc, CUtensorMap* map, const void* base, int64_t rows, int64_t H, int64_t ld,
              uint32_t box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)LM_BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

namespace {
// Dot product of two bf16 rows of length H by one warp (16-byte loads where the rows allow it,
// fp32 sums, a fixed shuffle tree): the logit of one vocabulary entry under one model.
__device__ __forceinline__ float warp_dot_bf16(const __nv_bfloat16* a, const __nv_bfloat16* b, int64_t H, int lane) {
  float acc = 0.f;
  const int64_t nvec = H / 8;
  const uint4* a4 = reinterpret_cast<const uint4*>(a);
  const uint4* b4 = reinterpret_cast<const uint4*>(b);
  for (int64_t i = lane; i < nvec; i += 32) {
    const uint4 x = a4[i], y = b4[i];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc = fmaf(Vec<JP_BF16>::get(x, e), Vec<JP_BF16>::get(y, e), acc);
  }
  for (int64_t i = nvec * 8 + lane; i < H; i += 32) acc = fmaf(__bfloat162float(a[i]), __bfloat162float(b[i]), acc);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  return acc;
}

// The records of the forward from two fused output-layer passes (Section 4.4.1: V_k is the
// union of the two top-k sets and Z_approx needs both models' probabilities on it): per row
// the two log-sum-exps, the sampled token's two log-probs, the two lists, and for every list
// entry the logit of the *other* model, one dot product of a hidden state with one row of
// that model's output matrix.  One warp per row.
__global__ void __launch_bounds__(128) fused_records_kernel(FusedRecordArgs A) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
  if (r >= A.T) return;
  const int k = A.k;
  const int32_t tok = A.tokens[r];
  const bool bad = tok < 0 || (int64_t)tok >= A.V;
  const bool valid = (A.mask == nullptr || A.mask[r] != 0) && !bad;
  if (lane == 0) {
    A.rec.flag[r] = valid ? kRowValid : 0;
    A.rec.lse_a[r] = valid ? A.lse_a[r] : 0.f; A.rec.lse_a_lo[r] = 0.f;
    A.rec.lse_p[r] = valid ? A.lse_p[r] : 0.f; A.rec.lse_p_lo[r] = 0.f;
    A.rec.lq[r] = valid ? A.lq[r] : 0.f;
    A.rec.lp[r] = valid ? A.lp[r] : 0.f;
    if (bad && (A.mask == nullptr || A.mask[r] != 0)) atomicAdd(&A.sc->n_bad_token, 1ull);
  }
  const __nv_bfloat16* ha = (const __nv_bfloat16*)A.hidden_a + r * A.ld_ha;
  const __nv_bfloat16* hp = (const __nv_bfloat16*)A.hidden_p + r * A.ld_hp;
  for (int j = 0; j < 2 * k; ++j) {
    const int64_t dst = r * (2 * k) + j;
    const bool from_actor = j < k;
    const int32_t idx = valid ? (from_actor ? A.idx_a[r * k + j] : A.idx_p[r * k + (j - k)]) : -1;
    float za = 0.f, zp = 0.f;
    if (idx >= 0) {                                           // uniform over the warp
      if (from_actor) {
        za = A.val_a[r * k + j];
        zp = warp_dot_bf16(hp, (const __nv_bfloat16*)A.weight_p + (int64_t)idx * A.ld_wp, A.H_p, lane);
      } else {
        zp = A.val_p[r * k + (j - k)];
        za = warp_dot_bf16(ha, (const __nv_bfloat16*)A.weight_a + (int64_t)idx * A.ld_wa, A.H_a, lane);
      }
    }
    if (lane == 0) { A.rec.idx[dst] = idx; A.rec.za[dst] = za; A.rec.zp[dst] = zp; }
  }
}
}  // namespace

cudaError_t launch_fused_records(const FusedRecordArgs& a, cudaStream_t s) {
  if (a.T <= 0) return cudaSuccess;
  fused_records_kernel<<<(unsigned)((a.T + 3) / 4), 128, 0, s>>>(a);
  return cudaGetLastError();
}

size_t lmhead_scratch_bytes(int64_t T, int k, int splits) {
  // part_s (double) first, then part_m, part_zx, part_val, part_idx
  return (size_t)splits * (size_t)T * (8 + 4 + 4 + (size_t)k * 8) + 256;
}

// CTA pairs whenever there are two row blocks to pair up (measured 2 to 13 % faster than single
// CTAs over hidden sizes 1024 .. 5120); a batch of at most 128 rows has nothing for a partner to do.
static bool lmhead_use_pairs(int64_t T) { return T > LM_BM; }

int lmhead_splits(int64_t T, int64_t V, int sms) {
  int64_t m_blocks = (T + LM_BM - 1) / LM_BM;
  if (lmhead_use_pairs(T)) m_blocks = (m_blocks + 1) / 2 * 2;
  const int n_tiles = (int)((V + LM_BN - 1) / LM_BN);
  int64_t s = m_blocks > 0 ? sms / m_blocks : 1;
  if (s < 1) s = 1;
  if (s > 32) s = 32;                       // the merge walks one split per lane
  if (s > n_tiles) s = n_tiles;
  const int tps = (int)((n_tiles + s - 1) / s);
  return (n_tiles + tps - 1) / tps;         // every split has at least one tile
}

template <bool PAIR, int KMAX>
static cudaError_t launch_lmhead_variant(dim3 grid, const CUtensorMap& map_a, const CUtensorMap& map_b, const LmArgs& a,
                                         cudaStream_t s) {
  const size_t smem = sizeof(LmSmemT<PAIR, KMAX>) + 1024;
  cudaError_t e = cudaFuncSetAttribute(lmhead_kernel<PAIR, KMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(LM_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = PAIR ? 2 : 1; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, lmhead_kernel<PAIR, KMAX>, map_a, map_b, a);
}

cudaError_t launch_lmhead(const void* hidden, int64_t ldh, const void* weight, int64_t ldw, const int32_t* tokens,
                          const uint8_t* mask, int64_t T, int64_t H, int64_t V, int k, int splits, void* scratch,
                          int32_t* status, float* out_lse, float* out_logp, int32_t* out_idx, float* out_val,
                          cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    enc = (EncodeTiledFn)fn;
  }
  CUtensorMap map_a, map_b;
  const bool pair = lmhead_use_pairs(T);
  if (!make_map(enc, &map_a, hidden, T, H, ldh, LM_BM) || !make_map(enc, &map_b, weight, V, H, ldw, pair ? LM_BN / 2 : LM_BN))
    return cudaErrorInvalidValue;
  LmArgs a{};
  a.tokens = tokens; a.mask = mask; a.T = T; a.H = H; a.V = V; a.k = k;
  a.n_tiles = (int)((V + LM_BN - 1) / LM_BN);
  a.splits = splits;
  a.tiles_per_split = (a.n_tiles + splits - 1) / splits;
  char* p = (char*)scratch;
  a.part_s = (double*)p; p += (size_t)splits * T * 8;
  a.part_m = (float*)p; p += (size_t)splits * T * 4;
  a.part_zx = (float*)p; p += (size_t)splits * T * 4;
  a.part_val = (float*)p; p += (size_t)splits * T * k * 4;
  a.part_idx = (int32_t*)p;
  a.status = status;
  cudaError_t e;
  const unsigned m_blocks = (unsigned)((T + LM_BM - 1) / LM_BM);
  if (pair) {
    // clusters of two CTAs along x: row blocks 2i and 2i + 1 (an odd count is rounded up: the extra
    // CTA works on rows beyond T, which read as zero and are never written)
    const dim3 grid((m_blocks + 1) / 2 * 2, (unsigned)splits);
    e = k <= 32 ? launch_lmhead_variant<true, 32>(grid, map_a, map_b, a, s) : launch_lmhead_variant<true, 64>(grid, map_a, map_b, a, s);
  } else {
    const dim3 grid(m_blocks, (unsigned)splits);
    e = k <= 32 ? launch_lmhead_variant<false, 32>(grid, map_a, map_b, a, s) : launch_lmhead_variant<false, 64>(grid, map_a, map_b, a, s);
  }
  if (e != cudaSuccess) return e;
  lmhead_merge_kernel<<<(unsigned)((T + 3) / 4), 128, 0, s>>>(a, out_lse, out_logp, out_idx, out_val);
  return cudaGetLastError();
}

}  // namespace jp
