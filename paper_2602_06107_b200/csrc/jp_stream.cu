// Row-streaming kernels: each valid row of the actor and policy logits is read
// from HBM once; the pass yields both log-sum-exps (online max / rescaled sum),
// the sampled token's logits and the two top-k lists (Section 4.4.1: V_k is the
// union of top-k(p_inf) and top-k(p_new)), each candidate carrying both logits.
// A second kernel sums the exact normaliser Z over the vocabulary (Eq. obrs_dist).
//
// Work split: persistent CTAs pull rows from an atomic counter; one CTA owns one
// row at a time; a thread owns 16-byte vectors strided by the CTA width, so every
// warp-level load is one contiguous 512-byte segment.
//
// Top-k: the total order is (logit desc, index asc), encoded in one 64-bit key.
// A threshold tau (the current k-th best key) filters the stream: one compare
// per 16-byte vector (its max against tau's logit) in the hot loop, exact key
// compares only for vectors that pass.  Survivors go to a shared-memory
// candidate buffer that is bitonic-sorted together with the current list when
// it fills, which tightens tau.  The first tile has no tau yet: the k-th
// largest of the per-thread maxima bounds it from below.
#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {

constexpr int NT = 256;                 // threads per CTA
constexpr int NWARP = NT / 32;
constexpr int UNROLL = 4;               // vectors per thread per tensor per tile
constexpr int PMAX = 512;               // list + candidate slots per tensor
constexpr int CTAS_PER_SM = 2;

struct __align__(16) StreamSmem {
  unsigned long long buf[2][PMAX];      // [0,K): current list, best first; [K,PMAX): candidates
  unsigned long long tau_key[2];
  int cnt[2];
  float red_m[2][NWARP];
  float red_s[2][NWARP];
  float warp_bound[2][NWARP];
  int row;
};

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

// r-th largest (1-based) of the 32 lane values: shuffle bitonic sort, descending.
__device__ __forceinline__ float warp_rth_largest(float v, int r, int lane) {
#pragma unroll
  for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      float o = __shfl_xor_sync(0xffffffffu, v, stride);
      bool lower = (lane & stride) == 0;
      bool desc = (lane & size) == 0;
      v = (lower == desc) ? fmaxf(v, o) : fminf(v, o);
    }
  }
  return __shfl_sync(0xffffffffu, v, r - 1);
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

// Element `e` (runtime) of a vector held as four words.
template <int DT>
__device__ __forceinline__ float vec_elem(uint32_t x, uint32_t y, uint32_t z, uint32_t w, int e) {
  if (DT == JP_BF16) {
    const int wi = e >> 1;
    uint32_t word = wi == 0 ? x : wi == 1 ? y : wi == 2 ? z : w;
    return __uint_as_float((e & 1) ? (word & 0xffff0000u) : (word << 16));
  }
  return __uint_as_float(e == 0 ? x : e == 1 ? y : e == 2 ? z : w);
}

// Warp-cooperative append.  `pass` marks the lanes whose vector may hold an entry
// that beats tau.  For each such lane the vector is broadcast, lanes 0..N-1 each
// test one entry exactly (64-bit key against tau) and the winners take
// consecutive slots of the CTA's candidate buffer.  Control flow is warp-uniform.
// `done` (owner lane's bits 0..N-1) marks entries appended earlier in this tile;
// the function returns the updated bits for the calling lane's own vector and
// sets `flag` when the CTA should merge (soft limit passed, or no slot left).
template <int DT>
__device__ __forceinline__ uint32_t push_warp(StreamSmem& sm, int t, const uint4& v, bool pass,
                                              uint32_t idx0, uint32_t V, unsigned long long tau,
                                              uint32_t done, int K, int lane, bool& flag) {
  constexpr int N = Vec<DT>::N;
  uint32_t mask = __ballot_sync(0xffffffffu, pass);
  const int cap = PMAX - K;
  const int soft = cap >> 1;
  while (mask) {
    const int L = __ffs(mask) - 1;
    mask &= mask - 1;
    const uint32_t x = __shfl_sync(0xffffffffu, v.x, L), y = __shfl_sync(0xffffffffu, v.y, L);
    const uint32_t z = __shfl_sync(0xffffffffu, v.z, L), w = __shfl_sync(0xffffffffu, v.w, L);
    const uint32_t i0 = __shfl_sync(0xffffffffu, idx0, L);
    const uint32_t dn = __shfl_sync(0xffffffffu, done, L);
    const uint32_t idx = i0 + lane;
    bool win = false;
    unsigned long long key = 0ull;
    if (lane < N && idx < V && !((dn >> lane) & 1u)) {
      key = make_key(vec_elem<DT>(x, y, z, w, lane), idx);
      win = key > tau;
    }
    const uint32_t wmask = __ballot_sync(0xffffffffu, win);
    if (wmask) {
      int base = 0;
      if (lane == 0) base = atomicAdd(&sm.cnt[t], __popc(wmask));
      base = __shfl_sync(0xffffffffu, base, 0);
      const int slot = base + __popc(wmask & ((1u << lane) - 1u));
      const bool stored = win && slot < cap;
      if (stored) sm.buf[t][K + slot] = key;
      const uint32_t smask = __ballot_sync(0xffffffffu, stored);
      if (lane == L) done |= smask;
      if (smask != wmask || base + __popc(wmask) > soft) flag = true;
    }
  }
  return done;
}

// Bitonic sort (descending) of buf[0..P) by ONE warp, then keep the best k, clear
// the rest and publish tau and the reset count.  P is a power of two >= 2.
__device__ __forceinline__ void warp_sort_list(unsigned long long* buf, int P, int k, int lane,
                                               unsigned long long* tau_out, int* cnt_out) {
  for (int size = 2; size <= P; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int j = lane; j < (P >> 1); j += 32) {
        const int lo = ((j & ~(stride - 1)) << 1) | (j & (stride - 1));
        const int hi = lo | stride;
        const bool desc = (lo & size) == 0;
        const unsigned long long a = buf[lo], b = buf[hi];
        if ((a < b) == desc) { buf[lo] = b; buf[hi] = a; }
      }
      __syncwarp();
    }
  }
  for (int i = k + lane; i < P; i += 32) buf[i] = 0ull;
  __syncwarp();
  if (lane == 0) { *tau_out = buf[k - 1]; *cnt_out = 0; }
}

// Folds the candidates of both tensors into their lists: warp 0 sorts the actor
// side, warp 1 the policy side, everyone else waits.  Called by all threads
// after a barrier that ordered every append before it; ends with a barrier.
__device__ __forceinline__ void merge_lists(StreamSmem& sm, int k, int K, int warp, int lane) {
  if (warp < 2) {
    const int cap = PMAX - K;
    const int n = min(sm.cnt[warp], cap);
    int P = K < 2 ? 2 : K;
    while (P < K + n) P <<= 1;
    if (n > 0) warp_sort_list(sm.buf[warp], P, k, lane, &sm.tau_key[warp], &sm.cnt[warp]);
    else if (lane == 0) sm.tau_key[warp] = sm.buf[warp][k - 1];
  }
  __syncthreads();
}

__device__ __forceinline__ float tau_value(unsigned long long key) {
  return key == 0ull ? JP_NEG_INF : key_value(key);
}

template <int DT>
__device__ __forceinline__ void load_tile(uint4 (&va)[UNROLL], uint4 (&vp)[UNROLL], const char* ra,
                                          const char* rp, int64_t v0, int64_t nvec, int tail,
                                          int tid) {
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    int64_t vi = v0 + (int64_t)j * NT + tid;
    if (vi < nvec) {
      va[j] = ldg_stream((const uint4*)ra + vi);
      vp[j] = ldg_stream((const uint4*)rp + vi);
    } else {
      va[j] = Vec<DT>::neg_inf();
      vp[j] = Vec<DT>::neg_inf();
      if (vi == nvec && tail > 0) {       // ragged end of the row: scalar loads, -inf padding
#pragma unroll
        for (int e = 0; e < Vec<DT>::N - 1; ++e) {
          if (e < tail) {
            Vec<DT>::set(va[j], e, Vec<DT>::load_scalar(ra, nvec * Vec<DT>::N + e));
            Vec<DT>::set(vp[j], e, Vec<DT>::load_scalar(rp, nvec * Vec<DT>::N + e));
          }
        }
      }
    }
  }
}

template <int DT, bool TOPK>
__global__ void __launch_bounds__(NT, CTAS_PER_SM) stream_kernel(StreamArgs A) {
  __shared__ StreamSmem sm;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int N = Vec<DT>::N;
  const int k = A.k;
  int K = 1;
  while (K < k) K <<= 1;
  const int64_t nvec = A.V / N;
  const int tail = (int)(A.V - nvec * N);
  const int64_t nvt = nvec + (tail > 0 ? 1 : 0);
  constexpr int64_t TILE = (int64_t)NT * UNROLL;

  if (TOPK) {
    for (int i = tid; i < 2 * PMAX; i += NT) (&sm.buf[0][0])[i] = 0ull;
    if (tid < 2) { sm.cnt[tid] = 0; sm.tau_key[tid] = 0ull; }
  }
  __syncthreads();

  for (;;) {
    if (tid == 0) sm.row = atomicAdd(&A.sc->row_counter, 1);
    __syncthreads();
    const int64_t row = sm.row;
    __syncthreads();
    if (row >= A.T) break;
    const int64_t rrow = A.record_offset + row;
    bool valid = A.mask == nullptr || A.mask[row] != 0;
    const int32_t x = valid ? A.tokens[row] : 0;
    if (valid && (x < 0 || (int64_t)x >= A.V)) {
      valid = false;
      if (tid == 0) atomicAdd(&A.sc->n_bad_token, 1ull);
    }
    if (!valid) {
      if (tid == 0) {
        A.rec.flag[rrow] = 0;
        A.rec.lse_a[rrow] = 0.f; A.rec.lse_p[rrow] = 0.f;
        A.rec.lq[rrow] = 0.f; A.rec.lp[rrow] = 0.f;
      }
      continue;
    }
    const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
    const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;

    Online oa{JP_NEG_INF, 0.f, 0ull}, op{JP_NEG_INF, 0.f, 0ull};
    unsigned long long tkey_a = 0ull, tkey_p = 0ull;
    float tval_a = JP_NEG_INF, tval_p = JP_NEG_INF;

    uint4 ca[UNROLL], cp[UNROLL], na[UNROLL], np_[UNROLL];
    load_tile<DT>(ca, cp, ra, rp, 0, nvec, tail, tid);
    int tile = 0;
    for (int64_t v0 = 0; v0 < nvt; v0 += TILE, ++tile) {
      const bool more = v0 + TILE < nvt;
      if (more) load_tile<DT>(na, np_, ra, rp, v0 + TILE, nvec, tail, tid);

      float vm_a[UNROLL], vm_p[UNROLL];
#pragma unroll
      for (int j = 0; j < UNROLL; ++j) {
        vm_a[j] = Vec<DT>::vmax(ca[j]);
        vm_p[j] = Vec<DT>::vmax(cp[j]);
        accumulate<DT>(ca[j], vm_a[j], oa);
        accumulate<DT>(cp[j], vm_p[j], op);
      }

      if (TOPK) {
        // Merge after tiles 0, 1, 3, 7, ... (whenever the number of tiles seen
        // doubles): the expected number of later candidates falls like 1/seen.
        bool force = ((tile + 1) & tile) == 0;
        if (tile == 0) {
          // No threshold yet.  With r = ceil(k / warps), the smallest over the
          // warps of each warp's r-th largest per-thread maximum has at least k
          // row entries at or above it, so it bounds the k-th best logit from below.
          float tm_a = vm_a[0], tm_p = vm_p[0];
#pragma unroll
          for (int j = 1; j < UNROLL; ++j) { tm_a = fmaxf(tm_a, vm_a[j]); tm_p = fmaxf(tm_p, vm_p[j]); }
          const int r = (k + NWARP - 1) / NWARP;
          float wa = warp_rth_largest(tm_a, r, lane);
          float wp = warp_rth_largest(tm_p, r, lane);
          if (lane == 0) { sm.warp_bound[0][warp] = wa; sm.warp_bound[1][warp] = wp; }
          __syncthreads();
          float ba = sm.warp_bound[0][0], bp = sm.warp_bound[1][0];
#pragma unroll
          for (int w = 1; w < NWARP; ++w) { ba = fminf(ba, sm.warp_bound[0][w]); bp = fminf(bp, sm.warp_bound[1][w]); }
          tval_a = ba; tval_p = bp;
          tkey_a = (unsigned long long)f32_order_bits(ba) << 32;   // below every entry with logit >= ba
          tkey_p = (unsigned long long)f32_order_bits(bp) << 32;
        }
        uint32_t pushed_a = 0u, pushed_p = 0u;
        for (;;) {
          bool flag = force;
          bool any_a = false, any_p = false;
#pragma unroll
          for (int j = 0; j < UNROLL; ++j) { any_a |= vm_a[j] >= tval_a; any_p |= vm_p[j] >= tval_p; }
          if (__any_sync(0xffffffffu, any_a)) {
#pragma unroll
            for (int j = 0; j < UNROLL; ++j) {
              const uint32_t idx0 = (uint32_t)((v0 + (int64_t)j * NT + tid) * N);
              const uint32_t d = push_warp<DT>(sm, 0, ca[j], vm_a[j] >= tval_a, idx0, (uint32_t)A.V, tkey_a,
                                               (pushed_a >> (j * N)) & ((1u << N) - 1u), K, lane, flag);
              pushed_a |= d << (j * N);
            }
          }
          if (__any_sync(0xffffffffu, any_p)) {
#pragma unroll
            for (int j = 0; j < UNROLL; ++j) {
              const uint32_t idx0 = (uint32_t)((v0 + (int64_t)j * NT + tid) * N);
              const uint32_t d = push_warp<DT>(sm, 1, cp[j], vm_p[j] >= tval_p, idx0, (uint32_t)A.V, tkey_p,
                                               (pushed_p >> (j * N)) & ((1u << N) - 1u), K, lane, flag);
              pushed_p |= d << (j * N);
            }
          }
          if (!__syncthreads_or(flag)) break;
          merge_lists(sm, k, K, warp, lane);
          tkey_a = sm.tau_key[0]; tkey_p = sm.tau_key[1];
          tval_a = tau_value(tkey_a); tval_p = tau_value(tkey_p);
          force = false;
        }
      }
      if (more) {
#pragma unroll
        for (int j = 0; j < UNROLL; ++j) { ca[j] = na[j]; cp[j] = np_[j]; }
      }
    }

    // ---- row epilogue: merge the per-thread (max, sum) pairs in a fixed tree
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
      sm.red_m[0][warp] = mL_a; sm.red_s[0][warp] = s_a;
      sm.red_m[1][warp] = mL_p; sm.red_s[1][warp] = s_p;
    }
    __syncthreads();
    if (TOPK) merge_lists(sm, k, K, warp, lane);          // folds whatever the last tiles appended
    if (tid < 2) {
      // log-sum-exp = ln2 (M + log2 S).  S = 2^e f with f in [1,2): logf(f) is good to an
      // ulp of a number below 0.7, and the large part (M + e) ln2 is formed in double, so
      // the published fp32 values are rounded once.
      float M = sm.red_m[tid][0];
      for (int w = 1; w < NWARP; ++w) M = fmaxf(M, sm.red_m[tid][w]);
      float S = 0.f;
      for (int w = 0; w < NWARP; ++w)
        if (sm.red_m[tid][w] != JP_NEG_INF) S += sm.red_s[tid][w] * exp2_int(sm.red_m[tid][w] - M);
      int e;
      const float f = 2.f * frexpf(S, &e);                // S = f * 2^(e-1)
      const double lse = ((double)M + (double)(e - 1)) * 0.6931471805599453 + (double)logf(f);
      const float lsef = (float)lse;
      const char* rowp = tid == 0 ? ra : rp;
      const float zx = Vec<DT>::load_scalar(rowp, x);
      const float lpx = (float)((double)zx - lse);
      if (tid == 0) { A.rec.lse_a[rrow] = lsef; A.rec.lq[rrow] = lpx; A.rec.flag[rrow] = 1; }
      else          { A.rec.lse_p[rrow] = lsef; A.rec.lp[rrow] = lpx; }
      if (!isfinite(lsef)) atomicAdd(&A.sc->n_nonfinite, 1ull);
    }
    if (TOPK) {
      if (tid < 2 * k) {
        int t = tid >= k;
        int j = tid - t * k;
        unsigned long long key = sm.buf[t][j];
        int64_t o = rrow * (2 * k) + tid;
        if (key != 0ull) {
          uint32_t idx = key_index(key);
          A.rec.idx[o] = (int32_t)idx;
          A.rec.za[o] = Vec<DT>::load_scalar(ra, idx);
          A.rec.zp[o] = Vec<DT>::load_scalar(rp, idx);
        } else {
          A.rec.idx[o] = -1; A.rec.za[o] = 0.f; A.rec.zp[o] = 0.f;
        }
      }
      __syncthreads();
      for (int i = tid; i < 2 * K; i += NT) sm.buf[i >= K][i - (i >= K) * K] = 0ull;
      if (tid < 2) sm.tau_key[tid] = 0ull;
    }
    __syncthreads();
  }
}

// Exact normaliser: Z_t = sum_v min(q_t(v), p_t(v)/lambda), one more pass over the
// row with the log-sum-exps known (Eq. obrs_dist; Appendix A, Z_C).
template <int DT>
__global__ void __launch_bounds__(NT, CTAS_PER_SM) exact_z_kernel(ExactZArgs A) {
  __shared__ float red[NWARP];
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
    for (int64_t v0 = 0; v0 < nvt; v0 += (int64_t)NT * UNROLL) {
      uint4 va[UNROLL], vp[UNROLL];
      load_tile<DT>(va, vp, ra, rp, v0, nvec, tail, tid);
#pragma unroll
      for (int j = 0; j < UNROLL; ++j) {
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
      for (int w = 0; w < NWARP; ++w) S += (double)red[w];
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

cudaError_t launch_stream(const StreamArgs& a, cudaStream_t s, int sms) {
  if (a.T <= 0) return cudaSuccess;
  const int grid = sms * CTAS_PER_SM;
  int g = (int)(a.T < grid ? a.T : grid);
  if (a.dtype == JP_BF16) {
    if (a.k > 0) stream_kernel<JP_BF16, true><<<g, NT, 0, s>>>(a);
    else stream_kernel<JP_BF16, false><<<g, NT, 0, s>>>(a);
  } else {
    if (a.k > 0) stream_kernel<JP_F32, true><<<g, NT, 0, s>>>(a);
    else stream_kernel<JP_F32, false><<<g, NT, 0, s>>>(a);
  }
  return cudaGetLastError();
}

cudaError_t launch_exact_z(const ExactZArgs& a, cudaStream_t s, int sms) {
  if (a.T <= 0) return cudaSuccess;
  const int grid = sms * CTAS_PER_SM;
  int g = (int)(a.T < grid ? a.T : grid);
  if (a.dtype == JP_BF16) exact_z_kernel<JP_BF16><<<g, NT, 0, s>>>(a);
  else exact_z_kernel<JP_F32><<<g, NT, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace jp
