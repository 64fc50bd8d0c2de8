// Vocabulary-parallel form of the forward pass (Section 4.4: the full-vocabulary pass over
// [tokens, vocabulary] logits is the memory bottleneck; here every device holds a slice of
// the vocabulary's columns).  A shard streams its columns once with the ordinary row
// kernel, which leaves per row the log-sum-exp of the slice and the slice's two top-k lists
// with both logits of every entry.  Those records are packed, exchanged between the shards
// by the caller, and merged here into the records of the whole vocabulary:
//   lse        = log sum_s exp(lse_s)                       (both tensors)
//   log-probs  = the owner shard's logits of the sampled token minus lse
//   top-k(p)   = the k best of the union of the shards' k best (the k best of the whole
//                vocabulary lie in it), same total order: higher logit first, equal
//                logits by lower index
// after which acceptance, Z_approx (Eq. z_approx over the union of the two lists), the
// batch calibration and the weights run from the records exactly as on one device.
#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {
namespace {

constexpr int VS_NT = 128;

__global__ void __launch_bounds__(256) vshard_localize_kernel(int64_t T, const int32_t* tokens, const uint8_t* mask,
                                                              int64_t vocab_offset, int64_t V_shard, int64_t V_total,
                                                              int32_t foreign, int32_t* tok_local,
                                                              uint8_t* mask_local, Scalars* sc) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= T) return;
  bool valid = mask == nullptr || mask[i] != 0;
  const int64_t x = tokens[i];
  if (valid && (x < 0 || x >= V_total)) {
    valid = false;
    if (sc) atomicAdd(&sc->n_bad_token, 1ull);
  }
  const int64_t loc = x - vocab_offset;
  const bool owner = valid && loc >= 0 && loc < V_shard;
  // Forward (foreign = 0): a shard that does not hold the sampled token streams the row all
  // the same; column 0 stands in for the token and the log-prob it yields is never used.
  // Backward (foreign = -1): no column of such a shard carries the one-hot term.
  tok_local[i] = owner ? (int32_t)loc : foreign;
  if (mask_local) mask_local[i] = valid ? (owner ? 2 : 1) : 0;
}

// One warp per row: the shard's records of the row as one packed line, stored at line
// line0 + r of every destination.  With one destination this is the local export; with one
// per shard (each the same place in a peer's gathered buffer, reachable by plain stores:
// peer-mapped device memory) the export is also the all-gather, pushed by the producer.
__global__ void __launch_bounds__(VS_NT) vshard_export_kernel(int64_t T, int k, Records rec, const void* za,
                                                              const void* zp, int64_t ld, int32_t dtype,
                                                              const int32_t* tok_local, const uint8_t* mask_local,
                                                              int64_t vocab_offset, VshardDests dests, int64_t line0) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * (VS_NT / 32) + (threadIdx.x >> 5);
  if (r >= T) return;
  const int64_t o = (line0 + r) * vshard_words(k);
  auto put = [&](int64_t w, float v) {
    for (int p = 0; p < dests.n; ++p) dests.dst[p][o + w] = v;
  };
  const bool flag = rec.flag[r] != 0;      // a non-finite slice travels as it is: the merged row is then non-finite too
  if (lane == 0) {
    const bool owner = flag && mask_local[r] == 2;
    float xa = 0.f, xp = 0.f;
    if (owner) {
      const int64_t x = tok_local[r];
      if (dtype == JP_BF16) {
        xa = Vec<JP_BF16>::load_scalar((const char*)za + r * ld * Vec<JP_BF16>::ESIZE, x);
        xp = Vec<JP_BF16>::load_scalar((const char*)zp + r * ld * Vec<JP_BF16>::ESIZE, x);
      } else {
        xa = Vec<JP_F32>::load_scalar((const char*)za + r * ld * Vec<JP_F32>::ESIZE, x);
        xp = Vec<JP_F32>::load_scalar((const char*)zp + r * ld * Vec<JP_F32>::ESIZE, x);
      }
    }
    put(0, __int_as_float(flag ? 1 : 0));
    put(1, __int_as_float(owner ? 1 : 0));
    put(2, flag ? rec.lse_a[r] : 0.f);
    put(3, flag ? rec.lse_a_lo[r] : 0.f);
    put(4, flag ? rec.lse_p[r] : 0.f);
    put(5, flag ? rec.lse_p_lo[r] : 0.f);
    put(6, xa);
    put(7, xp);
  }
  for (int j = lane; j < 2 * k; j += 32) {
    const int64_t e = r * (2 * k) + j;
    const int32_t idx = flag ? rec.idx[e] : -1;
    put(kVshardHeader + j, __int_as_float(idx >= 0 ? (int32_t)(idx + vocab_offset) : -1));
    put(kVshardHeader + 2 * k + j, idx >= 0 ? rec.za[e] : 0.f);
    put(kVshardHeader + 4 * k + j, idx >= 0 ? rec.zp[e] : 0.f);
  }
}

// One warp per row.  For each of the two lists the warp first copies every shard's k entries
// into shared memory as 64-bit (order bits, ~index) keys (all loads in flight at once), then
// lane s walks shard s's keys (and shards s + 32, ...: up to four per lane), which are sorted
// best first: every round the best of the lanes' current heads under the row kernel's order
// (higher logit first, equal logits by lower index; keys are distinct because the shards'
// columns are disjoint) is the next entry of the merged list, and the winning lane moves on.
// k rounds of one warp-wide maximum per list replace a rank count of every entry against every
// shard's list; where each merged entry came from is noted, and both logits of the entries are
// fetched at the end, again all at once.
__global__ void __launch_bounds__(VS_NT) vshard_merge_kernel(int n_shards, int my_shard, const float* g, int64_t T,
                                                             int k, Records rec, Scalars* sc, int warps_per_block) {
  extern __shared__ unsigned long long vs_smem[];            // per warp: n_shards * k keys, then k (shard, place) notes
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (warp >= warps_per_block) return;
  const int64_t r = (int64_t)blockIdx.x * warps_per_block + warp;
  if (r >= T) return;
  const int n = n_shards * k;
  unsigned long long* keys = vs_smem + (size_t)warp * (size_t)(n + (k + 1) / 2);
  uint32_t* from = reinterpret_cast<uint32_t*>(keys + n);    // (shard << 16) | place of merged entry j
  const int64_t W = vshard_words(k);
  auto line = [&](int s) { return g + ((int64_t)s * T + r) * W; };

  bool mine = true;
  for (int s = lane; s < n_shards; s += 32) mine = mine && __float_as_int(line(s)[0]) != 0;
  const bool all = __all_sync(0xffffffffu, mine);

  for (int t = 0; t < 2; ++t) {
    const int64_t dst0 = r * (2 * k) + (int64_t)t * k;
    if (!all) {
      for (int j = lane; j < k; j += 32) { rec.idx[dst0 + j] = -1; rec.za[dst0 + j] = 0.f; rec.zp[dst0 + j] = 0.f; }
      continue;
    }
    __syncwarp();
    for (int e = lane; e < n; e += 32) {
      const int s = e / k, j = e - s * k;
      const float* o = line(s);
      const int32_t idx = __float_as_int(o[kVshardHeader + t * k + j]);
      const float v = o[kVshardHeader + (t == 0 ? 2 * k : 4 * k) + t * k + j];
      keys[e] = idx >= 0 ? make_key(v, (uint32_t)idx) : 0ull;
    }
    __syncwarp();
    static_assert(kVshardMaxShards == 4 * 32, "four shards per lane");
    if (n_shards <= 32) {
      // one shard per lane: the head key stays in a register; the warp-wide maximum of the 64-bit
      // keys is two 32-bit reductions (high words, then low words among the lanes that tie on top)
      int head = 0;
      unsigned long long key = lane < n_shards ? keys[lane * k] : 0ull;
      for (int j = 0; j < k; ++j) {
        const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
        const uint32_t mhi = __reduce_max_sync(0xffffffffu, hi);
        const uint32_t mlo = __reduce_max_sync(0xffffffffu, hi == mhi ? lo : 0u);
        if (mhi == 0u && mlo == 0u) {                         // the shards hold fewer than k entries in all
          if (lane == 0) from[j] = 0xffffffffu;
          continue;
        }
        if (hi == mhi && lo == mlo) {                         // keys are distinct: exactly one lane
          from[j] = ((uint32_t)lane << 16) | (uint32_t)head;
          ++head;
          key = head < k ? keys[lane * k + head] : 0ull;
        }
      }
    } else {
      int head[4] = {0, 0, 0, 0};
      for (int j = 0; j < k; ++j) {
        unsigned long long key = 0ull;
        int which = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int s = lane + 32 * q;
          if (s < n_shards && head[q] < k) {
            const unsigned long long kq = keys[s * k + head[q]];
            if (kq > key) { key = kq; which = q; }
          }
        }
        const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
        const uint32_t mhi = __reduce_max_sync(0xffffffffu, hi);
        const uint32_t mlo = __reduce_max_sync(0xffffffffu, hi == mhi ? lo : 0u);
        if (mhi == 0u && mlo == 0u) {
          if (lane == 0) from[j] = 0xffffffffu;
          continue;
        }
        if (hi == mhi && lo == mlo) {
          int h = head[0];
#pragma unroll
          for (int q = 1; q < 4; ++q)
            if (q == which) h = head[q];
          from[j] = ((uint32_t)(lane + 32 * which) << 16) | (uint32_t)h;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (q == which) head[q] += 1;
        }
      }
    }
    __syncwarp();
    for (int j = lane; j < k; j += 32) {
      const uint32_t f = from[j];
      if (f == 0xffffffffu) {
        rec.idx[dst0 + j] = -1; rec.za[dst0 + j] = 0.f; rec.zp[dst0 + j] = 0.f;
      } else {
        const int s = (int)(f >> 16), h = (int)(f & 0xffffu);
        const float* o = line(s);
        rec.idx[dst0 + j] = __float_as_int(o[kVshardHeader + t * k + h]);
        rec.za[dst0 + j] = o[kVshardHeader + 2 * k + t * k + h];
        rec.zp[dst0 + j] = o[kVshardHeader + 4 * k + t * k + h];
      }
    }
  }

  if (lane == 0) {
    if (!all) {
      rec.flag[r] = 0;
      rec.lse_a[r] = 0.f; rec.lse_p[r] = 0.f; rec.lse_a_lo[r] = 0.f; rec.lse_p_lo[r] = 0.f;
      rec.lq[r] = 0.f; rec.lp[r] = 0.f;
    } else {
      double ma = -INFINITY, mp = -INFINITY, xa = 0.0, xp = 0.0;
      for (int s = 0; s < n_shards; ++s) {
        const float* o = line(s);
        ma = fmax(ma, (double)o[2] + (double)o[3]);
        mp = fmax(mp, (double)o[4] + (double)o[5]);
        if (__float_as_int(o[1]) != 0) { xa = (double)o[6]; xp = (double)o[7]; }
      }
      double sa = 0.0, sp = 0.0;
      for (int s = 0; s < n_shards; ++s) {
        const float* o = line(s);
        sa += exp(((double)o[2] + (double)o[3]) - ma);
        sp += exp(((double)o[4] + (double)o[5]) - mp);
      }
      const double la = ma + log(sa), lp = mp + log(sp);
      const float laf = (float)la, lpf = (float)lp;
      rec.lse_a[r] = laf; rec.lse_a_lo[r] = (float)(la - (double)laf);
      rec.lse_p[r] = lpf; rec.lse_p_lo[r] = (float)(lp - (double)lpf);
      rec.lq[r] = (float)(xa - la);
      rec.lp[r] = (float)(xp - lp);
      rec.flag[r] = kRowValid;      // a non-finite merged row is found and counted by the finalize step
    }
  }
}

}  // namespace

cudaError_t launch_vshard_localize(int64_t T, const int32_t* tokens, const uint8_t* mask, int64_t vocab_offset,
                                   int64_t V_shard, int64_t V_total, int32_t foreign, int32_t* tok_local,
                                   uint8_t* mask_local, Scalars* sc, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  vshard_localize_kernel<<<(unsigned)((T + 255) / 256), 256, 0, s>>>(T, tokens, mask, vocab_offset, V_shard, V_total,
                                                                   foreign, tok_local, mask_local, sc);
  return cudaGetLastError();
}

cudaError_t launch_vshard_export(int64_t T, int k, const Records& rec, const void* za, const void* zp, int64_t ld,
                                 int32_t dtype, const int32_t* tok_local, const uint8_t* mask_local,
                                 int64_t vocab_offset, const VshardDests& dests, int64_t line0, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  const int wpb = VS_NT / 32;
  vshard_export_kernel<<<(unsigned)((T + wpb - 1) / wpb), VS_NT, 0, s>>>(T, k, rec, za, zp, ld, dtype, tok_local,
                                                                        mask_local, vocab_offset, dests, line0);
  return cudaGetLastError();
}

cudaError_t launch_vshard_merge(int n_shards, int my_shard, const float* gathered, int64_t T, int k,
                                const Records& rec, Scalars* sc, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  // per warp: the keys of one list of every shard and a note per merged entry; at most 32 KB + 256 B
  const size_t per_warp = ((size_t)n_shards * k + (size_t)(k + 1) / 2) * sizeof(unsigned long long);
  int wpb = (int)((size_t)(48 * 1024) / per_warp);
  if (wpb > VS_NT / 32) wpb = VS_NT / 32;
  if (wpb < 1) return cudaErrorInvalidValue;                 // excluded by kVshardMaxEntries
  vshard_merge_kernel<<<(unsigned)((T + wpb - 1) / wpb), VS_NT, per_warp * wpb, s>>>(n_shards, my_shard, gathered, T, k,
                                                                                   rec, sc, wpb);
  return cudaGetLastError();
}

}  // namespace jp
