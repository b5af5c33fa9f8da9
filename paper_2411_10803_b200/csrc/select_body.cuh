// Dual criteria, key set and selection for ONE request, worked by a group of 256 threads
// (Eq. 9, Eq. 10; Sec. 3.3 key set).  Included by the stand-alone select kernel (one CTA per
// request) and by the single-launch filter kernel (the first eight warps of every CTA of the
// request's cluster).
//
// The per-token score is computed in fp32 with one rounding per operation (no fused
// multiply-add, IEEE division), because it decides which indices are kept.  Budget mode is a
// radix select over the order-preserving integer image of the score, followed by an
// index-ordered emit, so kept indices come out ascending and equal scores resolve to the
// lower index.
//
// Every thread owns a run of consecutive tokens and keeps their scores in registers; shared
// memory only holds the key-set bitmap, one 256-bin histogram and a few per-warp partials.
#pragma once

#include "mustdrop_internal.h"

namespace mustdrop {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMaxOwn = kMaxVis / kSelThreads;  // at most 16 consecutive tokens per thread

struct SelectParams {
  const float* g;
  const float* i;
  const int32_t* key_idx;
  const int32_t* key_cnt;
  int32_t* kept_idx;
  int32_t* kept_cnt;
  float* s_out;
  void* workspace;
  int32_t M, key_max, mode, criteria, budget, cap;
  float gamma, alpha;
  // a layer in a chain of pruning layers (all nullable): per-request token counts, original ids
  // in and out, and the key tokens' positions among the kept tokens
  const int32_t* vis_cnt;
  const int32_t* orig_in;
  int32_t* orig_out;
  int32_t* key_idx_out;
  int32_t* key_cnt_out;
  int32_t vis_start, N;                   // this request's sequence length = vis_start + its tokens + N
  int32_t gamma_default, alpha_default;   // 1: gamma = 1 / (the request's tokens), alpha = 2 / (its length)
};

struct SelectShared {
  uint32_t key[kMaxVis / 32];  // key-set bitmap
  int hist[256];
  double dsum[kSelWarps];
  int warp[kSelWarps];
  int wsuf[kSelWarps];
  uint32_t band[kSelWarps], bor[kSelWarps];   // per warp: AND / OR of the tokens' ordered score bits
  int pick[3];
  int nkey;
};

// How the 256 threads of a group meet: the whole CTA, or named barrier 1 when the group is a
// part of a larger CTA.
struct SelectSyncCta {
  static __device__ __forceinline__ void sync() { __syncthreads(); }
};
struct SelectSyncGroup {
  static __device__ __forceinline__ void sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
};

// Larger float <=> larger unsigned image (handles negative values and -0 as well).
__device__ __forceinline__ uint32_t ordered_bits(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix sum of one int per thread over the group; also returns the group total.
// Fixed order, so results never depend on scheduling.  Uses two barriers.
template <class Sync>
__device__ __noinline__ int group_exclusive_scan(int v, int tid, int* warp_sums /*[kSelWarps]*/, int* total) {
  const int lane = tid & 31, warp = tid >> 5;
  int inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, d);
    if (lane >= d) inc += t;
  }
  Sync::sync();  // protect warp_sums from the previous use
  if (lane == 31) warp_sums[warp] = inc;
  Sync::sync();
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kSelWarps; ++w) {
    int s = warp_sums[w];
    if (w < warp) base += s;
    tot += s;
  }
  *total = tot;
  return base + inc - v;
}


// Clears the group's shared state; touches no global data.  select_request's first group barrier
// orders the clear before every use, so no barrier is needed in between.
__device__ __forceinline__ void select_clear(SelectShared& s, int tid) {
  for (int w = tid; w < kMaxVis / 32; w += kSelThreads) s.key[w] = 0u;
  s.hist[tid] = 0;
  if (tid == 0) s.nkey = 0;
}

// Selection for request b.  `tid` is the thread's index in the group (0..255); OWN consecutive
// tokens per thread (1, 2, 4, 8 or 16; OWN * 256 >= M).  With write_out the group stores
// kept_idx / kept_cnt / s_out (and reports bad key indices); kept_list / kept_total, when not
// null, receive the same list and count (shared memory of the caller).
template <int OWN, class Sync>
__device__ __forceinline__ void select_request(const SelectParams& p, SelectShared& s, int b, int tid, bool write_out,
                                               int32_t* kept_list, int32_t* kept_total) {
  constexpr int kOwn = OWN;
  constexpr int own = OWN;
  static_assert(kSelThreads == 256, "one thread per radix bin");
  const int lane = tid & 31, warp = tid >> 5;
  const int ld = p.M;                                    // row length of g / i / s_out / orig_in
  const int M = p.vis_cnt ? clamp_vis_cnt(p.vis_cnt[b], p.M) : p.M;   // this request's tokens
  const int j0 = tid * own;                              // this thread's first token
  float gamma = p.gamma, alpha = p.alpha;
  if (p.vis_cnt != nullptr) {                            // thresholds that default follow the request's own sizes
    if (p.gamma_default) gamma = __fdiv_rn(1.0f, static_cast<float>(M));
    if (p.alpha_default) alpha = __fdiv_rn(2.0f, static_cast<float>(p.vis_start + M + p.N));
  }

  const float* g = p.g + static_cast<size_t>(b) * ld;
  const float* in = p.i + static_cast<size_t>(b) * ld;
  // the key-set loads are issued first so that their latency overlaps the score loads
  int key_c = 0, key_j = -1;
  if (p.key_max > 0) {
    key_c = p.key_cnt[b];
    if (tid < p.key_max) key_j = p.key_idx[static_cast<size_t>(b) * p.key_max + tid];
  }
  float gv[kOwn], iv[kOwn];
  double part = 0.0;
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    const int j = j0 + e;
    const bool ok = e < own && j < M;
    gv[e] = ok ? g[j] : 0.0f;
    iv[e] = ok ? in[j] : 0.0f;
    part += static_cast<double>(gv[e]);
  }
  // T = sum_j g[j] in double: per-thread runs, then a fixed shuffle tree, then the eight warps in order
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
  if (lane == 0) s.dsum[warp] = part;
  Sync::sync();   // also orders the bitmap clear before the key marks below
  // key set: mark distinct in-range indices
  if (p.key_max > 0) {
    const int c = key_c < p.key_max ? key_c : p.key_max;
    for (int t = tid; t < c; t += kSelThreads) {
      const int j = t == tid ? key_j : p.key_idx[static_cast<size_t>(b) * p.key_max + t];
      if (j >= 0 && j < M) {
        const uint32_t bit = 1u << (j & 31);
        if (!(atomicOr(&s.key[j >> 5], bit) & bit)) atomicAdd(&s.nkey, 1);   // count distinct keys
      } else {
        if (write_out) record_status(p.workspace, MUSTDROP_ERR_BAD_KEY_INDEX, b * 65536 + t);
      }
    }
  }
  double tsum = 0.0;
#pragma unroll
  for (int w = 0; w < kSelWarps; ++w) tsum += s.dsum[w];
  const float T = static_cast<float>(tsum);
  const float gt = __fmul_rn(gamma, T);

  // scores of the thread's tokens, as ordered integers
  uint32_t u[kOwn];
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    const int j = j0 + e;
    u[e] = 0u;
    if (e < own && j < M) {
      const float gj = __fdiv_rn(gv[e], gt);
      const float rj = __fdiv_rn(iv[e], alpha);
      float sc;
      if (p.criteria == MUSTDROP_CRIT_GLOBAL_ONLY) sc = gj;
      else if (p.criteria == MUSTDROP_CRIT_INDIVIDUAL_ONLY) sc = rj;
      else sc = (gj > rj) ? gj : rj;
      u[e] = ordered_bits(sc);
      if (write_out && p.s_out != nullptr) p.s_out[static_cast<size_t>(b) * ld + j] = sc;
    }
  }
  // Bits that all of the request's scores share need no radix pass (scores of one request lie
  // within a few powers of two: their top byte is the same for all, and a pass over it would be
  // every thread's atomics on one or two counters): AND and OR over the tokens, per warp here,
  // over the group behind the barrier below.
  uint32_t all_and = 0xffffffffu, all_or = 0u;
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    if (e < own && j0 + e < M) {
      all_and &= u[e];
      all_or |= u[e];
    }
  }
  all_and = __reduce_and_sync(0xffffffffu, all_and);
  all_or = __reduce_or_sync(0xffffffffu, all_or);
  if (lane == 0) {
    s.band[warp] = all_and;
    s.bor[warp] = all_or;
  }
  Sync::sync();   // key marks complete

  // per-token bits: bit e of `valid` = token exists, of `key` = in the key set, of `keep` = retained
  uint32_t valid = 0u, key = 0u, keep = 0u;
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    const int j = j0 + e;
    if (e < own && j < M) {
      valid |= 1u << e;
      if ((s.key[j >> 5] >> (j & 31)) & 1u) key |= 1u << e;
    }
  }
  const uint32_t cand = valid & ~key;

  if (p.mode == MUSTDROP_MODE_THRESHOLD) {
#pragma unroll
    for (int e = 0; e < kOwn; ++e) {
      if ((valid >> e) & 1u) {
        const bool in_d = gv[e] <= gt;            // Eq. 9
        const bool small = iv[e] < alpha;         // Eq. 10
        bool drop;
        if (p.criteria == MUSTDROP_CRIT_GLOBAL_ONLY) drop = in_d;
        else if (p.criteria == MUSTDROP_CRIT_INDIVIDUAL_ONLY) drop = small;
        else drop = in_d && small;
        if (!drop) keep |= 1u << e;
      }
    }
    keep |= key;
  } else {
    const int n_key = s.nkey;
    int want = p.budget - n_key;
    const int n_cand = M - n_key;
    want = want < n_cand ? want : n_cand;
    keep = key;
    if (want > 0) {
      // radix select of the want-th largest candidate: 8-bit digits from the highest bit in
      // which two tokens differ downwards (the bits above it are the same in every candidate)
      uint32_t g_and = 0xffffffffu, g_or = 0u;
#pragma unroll
      for (int w = 0; w < kSelWarps; ++w) {
        g_and &= s.band[w];
        g_or |= s.bor[w];
      }
      const uint32_t differ = g_and ^ g_or;
      const int hb = differ ? 31 - __clz(differ) : 7;                  // (all equal: one pass over the low byte)
      uint32_t mask = hb >= 31 ? 0u : ~((2u << hb) - 1u);               // the shared bits
      uint32_t prefix = g_and & mask;
      int remaining = want;
      // (kept as a real loop: the kernel runs once per launch from a cold instruction cache, so
      // code size, not instruction count, sets its latency)
#pragma unroll 1
      for (int shift = hb >= 7 ? hb - 7 : 0;; shift = shift > 8 ? shift - 8 : 0) {
#pragma unroll
        for (int e = 0; e < kOwn; ++e) {
          const bool act = ((cand >> e) & 1u) && (u[e] & mask) == prefix;
          if (act) atomicAdd(&s.hist[(u[e] >> shift) & 255u], 1);
        }
        Sync::sync();
        // digit d is the cut iff (#candidates with a larger digit) < remaining <= that + hist[d];
        // thread d owns bin d: suffix sums by warp shuffles, then across the eight warps
        const int here = s.hist[tid];
        s.hist[tid] = 0;   // ready for the next digit
        int suf = here;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int t = __shfl_down_sync(0xffffffffu, suf, d);
          if (lane + d < 32) suf += t;
        }
        if (lane == 0) s.wsuf[warp] = suf;
        Sync::sync();
        int above = suf - here;
#pragma unroll
        for (int w = 0; w < kSelWarps; ++w)
          if (w > warp) above += s.wsuf[w];
        if (above < remaining && remaining <= above + here) {
          s.pick[0] = tid;
          s.pick[1] = remaining - above;
          s.pick[2] = here;
        }
        Sync::sync();
        // (the lowest digit may reach over bits that are resolved already: they are the same in
        // every token still in the running, so the bins keep their order)
        prefix = (prefix & ~(255u << shift)) | (static_cast<uint32_t>(s.pick[0]) << shift);
        mask |= 255u << shift;
        remaining = s.pick[1];
        if (remaining == s.pick[2]) break;   // the whole bin is taken: lower digits cannot matter
        if (shift == 0) break;
      }
      // Over the resolved digits, prefix is the cut: larger tokens are kept, and `remaining` of
      // the tokens equal to it, lowest index first (all of them after an early exit).
      const bool all_equal_kept = remaining == s.pick[2];
      uint32_t eq = 0u;
#pragma unroll
      for (int e = 0; e < kOwn; ++e) {
        if ((cand >> e) & 1u) {
          const uint32_t v = u[e] & mask;
          if (v > prefix || (all_equal_kept && v == prefix)) keep |= 1u << e;
          else if (v == prefix) eq |= 1u << e;
        }
      }
      if (!all_equal_kept) {   // uniform over the block
        int eq_total;
        int eq_rank = group_exclusive_scan<Sync>(__popc(eq), tid, s.warp, &eq_total);
#pragma unroll
        for (int e = 0; e < kOwn; ++e) {
          if ((eq >> e) & 1u) {
            if (eq_rank < remaining) keep |= 1u << e;
            ++eq_rank;
          }
        }
      }
    }
  }

  // index-ordered emit
  int total;
  int pos = group_exclusive_scan<Sync>(__popc(keep), tid, s.warp, &total);
  // a chain of layers also wants the kept tokens' original ids and where the key tokens went
  const bool emit_keys = p.key_idx_out != nullptr && p.key_max > 0;   // uniform over the group
  int key_pos = 0, key_total = 0;
  if (emit_keys) key_pos = group_exclusive_scan<Sync>(__popc(key & keep), tid, s.warp, &key_total);
  int32_t* out = p.kept_idx + static_cast<size_t>(b) * p.cap;
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    if ((keep >> e) & 1u) {
      if (pos < p.cap) {
        if (write_out) {
          out[pos] = j0 + e;
          if (p.orig_out != nullptr)
            p.orig_out[static_cast<size_t>(b) * p.cap + pos] =
                p.orig_in != nullptr ? p.orig_in[static_cast<size_t>(b) * ld + j0 + e] : j0 + e;
          if (emit_keys && ((key >> e) & 1u) && key_pos < p.key_max)
            p.key_idx_out[static_cast<size_t>(b) * p.key_max + key_pos] = pos;
        }
        if (kept_list != nullptr) kept_list[pos] = j0 + e;
      }
      if ((key >> e) & 1u) ++key_pos;
      ++pos;
    }
  }
  if (tid == 0) {
    if (write_out) {
      p.kept_cnt[b] = total;
      if (p.key_cnt_out != nullptr) p.key_cnt_out[b] = emit_keys ? (key_total < p.key_max ? key_total : p.key_max) : 0;
    }
    if (kept_total != nullptr) *kept_total = total;
  }
}

}  // namespace mustdrop
