// Dual criteria, key set and selection: one CTA per request (Eq. 9, Eq. 10; Sec. 3.3 key set).
//
// The per-token score is computed in fp32 with one rounding per operation (no fused
// multiply-add, IEEE division), because it decides which indices are kept.  Budget mode is a
// radix select over the order-preserving integer image of the score, followed by an
// index-ordered emit, so kept indices come out ascending and equal scores resolve to the
// lower index.
//
// Every thread owns a run of consecutive tokens and keeps their scores in registers; shared
// memory only holds the key-set bitmap, one 256-bin histogram and a few per-warp partials.
#include "mustdrop_internal.h"

namespace mustdrop {
namespace {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMaxOwn = kMaxVis / kSelThreads;  // at most 16 consecutive tokens per thread

// Larger float <=> larger unsigned image (handles negative values and -0 as well).
__device__ __forceinline__ uint32_t ordered_bits(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix sum of one int per thread over the block; also returns the block total.
// Fixed order, so results never depend on scheduling.  Uses two barriers.
__device__ __noinline__ int block_exclusive_scan(int v, int* warp_sums /*[kSelWarps]*/, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, d);
    if (lane >= d) inc += t;
  }
  __syncthreads();  // protect warp_sums from the previous use
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
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

#ifdef MUSTDROP_TRACE
#define SEL_STAMP(ev) do { if (threadIdx.x == 0 && blockIdx.x == 0 && p.workspace) { \
  reinterpret_cast<long long*>(static_cast<unsigned char*>(p.workspace) + 2048)[ev] = clock64(); } } while (0)
#else
#define SEL_STAMP(ev) ((void)0)
#endif

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
};

// OWN: consecutive tokens per thread (1, 2, 4, 8 or 16; OWN * 256 >= M).
template <int OWN>
__global__ void __launch_bounds__(kSelThreads) select_kernel(SelectParams p) {
  constexpr int kOwn = OWN;
  __shared__ uint32_t s_key[kMaxVis / 32];  // key-set bitmap
  __shared__ int s_hist[256];
  __shared__ double s_dsum[kSelWarps];
  __shared__ int s_warp[kSelWarps];
  __shared__ int s_wsuf[kSelWarps];
  __shared__ int s_pick[3];
  __shared__ int s_nkey;
  static_assert(kSelThreads == 256, "one thread per radix bin");

  const int b = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int M = p.M;
  constexpr int own = OWN;
  const int j0 = tid * own;                              // this thread's first token

  // Work that touches no global data, then let the next kernel start its prologue and wait for
  // the kernel that produced g / i.
  SEL_STAMP(0);
  MD_PIPE(p.workspace, 1, false, false);
  for (int w = tid; w < kMaxVis / 32; w += kSelThreads) s_key[w] = 0u;
  s_hist[tid] = 0;
  if (tid == 0) s_nkey = 0;
  pdl_launch_dependents();
  pdl_wait();
  SEL_STAMP(1);

  const float* g = p.g + static_cast<size_t>(b) * M;
  const float* in = p.i + static_cast<size_t>(b) * M;
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
  if (lane == 0) s_dsum[warp] = part;
  SEL_STAMP(2);
  __syncthreads();   // also orders the bitmap clear before the key marks below
  SEL_STAMP(3);
  // key set: mark distinct in-range indices
  if (p.key_max > 0) {
    const int c = key_c < p.key_max ? key_c : p.key_max;
    for (int t = tid; t < c; t += kSelThreads) {
      const int j = t == tid ? key_j : p.key_idx[static_cast<size_t>(b) * p.key_max + t];
      if (j >= 0 && j < M) {
        const uint32_t bit = 1u << (j & 31);
        if (!(atomicOr(&s_key[j >> 5], bit) & bit)) atomicAdd(&s_nkey, 1);   // count distinct keys
      } else {
        record_status(p.workspace, MUSTDROP_ERR_BAD_KEY_INDEX, b * 65536 + t);
      }
    }
  }
  double tsum = 0.0;
#pragma unroll
  for (int w = 0; w < kSelWarps; ++w) tsum += s_dsum[w];
  const float T = static_cast<float>(tsum);
  const float gt = __fmul_rn(p.gamma, T);

  // scores of the thread's tokens, as ordered integers
  uint32_t u[kOwn];
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    const int j = j0 + e;
    u[e] = 0u;
    if (e < own && j < M) {
      const float gj = __fdiv_rn(gv[e], gt);
      const float rj = __fdiv_rn(iv[e], p.alpha);
      float s;
      if (p.criteria == MUSTDROP_CRIT_GLOBAL_ONLY) s = gj;
      else if (p.criteria == MUSTDROP_CRIT_INDIVIDUAL_ONLY) s = rj;
      else s = (gj > rj) ? gj : rj;
      u[e] = ordered_bits(s);
      if (p.s_out != nullptr) p.s_out[static_cast<size_t>(b) * M + j] = s;
    }
  }
  SEL_STAMP(4);
  __syncthreads();   // key marks complete
  SEL_STAMP(5);

  // per-token bits: bit e of `valid` = token exists, of `key` = in the key set, of `keep` = retained
  uint32_t valid = 0u, key = 0u, keep = 0u;
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    const int j = j0 + e;
    if (e < own && j < M) {
      valid |= 1u << e;
      if ((s_key[j >> 5] >> (j & 31)) & 1u) key |= 1u << e;
    }
  }
  const uint32_t cand = valid & ~key;

  if (p.mode == MUSTDROP_MODE_THRESHOLD) {
#pragma unroll
    for (int e = 0; e < kOwn; ++e) {
      if ((valid >> e) & 1u) {
        const bool in_d = gv[e] <= gt;            // Eq. 9
        const bool small = iv[e] < p.alpha;       // Eq. 10
        bool drop;
        if (p.criteria == MUSTDROP_CRIT_GLOBAL_ONLY) drop = in_d;
        else if (p.criteria == MUSTDROP_CRIT_INDIVIDUAL_ONLY) drop = small;
        else drop = in_d && small;
        if (!drop) keep |= 1u << e;
      }
    }
    keep |= key;
  } else {
    const int n_key = s_nkey;
    SEL_STAMP(6);
    int want = p.budget - n_key;
    const int n_cand = M - n_key;
    want = want < n_cand ? want : n_cand;
    keep = key;
    if (want > 0) {
      // radix select of the want-th largest candidate: four 8-bit digits from the top
      uint32_t prefix = 0, mask = 0;
      int remaining = want;
      // (kept as a real loop: the kernel runs once per launch from a cold instruction cache, so
      // code size, not instruction count, sets its latency)
#pragma unroll 1
      for (int shift = 24; shift >= 0; shift -= 8) {
#pragma unroll
        for (int e = 0; e < kOwn; ++e) {
          const bool act = ((cand >> e) & 1u) && (u[e] & mask) == prefix;
          if (act) atomicAdd(&s_hist[(u[e] >> shift) & 255u], 1);
        }
        if (shift == 16) SEL_STAMP(13);
        __syncthreads();
        if (shift == 16) SEL_STAMP(14);
        // digit d is the cut iff (#candidates with a larger digit) < remaining <= that + hist[d];
        // thread d owns bin d: suffix sums by warp shuffles, then across the eight warps
        const int here = s_hist[tid];
        s_hist[tid] = 0;   // ready for the next digit
        int suf = here;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int t = __shfl_down_sync(0xffffffffu, suf, d);
          if (lane + d < 32) suf += t;
        }
        if (lane == 0) s_wsuf[warp] = suf;
        if (shift == 16) SEL_STAMP(15);
        __syncthreads();
        if (shift == 16) SEL_STAMP(16);
        int above = suf - here;
#pragma unroll
        for (int w = 0; w < kSelWarps; ++w)
          if (w > warp) above += s_wsuf[w];
        if (above < remaining && remaining <= above + here) {
          s_pick[0] = tid;
          s_pick[1] = remaining - above;
          s_pick[2] = here;
        }
        __syncthreads();
        SEL_STAMP(7 + (24 - shift) / 8);
        prefix |= static_cast<uint32_t>(s_pick[0]) << shift;
        mask |= 255u << shift;
        remaining = s_pick[1];
        if (remaining == s_pick[2]) break;   // the whole bin is taken: lower digits cannot matter
      }
      // Over the resolved digits, prefix is the cut: larger tokens are kept, and `remaining` of
      // the tokens equal to it, lowest index first (all of them after an early exit).
      const bool all_equal_kept = remaining == s_pick[2];
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
        int eq_rank = block_exclusive_scan(__popc(eq), s_warp, &eq_total);
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

  SEL_STAMP(11);
  // index-ordered emit
  int total;
  int pos = block_exclusive_scan(__popc(keep), s_warp, &total);
  int32_t* out = p.kept_idx + static_cast<size_t>(b) * p.cap;
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    if ((keep >> e) & 1u) {
      if (pos < p.cap) out[pos] = j0 + e;
      ++pos;
    }
  }
  if (tid == 0) p.kept_cnt[b] = total;
  MD_PIPE(p.workspace, 1, true, false);
  SEL_STAMP(12);
}

}  // namespace

cudaError_t launch_select(const mustdrop_plan& plan, const float* g, const float* i, const int32_t* key_idx,
                          const int32_t* key_cnt, int32_t* kept_idx, int32_t* kept_cnt, float* s_out,
                          void* workspace, cudaStream_t stream) {
  const Resolved& r = plan.r;
  SelectParams p;
  p.g = g; p.i = i; p.key_idx = key_idx; p.key_cnt = key_cnt; p.kept_idx = kept_idx; p.kept_cnt = kept_cnt;
  p.s_out = s_out; p.workspace = workspace;
  p.M = r.M; p.key_max = r.key_max; p.mode = r.mode; p.criteria = r.criteria; p.budget = r.budget; p.cap = r.cap;
  p.gamma = r.gamma; p.alpha = r.alpha;
  const int own = (r.M + kSelThreads - 1) / kSelThreads;
  static_assert(kMaxOwn == 16, "dispatch below covers up to 16 tokens per thread");
  if (own <= 1) return launch_pdl(select_kernel<1>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
  if (own <= 2) return launch_pdl(select_kernel<2>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
  if (own <= 4) return launch_pdl(select_kernel<4>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
  if (own <= 8) return launch_pdl(select_kernel<8>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
  return launch_pdl(select_kernel<16>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
}

}  // namespace mustdrop
