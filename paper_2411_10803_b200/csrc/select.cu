// Dual criteria, key set and selection: one CTA per request (Eq. 9, Eq. 10; Sec. 3.3 key set).
//
// The per-token score is computed in fp32 with one rounding per operation (no fused
// multiply-add, IEEE division), because it decides which indices are kept.  Budget mode is a
// radix select over the order-preserving integer image of the score, followed by an
// index-ordered emit, so kept indices come out ascending and equal scores resolve to the
// lower index.
#include "mustdrop_internal.h"

namespace mustdrop {
namespace {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kChunk = kMaxVis / kSelThreads;  // 16 consecutive tokens per thread in the ordered passes

// Larger float <=> larger unsigned image (handles negative values and -0 as well).
__device__ __forceinline__ uint32_t ordered_bits(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix sum of one int per thread over the block; also returns the block total.
// Fixed order, so results never depend on scheduling.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums /*[kSelWarps]*/, int* total) {
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

__global__ void __launch_bounds__(kSelThreads) select_kernel(SelectParams p) {
  __shared__ uint32_t s_bits[kMaxVis];      // ordered image of the score
  __shared__ uint8_t s_flag[kMaxVis];       // bit0: in key set, bit1: keep
  __shared__ int s_hist[256];
  __shared__ double s_dsum[kSelWarps];
  __shared__ int s_warp[kSelWarps];
  __shared__ int s_pick[2];
  __shared__ int s_wsuf[kSelWarps];
  static_assert(kSelThreads == 256, "one thread per radix bin");

  const int b = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int M = p.M;
  // Programmatic dependent launch: let the next kernel start its prologue, then wait until the
  // kernel that produced g / i has finished and its writes are visible.
  pdl_launch_dependents();
  pdl_wait();
  const float* g = p.g + static_cast<size_t>(b) * M;
  const float* in = p.i + static_cast<size_t>(b) * M;

  // T = sum_j g[j] in double; thread-strided partial sums, then a fixed shuffle tree.
  double part = 0.0;
  for (int j = tid; j < M; j += kSelThreads) part += static_cast<double>(g[j]);
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
  if (lane == 0) s_dsum[warp] = part;
  for (int j = tid; j < M; j += kSelThreads) s_flag[j] = 0;
  __syncthreads();
  double tsum = 0.0;
#pragma unroll
  for (int w = 0; w < kSelWarps; ++w) tsum += s_dsum[w];
  const float T = static_cast<float>(tsum);
  const float gt = __fmul_rn(p.gamma, T);

  // key set: mark distinct in-range indices
  if (p.key_max > 0) {
    int c = p.key_cnt[b];
    c = c < p.key_max ? c : p.key_max;
    for (int t = tid; t < c; t += kSelThreads) {
      int j = p.key_idx[static_cast<size_t>(b) * p.key_max + t];
      if (j >= 0 && j < M) s_flag[j] = 1;
      else record_status(p.workspace, MUSTDROP_ERR_BAD_KEY_INDEX, b * 65536 + t);
    }
  }
  // scores
  for (int j = tid; j < M; j += kSelThreads) {
    const float gj = __fdiv_rn(g[j], gt);
    const float rj = __fdiv_rn(in[j], p.alpha);
    float s;
    if (p.criteria == MUSTDROP_CRIT_GLOBAL_ONLY) s = gj;
    else if (p.criteria == MUSTDROP_CRIT_INDIVIDUAL_ONLY) s = rj;
    else s = (gj > rj) ? gj : rj;
    s_bits[j] = ordered_bits(s);
    if (p.s_out != nullptr) p.s_out[static_cast<size_t>(b) * M + j] = s;
  }
  __syncthreads();

  const int j0 = tid * kChunk;  // this thread's run of consecutive tokens in the ordered passes

  if (p.mode == MUSTDROP_MODE_THRESHOLD) {
    for (int j = tid; j < M; j += kSelThreads) {
      const bool in_d = g[j] <= gt;            // Eq. 9
      const bool small = in[j] < p.alpha;      // Eq. 10
      bool drop;
      if (p.criteria == MUSTDROP_CRIT_GLOBAL_ONLY) drop = in_d;
      else if (p.criteria == MUSTDROP_CRIT_INDIVIDUAL_ONLY) drop = small;
      else drop = in_d && small;
      if ((s_flag[j] & 1) || !drop) s_flag[j] |= 2;
    }
  } else {
    // number of distinct keys
    int nk = 0;
    for (int j = tid; j < M; j += kSelThreads) nk += (s_flag[j] & 1);
    int n_key;
    (void)block_exclusive_scan(nk, s_warp, &n_key);
    int want = p.budget - n_key;
    const int n_cand = M - n_key;
    want = want < n_cand ? want : n_cand;
    if (want > 0) {
      // radix select of the want-th largest candidate: four 8-bit digits from the top
      uint32_t prefix = 0, mask = 0;
      int remaining = want;
      for (int shift = 24; shift >= 0; shift -= 8) {
        for (int t = tid; t < 256; t += kSelThreads) s_hist[t] = 0;
        __syncthreads();
        for (int j = tid; j < M; j += kSelThreads) {
          const uint32_t u = s_bits[j];
          if (!(s_flag[j] & 1) && (u & mask) == prefix) atomicAdd(&s_hist[(u >> shift) & 255u], 1);
        }
        __syncthreads();
        // digit d is the cut iff (#candidates with a larger digit) < remaining <= that + hist[d];
        // thread d owns bin d: suffix sums by warp shuffles, then across the eight warps
        {
          const int here = s_hist[tid];
          int suf = here;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_down_sync(0xffffffffu, suf, d);
            if (lane + d < 32) suf += t;
          }
          if (lane == 0) s_wsuf[warp] = suf;
          __syncthreads();
          int above = suf - here;
#pragma unroll
          for (int w = 0; w < kSelWarps; ++w)
            if (w > warp) above += s_wsuf[w];
          if (above < remaining && remaining <= above + here) {
            s_pick[0] = tid;
            s_pick[1] = remaining - above;
          }
        }
        __syncthreads();
        prefix |= static_cast<uint32_t>(s_pick[0]) << shift;
        mask |= 255u << shift;
        remaining = s_pick[1];
        __syncthreads();
      }
      // prefix is now the cut value; `remaining` tokens equal to it are taken, lowest index first
      int eq = 0;
      for (int t = 0; t < kChunk; ++t) {
        const int j = j0 + t;
        if (j < M && !(s_flag[j] & 1) && s_bits[j] == prefix) ++eq;
      }
      int eq_total;
      int eq_rank = block_exclusive_scan(eq, s_warp, &eq_total);
      for (int t = 0; t < kChunk; ++t) {
        const int j = j0 + t;
        if (j >= M) break;
        const uint8_t f = s_flag[j];
        if (f & 1) continue;
        const uint32_t u = s_bits[j];
        if (u > prefix) s_flag[j] = f | 2;
        else if (u == prefix) {
          if (eq_rank < remaining) s_flag[j] = f | 2;
          ++eq_rank;
        }
      }
    }
    __syncthreads();
    for (int j = tid; j < M; j += kSelThreads)
      if (s_flag[j] & 1) s_flag[j] |= 2;
  }
  __syncthreads();

  // index-ordered emit
  int cnt = 0;
  for (int t = 0; t < kChunk; ++t) {
    const int j = j0 + t;
    if (j < M && (s_flag[j] & 2)) ++cnt;
  }
  int total;
  int pos = block_exclusive_scan(cnt, s_warp, &total);
  int32_t* out = p.kept_idx + static_cast<size_t>(b) * p.cap;
  for (int t = 0; t < kChunk; ++t) {
    const int j = j0 + t;
    if (j < M && (s_flag[j] & 2)) {
      if (pos < p.cap) out[pos] = j;
      ++pos;
    }
  }
  if (tid == 0) p.kept_cnt[b] = total;
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
  return launch_pdl(select_kernel, dim3(r.B), dim3(kSelThreads), 0, stream, p);
}

}  // namespace mustdrop
