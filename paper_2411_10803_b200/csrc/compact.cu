// Gather-compaction of the retained tokens: hidden rows and per-head K / V rows are copied
// as 16-byte vectors into dense outputs (the pruned tokens leave the sequence and the KV
// cache; Table 3 counts the vision tokens that remain in the cache).
//
// In rebuild mode the outputs hold the request's whole next sequence, packed: the prefix rows,
// the kept vision rows, then its text rows (which sit directly behind its own vision tokens in
// the source) - the input layout of the next pruning layer.
//
// Work unit: one CTA per (output row r, request b, tensor).  A hidden row is `hidden` bf16
// contiguous; a K or V "row" is H pieces of 256 bytes, one per head.  Every thread keeps
// several independent 16-byte loads in flight before storing.
#include "mustdrop_internal.h"

namespace mustdrop {
namespace {

constexpr int kCompactThreads = 256;
constexpr int kUnroll = 4;

struct CompactParams {
  const int32_t* kept_idx;
  const int32_t* kept_cnt;
  const uint4* src[3];   // hidden, k, v
  uint4* dst[3];
  void* workspace;
  const int32_t* vis_cnt;   // [B] or null: vision tokens the request holds (rebuild: where its text rows start)
  int32_t rebuild, N, out_rows;
  int32_t cap, M, vis_start, H, hidden_vecs;  // hidden_vecs = hidden / 8
  // strides in 16-byte vectors
  int64_t hid_sb, hid_sl, k_sb, k_sh, k_sl, v_sb, v_sh, v_sl;
};

// Source rows are read once: no L1 allocation, first in line for L2 eviction.
__device__ __forceinline__ uint4 ld_stream(const uint4* p, uint64_t policy) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p), "l"(policy));
  return v;
}

__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

__global__ void __launch_bounds__(kCompactThreads) compact_kernel(CompactParams p) {
  const int r = blockIdx.x, b = blockIdx.y, which = blockIdx.z;
  MD_PIPE(p.workspace, 2, false, false);
  pdl_launch_dependents();
  pdl_wait();   // kept_idx / kept_cnt come from the previous kernel in the stream
  if (p.src[which] == nullptr) return;
  // a count outside [0, cap] is not trusted: clamped, and recorded (a negative one marks a request
  // whose selection failed: nothing of it is copied)
  const int cnt_raw = p.kept_cnt[b];
  const int n_kept = min(max(cnt_raw, 0), p.cap);
  if (cnt_raw != n_kept && threadIdx.x == 0 && r == 0)
    record_status(p.workspace, MUSTDROP_ERR_BAD_KEY_INDEX, b * 65536 + 65535);
  if (cnt_raw < 0) return;
  int64_t row;        // source row
  int out_row = r;    // destination row
  if (!p.rebuild || (r >= p.vis_start && r < p.vis_start + p.cap)) {
    const int rk = p.rebuild ? r - p.vis_start : r;          // kept-row number
    if (rk >= n_kept) return;
    const int j = p.kept_idx[static_cast<size_t>(b) * p.cap + rk];
    if (j < 0 || j >= p.M) {
      if (threadIdx.x == 0) record_status(p.workspace, MUSTDROP_ERR_BAD_KEY_INDEX, b * 65536 + (rk & 65535));
      return;
    }
    row = p.vis_start + j;
  } else if (r < p.vis_start) {
    row = r;                                                 // prefix row, copied through
  } else {
    const int t = r - p.vis_start - p.cap;                   // text row t
    const int Mb = p.vis_cnt ? clamp_vis_cnt(p.vis_cnt[b], p.M) : p.M;
    row = p.vis_start + Mb + t;
    out_row = p.vis_start + n_kept + t;
  }
  uint64_t once;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(once));
  if (which == 0) {
    const uint4* src = p.src[0] + b * p.hid_sb + row * p.hid_sl;
    uint4* dst = p.dst[0] + (static_cast<int64_t>(b) * p.out_rows + out_row) * p.hidden_vecs;
    const int n = p.hidden_vecs;
    for (int base = 0; base < n; base += kCompactThreads * kUnroll) {
      uint4 v[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int x = base + u * kCompactThreads + threadIdx.x;
        if (x < n) v[u] = ld_stream(src + x, once);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int x = base + u * kCompactThreads + threadIdx.x;
        if (x < n) st_stream(dst + x, v[u]);
      }
    }
  } else {
    const bool is_k = which == 1;
    const int64_t sb = is_k ? p.k_sb : p.v_sb, sh = is_k ? p.k_sh : p.v_sh, sl = is_k ? p.k_sl : p.v_sl;
    const uint4* src = p.src[which] + b * sb + row * sl;
    uint4* dst = p.dst[which] + (static_cast<int64_t>(b) * p.H * p.out_rows + out_row) * 16;
    const int n = p.H * 16;  // 16 vectors of 16 bytes per head row
    for (int base = 0; base < n; base += kCompactThreads * kUnroll) {
      uint4 v[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int x = base + u * kCompactThreads + threadIdx.x;
        if (x < n) v[u] = ld_stream(src + (x >> 4) * sh + (x & 15), once);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int x = base + u * kCompactThreads + threadIdx.x;
        if (x < n) st_stream(dst + static_cast<int64_t>(x >> 4) * p.out_rows * 16 + (x & 15), v[u]);
      }
    }
  }
  MD_PIPE(p.workspace, 2, true, false);
}

}  // namespace

cudaError_t launch_compact(const mustdrop_plan& plan, const int32_t* kept_idx, const int32_t* kept_cnt,
                           const void* hidden, const void* k, const void* v, void* hidden_out, void* k_out,
                           void* v_out, void* workspace, cudaStream_t stream, const int32_t* vis_cnt) {
  const Resolved& r = plan.r;
  CompactParams p;
  p.kept_idx = kept_idx; p.kept_cnt = kept_cnt;
  p.src[0] = static_cast<const uint4*>(hidden); p.src[1] = static_cast<const uint4*>(k);
  p.src[2] = static_cast<const uint4*>(v);
  p.dst[0] = static_cast<uint4*>(hidden_out); p.dst[1] = static_cast<uint4*>(k_out);
  p.dst[2] = static_cast<uint4*>(v_out);
  p.workspace = workspace;
  p.vis_cnt = vis_cnt; p.rebuild = r.rebuild; p.N = r.N; p.out_rows = r.out_rows;
  p.cap = r.cap; p.M = r.M; p.vis_start = r.vis_start; p.H = r.H; p.hidden_vecs = r.hidden / 8;
  p.hid_sb = r.hid_sb / 8; p.hid_sl = r.hid_sl / 8;
  p.k_sb = r.k_sb / 8; p.k_sh = r.k_sh / 8; p.k_sl = r.k_sl / 8;
  p.v_sb = r.v_sb / 8; p.v_sh = r.v_sh / 8; p.v_sl = r.v_sl / 8;
  dim3 grid(r.out_rows, r.B, 3);
  return launch_pdl(compact_kernel, grid, dim3(kCompactThreads), 0, stream, p);
}

}  // namespace mustdrop
