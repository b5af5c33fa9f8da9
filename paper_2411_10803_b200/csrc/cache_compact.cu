// Decoding-stage cache compaction (Sec. 3.5, output-aware cache policy): the layers that follow
// the second one keep, of the vision tokens, only S_few - the set still retained after the last
// pruning layer.  One launch rebuilds the K and V caches of all those layers:
//   out[y][b][h] = [ prefix rows ; rows of the tokens in S_few[b] ; tail rows (text) ]
// A layer's cache lists the vision tokens it holds by original id (ascending), so a token of
// S_few is located in it by binary search.
//
// Work unit: one CTA per (output row, request, layer); it copies the row's 256-byte pieces of
// all heads, for K and for V, as 16-byte vectors with several loads in flight per thread.
#include "mustdrop_internal.h"

namespace mustdrop {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;

struct CacheParams {
  const uint4* src[2];   // k_cache, v_cache  [Lyr,B,H,R,16 vectors]
  uint4* dst[2];         // k_out, v_out      [Lyr,B,H,rows_out,16 vectors]
  const int32_t* layer_ids;   // [Lyr,B,ids_max] original ids held by the layer, ascending
  const int32_t* layer_cnt;   // [Lyr,B]
  const int32_t* s_few;       // [B,cap] original ids, ascending
  const int32_t* s_few_cnt;   // [B]
  void* workspace;
  int32_t B, H, rows_in, rows_out, vis_start, n_tail, ids_max, cap;
};

__device__ __forceinline__ uint4 ld_once(const uint4* p, uint64_t policy) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p), "l"(policy));
  return v;
}
__device__ __forceinline__ void st_once(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

__global__ void __launch_bounds__(kThreads) cache_compact_kernel(CacheParams p) {
  const int r = blockIdx.x, b = blockIdx.y, y = blockIdx.z;
  pdl_launch_dependents();
  pdl_wait();   // S_few comes from the last pruning layer's selection
  const int n_few = min(max(p.s_few_cnt[b], 0), p.cap);
  const int n_held = min(max(p.layer_cnt[static_cast<size_t>(y) * p.B + b], 0), p.ids_max);
  int src_row, dst_row;
  if (r < p.vis_start) {
    src_row = dst_row = r;                                   // prefix
  } else if (r < p.vis_start + p.cap) {
    const int rk = r - p.vis_start;
    if (rk >= n_few) return;
    const int want = p.s_few[static_cast<size_t>(b) * p.cap + rk];
    const int32_t* ids = p.layer_ids + (static_cast<size_t>(y) * p.B + b) * p.ids_max;
    int lo = 0, hi = n_held;                                 // first position with ids[pos] >= want
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (ids[mid] < want) lo = mid + 1; else hi = mid;
    }
    if (lo >= n_held || ids[lo] != want) {                   // the layer does not hold the token: row skipped
      if (threadIdx.x == 0) record_status(p.workspace, MUSTDROP_ERR_BAD_KEY_INDEX, b * 65536 + (rk & 65535));
      return;
    }
    src_row = p.vis_start + lo;
    dst_row = r;
  } else {
    const int t = r - p.vis_start - p.cap;                   // tail row t
    src_row = p.vis_start + n_held + t;
    dst_row = p.vis_start + n_few + t;
  }
  uint64_t once;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(once));
  const int64_t plane_in = static_cast<int64_t>(p.rows_in) * 16, plane_out = static_cast<int64_t>(p.rows_out) * 16;
  const int64_t base_in = (static_cast<int64_t>(y) * p.B + b) * p.H * plane_in + static_cast<int64_t>(src_row) * 16;
  const int64_t base_out = (static_cast<int64_t>(y) * p.B + b) * p.H * plane_out + static_cast<int64_t>(dst_row) * 16;
  const int n = p.H * 16 * 2;   // 16 vectors per head row, K then V
  for (int base = 0; base < n; base += kThreads * kUnroll) {
    uint4 v[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int x = base + u * kThreads + threadIdx.x;
      if (x < n) {
        const int which = x >= p.H * 16, xx = which ? x - p.H * 16 : x;
        const uint4* s = which ? p.src[1] : p.src[0];
        if (s != nullptr) v[u] = ld_once(s + base_in + (xx >> 4) * plane_in + (xx & 15), once);
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int x = base + u * kThreads + threadIdx.x;
      if (x < n) {
        const int which = x >= p.H * 16, xx = which ? x - p.H * 16 : x;
        uint4* d = which ? p.dst[1] : p.dst[0];
        if (d != nullptr) st_once(d + base_out + (xx >> 4) * plane_out + (xx & 15), v[u]);
      }
    }
  }
}

inline bool aligned16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; }

}  // namespace
}  // namespace mustdrop

extern "C" mustdrop_status_t mustdrop_cache_compact(const mustdrop_cache_config_t* c, const void* k_cache,
                                                    const void* v_cache, const int32_t* layer_ids,
                                                    const int32_t* layer_cnt, const int32_t* s_few,
                                                    const int32_t* s_few_cnt, void* k_out, void* v_out,
                                                    void* workspace, void* cuda_stream) {
  using namespace mustdrop;
  if (c == nullptr || layer_ids == nullptr || layer_cnt == nullptr || s_few == nullptr || s_few_cnt == nullptr)
    return MUSTDROP_ERR_INVALID_ARG;
  if (c->n_layers <= 0 || c->batch <= 0 || c->n_heads <= 0 || c->rows_in <= 0 || c->vis_start < 0 || c->n_tail < 0 ||
      c->ids_max <= 0 || c->cap <= 0 || c->cap > c->ids_max)
    return MUSTDROP_ERR_INVALID_ARG;
  if (c->head_dim != kHeadDim || c->batch > 65535 || c->n_layers > 65535) return MUSTDROP_ERR_UNSUPPORTED;
  if (static_cast<int64_t>(c->vis_start) + c->ids_max + c->n_tail > c->rows_in) return MUSTDROP_ERR_INVALID_ARG;
  if ((k_cache == nullptr) != (k_out == nullptr) || (v_cache == nullptr) != (v_out == nullptr))
    return MUSTDROP_ERR_INVALID_ARG;
  const void* ptrs[] = {k_cache, v_cache, layer_ids, layer_cnt, s_few, s_few_cnt, k_out, v_out, workspace};
  for (const void* q : ptrs)
    if (q != nullptr && !aligned16(q)) return MUSTDROP_ERR_INVALID_ARG;
  if (k_cache == nullptr && v_cache == nullptr) return MUSTDROP_OK;
  CacheParams p;
  p.src[0] = static_cast<const uint4*>(k_cache); p.src[1] = static_cast<const uint4*>(v_cache);
  p.dst[0] = static_cast<uint4*>(k_out); p.dst[1] = static_cast<uint4*>(v_out);
  p.layer_ids = layer_ids; p.layer_cnt = layer_cnt; p.s_few = s_few; p.s_few_cnt = s_few_cnt;
  p.workspace = workspace;
  p.B = c->batch; p.H = c->n_heads; p.rows_in = c->rows_in;
  p.rows_out = c->vis_start + c->cap + c->n_tail;
  p.vis_start = c->vis_start; p.n_tail = c->n_tail; p.ids_max = c->ids_max; p.cap = c->cap;
  dim3 grid(static_cast<unsigned>(p.rows_out), static_cast<unsigned>(c->batch), static_cast<unsigned>(c->n_layers));
  cudaError_t e = launch_pdl(cache_compact_kernel, grid, dim3(kThreads), 0, static_cast<cudaStream_t>(cuda_stream), p);
  if (e != cudaSuccess) {
    set_last_cuda_error(e);
    return MUSTDROP_ERR_CUDA;
  }
  return MUSTDROP_OK;
}
