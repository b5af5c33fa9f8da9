// Dual criteria, key set and selection: one CTA per request (Eq. 9, Eq. 10; Sec. 3.3 key set).
//
// The per-token score is computed in fp32 with one rounding per operation (no fused
// multiply-add, IEEE division), because it decides which indices are kept.  Budget mode is a
// radix select over the order-preserving integer image of the score, followed by an
// index-ordered emit, so kept indices come out ascending and equal scores resolve to the
// lower index.
//
// The work of a request is in select_body.cuh; this file is the stand-alone kernel around it.
#include "select_body.cuh"

namespace mustdrop {
namespace {

template <int OWN>
__global__ void __launch_bounds__(kSelThreads) select_kernel(SelectParams p) {
  __shared__ SelectShared s;
  const int tid = threadIdx.x;
  // Work that touches no global data, then let the next kernel start its prologue and wait for
  // the kernel that produced g / i.
  MD_PIPE(p.workspace, 1, false, false);
  select_clear(s, tid);
  pdl_launch_dependents();
  pdl_wait();
  select_request<OWN, SelectSyncCta>(p, s, blockIdx.x, tid, true, nullptr, nullptr);
  MD_PIPE(p.workspace, 1, true, false);
}

}  // namespace

cudaError_t launch_select(const mustdrop_plan& plan, const float* g, const float* i, const int32_t* key_idx,
                          const int32_t* key_cnt, int32_t* kept_idx, int32_t* kept_cnt, float* s_out,
                          void* workspace, cudaStream_t stream, const LayerArgs& la) {
  const Resolved& r = plan.r;
  SelectParams p;
  p.g = g; p.i = i; p.key_idx = key_idx; p.key_cnt = key_cnt; p.kept_idx = kept_idx; p.kept_cnt = kept_cnt;
  p.s_out = s_out; p.workspace = workspace;
  p.M = r.M; p.key_max = r.key_max; p.mode = r.mode; p.criteria = r.criteria; p.budget = r.budget; p.cap = r.cap;
  p.gamma = r.gamma; p.alpha = r.alpha;
  p.vis_cnt = la.vis_cnt; p.orig_in = la.orig_in; p.orig_out = la.orig_out;
  p.key_idx_out = la.key_idx_out; p.key_cnt_out = la.key_cnt_out;
  p.vis_start = r.vis_start; p.N = r.N; p.gamma_default = r.gamma_default; p.alpha_default = r.alpha_default;
  const int own = (r.M + kSelThreads - 1) / kSelThreads;
  static_assert(kMaxOwn == 16, "dispatch below covers up to 16 tokens per thread");
  if (own <= 1) return launch_pdl(select_kernel<1>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
  if (own <= 2) return launch_pdl(select_kernel<2>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
  if (own <= 4) return launch_pdl(select_kernel<4>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
  if (own <= 8) return launch_pdl(select_kernel<8>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
  return launch_pdl(select_kernel<16>, dim3(r.B), dim3(kSelThreads), 0, stream, p);
}

}  // namespace mustdrop
