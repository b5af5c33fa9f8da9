// C-ABI layer: configuration checks, plan object, argument checks, kernel dispatch.
// The operations themselves are defined by Sec. 3.4 (Eq. 8-10) of the paper; see mustdrop.h.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <set>
#include <utility>

#include "mustdrop_internal.h"

namespace {

thread_local int32_t g_last_cuda_error = 0;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline mustdrop_status_t cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int32_t>(e);
  return MUSTDROP_ERR_CUDA;
}

inline bool valid_plan(const mustdrop_plan_t* p) { return p != nullptr && p->magic == mustdrop::kPlanMagic; }

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

namespace mustdrop {
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = static_cast<int32_t>(e); }

cudaError_t ensure_kernel_attributes(const void* kernel, bool nonportable_cluster) {
  static std::mutex mu;
  static std::set<std::pair<const void*, int>> done;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  const auto key = std::make_pair(kernel, dev);
  if (done.count(key)) return cudaSuccess;
  cudaFuncAttributes fa;
  e = cudaFuncGetAttributes(&fa, kernel);
  if (e != cudaSuccess) return e;
  int optin = 0;
  e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           optin - static_cast<int>(fa.sharedSizeBytes));
  if (e != cudaSuccess) return e;
  if (nonportable_cluster) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  done.insert(key);
  return cudaSuccess;
}
}  // namespace mustdrop

extern "C" {

mustdrop_status_t mustdrop_filter_plan(const mustdrop_config_t* c, mustdrop_plan_t** plan_out,
                                       size_t* workspace_bytes) {
  using namespace mustdrop;
  if (c == nullptr || plan_out == nullptr || workspace_bytes == nullptr) return MUSTDROP_ERR_INVALID_ARG;
  *plan_out = nullptr;
  *workspace_bytes = 0;
  if (c->batch <= 0 || c->n_heads <= 0 || c->head_dim <= 0 || c->hidden <= 0 || c->seq_len <= 0 ||
      c->n_vis <= 0 || c->n_txt <= 0 || c->vis_start < 0 || c->txt_start < 0 || c->key_max < 0 ||
      (c->flags & ~(MUSTDROP_FLAG_REBUILD_SEQUENCE | MUSTDROP_FLAG_PER_HEAD_MAX | MUSTDROP_FLAG_INPUTS_READY)) != 0)
    return MUSTDROP_ERR_INVALID_ARG;
  if (c->debug_score_variant < MUSTDROP_DEBUG_VARIANT_AUTO || c->debug_score_variant > MUSTDROP_DEBUG_VARIANT_GRID ||
      c->debug_cluster < 0 || c->debug_cluster > (c->debug_score_variant == MUSTDROP_DEBUG_VARIANT_GRID ? 32 : 16) || (c->debug_filter_staged & ~1) != 0 || c->debug_wait_cycles < 0)
    return MUSTDROP_ERR_INVALID_ARG;
  // the vision span precedes the text span and both lie inside the sequence
  if (static_cast<int64_t>(c->vis_start) + c->n_vis > c->txt_start ||
      static_cast<int64_t>(c->txt_start) + c->n_txt > c->seq_len)
    return MUSTDROP_ERR_INVALID_ARG;
  if ((c->flags & MUSTDROP_FLAG_REBUILD_SEQUENCE) &&
      (c->txt_start != c->vis_start + c->n_vis || c->seq_len != c->txt_start + c->n_txt))
    return MUSTDROP_ERR_INVALID_ARG;
  if (c->causal != 0 && c->causal != 1) return MUSTDROP_ERR_INVALID_ARG;
  if (c->mode != MUSTDROP_MODE_BUDGET && c->mode != MUSTDROP_MODE_THRESHOLD) return MUSTDROP_ERR_INVALID_ARG;
  if (c->criteria < MUSTDROP_CRIT_DUAL || c->criteria > MUSTDROP_CRIT_INDIVIDUAL_ONLY)
    return MUSTDROP_ERR_INVALID_ARG;
  if (!(c->scale >= 0.0f) || !std::isfinite(c->scale)) return MUSTDROP_ERR_INVALID_ARG;
  if (!(c->gamma >= 0.0f) || !std::isfinite(c->gamma) || !(c->alpha >= 0.0f) || !std::isfinite(c->alpha))
    return MUSTDROP_ERR_INVALID_ARG;
  const int64_t strides[] = {c->k_stride_b, c->k_stride_h, c->k_stride_l, c->v_stride_b,
                             c->v_stride_h, c->v_stride_l, c->hid_stride_b, c->hid_stride_l};
  for (int64_t s : strides)
    if (s < 0) return MUSTDROP_ERR_INVALID_ARG;
  if (c->batch > 65535) return MUSTDROP_ERR_UNSUPPORTED;
  if (c->head_dim != kHeadDim || c->n_txt > kMaxTxt || c->n_vis > kMaxVis || (c->hidden % 8) != 0)
    return MUSTDROP_ERR_UNSUPPORTED;
  for (int64_t s : strides)
    if (s % 8 != 0) return MUSTDROP_ERR_UNSUPPORTED;
  if (c->mode == MUSTDROP_MODE_BUDGET) {
    if (c->budget <= 0 || c->budget > c->n_vis || c->budget < c->key_max) return MUSTDROP_ERR_BUDGET;
  }

  mustdrop_plan_t* p = new (std::nothrow) mustdrop_plan_t();
  if (p == nullptr) return MUSTDROP_ERR_INVALID_ARG;
  p->magic = kPlanMagic;
  p->config = *c;
  Resolved& r = p->r;
  r.B = c->batch; r.H = c->n_heads; r.D = c->head_dim; r.hidden = c->hidden; r.L = c->seq_len;
  r.vis_start = c->vis_start; r.M = c->n_vis; r.txt_start = c->txt_start; r.N = c->n_txt;
  r.causal = c->causal; r.mode = c->mode; r.criteria = c->criteria; r.budget = c->budget;
  r.key_max = c->key_max;
  r.cap = (c->mode == MUSTDROP_MODE_BUDGET) ? c->budget : c->n_vis;
  r.rebuild = (c->flags & MUSTDROP_FLAG_REBUILD_SEQUENCE) ? 1 : 0;
  r.per_head_max = (c->flags & MUSTDROP_FLAG_PER_HEAD_MAX) ? 1 : 0;
  r.inputs_ready = (c->flags & MUSTDROP_FLAG_INPUTS_READY) ? 1 : 0;
  r.wait_cycles = c->debug_wait_cycles;
  r.out_rows = r.rebuild ? c->vis_start + r.cap + c->n_txt : r.cap;
  r.gamma_default = c->gamma == 0.0f;
  r.alpha_default = c->alpha == 0.0f;
  r.scale = (c->scale == 0.0f) ? 1.0f / sqrtf(static_cast<float>(c->head_dim)) : c->scale;
  r.scale_log2e = r.scale * 1.4426950408889634f;
  r.gamma = (c->gamma == 0.0f) ? 1.0f / static_cast<float>(c->n_vis) : c->gamma;
  r.alpha = (c->alpha == 0.0f) ? 2.0f / static_cast<float>(c->seq_len) : c->alpha;
  r.k_sl = c->k_stride_l ? c->k_stride_l : c->head_dim;
  r.k_sh = c->k_stride_h ? c->k_stride_h : static_cast<int64_t>(c->seq_len) * r.k_sl;
  r.k_sb = c->k_stride_b ? c->k_stride_b : static_cast<int64_t>(c->n_heads) * r.k_sh;
  r.v_sl = c->v_stride_l ? c->v_stride_l : c->head_dim;
  r.v_sh = c->v_stride_h ? c->v_stride_h : static_cast<int64_t>(c->seq_len) * r.v_sl;
  r.v_sb = c->v_stride_b ? c->v_stride_b : static_cast<int64_t>(c->n_heads) * r.v_sh;
  r.hid_sl = c->hid_stride_l ? c->hid_stride_l : c->hidden;
  r.hid_sb = c->hid_stride_b ? c->hid_stride_b : static_cast<int64_t>(c->seq_len) * r.hid_sl;
  if (r.k_sl < c->head_dim || r.v_sl < c->head_dim || r.hid_sl < c->hidden) {
    delete p;
    return MUSTDROP_ERR_INVALID_ARG;
  }

  // The device is only consulted for the SM count; a box without a GPU still gets a plan.
  p->device = -1;
  p->sm_count = 148;
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) {
      p->device = dev;
      p->sm_count = sms;
    }
  }
  (void)cudaGetLastError();

  // Score kernel: the fused single-pass kernel where its geometry covers the shape, else the
  // two-pass kernel.  The configuration's debug_score_variant / debug_cluster override the choice.
  p->score_variant = kScoreTwoPassMma;
  {
    const bool want = c->debug_score_variant != MUSTDROP_DEBUG_VARIANT_AUTO;   // a variant is forced
    const int forced_cluster = c->debug_cluster;
    const bool allow_fused = c->debug_score_variant != MUSTDROP_DEBUG_VARIANT_TWO_PASS;
    const bool force_split = c->debug_score_variant == MUSTDROP_DEBUG_VARIANT_ROW_SPLIT;
    const bool force_grid = c->debug_score_variant == MUSTDROP_DEBUG_VARIANT_GRID;
    const double k_mb = 256.0e-6 * r.B * r.H * r.L;
    const double two_pass_us = k_mb * (0.6 + 0.7 * r.N / 128.0);   // the two-pass kernel's measured rate
    double chosen_us = two_pass_us;
    p->row_split = 0;
    if (allow_fused && !force_split && !force_grid && plan_score_fused(r, p->sm_count, forced_cluster, &p->fused)) {
      p->score_variant = kScoreFusedCluster;
      chosen_us = p->fused.est_us;
      // A fused plan that had to fall back to few statistics slots (sequences needing clusters of
      // more than 8 CTAs) can be slower than reading K twice: compare with the two-pass kernel
      // unless the variant is forced.
      const bool tight = p->fused.n_slot < 2 * p->fused.n_buf;
      if (tight && !want && forced_cluster == 0 && p->fused.est_us > two_pass_us) {
        p->score_variant = kScoreTwoPassMma;
        chosen_us = two_pass_us;
      }
    }
    // More than 64 text rows fill all 128 tensor-memory lanes with one key range, which halves the
    // keys a CTA can take.  Alternative: two launches over the same keys, text rows 0..63 and the
    // rest, each with the two-tile layout (twice the keys per CTA); the second adds its column
    // sums to / takes the maximum with the first's.  Taken when estimated faster than the above.
    // (Not with the per-head reading of Eq. 10: its maxima run over ALL text rows of a head before
    // the head mean, which two launches over disjoint rows cannot combine afterwards.)
    if (allow_fused && r.N > 64 && !r.per_head_max && !force_grid) {
      mustdrop::FusedGeometry ga, gb;
      // clusters small enough for both launches to be resident at once, if such a plan exists
      const int fit = p->sm_count / (2 * r.B);
      bool ok = fit >= 1 && plan_score_fused(r, p->sm_count, forced_cluster, &ga, 0, 64, fit) &&
                plan_score_fused(r, p->sm_count, forced_cluster, &gb, 64, r.N - 64, fit);
      if (!ok)
        ok = plan_score_fused(r, p->sm_count, forced_cluster, &ga, 0, 64) &&
             plan_score_fused(r, p->sm_count, forced_cluster, &gb, 64, r.N - 64);
      if (ok) {
        const bool together = r.B * (ga.cluster + gb.cluster) <= p->sm_count;   // both launches resident at once
        const double split_us = together ? 1.15 * (ga.est_us > gb.est_us ? ga.est_us : gb.est_us) : ga.est_us + gb.est_us;
        if (force_split || (!want && forced_cluster == 0 && split_us < chosen_us)) {
          p->score_variant = kScoreFusedCluster;
          p->row_split = 1;
          p->fused = ga;
          p->fused_b = gb;
        }
      }
    }
    // Small batches of long sequences: the same kernel without clusters - every CTA of the batch
    // resident at once, as many per request as the SMs allow, statistics through global memory.
    // Taken when estimated faster than what was chosen above.
    if (allow_fused && !force_split && (force_grid || (!want && forced_cluster == 0))) {
      mustdrop::FusedGeometry gg;
      if (plan_score_grid(r, p->sm_count, force_grid ? forced_cluster : 0, &gg) &&
          (force_grid || gg.est_us < (p->row_split ? 1e30 : chosen_us) * 0.9 ||
           (p->row_split && gg.est_us < 1.15 * (p->fused.est_us > p->fused_b.est_us ? p->fused.est_us : p->fused_b.est_us)))) {
        p->score_variant = kScoreFusedCluster;
        p->row_split = 0;
        p->fused = gg;
      }
    }
    // mustdrop_filter: one launch where the fused kernel covers the shape and a kept row fits its
    // shared-memory ring; debug_filter_staged forces the separate launches.
    p->filter_single = 0;
    if (p->score_variant == kScoreFusedCluster && !c->debug_filter_staged &&
        plan_filter_single(r, p->row_split ? p->fused_b : p->fused, &p->filter))
      p->filter_single = 1;
  }
  size_t off = kWsStatusBytes;
  p->ws_rowstats_off = off;
  off += round_up(sizeof(float) * 2 * static_cast<size_t>(r.B) * r.H * r.N, 256);
#ifdef MUSTDROP_TRACE
  // trace builds stamp into the workspace from byte 4096 on (up to 32 CTAs per request): keep the
  // regions the kernels really use clear of that
  if (off < 4096 + static_cast<size_t>(r.B) * 32 * r.H * 16 * 8) off = round_up(4096 + static_cast<size_t>(r.B) * 32 * r.H * 16 * 8, 256);
#endif
  p->ws_gx_cnt_off = p->ws_gx_stats_off = off;
  if (p->score_variant == kScoreFusedCluster && p->fused.gx) {
    p->ws_gx_cnt_off = off;
    off += round_up(sizeof(uint32_t) * (static_cast<size_t>(r.B) * r.H + 3 * static_cast<size_t>(r.B)), 256);
    p->ws_gx_stats_off = off;
    off += round_up(grid_plan_stats_bytes(r, p->fused), 256);
  }
  p->ws_bytes = off;
  p->map_cache = map_cache_create();
  *workspace_bytes = p->ws_bytes;
  *plan_out = p;
  return MUSTDROP_OK;
}

mustdrop_status_t mustdrop_plan_destroy(mustdrop_plan_t* plan) {
  if (plan == nullptr) return MUSTDROP_OK;
  if (!valid_plan(plan)) return MUSTDROP_ERR_INVALID_ARG;
  plan->magic = 0;
  mustdrop::map_cache_destroy(plan->map_cache);
  delete plan;
  return MUSTDROP_OK;
}

mustdrop_status_t mustdrop_score(const mustdrop_plan_t* plan, const void* q_text, const void* k, float* g_out,
                                 float* i_out, void* workspace, void* cuda_stream) {
  if (!valid_plan(plan) || q_text == nullptr || k == nullptr || g_out == nullptr || i_out == nullptr)
    return MUSTDROP_ERR_INVALID_ARG;
  if (workspace == nullptr) return MUSTDROP_ERR_WORKSPACE;
  if (!aligned16(q_text) || !aligned16(k) || !aligned16(g_out) || !aligned16(i_out) || !aligned16(workspace))
    return MUSTDROP_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  if (plan->score_variant == mustdrop::kScoreFusedCluster) {
    e = mustdrop::launch_score_fused(*plan, q_text, k, g_out, i_out, workspace, stream);
  } else {
    void* rowstats = static_cast<unsigned char*>(workspace) + plan->ws_rowstats_off;
    e = mustdrop::launch_score_two_pass(*plan, q_text, k, g_out, i_out, rowstats, stream);
  }
  return e == cudaSuccess ? MUSTDROP_OK : cuda_fail(e);
}

mustdrop_status_t mustdrop_select(const mustdrop_plan_t* plan, const float* g, const float* i,
                                  const int32_t* key_idx, const int32_t* key_cnt, int32_t* kept_idx,
                                  int32_t* kept_cnt, float* s_out, void* workspace, void* cuda_stream) {
  if (!valid_plan(plan) || g == nullptr || i == nullptr || kept_idx == nullptr || kept_cnt == nullptr)
    return MUSTDROP_ERR_INVALID_ARG;
  if (plan->r.key_max > 0 && (key_idx == nullptr || key_cnt == nullptr)) return MUSTDROP_ERR_INVALID_ARG;
  if (workspace == nullptr) return MUSTDROP_ERR_WORKSPACE;
  if (!aligned16(g) || !aligned16(i) || !aligned16(kept_idx) || !aligned16(kept_cnt) || !aligned16(workspace) ||
      (key_idx && !aligned16(key_idx)) || (key_cnt && !aligned16(key_cnt)) || (s_out && !aligned16(s_out)))
    return MUSTDROP_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e =
      mustdrop::launch_select(*plan, g, i, key_idx, key_cnt, kept_idx, kept_cnt, s_out, workspace, stream);
  return e == cudaSuccess ? MUSTDROP_OK : cuda_fail(e);
}

mustdrop_status_t mustdrop_compact(const mustdrop_plan_t* plan, const int32_t* kept_idx, const int32_t* kept_cnt,
                                   const void* hidden, const void* k, const void* v, void* hidden_out,
                                   void* k_out, void* v_out, void* workspace, void* cuda_stream) {
  if (!valid_plan(plan) || kept_idx == nullptr || kept_cnt == nullptr) return MUSTDROP_ERR_INVALID_ARG;
  if ((hidden == nullptr) != (hidden_out == nullptr) || (k == nullptr) != (k_out == nullptr) ||
      (v == nullptr) != (v_out == nullptr))
    return MUSTDROP_ERR_INVALID_ARG;
  const void* ptrs[] = {kept_idx, kept_cnt, hidden, k, v, hidden_out, k_out, v_out, workspace};
  for (const void* q : ptrs)
    if (q != nullptr && !aligned16(q)) return MUSTDROP_ERR_INVALID_ARG;
  if (hidden == nullptr && k == nullptr && v == nullptr) return MUSTDROP_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = mustdrop::launch_compact(*plan, kept_idx, kept_cnt, hidden, k, v, hidden_out, k_out, v_out,
                                           workspace, stream);
  return e == cudaSuccess ? MUSTDROP_OK : cuda_fail(e);
}

mustdrop_status_t mustdrop_filter(const mustdrop_plan_t* plan, const void* q_text, const void* k, const void* v,
                                  const void* hidden, const int32_t* key_idx, const int32_t* key_cnt, float* g_out,
                                  float* i_out, float* s_out, int32_t* kept_idx, int32_t* kept_cnt,
                                  void* hidden_out, void* k_out, void* v_out, void* workspace, void* cuda_stream) {
  if (!valid_plan(plan) || q_text == nullptr || k == nullptr || g_out == nullptr || i_out == nullptr ||
      kept_idx == nullptr || kept_cnt == nullptr)
    return MUSTDROP_ERR_INVALID_ARG;
  if (plan->r.key_max > 0 && (key_idx == nullptr || key_cnt == nullptr)) return MUSTDROP_ERR_INVALID_ARG;
  if ((hidden == nullptr) != (hidden_out == nullptr) || (v == nullptr) != (v_out == nullptr))
    return MUSTDROP_ERR_INVALID_ARG;
  if (workspace == nullptr) return MUSTDROP_ERR_WORKSPACE;
  const void* ptrs[] = {q_text, k, v, hidden, key_idx, key_cnt, g_out, i_out, s_out, kept_idx, kept_cnt,
                        hidden_out, k_out, v_out, workspace};
  for (const void* q : ptrs)
    if (q != nullptr && !aligned16(q)) return MUSTDROP_ERR_INVALID_ARG;
  if (plan->filter_single) {
    cudaError_t e = mustdrop::launch_filter_fused(*plan, q_text, k, v, hidden, key_idx, key_cnt, g_out, i_out, s_out,
                                                  kept_idx, kept_cnt, hidden_out, k_out, v_out, workspace,
                                                  static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? MUSTDROP_OK : cuda_fail(e);
  }
  mustdrop_status_t st = mustdrop_score(plan, q_text, k, g_out, i_out, workspace, cuda_stream);
  if (st != MUSTDROP_OK) return st;
  st = mustdrop_select(plan, g_out, i_out, key_idx, key_cnt, kept_idx, kept_cnt, s_out, workspace, cuda_stream);
  if (st != MUSTDROP_OK) return st;
  return mustdrop_compact(plan, kept_idx, kept_cnt, hidden, k_out != nullptr ? k : nullptr, v, hidden_out, k_out,
                          v_out, workspace, cuda_stream);
}

mustdrop_status_t mustdrop_filter_layer(const mustdrop_plan_t* plan, const mustdrop_layer_io_t* io, void* workspace,
                                        void* cuda_stream) {
  if (!valid_plan(plan) || io == nullptr) return MUSTDROP_ERR_INVALID_ARG;
  if (io->q_text == nullptr || io->k == nullptr || io->g_out == nullptr || io->i_out == nullptr ||
      io->kept_idx == nullptr || io->kept_cnt == nullptr)
    return MUSTDROP_ERR_INVALID_ARG;
  const mustdrop::Resolved& r = plan->r;
  if (r.key_max > 0 && (io->key_idx == nullptr || io->key_cnt == nullptr)) return MUSTDROP_ERR_INVALID_ARG;
  if ((io->hidden == nullptr) != (io->hidden_out == nullptr) || (io->v == nullptr) != (io->v_out == nullptr))
    return MUSTDROP_ERR_INVALID_ARG;
  if ((io->key_idx_out == nullptr) != (io->key_cnt_out == nullptr)) return MUSTDROP_ERR_INVALID_ARG;
  // a ragged batch packs each request's text directly behind its own vision tokens
  if (io->vis_cnt != nullptr && (r.txt_start != r.vis_start + r.M || r.L != r.txt_start + r.N))
    return MUSTDROP_ERR_INVALID_ARG;
  if (workspace == nullptr) return MUSTDROP_ERR_WORKSPACE;
  const void* ptrs[] = {io->q_text, io->k, io->v, io->hidden, io->key_idx, io->key_cnt, io->vis_cnt, io->orig_idx,
                        io->g_out, io->i_out, io->s_out, io->kept_idx, io->kept_cnt, io->orig_out, io->key_idx_out,
                        io->key_cnt_out, io->hidden_out, io->k_out, io->v_out, workspace};
  for (const void* q : ptrs)
    if (q != nullptr && !aligned16(q)) return MUSTDROP_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  mustdrop::LayerArgs la;
  la.vis_cnt = io->vis_cnt; la.orig_in = io->orig_idx; la.orig_out = io->orig_out;
  la.key_idx_out = io->key_idx_out; la.key_cnt_out = io->key_cnt_out;
  cudaError_t e;
  if (plan->filter_single) {
    e = mustdrop::launch_filter_fused(*plan, io->q_text, io->k, io->v, io->hidden, io->key_idx, io->key_cnt, io->g_out,
                                      io->i_out, io->s_out, io->kept_idx, io->kept_cnt, io->hidden_out, io->k_out,
                                      io->v_out, workspace, stream, la);
    return e == cudaSuccess ? MUSTDROP_OK : cuda_fail(e);
  }
  if (plan->score_variant == mustdrop::kScoreFusedCluster) {
    e = mustdrop::launch_score_fused(*plan, io->q_text, io->k, io->g_out, io->i_out, workspace, stream, la.vis_cnt);
  } else {
    void* rowstats = static_cast<unsigned char*>(workspace) + plan->ws_rowstats_off;
    e = mustdrop::launch_score_two_pass(*plan, io->q_text, io->k, io->g_out, io->i_out, rowstats, stream, la.vis_cnt);
  }
  if (e != cudaSuccess) return cuda_fail(e);
  e = mustdrop::launch_select(*plan, io->g_out, io->i_out, io->key_idx, io->key_cnt, io->kept_idx, io->kept_cnt,
                              io->s_out, workspace, stream, la);
  if (e != cudaSuccess) return cuda_fail(e);
  if (io->hidden_out == nullptr && io->k_out == nullptr && io->v_out == nullptr) return MUSTDROP_OK;
  e = mustdrop::launch_compact(*plan, io->kept_idx, io->kept_cnt, io->hidden, io->k_out != nullptr ? io->k : nullptr,
                               io->v, io->hidden_out, io->k_out, io->v_out, workspace, stream, la.vis_cnt);
  return e == cudaSuccess ? MUSTDROP_OK : cuda_fail(e);
}

int32_t mustdrop_plan_filter_launches(const mustdrop_plan_t* plan) {
  if (!valid_plan(plan)) return -1;
  if (plan->filter_single) return plan->row_split ? 2 : 1;
  return plan->score_variant == mustdrop::kScoreTwoPassMma ? 4 : (plan->row_split ? 4 : 3);
}

mustdrop_status_t mustdrop_device_status(const mustdrop_plan_t* plan, const void* workspace, void* cuda_stream,
                                         int32_t* code_out, int32_t* detail_out) {
  if (!valid_plan(plan) || code_out == nullptr) return MUSTDROP_ERR_INVALID_ARG;
  if (workspace == nullptr) return MUSTDROP_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int32_t host[2] = {0, 0};
  cudaError_t e = cudaMemcpyAsync(host, workspace, sizeof(host), cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail(e);
  *code_out = host[0];
  if (detail_out != nullptr) *detail_out = host[1];
  return MUSTDROP_OK;
}

const char* mustdrop_status_string(mustdrop_status_t s) {
  switch (s) {
    case MUSTDROP_OK: return "ok";
    case MUSTDROP_ERR_INVALID_ARG: return "invalid argument";
    case MUSTDROP_ERR_UNSUPPORTED: return "unsupported configuration";
    case MUSTDROP_ERR_BUDGET: return "budget smaller than the key set capacity or larger than n_vis";
    case MUSTDROP_ERR_WORKSPACE: return "workspace missing";
    case MUSTDROP_ERR_CUDA: return "CUDA runtime error";
    case MUSTDROP_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case MUSTDROP_ERR_BAD_KEY_INDEX: return "index outside [0, n_vis) ignored";
    case MUSTDROP_ERR_SCRATCH_LIMIT:
      return "batch * n_heads * n_txt exceeds the built-in scratch of mustdrop_score_static (524288 rows)";
  }
  return "unknown status";
}

int32_t mustdrop_last_cuda_error(void) { return g_last_cuda_error; }

const char* mustdrop_plan_score_variant(const mustdrop_plan_t* plan) {
  if (!valid_plan(plan)) return "invalid plan";
  switch (plan->score_variant) {
    case mustdrop::kScoreTwoPassMma: return "two_pass_mma";
    case mustdrop::kScoreFusedCluster: return "fused_cluster_tcgen05";
  }
  return "unknown";
}

int32_t mustdrop_plan_describe(const mustdrop_plan_t* plan, char* buf, size_t n) {
  if (!valid_plan(plan)) return -1;
  char text[256];
  int len;
  if (plan->score_variant == mustdrop::kScoreFusedCluster) {
    const mustdrop::FusedGeometry& g = plan->row_split ? plan->fused_b : plan->fused;
    if (g.gx)
      len = std::snprintf(text, sizeof(text),
                          "fused tcgen05 score: grid plan (statistics through global memory), %d CTAs per request, "
                          "%d keys per CTA, stages %d, %d tensor-memory buffers, %d statistics slots; filter = %d launch(es)",
                          g.cluster, g.tk, g.n_q, g.n_buf, g.n_slot, mustdrop_plan_filter_launches(plan));
    else
      len = std::snprintf(text, sizeof(text),
                          "fused tcgen05 score%s: cluster %d, %d keys per CTA, %s %d/%d, %d tensor-memory buffers, "
                          "%d statistics slots, %d clusters resident; filter = %d launch(es)",
                          plan->row_split ? " (text rows in two launches; second launch)" : "", g.cluster, g.tk,
                          g.split ? "query/key-half rings" : "stages", g.n_q, g.split ? g.n_k : 0, g.n_buf, g.n_slot,
                          g.resident, mustdrop_plan_filter_launches(plan));
  } else {
    len = std::snprintf(text, sizeof(text), "two-pass mma.sync score; filter = %d launch(es)",
                        mustdrop_plan_filter_launches(plan));
  }
  if (buf != nullptr && n > 0) std::snprintf(buf, n, "%s", text);
  return len;
}

}  // extern "C"
