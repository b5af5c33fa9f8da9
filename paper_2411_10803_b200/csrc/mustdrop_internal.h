// Internal declarations shared by the C-ABI layer and the kernel translation units.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "mustdrop.h"

namespace mustdrop {

constexpr int kHeadDim = 128;
constexpr int kMaxTxt = 128;
constexpr int kMaxVis = 4096;

// Workspace layout (bytes).  The first 256 bytes hold the device status word:
//   int32 code, int32 detail.  Everything after is kernel scratch.
constexpr size_t kWsStatusBytes = 256;

enum ScoreVariant : int32_t {
  kScoreTwoPassMma = 0,   // row statistics pass + accumulate pass, warp-level mma
  kScoreFusedCluster = 1, // one pass: tcgen05 MMA + TMA, key range split over a thread-block cluster
};

// Launch geometry of the fused score kernel.
struct FusedGeometry {
  int32_t halves;     // 2: two M=64 tiles per head (N <= 64); 1: one M=128 tile
  int32_t cluster;    // CTAs per request
  int32_t tk;         // keys per CTA
  int32_t cpl;        // tensor-memory columns per lane and head (= tk / halves)
  int32_t n_q, n_k;   // whole stages: n_q of them (n_k unused); split: rings of n_q query tiles and n_k key half-tiles
  int32_t split;      // 1: split rings
  int32_t n_buf;      // tensor-memory buffers
  int32_t n_slot;     // statistics slots: 2 x n_buf, or 2d (d = 2 or 1) with the exp warps held within d heads of the add warps
  int32_t ach;        // chunks of 16 columns per accumulating thread (kernel variant: 5 or 10)
  int32_t row0, n_rows;   // the text rows this geometry's launch covers
  int32_t gx;         // 1: grid plan - the request's CTAs are ordinary CTAs of the grid (cluster = their number) and
                      //    exchange their statistics through global memory
  int32_t resident;   // clusters the device can hold at once (0: not asked)
  float est_us;       // the planner's estimate of the score time
  size_t smem_bytes;  // dynamic shared memory
};

// Shared-memory plan of the selection / gather tail of the single-launch filter kernel.
struct FilterGeometry {
  size_t smem_bytes;   // dynamic shared memory of the launch (>= the score geometry's)
  int32_t slot_bytes;  // one kept row: hidden row + K pieces + V pieces of all heads
  int32_t n_slot;      // rows in flight per CTA
};

struct Resolved {
  int32_t B, H, D, hidden, L, vis_start, M, txt_start, N;
  int32_t causal, mode, criteria, budget, key_max, cap;
  int32_t per_head_max;   // Eq. 10 per head, then the head mean
  int32_t inputs_ready;   // the caller promises q_text / k were complete before the stream's previous kernel began
  int32_t wait_cycles;    // > 0: the fused kernel's role waits give up after this many cycles (debugging)
  int32_t rebuild;        // outputs hold [prefix ; kept vision ; text] instead of the kept vision rows only
  int32_t out_rows;       // rows per request (and head) of hidden_out / k_out / v_out
  int32_t gamma_default, alpha_default;   // thresholds follow each request's own sizes (ragged batches)
  float scale, scale_log2e, gamma, alpha;
  int64_t k_sb, k_sh, k_sl, v_sb, v_sh, v_sl, hid_sb, hid_sl;
};

// Optional per-call arguments of a layer in a chain of pruning layers (all device pointers, all nullable).
struct LayerArgs {
  const int32_t* vis_cnt = nullptr;     // [B] vision tokens each request actually holds (<= n_vis)
  const int32_t* orig_in = nullptr;     // [B, n_vis] original id of each current vision token (null: identity)
  int32_t* orig_out = nullptr;          // [B, cap] original ids of the kept tokens
  int32_t* key_idx_out = nullptr;       // [B, key_max] positions of the key tokens among the kept tokens
  int32_t* key_cnt_out = nullptr;       // [B]
};

// Number of vision tokens of request b: the plan's n_vis, or vis_cnt[b] clamped to [1, n_vis].
__host__ __device__ inline int32_t clamp_vis_cnt(int32_t v, int32_t M) { return v < 1 ? 1 : (v > M ? M : v); }

// Encoded tensor maps of recent calls (defined with the fused kernel's launch code).
struct MapCache;
MapCache* map_cache_create();
void map_cache_destroy(MapCache* c);

}  // namespace mustdrop

struct mustdrop_plan {
  uint32_t magic;
  mustdrop_config_t config;
  mustdrop::Resolved r;
  int32_t device;
  int32_t sm_count;
  int32_t score_variant;
  size_t ws_bytes;
  size_t ws_rowstats_off;   // float2 [B,H,N]: (row max in log2 units, 1 / row sum)
  size_t ws_gx_cnt_off;     // grid plans: uint32 counters [B H + 3 B], zero between calls
  size_t ws_gx_stats_off;   // grid plans: float2 [B,H,CTAs per request,rows,pairs]
  mustdrop::FusedGeometry fused;
  int32_t row_split;        // 1: the text rows are scored by two launches (fused: rows 0..63, fused_b: the rest)
  mustdrop::FusedGeometry fused_b;
  int32_t filter_single;    // 1: mustdrop_filter is one launch of the fused kernel with its tail
  mustdrop::FilterGeometry filter;
  mustdrop::MapCache* map_cache;   // guarded by its own lock; null: every call encodes its maps
};

namespace mustdrop {

constexpr uint32_t kPlanMagic = 0x4d445250u;  // "MDRP"

// Each launcher enqueues on `stream` and returns the launch error (cudaGetLastError).
cudaError_t launch_score_two_pass(const mustdrop_plan& p, const void* q_text, const void* k,
                                  float* g_out, float* i_out, void* rowstats, cudaStream_t stream,
                                  const int32_t* vis_cnt = nullptr);
bool plan_score_fused(const Resolved& r, int sm_count, int forced_cluster, FusedGeometry* out, int row0 = 0,
                      int n_rows = 0, int max_cluster = 0);
// Grid plan of the same kernel (all CTAs of the batch resident at once, statistics through global
// memory); false when the batch leaves fewer than two CTAs per request or the shape does not fit.
bool plan_score_grid(const Resolved& r, int sm_count, int forced_ctas, FusedGeometry* out);
size_t grid_plan_stats_bytes(const Resolved& r, const FusedGeometry& g);
cudaError_t launch_score_fused(const mustdrop_plan& p, const void* q_text, const void* k, float* g_out,
                               float* i_out, void* workspace, cudaStream_t stream, const int32_t* vis_cnt = nullptr);
bool plan_filter_single(const Resolved& r, const FusedGeometry& geo, FilterGeometry* out);
cudaError_t launch_filter_fused(const mustdrop_plan& p, const void* q_text, const void* k, const void* v,
                                const void* hidden, const int32_t* key_idx, const int32_t* key_cnt, float* g_out,
                                float* i_out, float* s_out, int32_t* kept_idx, int32_t* kept_cnt, void* hidden_out,
                                void* k_out, void* v_out, void* workspace, cudaStream_t stream,
                                const LayerArgs& la = LayerArgs());
cudaError_t launch_select(const mustdrop_plan& p, const float* g, const float* i, const int32_t* key_idx,
                          const int32_t* key_cnt, int32_t* kept_idx, int32_t* kept_cnt, float* s_out,
                          void* workspace, cudaStream_t stream, const LayerArgs& la = LayerArgs());
cudaError_t launch_compact(const mustdrop_plan& p, const int32_t* kept_idx, const int32_t* kept_cnt,
                           const void* hidden, const void* k, const void* v, void* hidden_out, void* k_out,
                           void* v_out, void* workspace, cudaStream_t stream, const int32_t* vis_cnt = nullptr);

// Launch attributes of a kernel, set ONCE per device and never changed afterwards (so that host
// threads with different plans cannot interleave a set with a launch): the largest dynamic shared
// memory the device grants next to the kernel's static part and, if asked, the opt-in to clusters
// of more than 8 CTAs.
cudaError_t ensure_kernel_attributes(const void* kernel, bool nonportable_cluster);

// Remember the cudaError_t of a failed runtime call for mustdrop_last_cuda_error (per thread).
void set_last_cuda_error(cudaError_t e);

// Programmatic dependent launch.  Every kernel of the library is launched with the
// programmatic-stream-serialization attribute: it may start while its predecessor in the stream
// is still running, does work that touches no global data, and then calls pdl_wait(), which
// returns once the predecessor grids have completed and their writes are visible.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename Kernel, typename... Args>
inline cudaError_t launch_pdl(Kernel kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// Optional pipeline tracing (compiled in only with -DMUSTDROP_TRACE): first CTA start and last
// CTA end of every kernel, per step, as global-timer values in the workspace (bytes 3072..4095:
// [counter][step % 20][kernel 0..2][start, end]).
#ifdef MUSTDROP_TRACE
__device__ __forceinline__ unsigned long long md_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void md_pipe_stamp(void* workspace, int kernel, bool is_end, bool new_step) {
  if (workspace == nullptr || threadIdx.x != 0) return;
  unsigned long long* base = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(workspace) + 3072);
  unsigned long long step = *reinterpret_cast<volatile unsigned long long*>(base);
  if (new_step && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) step = atomicAdd(base, 1ull) + 1ull;
  else if (new_step) return;   // only one CTA opens a step; the others stamp at their end
  unsigned long long* slot = base + 1 + ((step % 20ull) * 3ull + kernel) * 2ull;
  if (is_end) atomicMax(slot + 1, md_now());
  else atomicMin(slot, md_now());
}
#define MD_PIPE(ws, kernel, is_end, new_step) md_pipe_stamp((ws), (kernel), (is_end), (new_step))
#else
#define MD_PIPE(ws, kernel, is_end, new_step) ((void)0)
#endif

// Device-side helper: record the first device-detected condition (never traps).
__device__ __forceinline__ void record_status(void* workspace, int32_t code, int32_t detail) {
  if (workspace == nullptr) return;
  int32_t* w = reinterpret_cast<int32_t*>(workspace);
  if (atomicCAS(w, 0, code) == 0) w[1] = detail;
}

}  // namespace mustdrop
