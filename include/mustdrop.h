/*
 * mustdrop.h - C ABI of the B200 (sm_100a) vision-token filter.
 *
 * The library implements the prefill-stage, text-guided dual-attention filtering of vision
 * tokens of MustDrop (arXiv 2411.10803, Sec. 3.4 "Dual-Attention Filtering Guided by
 * Language") as a batched operation at one pruning layer:
 *
 *     mustdrop_score    text-query x key attention -> per-vision-token importance (Eq. 1, 8, 10)
 *     mustdrop_select   dual criteria + key set -> retained indices             (Eq. 9, 10, Sec. 3.3)
 *     mustdrop_compact  gather the retained hidden states and per-head K/V     (Table 3: tokens in the KV cache)
 *
 * Conventions shared by all calls
 *   - Pointers marked (host) are plain host memory.  Every other data pointer is DEVICE
 *     memory, 16-byte aligned, allocated and freed by the caller.  The library allocates only
 *     the host-side plan; it never allocates device memory and never synchronises, except
 *     mustdrop_device_status.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls enqueue work and return; issuing score, select, compact in that order on one
 *     stream is the whole protocol.  Every kernel waits for the work that precedes it in the
 *     stream before it reads an input or writes an output (only its set-up overlaps the end of
 *     its predecessor), so inputs may come from the kernel enqueued just before the call.
 *   - Host-detectable problems return a non-OK status and launch nothing.  Conditions only
 *     the device can see (a key index outside [0, n_vis)) are recorded in a status word in
 *     the workspace and never trap.
 *   - Sequence layout (Sec. 3.1, "Prefilling"): the n_vis vision tokens occupy positions
 *     [vis_start, vis_start+n_vis), the n_txt text tokens [txt_start, txt_start+n_txt),
 *     vis_start+n_vis <= txt_start, txt_start+n_txt <= seq_len.
 *   - A plan's configuration is immutable.  Calls from several host threads are safe when they
 *     use distinct workspaces (launch attributes of the kernels are set once per device, and the
 *     plan's cache of encoded tensor maps is guarded by a lock).
 *   - A request whose result is invalid because a bounded wait inside the one-launch filter
 *     kernel ran out gets kept_cnt[b] = -1 (and MUSTDROP_ERR_TIMEOUT in the device status word);
 *     its other outputs are unspecified.
 */
#ifndef MUSTDROP_H_
#define MUSTDROP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mustdrop_plan mustdrop_plan_t; /* opaque, host memory, owned by the library */

typedef enum {
  MUSTDROP_OK = 0,
  MUSTDROP_ERR_INVALID_ARG = 1,   /* null or misaligned pointer, non-positive size, bad span, bad threshold */
  MUSTDROP_ERR_UNSUPPORTED = 2,   /* head_dim != 128, n_txt > 128, n_vis > 4096, odd strides */
  MUSTDROP_ERR_BUDGET = 3,        /* budget < key_max or budget > n_vis (BUDGET mode) */
  MUSTDROP_ERR_WORKSPACE = 4,     /* null workspace */
  MUSTDROP_ERR_CUDA = 5,          /* a CUDA runtime call failed; see mustdrop_last_cuda_error */
  MUSTDROP_ERR_TIMEOUT = 6,       /* device status only: a bounded wait inside a kernel ran out */
  MUSTDROP_ERR_BAD_KEY_INDEX = 7, /* device status only: an index outside [0, n_vis) was ignored */
  MUSTDROP_ERR_SCRATCH_LIMIT = 8  /* mustdrop_score_static: batch * n_heads * n_txt exceeds the built-in scratch */
} mustdrop_status_t;

typedef enum { MUSTDROP_MODE_BUDGET = 0, MUSTDROP_MODE_THRESHOLD = 1 } mustdrop_mode_t;

/* Which criteria decide (Table 4, rows b, c, d). */
typedef enum {
  MUSTDROP_CRIT_DUAL = 0,
  MUSTDROP_CRIT_GLOBAL_ONLY = 1,
  MUSTDROP_CRIT_INDIVIDUAL_ONLY = 2
} mustdrop_criteria_t;

/*
 * MUSTDROP_FLAG_REBUILD_SEQUENCE: the compacted outputs hold the request's whole next sequence
 * instead of the kept vision rows only: the vis_start prefix rows, the kept vision rows, then
 * the n_txt text rows, packed without a gap - the input layout of the next pruning layer
 * (the paper's overview has the filter applied gradually at several layers, each on what the
 * layer before it kept).
 * Outputs then have vis_start + cap + n_txt rows per request (and head); rows behind a
 * request's own end are left untouched.  Requires txt_start == vis_start + n_vis and
 * seq_len == txt_start + n_txt.
 */
#define MUSTDROP_FLAG_REBUILD_SEQUENCE 1

/*
 * MUSTDROP_FLAG_PER_HEAD_MAX: the other reading of Eq. 10 over attention heads, which the paper
 * leaves open: i_out[b][j] = mean over heads of ( max over text tokens of p^h[i][vis_start + j] )
 * instead of the maximum of the head-mean attention.  g_out (Eq. 8) is the same under both.
 * (On the fused kernel each head's maximum is rounded to 11 significant bits before the mean over
 * heads is taken in fp32: at most 5e-4 relative, inside the 2e-3 the scores are held to.)
 */
#define MUSTDROP_FLAG_PER_HEAD_MAX 2

/*
 * MUSTDROP_FLAG_INPUTS_READY: a promise by the caller that q_text and k were completely written,
 * and visible to the device, before the kernel that PRECEDES this call in the stream started
 * (e.g. they were produced several kernels earlier, or uploaded and synchronised).  The score
 * part then starts streaming keys without waiting for that predecessor to finish, so the
 * beginning of one call overlaps the end of the call before it.  Without the flag (the default)
 * nothing is read before all earlier work in the stream has completed.  Outputs are always
 * written after that wait.  Ignored when vis_cnt is given to mustdrop_filter_layer.
 */
#define MUSTDROP_FLAG_INPUTS_READY 4

typedef struct {
  int32_t batch;      /* B, independent requests */
  int32_t n_heads;    /* H */
  int32_t head_dim;   /* D, must be 128 */
  int32_t hidden;     /* elements per hidden-state row (any positive multiple of 8) */
  int32_t seq_len;    /* L */
  int32_t vis_start;  /* first vision position */
  int32_t n_vis;      /* M, 1..4096 */
  int32_t txt_start;  /* first text position */
  int32_t n_txt;      /* N, 1..128 */
  int32_t causal;     /* 1: text query i attends keys 0..txt_start+i (the model's prefill mask); 0: all L keys */
  float   scale;      /* logit scale; 0 => 1/sqrt(head_dim) (Eq. 1) */
  int32_t mode;       /* mustdrop_mode_t */
  int32_t criteria;   /* mustdrop_criteria_t */
  int32_t budget;     /* Kp: tokens kept per request in BUDGET mode, key set included */
  float   gamma;      /* Eq. 9 threshold; 0 => 1/n_vis */
  float   alpha;      /* Eq. 10 threshold; 0 => 2/seq_len */
  int32_t key_max;    /* capacity of key_idx per request; 0 = no key set */
  int32_t flags;      /* bit set of MUSTDROP_FLAG_*; other bits must be 0 */
  /* Strides in ELEMENTS (bf16); 0 => contiguous.  Head rows themselves are contiguous
   * (head_dim elements).  Every stride must be a multiple of 8 (16 bytes). */
  int64_t k_stride_b, k_stride_h, k_stride_l;       /* K      [B,H,L,D] */
  int64_t v_stride_b, v_stride_h, v_stride_l;       /* V      [B,H,L,D] */
  int64_t hid_stride_b, hid_stride_l;               /* hidden [B,L,hidden] */
  /* Debugging overrides of the planner, for tests and sweeps.  All 0 in normal use. */
  int32_t debug_score_variant;  /* mustdrop_debug_variant_t: force a score kernel */
  int32_t debug_cluster;        /* 1..16: force the fused kernel's cluster size */
  int32_t debug_filter_staged;  /* 1: mustdrop_filter enqueues the separate kernels even where one launch would do */
  int32_t debug_wait_cycles;    /* > 0: waits between the warp roles of the fused kernel give up after this many
                                   SM clock cycles instead of ~0.1 s (used to exercise the time-out path) */
} mustdrop_config_t;

typedef enum {
  MUSTDROP_DEBUG_VARIANT_AUTO = 0,
  MUSTDROP_DEBUG_VARIANT_TWO_PASS = 1,   /* the general-shape two-pass kernel */
  MUSTDROP_DEBUG_VARIANT_FUSED = 2,      /* the one-pass tcgen05 kernel, whatever the cost model says */
  MUSTDROP_DEBUG_VARIANT_ROW_SPLIT = 3,  /* the one-pass kernel with the text rows scored by two launches */
  MUSTDROP_DEBUG_VARIANT_GRID = 4        /* the one-pass kernel without clusters: statistics exchanged through global
                                            memory (debug_cluster then gives the CTAs per request, up to 32) */
} mustdrop_debug_variant_t;

/*
 * Validate a configuration and build a plan (host only; nothing is launched).
 * config, plan_out and workspace_bytes are (host).  `*workspace_bytes` receives the size of
 * the device workspace the other calls need (>= 256, a multiple of 256).  The workspace must
 * be zeroed once before first use (its first bytes are the device status word, and some plans
 * keep counters in it); after that the calls keep it consistent - except after a device status
 * of MUSTDROP_ERR_TIMEOUT, when it has to be zeroed again before it is reused.  The plan records the CUDA device current at this call.
 */
mustdrop_status_t mustdrop_filter_plan(const mustdrop_config_t *config, mustdrop_plan_t **plan_out,
                                       size_t *workspace_bytes);

mustdrop_status_t mustdrop_plan_destroy(mustdrop_plan_t *plan);

/*
 * Importance of every vision token (Sec. 3.4).
 *   z^h[i][l] = scale * <q_text[b][h][i], k[b][h][l]>                      (Eq. 1)
 *   p^h[i][.] = softmax over the keys visible to text query i (all vision keys, and the text
 *               keys up to and including its own when causal)             (Eq. 1, "attention map")
 *   a[i][j]   = mean over heads of p^h[i][vis_start + j]
 *   g_out[b][j] = sum_i a[i][j]                                            (Eq. 8)
 *   i_out[b][j] = max_i a[i][j]                                            (Eq. 10)
 * q_text bf16 [B,H,N,D] contiguous; k bf16 [B,H,L,D] (plan strides); g_out, i_out fp32 [B,M].
 * fp32 accumulation from bf16 inputs.
 */
mustdrop_status_t mustdrop_score(const mustdrop_plan_t *plan, const void *q_text, const void *k,
                                 float *g_out, float *i_out, void *workspace, void *cuda_stream);

/*
 * mustdrop_score for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above.  It always runs the two-pass
 * kernel, so its results equal mustdrop_score's up to the rounding order of fp32 sums.)
 *
 * Who needs it: code running where cudaMalloc is not an option - inside an engine whose pool
 * allocator owns the whole device heap, in a plug-in that must leave the host application's
 * allocator alone, or after a process has fixed its memory budget.  Such a caller has no
 * workspace to pass, so this call keeps its scratch (the per-row softmax statistics) in a
 * fixed 4 MiB array inside the library image; every GPU that loads the library holds that
 * array until the process exits.  The call itself allocates nothing and frees nothing.
 *
 * Limit: batch * n_heads * n_txt <= mustdrop_score_static_max_rows() (524288); a larger plan
 * is refused with MUSTDROP_ERR_SCRATCH_LIMIT and nothing is launched.
 * Sharing: all calls on a device use the same array.  Nothing in it has to start at zero
 * (each call overwrites every entry it later reads), but two calls that overlap on the GPU
 * (different streams, or different host threads without ordering) race on it and must be
 * serialised by the caller.  Calls on one stream are safe.
 * First call: the first call on each device looks up the array's device address (the device
 * must be current); make that first call outside any stream capture.
 * Arguments and results are those of mustdrop_score, without the workspace.
 */
mustdrop_status_t mustdrop_score_static(const mustdrop_plan_t *plan, const void *q_text, const void *k,
                                        float *g_out, float *i_out, void *cuda_stream);

/* Largest batch * n_heads * n_txt that mustdrop_score_static accepts. */
size_t mustdrop_score_static_max_rows(void);

/*
 * Dual criteria, key set and selection (Eq. 9, Eq. 10; the key set O of Sec. 3.3 is always kept).
 *   T = sum_j g[j];  gt = gamma * T;  D = { j : g[j] <= gt }               (Eq. 9)
 *   THRESHOLD mode: token j is dropped iff j in D and i[j] < alpha and j not in O.
 *   BUDGET mode: s[j] = max(g[j]/gt, i[j]/alpha) (fp32, one rounding per operation); O is kept,
 *   then the tokens with the largest s, lower index first among equals, until exactly
 *   `budget` tokens are kept.  GLOBAL_ONLY / INDIVIDUAL_ONLY use one of the two terms.
 * g, i fp32 [B,M]; key_idx int32 [B,key_max] vision-relative (entries outside [0,M) and repeats
 * are ignored, the former also recorded as MUSTDROP_ERR_BAD_KEY_INDEX), key_cnt int32 [B];
 * both may be NULL when key_max == 0.
 * kept_idx int32 [B,cap], cap = budget (BUDGET) or n_vis (THRESHOLD): strictly ascending,
 * vision-relative; entries at and beyond kept_cnt[b] are left untouched.  kept_cnt int32 [B].
 * s_out: NULL or fp32 [B,M], receives s.
 */
mustdrop_status_t mustdrop_select(const mustdrop_plan_t *plan, const float *g, const float *i,
                                  const int32_t *key_idx, const int32_t *key_cnt,
                                  int32_t *kept_idx, int32_t *kept_cnt, float *s_out,
                                  void *workspace, void *cuda_stream);

/*
 * Gather-compaction of the retained tokens (pruned tokens leave the sequence and the KV
 * cache; Table 3).  For r < kept_cnt[b]:
 *   hidden_out[b][r][:]  = hidden[b][vis_start + kept_idx[b][r]][:]
 *   k_out[b][h][r][:]    = k[b][h][vis_start + kept_idx[b][r]][:]          (v likewise)
 * hidden bf16 [B,L,hidden], k, v bf16 [B,H,L,D] (plan strides); outputs contiguous
 * hidden_out [B,cap,hidden], k_out, v_out [B,H,cap,D].  Rows r >= kept_cnt[b] are left
 * untouched.  Any of the three (source, destination) pairs may be NULL together to skip it.
 * An index outside [0, n_vis) is skipped and, when workspace is not NULL, recorded in its
 * device status word.  A kept_cnt[b] above cap is clamped to cap; a negative one (a request
 * marked invalid) copies nothing for that request; both are recorded the same way.
 */
mustdrop_status_t mustdrop_compact(const mustdrop_plan_t *plan, const int32_t *kept_idx,
                                   const int32_t *kept_cnt, const void *hidden, const void *k,
                                   const void *v, void *hidden_out, void *k_out, void *v_out,
                                   void *workspace, void *cuda_stream);

/*
 * The whole filtering step of one pruning layer in one call (Sec. 3.4: Eq. 8-10 on the text-to-
 * vision attention, the key set of Sec. 3.3 kept, pruned tokens removed from the sequence and
 * the KV cache): mustdrop_score, then mustdrop_select on its outputs, then mustdrop_compact with
 * the selected indices.  Results are those of the three calls made in that order on one stream;
 * g_out, i_out, (s_out), kept_idx and kept_cnt are all written.
 *
 * Where the plan's score kernel is the fused one and a kept row (hidden row + K + V pieces of all
 * heads) fits its shared-memory ring, this is ONE kernel launch: the thread-block cluster that
 * scored a request also selects its tokens and gathers them, so a request's copy starts while
 * other requests are still being scored.  Otherwise it enqueues the separate kernels.
 * mustdrop_plan_filter_launches tells which (1, or the number of separate launches).
 *
 * Arguments as in the three calls (all device pointers, 16-byte aligned): q_text, k required;
 * (hidden, hidden_out) and (v, v_out) may each be NULL together; k_out may be NULL to leave K
 * uncopied; s_out may be NULL; key_idx / key_cnt may be NULL when key_max == 0.
 * Errors as in the three calls; nothing is launched when an argument is refused.
 */
mustdrop_status_t mustdrop_filter(const mustdrop_plan_t *plan, const void *q_text, const void *k,
                                  const void *v, const void *hidden, const int32_t *key_idx,
                                  const int32_t *key_cnt, float *g_out, float *i_out, float *s_out,
                                  int32_t *kept_idx, int32_t *kept_cnt, void *hidden_out, void *k_out,
                                  void *v_out, void *workspace, void *cuda_stream);

/*
 * One pruning layer of a chain of layers (Sec. 3.4: the filter is applied at successive layers,
 * each on the tokens the previous one kept; after the spatial merge of Sec. 3.3 requests hold
 * different numbers of vision tokens; the set left after the last layer is the S_few of the
 * decoding-stage cache policy, Sec. 3.5).  mustdrop_filter with four optional additions, all
 * device pointers, each may be NULL:
 *   vis_cnt  int32 [B]       vision tokens request b actually holds, 1..n_vis (values outside
 *                            are clamped).  Its text tokens then sit directly behind them, at
 *                            rows vis_start + vis_cnt[b] .. + n_txt of k / v / hidden; later rows
 *                            are padding and are never read.  Scores of the absent tokens come
 *                            out 0, they are never selected, a request with fewer tokens than the
 *                            budget keeps them all, and thresholds left at 0 default per request
 *                            (gamma = 1 / vis_cnt[b], alpha = 2 / (vis_start + vis_cnt[b] + n_txt)).
 *                            Needs txt_start == vis_start + n_vis and seq_len == txt_start + n_txt.
 *                            May be the kept_cnt an earlier call on the same stream wrote.
 *   orig_idx int32 [B,n_vis] original id of every current vision token (NULL: 0, 1, 2, ...)
 *   orig_out int32 [B,cap]   receives the original ids of the kept tokens, ascending: the next
 *                            layer's orig_idx; after the last layer, S_few
 *   key_idx_out int32 [B,key_max], key_cnt_out int32 [B]
 *                            positions of the key tokens among the kept tokens: the next layer's
 *                            key_idx / key_cnt
 * With MUSTDROP_FLAG_REBUILD_SEQUENCE the outputs of one layer are laid out as the inputs of the
 * next (vis_cnt = this layer's kept_cnt).  One kernel launch where mustdrop_filter is one.
 */
typedef struct {
  const void *q_text, *k, *v, *hidden;       /* as in mustdrop_filter */
  const int32_t *key_idx, *key_cnt;
  const int32_t *vis_cnt, *orig_idx;
  float *g_out, *i_out, *s_out;
  int32_t *kept_idx, *kept_cnt;
  int32_t *orig_out, *key_idx_out, *key_cnt_out;
  void *hidden_out, *k_out, *v_out;
} mustdrop_layer_io_t;

mustdrop_status_t mustdrop_filter_layer(const mustdrop_plan_t *plan, const mustdrop_layer_io_t *io /* (host) */,
                                        void *workspace, void *cuda_stream);

/*
 * Decoding-stage cache compaction (Sec. 3.5, output-aware cache policy: the layers following
 * the second one keep, of the vision tokens, only S_few - the tokens still retained after the
 * last pruning layer).  One launch rebuilds the K and V caches of n_layers such layers.
 *   k_cache, v_cache bf16 [n_layers, B, H, rows_in, D] contiguous: layer y of request b holds
 *       vis_start prefix rows, then the vision tokens listed in layer_ids[y][b][0 .. layer_cnt[y][b])
 *       (original ids, strictly ascending), then n_tail further rows (text);
 *   layer_ids int32 [n_layers, B, ids_max], layer_cnt int32 [n_layers, B];
 *   s_few int32 [B, cap] original ids, ascending (the last layer's orig_out), s_few_cnt int32 [B];
 *   k_out, v_out bf16 [n_layers, B, H, vis_start + cap + n_tail, D]: prefix rows, the rows of the
 *       tokens of S_few in order, the tail rows directly behind them; later rows are untouched.
 * A token of S_few that a layer does not hold is skipped and recorded as
 * MUSTDROP_ERR_BAD_KEY_INDEX in the status word of `workspace` (>= 256 zeroed bytes, may be NULL).
 * (k_cache, k_out) or (v_cache, v_out) may be NULL together.  vis_start + ids_max + n_tail <= rows_in,
 * cap <= ids_max, head_dim == 128.
 */
typedef struct {
  int32_t n_layers, batch, n_heads, head_dim;
  int32_t rows_in, vis_start, n_tail, ids_max, cap;
} mustdrop_cache_config_t;

mustdrop_status_t mustdrop_cache_compact(const mustdrop_cache_config_t *config /* (host) */, const void *k_cache,
                                         const void *v_cache, const int32_t *layer_ids,
                                         const int32_t *layer_cnt, const int32_t *s_few,
                                         const int32_t *s_few_cnt, void *k_out, void *v_out,
                                         void *workspace, void *cuda_stream);

/*
 * Local Spatial Merging of the vision encoder's tokens (Sec. 3.3, Eq. 5).  The grid x grid
 * tokens of an image (raster order) are cut into non-overlapping window x window squares; a
 * square whose mean cosine similarity over its unordered token pairs exceeds tau is replaced by
 * the plain average of its tokens, placed at the square's first slot; the surviving tokens are
 * packed in raster order.  (The paper states neither the similarity measure nor tau nor the
 * weights: cosine, caller's tau, uniform weights are this library's reading.)
 *   tokens bf16 [B, grid*grid, channels]; merged bf16 [B, grid*grid, channels] receives the
 *   merged_cnt[b] surviving rows of image b (later rows untouched); slots int32 [B, grid*grid]
 *   the slot each surviving row came from; merged_cnt int32 [B] (the vis_cnt of
 *   mustdrop_filter_layer); window_sim fp32 [B, (grid/window)^2] or NULL receives the similarities.
 * fp32 accumulation; an average is rounded once to bf16.  window must be 2, grid even,
 * grid*grid <= 4096, channels a multiple of 8 (else MUSTDROP_ERR_UNSUPPORTED).
 */
mustdrop_status_t mustdrop_spatial_merge(int32_t batch, int32_t grid, int32_t window, int32_t channels,
                                         float tau, const void *tokens, void *merged, int32_t *slots,
                                         int32_t *merged_cnt, float *window_sim, void *cuda_stream);

/*
 * Key Retaining (Sec. 3.3, Eq. 6-7): a_cls = mean over heads of softmax(q_cls k^T / sqrt(head_dim))
 * over the n_tokens patch tokens; O = { j : a_cls[j] > mu }.  The paper calls mu "adaptive" and
 * gives no rule; here mu = Q3 + 1.5 (Q3 - Q1) of a_cls (Tukey's upper fence, linearly interpolated
 * quartiles).
 *   q_cls bf16 [B, H, head_dim]; k bf16 [B, H, n_tokens, head_dim] contiguous;
 *   key_idx int32 [B, key_max] receives O ascending (if O has more than key_max members, the
 *   key_max lowest indices), key_cnt int32 [B] the number stored - the key_idx / key_cnt of the
 *   filter calls; a_cls fp32 [B, n_tokens] and mu_out fp32 [B] may be NULL.
 * head_dim a multiple of 8 up to 256, n_tokens <= 4096.
 */
mustdrop_status_t mustdrop_key_set(int32_t batch, int32_t n_heads, int32_t head_dim, int32_t n_tokens,
                                   int32_t key_max, const void *q_cls, const void *k, float *a_cls,
                                   float *mu_out, int32_t *key_idx, int32_t *key_cnt, void *cuda_stream);

/* Kernel launches one mustdrop_filter call enqueues for this plan (-1: invalid plan). */
int32_t mustdrop_plan_filter_launches(const mustdrop_plan_t *plan);

/*
 * Read the device status word of a workspace (synchronises `cuda_stream`).
 * code_out (host) receives MUSTDROP_OK or the first device-detected condition, detail_out
 * (host, may be NULL) an operation-specific detail (BAD_KEY_INDEX: request * 65536 + slot).
 */
mustdrop_status_t mustdrop_device_status(const mustdrop_plan_t *plan, const void *workspace,
                                         void *cuda_stream, int32_t *code_out, int32_t *detail_out);

/* Static description of a status code. */
const char *mustdrop_status_string(mustdrop_status_t status);

/* cudaError_t value of the last failed CUDA call made by this library on this thread (0 if none). */
int32_t mustdrop_last_cuda_error(void);

/* Name of the score kernel variant the plan selected (static string; for logs and benchmarks). */
const char *mustdrop_plan_score_variant(const mustdrop_plan_t *plan);

/*
 * One-line description of what the plan will launch (kernel variant, cluster size, keys per CTA,
 * stages, buffers), for logs and benchmarks.  buf (host) receives at most n bytes including the
 * terminating zero; returns the length the full text needs.
 */
int32_t mustdrop_plan_describe(const mustdrop_plan_t *plan, char *buf /* (host) */, size_t n);

#ifdef __cplusplus
}
#endif
#endif /* MUSTDROP_H_ */
