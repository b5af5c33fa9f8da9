// Importance scores in ONE pass over the keys (Eq. 1, Eq. 8, Eq. 10), sm_100a only.
//
// A thread-block cluster owns one request and splits its L keys over its CTAs; each CTA loops
// over the heads.  Warp roles inside a CTA (16 warps):
//   TMA warp      stages the CTA's K rows and the head's text queries in shared memory;
//   MMA warp      one thread issues tcgen05 MMAs (bf16 in, fp32 logits in tensor memory);
//   8 exp warps   read the logits with text queries on the TMEM lanes (a thread owns one text row
//                 and a run of key columns, so row maxima and sums are in-thread), write the
//                 exponentials back to tensor memory and send their (max, sum) pairs to every
//                 CTA of the cluster with asynchronous distributed-shared-memory stores that
//                 count on the receiver's mbarrier;
//   4 add warps   once all pairs of a head have arrived, normalise the exponentials and add them
//                 into per-thread head sums that live in registers for the whole kernel.
// Three to eight tensor-memory buffers (as many as the columns per head allow) keep the MMA, exp
// and add stages of consecutive heads in flight.
// After the last head the head mean is reduced over the text rows into G (column sum) and
// I (column max).  K is read once; nothing goes through global scratch.
//
// Lane layouts.  N <= 64: two M=64 MMAs per head write the two halves of the CTA's key range
// to the lower and upper 16 lanes of every 32-lane TMEM quadrant, so all 128 lanes carry one of
// 64 text rows.  N > 64: one M=128 MMA, lane = text row.
//
// Every wait on an mbarrier is bounded; when a wait runs out the CTA records
// MUSTDROP_ERR_TIMEOUT in the workspace status word, stops working and goes to the common exit
// (which still frees tensor memory and joins the cluster barrier).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>

#include "mustdrop_internal.h"
#include "select_body.cuh"

namespace mustdrop {
namespace {

constexpr int kExpWarps = 8;                // warps 0-7: 4 TMEM lane quadrants x 2 column groups
constexpr int kColGroups = 2;
constexpr float kPhScale = 16384.0f;        // per-head maxima travel as fp16 times 2^14
constexpr int kAddWarps = 4;                // warps 8-11: one per lane quadrant, all columns
constexpr int kExpThreads = kExpWarps * 32;
constexpr int kAddThreads = kAddWarps * 32;
constexpr int kTmaWarp = kExpWarps + kAddWarps;   // warp 12
constexpr int kMmaWarp = kTmaWarp + 1;            // warp 13; warps 14-15 only fill the last warpgroup
constexpr int kThreads = 16 * 32;
constexpr int kChunk = 16;                  // TMEM columns per tcgen05.ld / st
constexpr int kMaxCluster = 16;               // beyond 8 the cluster size is non-portable (opt-in per kernel)
constexpr int kMaxQBufs = 4;                  // shared-memory ring of text-query tiles (one per head)
constexpr int kMaxKBufs = 8;                  // shared-memory ring of key half-tiles (HALVES per head)
constexpr int kMinBufs = 3;                 // tensor-memory buffers: MMA, exp and add stages in flight (two for 176-column tiles) ...
constexpr int kMaxBufs = 8;                 // ... more when the columns per head allow, to hide the per-head latency chain
constexpr int kMaxSlots = 2 * kMaxBufs;     // statistics slots = 2 x buffers: a peer's exp warps run at most that far ahead of our add warps
constexpr int kTmemCols = 512;
constexpr int kMaxGatherSlots = 8;         // rows in flight per CTA in the gather tail of the filter kernel
constexpr int kKeptListBytes = kMaxVis * 4; // the request's kept indices, at the start of dynamic shared memory
constexpr long long kWaitCycles = 200000000LL;   // ~0.1 s at 2 GHz; no legitimate wait comes near it

struct FusedParams {
  float* g_out;
  float* i_out;
  void* workspace;
  const int32_t* vis_cnt;             // [B] or null: vision tokens the request holds; its text keys follow them
  int32_t H, N, L, M, vis_start, txt_start, causal;
  int32_t n_txt;                      // all text rows of the request (N is this launch's share)
  int32_t row0, combine;              // this launch covers text rows row0 .. row0 + N - 1; combine: add to / max with what g_out / i_out hold
  int32_t cluster, tk, cpl;           // CTAs per request, keys per CTA, columns per TMEM lane
  int32_t n_q, n_k;                   // whole stages: n_q of them; split: ring sizes of query tiles and key half-tiles
  int32_t split;
  int32_t n_buf, n_slot;              // tensor-memory buffers, statistics slots (2 * n_buf, or 4 when tight)
  int32_t tight;                      // d = 1 or 2: the exp warps start head h only when the add warps are done with head h - d (0: no such rule)
  // Statistics exchange through global memory instead of distributed shared memory ("grid" plans:
  // the CTAs of a request are ordinary CTAs of the grid, any number of them, all resident at once).
  int32_t gx;                         // 1: grid plan (cluster = CTAs per request, launched without a cluster)
  float2* gx_stats;                   // [B][H][CTAs per request][rows][pairs] (stabiliser, sum)
  uint32_t* gx_cnt;                   // [B*H] CTAs that published a head, [B] scores stored, [B] barrier passed, [B] CTAs that left; zero between calls
  int32_t per_head;                   // 1: i_out = head mean of the per-head maxima over the text rows (PH instantiations)
  int32_t early_inputs;               // 1: q_text / k may be read before the stream's earlier work has completed (caller's promise)
  long long wait_cycles;              // clock cycles after which a wait between the warp roles gives up
  float scale_log2e, inv_heads;
};

// Tail of the single-launch filter kernel: selection and gather-compaction of the request by
// the cluster that scored it.
struct FilterTail {
  SelectParams sel;              // g / i are the score outputs of this launch
  const unsigned char* hidden;   // null: tensor not copied
  unsigned char* hidden_out;
  int64_t hid_sb, hid_sl;        // bytes
  int32_t hidden_bytes;          // bytes of a hidden row (0 when not copied)
  int32_t hidden_pad;            // the same rounded up to 128 (alignment of the tensor copies behind it)
  int32_t kv_bytes;              // bytes of a K (or V) row over all heads = H * 256
  int32_t has_k, has_v;
  int32_t slot_bytes, n_slot;    // gather ring in dynamic shared memory
  int32_t vis_start;
  int32_t rebuild, N, out_rows;  // rebuild: outputs are [prefix ; kept vision ; text] (out_rows rows per request)
};

// ---- small PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Grid plans: release / acquire on a counter in global memory.
__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Bounded wait until a counter has reached its target (same give-up rules as mbar_wait).
__device__ __forceinline__ bool count_wait(const uint32_t* p, uint32_t target, volatile int* abort_flag, long long limit) {
  if (ld_acquire_gpu(p) >= target) return true;
  const long long t0 = clock64();
  while (ld_acquire_gpu(p) < target) {
    if (*abort_flag != 0 || clock64() - t0 > limit) {
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag) when the wait ran out or the
// CTA has already given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag != 0 || clock64() - t0 > limit) {
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t cta_rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(cta_rank));
  return r;
}
// Asynchronous store of 8 bytes into (possibly another CTA's) shared memory; its arrival is
// counted on the mbarrier of the destination CTA, so no fence or separate arrive is needed.
__device__ __forceinline__ void st_async_f32x2(uint32_t addr, float a, float b, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];" ::"r"(addr),
               "f"(a), "f"(b), "r"(bar)
               : "memory");
}
// Barrier over all threads of the CTA, counted per thread: warps whose lanes took different
// roles (one lane drives the copies or the MMAs, the others only wait) may arrive diverged.
__device__ __forceinline__ void cta_sync() { asm volatile("barrier.sync 0, %0;" ::"n"(kThreads) : "memory"); }
__device__ __forceinline__ void st_remote_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}
// The same copy with an L2 eviction-priority hint (keys are read exactly once: evict them first,
// so that they do not push out data other kernels left in L2).
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                                 uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar), "l"(policy)
      : "memory");
}
// Bulk copies of the gather tail: a contiguous row (1-D) or one token's pieces over all heads
// (4-D box 128 x 1 x H x 1) from global to shared memory, and back out to the dense outputs.
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void bulk_store_1d(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::"l"(map),
               "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  return policy;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
}
// The same store under a predicate that must be uniform over the warp (no branch around it).
__device__ __forceinline__ void tc_st16_if(bool go, uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %17, 0;\n\t"
      "@p tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};\n\t}"
      ::"r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
        "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
        "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15])), "r"(taddr), "r"(static_cast<uint32_t>(go))
      : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::"r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
        "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
        "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15])), "r"(taddr)
      : "memory");
}
// Two fp32 operations per instruction (packed in a 64-bit register pair): the exp and add warps'
// loops are as much bound by the number of instructions they issue as by any unit.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Shared-memory matrix descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups
// 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return static_cast<uint64_t>((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// Optional timeline tracing (compiled out unless MUSTDROP_TRACE is defined): one global-timer
// stamp per (CTA, head, event) into the scratch part of the workspace.
#ifdef MUSTDROP_TRACE
__device__ __forceinline__ void trace_stamp(void* workspace, int n_heads, int h, int ev) {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(workspace) + 4096)
      [(static_cast<size_t>(blockIdx.x) * n_heads + h) * 16 + ev] = t;
}
#define MD_TRACE(h, ev) trace_stamp(p.workspace, p.H, (h), (ev))
#else
#define MD_TRACE(h, ev) ((void)0)
#endif

// Rare path of the exp warps (kept out of line so that the hot loop stays small): the `count`
// chunks already stored at first, first + stride, ... are multiplied by this lane's factor.
// Called by all lanes of a warp together.
__device__ __forceinline__ void rescale_stored(uint32_t first, uint32_t stride, int count, float fac) {
  tc_wait_st();
  for (int u = 0; u < count; ++u) {
    float old[kChunk];
    tc_ld16(first + stride * u, old);
    tc_wait_ld();
#pragma unroll
    for (int j = 0; j < kChunk; ++j) old[j] *= fac;
    tc_st16(first + stride * u, old);
  }
}

// The careful way through the chunks t_begin .. t_end - 1 of a thread (first + stride * t in
// tensor memory), out of line as well: a chunk lay so far above the row's stabiliser that the sum
// left its range, so from that chunk on nothing was stored.  Per chunk: its logits are taken
// again, the stabiliser moves up to their maximum if that is larger, the chunks stored before it
// are rescaled, the chunk's exponentials are computed and stored.  nvis0 - nvis_step * t columns of
// chunk t are visible to this lane.  Returns the final stabiliser and the row's running sum.
struct RedoResult {
  float mx, l;
};
__device__ __forceinline__ RedoResult redo_rest(uint32_t first, uint32_t stride, int t_begin, int t_end, int nvis0, int nvis_step,
                                             float scale_log2e, bool two_halves, float mx, float l) {
  for (int t = t_begin; t < t_end; ++t) {
    const int nvis = nvis0 - nvis_step * t;
    float zc[kChunk];
    tc_ld16(first + stride * t, zc);
    tc_wait_ld();
    float cm = -INFINITY;
#pragma unroll
    for (int j = 0; j < kChunk; ++j) {
      zc[j] = (j < nvis) ? zc[j] : -INFINITY;
      cm = fmaxf(cm, zc[j]);
    }
    cm *= scale_log2e;
    if (two_halves) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 16));   // one stabiliser per row
    const float up = fmaxf(mx, cm);
    const float sub = (up == -INFINITY) ? 0.0f : up;     // a lane with nothing visible so far keeps 0
    // (a lane whose stabiliser stays, or that has stored nothing but zeros so far, multiplies by 1)
    const float fac = (up == mx || mx == -INFINITY) ? 1.0f : ex2(mx - up);
    if (__any_sync(0xffffffffu, fac != 1.0f)) rescale_stored(first, stride, t, fac);   // (all lanes take part)
    float part[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
    for (int j = 0; j < kChunk; ++j) {
      const float e = ex2(fmaf(zc[j], scale_log2e, -sub));
      zc[j] = e;
      part[j & 3] += e;
    }
    tc_st16(first + stride * t, zc);
    l = l * fac + ((part[0] + part[1]) + (part[2] + part[3]));
    mx = up;
  }
  return RedoResult{mx, l};
}

struct __align__(8) Barriers {
  uint64_t qfull[kMaxQBufs];     // TMA -> MMA: query tile of a head has landed
  uint64_t qempty[kMaxQBufs];    // MMA -> TMA: query tile consumed
  uint64_t full[kMaxKBufs];      // TMA -> MMA: key half-tile has landed
  uint64_t empty[kMaxKBufs];     // MMA -> TMA: key half-tile consumed
  uint64_t tfull[kMaxBufs];      // MMA -> exp warps: logits of a head are in tensor memory
  uint64_t eready[kMaxBufs];     // exp -> add warps: exponentials of a head are in tensor memory
  uint64_t tempty[kMaxBufs];     // add warps -> MMA: tensor-memory buffer free
  uint64_t sfull[kMaxSlots];    // all CTAs' (max, sum) pairs of a head have arrived
  uint64_t fin;                  // add warps meet before / after staging the head sums
  uint64_t ph;                   // add warps meet once per head (per-head maxima of Eq. 10)
  uint64_t gsent[kMaxBufs];      // grid plans: exp warps -> publishing thread: this CTA's pairs of a head are in global memory
  uint64_t gfull[kMaxGatherSlots];   // filter tail: a gathered row has landed in its slot
};

// Tensor maps of the gather tail (used only by the FILTER instantiations).
struct GatherMaps {
  CUtensorMap k_src, v_src, k_dst, v_dst;
};

// ---- the filter tail ------------------------------------------------------------------------------
// Both parts run once per CTA after the score part.  Functions of their own for reading only: they
// are inlined (as real calls - like any call in this kernel - they slowed the gather by a third).

// Selection of request b by the 256 threads of the exp warps (tid = 0..255); rank 0 of the
// request's CTAs stores the list, every CTA keeps it in its shared memory.
__device__ __forceinline__ void filter_select(const SelectParams& sel, SelectShared& sel_sh, int b, int tid, bool writer,
                                           int32_t* kept_list, int32_t* kept_total) {
  select_clear(sel_sh, tid);
  const int own = (sel.M + kSelThreads - 1) / kSelThreads;
  if (own <= 1) select_request<1, SelectSyncGroup>(sel, sel_sh, b, tid, writer, kept_list, kept_total);
  else if (own <= 2) select_request<2, SelectSyncGroup>(sel, sel_sh, b, tid, writer, kept_list, kept_total);
  else if (own <= 4) select_request<4, SelectSyncGroup>(sel, sel_sh, b, tid, writer, kept_list, kept_total);
  else if (own <= 8) select_request<8, SelectSyncGroup>(sel, sel_sh, b, tid, writer, kept_list, kept_total);
  else select_request<16, SelectSyncGroup>(sel, sel_sh, b, tid, writer, kept_list, kept_total);
}

// Gather of the request's kept rows, driven by ONE thread of the CTA: row r of the compacted
// outputs is copied by CTA r mod cluster.
__device__ __forceinline__ void filter_gather(const FilterTail& ft, const GatherMaps& gm, uint64_t* gfull, volatile int* abort_flag,
                                           const int32_t* kept_list, int kept_total_s, uint32_t stage_base, int rank, int b,
                                           int Mb, int cluster, void* workspace) {
  // One thread drives the copies: rows are loaded into a ring of shared-memory slots by bulk
  // copies that count on the slot's mbarrier, and stored from there by bulk copies tracked in
  // bulk groups.  Loads run n_slot - 2 rows ahead of the stores.
  fence_proxy_async();   // earlier generic-proxy accesses to the slots precede the async-proxy writes
  const int total = kept_total_s < ft.sel.cap ? kept_total_s : ft.sel.cap;
  const int C = cluster;
  // items: the kept vision rows, then (rebuild) the prefix rows and the request's text rows
  const int n_items = total + (ft.rebuild ? ft.vis_start + ft.N : 0);
  const int n_mine = n_items > rank ? (n_items - rank + C - 1) / C : 0;
  const int S = ft.n_slot, ahead = S - 2;
  const uint32_t ring = stage_base + kKeptListBytes;
  const uint32_t payload = static_cast<uint32_t>(ft.hidden_bytes) + static_cast<uint32_t>(ft.has_k + ft.has_v) * ft.kv_bytes;
  const uint64_t once = l2_evict_first_policy();
  // item -> (source row, destination row)
  auto src_row = [&](int it) {
    if (it < total) return ft.vis_start + kept_list[it];
    const int x = it - total;
    return x < ft.vis_start ? x : ft.vis_start + Mb + (x - ft.vis_start);
  };
  auto dst_row = [&](int it) {
    if (!ft.rebuild) return it;
    if (it < total) return ft.vis_start + it;
    const int x = it - total;
    return x < ft.vis_start ? x : ft.vis_start + total + (x - ft.vis_start);
  };
  bool ok = true;
  int loaded = 0;
  for (int i = 0; i < n_mine + ahead && ok; ++i) {
    if (i < n_mine) {
      const int slot = i % S;
      if (i >= S) bulk_wait_read_1();   // the stores of item i - S have finished reading the slot
      const int row = src_row(rank + i * C);
      const uint32_t bar = smem_u32(&gfull[slot]);
      uint32_t dst = ring + static_cast<uint32_t>(slot) * ft.slot_bytes;
      mbar_expect_tx(bar, payload);
      if (ft.hidden_bytes > 0) {
        bulk_load_1d(dst, ft.hidden + b * ft.hid_sb + row * ft.hid_sl, ft.hidden_bytes, bar, once);
        dst += ft.hidden_pad;
      }
      if (ft.has_k) {
        tma_load_4d_hint(dst, &gm.k_src, 0, row, 0, b, bar, once);
        dst += ft.kv_bytes;
      }
      if (ft.has_v) tma_load_4d_hint(dst, &gm.v_src, 0, row, 0, b, bar, once);
      loaded = i + 1;
    }
    const int c = i - ahead;
    if (c >= 0) {
      const int slot = c % S;
      if (!mbar_wait(smem_u32(&gfull[slot]), static_cast<uint32_t>(c / S) & 1u, abort_flag, kWaitCycles)) { ok = false; break; }
      const int r = dst_row(rank + c * C);
      uint32_t src = ring + static_cast<uint32_t>(slot) * ft.slot_bytes;
      if (ft.hidden_bytes > 0) {
        bulk_store_1d(ft.hidden_out + (static_cast<int64_t>(b) * ft.out_rows + r) * ft.hidden_bytes, src, ft.hidden_bytes);
        src += ft.hidden_pad;
      }
      if (ft.has_k) {
        tma_store_4d(&gm.k_dst, 0, r, 0, b, src);
        src += ft.kv_bytes;
      }
      if (ft.has_v) tma_store_4d(&gm.v_dst, 0, r, 0, b, src);
      bulk_commit();
    }
  }
  if (!ok) {
    // gave up: still leave only when every load this thread started has landed (bounded)
    record_status(workspace, MUSTDROP_ERR_TIMEOUT, blockIdx.x);
    ft.sel.kept_cnt[b] = -1;   // some of this request's rows were not copied
    for (int i = (loaded > S ? loaded - S : 0); i < loaded; ++i) {
      const uint32_t bar = smem_u32(&gfull[i % S]);
      const long long t0 = clock64();
      while (!mbar_try_wait(bar, static_cast<uint32_t>(i / S) & 1u) && clock64() - t0 < kWaitCycles) {}
    }
  }
  bulk_wait_all();   // the stores have been written before the CTA (and its shared memory) goes away
}

// HALVES: 2 = two M=64 tiles per head (N <= 64), 1 = one M=128 tile.
// ACH: chunks (of 16 columns) an add thread may own; an exp thread owns up to (ACH+1)/2.
// FILTER: after the scores, the cluster also selects the request's tokens and gathers them.
// PH: the other reading of Eq. 10 - per head the column maximum over the text rows, then the head
//     mean - computed by the add warps from the same normalised probabilities (G is unchanged).
template <int HALVES, int ACH, bool FILTER, bool PH>
__global__ void __launch_bounds__(kThreads, 1)
score_fused_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                   const FusedParams p, const __grid_constant__ GatherMaps gm, const __grid_constant__ FilterTail ft) {
  constexpr int NROWS = 128 / HALVES;            // text rows carried by the TMEM lanes
  // The two exp warps of a lane quadrant ALTERNATE heads (group g = 0, 1 takes the heads g,
  // g + 2, ...): two heads are in the exp stage at a time, so what a head costs besides its chunk
  // loop - waiting for its MMAs, the first chunk's load and maximum, the hand-over, the statistics
  // stores - runs under the other group's loop.  (Splitting every head's chunks over the two warps
  // instead left those 0.7 us per head on the path of every head: 7 % of a step at the target point.)
  constexpr bool kRealloc = ACH > 5;             // move registers from the other warpgroups to the add warps

  extern __shared__ __align__(1024) unsigned char smem_dyn[];
  __shared__ Barriers bars;
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_flag_s;          // this CTA gave up a wait
  __shared__ int cluster_abort_s;       // some CTA of the cluster did (written by that CTA before the exit barrier)

  volatile int* abort_flag = &abort_flag_s;
  const long long wait_limit = p.wait_cycles;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = p.gx ? blockIdx.x % static_cast<uint32_t>(p.cluster) : cluster_cta_rank();
  const int b = blockIdx.x / p.cluster;
  MD_PIPE(p.workspace, 0, false, true);
  if (threadIdx.x == 0) MD_TRACE(0, 8);    // (CTA-level stamps use the event slots 8.. of head 0) kernel entry
  // dynamic shared memory: [n_q query tiles][n_k key half-tiles][stats: n_slot x cluster x NROWS float2]
  // A tile is two slabs of 64 elements (128 bytes per row, 128-byte swizzle), rows contiguous per slab.
  // Two layouts of the staging area: whole stages (a head's query tile and all its keys, n_q of
  // them, recycled together), or - where shared memory is short - a ring of n_q query tiles and a
  // ring of n_k key half-tiles recycled on their own (p.split).
  constexpr uint32_t q_bytes = NROWS * 256u;
  const uint32_t kh_bytes = static_cast<uint32_t>(p.cpl) * 256u;
  const uint32_t stage_bytes = static_cast<uint32_t>(NROWS + p.tk) * 256u;
  const uint32_t stage_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const uint32_t k_base = stage_base + static_cast<uint32_t>(p.n_q) * q_bytes;
  unsigned char* stage_ptr = smem_dyn + (stage_base - smem_u32(smem_dyn));
  const size_t staging = p.split ? static_cast<size_t>(p.n_q) * q_bytes + static_cast<size_t>(p.n_k) * kh_bytes
                                 : static_cast<size_t>(p.n_q) * stage_bytes;
  float2* stats = reinterpret_cast<float2*>(stage_ptr + staging);
  // pairs per slot: one (max, sum) pair per text row and CTA
  const uint32_t slot_pairs = static_cast<uint32_t>(p.cluster) * NROWS;
  // PH only: [2][4 add warps][tk] per-head column maxima of each warp's text rows, double-buffered over heads
  float* const ph_stage = reinterpret_cast<float*>(stats + static_cast<size_t>(p.n_slot) * slot_pairs);
  // grid plans only: [n_buf][rows] the pairs of this CTA's own exp warps, per tensor-memory buffer
  float2* const own_pairs = reinterpret_cast<float2*>(ph_stage + (PH ? 2 * kAddWarps * p.tk : 0));

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    cluster_abort_s = 0;
    for (int s = 0; s < kMaxQBufs; ++s) { mbar_init(smem_u32(&bars.qfull[s]), 1); mbar_init(smem_u32(&bars.qempty[s]), 1); }
    for (int s = 0; s < kMaxKBufs; ++s) { mbar_init(smem_u32(&bars.full[s]), 1); mbar_init(smem_u32(&bars.empty[s]), 1); }
    for (int s = 0; s < kMaxBufs; ++s) {
      mbar_init(smem_u32(&bars.tfull[s]), 1);
      mbar_init(smem_u32(&bars.eready[s]), kExpWarps / kColGroups);   // (the four warps of the head's group)
      mbar_init(smem_u32(&bars.tempty[s]), kAddWarps);
    }
    // (grid plans: the 32 lanes of the fetch warp each arrive once their copies have landed)
    for (int s = 0; s < kMaxSlots; ++s) mbar_init(smem_u32(&bars.sfull[s]), p.gx ? 32 : 1);
    mbar_init(smem_u32(&bars.fin), kAddThreads);
    mbar_init(smem_u32(&bars.ph), kAddThreads);
    for (int s = 0; s < kMaxBufs; ++s) mbar_init(smem_u32(&bars.gsent[s]), kExpWarps / kColGroups);
    for (int s = 0; s < kMaxGatherSlots; ++s) mbar_init(smem_u32(&bars.gfull[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // every CTA's barriers are initialised before any remote store counts on them
  tc_fence_after();
  // Let the next kernel in the stream begin its prologue.  Everything up to here touched no
  // global data; the copy thread waits for the stream's earlier work before its first load (its
  // inputs may come from the kernel just before this one), the other roles before their stores.
  pdl_launch_dependents();
  if (threadIdx.x == 0) MD_TRACE(0, 9);    // prologue done
  const uint32_t tmem_base = tmem_base_holder;
  // This request's own sequence.  In a ragged batch the token count comes from an earlier
  // kernel in the stream (the previous layer's selection), so it is read after the wait.
  int Mb = p.M, Lb = p.L, txt_start = p.txt_start;
  if (p.vis_cnt != nullptr) {
    pdl_wait();
    Mb = clamp_vis_cnt(p.vis_cnt[b], p.M);
    txt_start = p.vis_start + Mb;
    Lb = txt_start + p.n_txt;
  }

  // End of the score part, executed by every thread: tensor memory freed, and no CTA goes on
  // while a peer may still write into its shared memory.  The cluster barrier also orders every
  // CTA's g_out / i_out stores before what the filter tail loads.  (In the filter kernel each
  // warp role calls this from its own branch and continues there with its part of the tail, so
  // every role keeps the register count setmaxnreg gave it; no second setmaxnreg is needed.)
  __shared__ int32_t kept_total_s;
  auto common_exit = [&]() {
    __syncwarp();   // a warp whose lane 0 had a role of its own is whole again before the aligned instructions below
    tc_fence_before();
    cta_sync();
    if (p.gx) {
      // grid plan: the request's CTAs are no cluster.  In the filter kernel they meet through a
      // counter in global memory: every CTA's scores are stored before any CTA selects.  (A CTA
      // that gives up tells nobody: its peers run into their own limits.)
      if (threadIdx.x == 0) {
        const size_t n_req = gridDim.x / p.cluster;
        if (*abort_flag == 0) {
          // every CTA has seen all of its heads complete when it gets here: the last one of the
          // request to do so clears the heads' counters for the next call (one counted visit per
          // CTA instead of one per head, whose returned value the fetch warp would have to wait for)
          uint32_t* const left = p.gx_cnt + n_req * p.H + 2 * n_req + b;
          if (atomicAdd(left, 1u) == static_cast<uint32_t>(p.cluster) - 1u) {
            for (int hh = 0; hh < p.H; ++hh) p.gx_cnt[static_cast<size_t>(b) * p.H + hh] = 0u;
            *left = 0u;
          }
        }
        if (FILTER && *abort_flag == 0) {
          uint32_t* const stored = p.gx_cnt + n_req * p.H + b;
          uint32_t* const passed = stored + n_req;
          __threadfence();
          atomicAdd(stored, 1u);
          if (count_wait(stored, static_cast<uint32_t>(p.cluster), abort_flag, wait_limit) &&
              atomicAdd(passed, 1u) == static_cast<uint32_t>(p.cluster) - 1u) {
            *stored = 0u;   // the last one through leaves the counters as the next call expects them
            *passed = 0u;
          }
        }
        if (*abort_flag != 0) {
          record_status(p.workspace, MUSTDROP_ERR_TIMEOUT, blockIdx.x);
          cluster_abort_s = 1;
        }
      }
      cta_sync();
    } else if (threadIdx.x == 0 && *abort_flag != 0) {
      record_status(p.workspace, MUSTDROP_ERR_TIMEOUT, blockIdx.x);
      for (int c = 0; c < p.cluster; ++c) st_remote_u32(map_to_cta(smem_u32(&cluster_abort_s), c), 1u);
    }
    if (warp == kMmaWarp) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
    cluster_sync_all();   // (release / acquire: a peer's flag store above is visible behind it)
    if (threadIdx.x == 0) MD_TRACE(0, 11);   // score part left
    MD_PIPE(p.workspace, 0, true, false);
  };
  // After common_exit: did any CTA of the cluster give up?  (Stable by then: same answer in every thread.)
  auto cluster_gave_up = [&]() { return *reinterpret_cast<volatile int*>(&cluster_abort_s) != 0; };
  // The way out after a give-up, taken by every thread of every CTA of the cluster.  A peer's
  // asynchronous statistics stores may still be on their way into this CTA's shared memory: give
  // them time to land and meet once more, so that no CTA's shared memory goes away under them.
  auto leave_after_give_up = [&](int32_t* kept_cnt) {
    if (kept_cnt != nullptr && (rank == 0 || p.gx) && threadIdx.x == 0) {
      pdl_wait();
      kept_cnt[b] = -1;   // this request's result is invalid
    }
    const long long t0 = clock64();
    while (clock64() - t0 < 40000) {}
    __syncwarp();
    cluster_sync_all();
  };
  int32_t* const kept_list = reinterpret_cast<int32_t*>(stage_ptr);   // filter tail: the request's kept indices

  if (warp >= kTmaWarp) {
    if (kRealloc) asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    if (warp == kTmaWarp && lane == 0) {
      // ---------------- TMA producer ----------------
      const int key0 = static_cast<int>(rank) * p.tk;
      const uint64_t stream_once = l2_evict_first_policy();
      if (!p.early_inputs) pdl_wait();   // q_text / k may be the output of the kernel just before this one
      if (p.split) {
        int q_issued = 0, k_issued = 0;   // tiles started so far
        bool ok = true;
        for (int h = 0; h < p.H && ok; ++h) {
          const int qi = h % p.n_q;
          if (!mbar_wait(smem_u32(&bars.qempty[qi]), (static_cast<uint32_t>(h / p.n_q) & 1u) ^ 1u, abort_flag, wait_limit)) break;
          const uint32_t qfull = smem_u32(&bars.qfull[qi]);
          const uint32_t q_dst = stage_base + qi * q_bytes;
          mbar_expect_tx(qfull, q_bytes);
          MD_TRACE(h, 0);
          tma_load_4d(q_dst, &q_map, 0, 0, h, b, qfull);
          tma_load_4d(q_dst + NROWS * 128u, &q_map, 64, 0, h, b, qfull);
          q_issued = h + 1;
  #pragma unroll
          for (int hv = 0; hv < HALVES; ++hv) {
            const int ki = k_issued % p.n_k;
            if (!mbar_wait(smem_u32(&bars.empty[ki]), (static_cast<uint32_t>(k_issued / p.n_k) & 1u) ^ 1u, abort_flag, wait_limit)) {
              ok = false;
              break;
            }
            const uint32_t full = smem_u32(&bars.full[ki]);
            const uint32_t k_dst = k_base + ki * kh_bytes;
            mbar_expect_tx(full, kh_bytes);
            tma_load_4d_hint(k_dst, &k_map, 0, key0 + hv * p.cpl, h, b, full, stream_once);
            tma_load_4d_hint(k_dst + p.cpl * 128u, &k_map, 64, key0 + hv * p.cpl, h, b, full, stream_once);
            ++k_issued;
          }
        }
        // Leave only when every copy this thread started has landed (bounded).
        for (int x = (q_issued > p.n_q ? q_issued - p.n_q : 0); x < q_issued; ++x) {
          const uint32_t bar = smem_u32(&bars.qfull[x % p.n_q]);
          const uint32_t ph = static_cast<uint32_t>(x / p.n_q) & 1u;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar, ph) && clock64() - t0 < kWaitCycles) {}
        }
        for (int x = (k_issued > p.n_k ? k_issued - p.n_k : 0); x < k_issued; ++x) {
          const uint32_t bar = smem_u32(&bars.full[x % p.n_k]);
          const uint32_t ph = static_cast<uint32_t>(x / p.n_k) & 1u;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar, ph) && clock64() - t0 < kWaitCycles) {}
        }
      } else {
        int issued = 0;
        for (int h = 0; h < p.H; ++h) {
          const int s = h % p.n_q;
          const uint32_t ph = static_cast<uint32_t>(h / p.n_q) & 1u;
          if (!mbar_wait(smem_u32(&bars.empty[s]), ph ^ 1u, abort_flag, wait_limit)) break;
          const uint32_t full = smem_u32(&bars.full[s]);
          const uint32_t q_dst = stage_base + s * stage_bytes;
          const uint32_t k_dst = q_dst + NROWS * 256u;
          mbar_expect_tx(full, stage_bytes);
          MD_TRACE(h, 0);
  #pragma unroll
          for (int slab = 0; slab < 2; ++slab) {
            tma_load_4d(q_dst + slab * (NROWS * 128u), &q_map, slab * 64, 0, h, b, full);
  #pragma unroll
            for (int hv = 0; hv < HALVES; ++hv)
              tma_load_4d_hint(k_dst + slab * (p.tk * 128u) + hv * (p.cpl * 128u), &k_map, slab * 64, key0 + hv * p.cpl,
                               h, b, full, stream_once);
          }
          issued = h + 1;
        }
        // Leave only when every copy this thread started has landed (bounded).
        for (int h = (issued > p.n_q ? issued - p.n_q : 0); h < issued; ++h) {
          const uint32_t bar = smem_u32(&bars.full[h % p.n_q]);
          const uint32_t ph = static_cast<uint32_t>(h / p.n_q) & 1u;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar, ph) && clock64() - t0 < kWaitCycles) {}
        }
      }
#ifdef MUSTDROP_TRACE
    } else if (warp == kTmaWarp && lane == 1 && !p.split) {
      // trace build only: an onlooker that stamps the moment a stage's copies have landed (it tests
      // the barrier's phase and changes nothing; the MMA thread's own stamp comes when its turn does)
      for (int h = 0; h < p.H; ++h) {
        const uint32_t bar = smem_u32(&bars.full[h % p.n_q]);
        const uint32_t ph = static_cast<uint32_t>(h / p.n_q) & 1u;
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, ph) && clock64() - t0 < kWaitCycles && *abort_flag == 0) {}
        MD_TRACE(h, 14);
      }
#endif
    } else if (warp == kMmaWarp && lane == 0) {
      // ---------------- MMA issuer ----------------
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(p.cpl >> 3) << 17) |
                             (static_cast<uint32_t>(NROWS >> 4) << 24);
      int committed = -1;   // last head whose MMAs were committed to its tfull barrier
      if (p.split) {
        int k_used = 0;
        bool ok = true;
        for (int h = 0; h < p.H && ok; ++h) {
          const int qi = h % p.n_q, buf = h % p.n_buf;
          const uint32_t bph = static_cast<uint32_t>(h / p.n_buf) & 1u;
          if (!mbar_wait(smem_u32(&bars.qfull[qi]), static_cast<uint32_t>(h / p.n_q) & 1u, abort_flag, wait_limit)) break;
          MD_TRACE(h, 1);
          if (!mbar_wait(smem_u32(&bars.tempty[buf]), bph ^ 1u, abort_flag, wait_limit)) break;
          MD_TRACE(h, 2);
          const uint32_t q_src = stage_base + qi * q_bytes;
  #pragma unroll
          for (int hv = 0; hv < HALVES; ++hv) {
            const int ki = k_used % p.n_k;
            if (!mbar_wait(smem_u32(&bars.full[ki]), static_cast<uint32_t>(k_used / p.n_k) & 1u, abort_flag, wait_limit)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t k_src = k_base + ki * kh_bytes;
            // the second M=64 tile goes to the upper 16 lanes of every TMEM quadrant
            const uint32_t d = tmem_base + static_cast<uint32_t>(buf * p.cpl) + (hv ? (16u << 16) : 0u);
  #pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t slab = ks >> 2, koff = (ks & 3) * 32u;
              const uint64_t ad = smem_desc(q_src + slab * (NROWS * 128u) + koff);
              const uint64_t bd = smem_desc(k_src + slab * (p.cpl * 128u) + koff);
              tc_mma(d, ad, bd, idesc, ks > 0 ? 1u : 0u);
            }
            tc_commit(smem_u32(&bars.empty[ki]));   // this half-tile may be refilled once its MMAs are done
            ++k_used;
          }
          if (!ok) break;
          tc_commit(smem_u32(&bars.qempty[qi]));
          tc_commit(smem_u32(&bars.tfull[buf]));
          committed = h;
        }
      } else {
        for (int h = 0; h < p.H; ++h) {
          const int s = h % p.n_q, buf = h % p.n_buf;
          const uint32_t ph = static_cast<uint32_t>(h / p.n_q) & 1u;
          const uint32_t bph = static_cast<uint32_t>(h / p.n_buf) & 1u;
          if (!mbar_wait(smem_u32(&bars.full[s]), ph, abort_flag, wait_limit)) break;
          MD_TRACE(h, 1);
          if (!mbar_wait(smem_u32(&bars.tempty[buf]), bph ^ 1u, abort_flag, wait_limit)) break;
          MD_TRACE(h, 2);
          tc_fence_after();
          const uint32_t q_src = stage_base + s * stage_bytes;
          const uint32_t k_src = q_src + NROWS * 256u;
  #pragma unroll
          for (int hv = 0; hv < HALVES; ++hv) {
            // the second M=64 tile goes to the upper 16 lanes of every TMEM quadrant
            const uint32_t d = tmem_base + static_cast<uint32_t>(buf * p.cpl) + (hv ? (16u << 16) : 0u);
  #pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t slab = ks >> 2, koff = (ks & 3) * 32u;
              const uint64_t ad = smem_desc(q_src + slab * (NROWS * 128u) + koff);
              const uint64_t bd = smem_desc(k_src + slab * (p.tk * 128u) + hv * (p.cpl * 128u) + koff);
              tc_mma(d, ad, bd, idesc, ks > 0 ? 1u : 0u);
            }
          }
          tc_commit(smem_u32(&bars.empty[s]));
          tc_commit(smem_u32(&bars.tfull[buf]));
          committed = h;
        }
      }
      if (*abort_flag != 0 && committed >= 0) {
        // gave up: leave only when the MMAs already issued have finished writing tensor memory (bounded)
        const uint32_t bar = smem_u32(&bars.tfull[committed % p.n_buf]);
        const uint32_t ph = static_cast<uint32_t>(committed / p.n_buf) & 1u;
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, ph) && clock64() - t0 < kWaitCycles) {}
      }
    }
    if (warp == kMmaWarp + 1 && p.gx) {
      // ---------------- statistics fetch warp (grid plans) ----------------
      // Per head: wait until every CTA of the request has published its pairs (a counter in global
      // memory), then copy the head's block of pairs from global memory (L2) into a statistics slot
      // with asynchronous copies that arrive on the slot's barrier - the add warps find their
      // statistics in shared memory exactly as with a cluster, and the round trips to L2 are off
      // their path.  A slot is reused once the add warps are done with the head that used it.
      pdl_wait();   // the counters belong to the workspace: an earlier call may still be resetting them
      const uint32_t target = static_cast<uint32_t>(p.cluster);   // one counted release per CTA and head
      const uint32_t slot_bytes_gx = slot_pairs * 8u;
      int ready = 0;   // heads below this one are known to be published by every CTA of the request
      for (int h = 0; h < p.H; ++h) {
        const int slot = h % p.n_slot;
        if (h >= p.n_slot) {
          const int u = h - p.n_slot;
          if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tempty[u % p.n_buf]),
                                                 static_cast<uint32_t>(u / p.n_buf) & 1u, abort_flag, wait_limit)))
            break;
        }
        const size_t bh = static_cast<size_t>(b) * p.H + h;
        if (h >= ready) {
          // one round trip tells about 32 heads: lane i looks at the counter of head h + i, and
          // the run of complete heads from h on is taken in one go
          const uint32_t* const mine = p.gx_cnt + static_cast<size_t>(b) * p.H + (h + lane < p.H ? h + lane : p.H - 1);
          const long long t0 = clock64();
          bool ok = true;
          for (;;) {
            const bool full = ld_acquire_gpu(mine) >= target;
            const unsigned not_full = __ballot_sync(0xffffffffu, !(full && h + lane < p.H));
            const int run = not_full == 0u ? 32 : __ffs(not_full) - 1;
            if (run > 0) { ready = h + run; break; }
            if (*abort_flag != 0 || clock64() - t0 > wait_limit) { *abort_flag = 1; ok = false; }
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
          }
          if (!ok) break;
        }
        const unsigned char* const src = reinterpret_cast<const unsigned char*>(p.gx_stats + bh * slot_pairs);
        const uint32_t dst = smem_u32(stats + static_cast<size_t>(slot) * slot_pairs);
        for (uint32_t off = lane * 16u; off < slot_bytes_gx; off += 32u * 16u)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + off), "l"(src + off) : "memory");
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&bars.sfull[slot])) : "memory");
      }
      asm volatile("cp.async.wait_all;" ::: "memory");   // no copy of this warp is in flight when the CTA leaves
    } else if (warp == kMmaWarp + 2 && p.gx) {
      // ---------------- publishing warp (grid plans) ----------------
      // Once all exp warps of this CTA have left their pairs of a head in shared memory: merge the
      // pairs of each row into one, store it to global memory, then one fence and one counted
      // release for the CTA - the round trip of the fence is off the exp warps' path.
      pdl_wait();   // global memory of the workspace: not before the stream's earlier work is done
      for (int h = 0; h < p.H; ++h) {
        const int buf = h % p.n_buf;
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.gsent[buf]), static_cast<uint32_t>(h / p.n_buf) & 1u,
                                               abort_flag, wait_limit)))
          break;
        const size_t bh = static_cast<size_t>(b) * p.H + h;
        float2* const dst = p.gx_stats + (bh * p.cluster + rank) * NROWS;
        for (int r = lane; r < NROWS; r += 32) {
          dst[r] = own_pairs[buf * NROWS + r];
        }
        __syncwarp();
        if (lane == 0) {
          __threadfence();
          atomicAdd(p.gx_cnt + bh, 1u);
        }
      }
    }
    if constexpr (FILTER) {
      // filter tail, TMA / MMA warps: nothing to do but to meet the others
      common_exit();
      if (cluster_gave_up()) { leave_after_give_up(ft.sel.kept_cnt); return; }
      cta_sync();   // pairs with the barrier after the selection
      return;
    }
  } else if (warp < kExpWarps) {
    // ---------------- exp warps ----------------
    if (kRealloc) asm volatile("setmaxnreg.dec.sync.aligned.u32 112;");
    const int q = warp & 3, g = warp >> 2;
    const int half = (HALVES == 2) ? (lane >> 4) : 0;
    const int row = (HALVES == 2) ? (16 * q + (lane & 15)) : (32 * q + lane);
    const uint32_t lane_addr = static_cast<uint32_t>(32 * q) << 16;
    const int total_chunks = p.cpl / kChunk;
    // chunks g, g+2, ... of every head, or all chunks of every second head (uniform per warp)
    const int my_chunks = total_chunks;
    auto chunk_of = [&](int t) { return t; };
    const int key_lane0 = static_cast<int>(rank) * p.tk + half * p.cpl;        // key of this lane's column 0
    int lim = p.causal ? (txt_start + p.row0 + row + 1) : Lb;                  // keys below lim are visible
    lim = (lim < Lb ? lim : Lb) - key_lane0;                                   // ... as a column count of this lane
    // Masking.  A lane sees the first `lim` of its columns (causal rows, end of the sequence); the
    // hidden ones are text keys or lie beyond the sequence, i.e. never columns of the output, so all
    // that matters about them is that they stay out of the row's sum.  A chunk is visible to a lane
    // in full (nothing to do), not at all (its exponents are formed with scale 0 and addend -inf,
    // and the lane's sum of that chunk is dropped), or in part: the chunks partly visible to some
    // lane of the warp - [mix_lo, mix_hi), one or two per head and only in the CTA that holds the
    // causal triangle or the end of the sequence - get their hidden logits overwritten before the loop.
    const bool partial = lim > 0 && lim < p.cpl;
    int lim_lo = partial ? lim : (1 << 30), lim_hi = partial ? lim : 0;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
      const int a = __shfl_xor_sync(0xffffffffu, lim_lo, d), c = __shfl_xor_sync(0xffffffffu, lim_hi, d);
      lim_lo = a < lim_lo ? a : lim_lo;
      lim_hi = c > lim_hi ? c : lim_hi;
    }
    // chunk c (columns 16c .. 16c + 15) is partly visible to a lane only if 16c < lim < 16c + 16
    const int mix_lo = lim_lo / kChunk;
    const int mix_hi = (lim_hi + kChunk - 1) / kChunk;
    const bool sender = (half == 0);           // with two halves, lanes s and s+16 share a row: the lower one sends
    const uint32_t pair_idx = rank * NROWS + row;                              // this thread's pair in a slot

    for (int h = g; h < p.H; h += kColGroups) {
      const int buf = h % p.n_buf;
      const uint32_t bph = static_cast<uint32_t>(h / p.n_buf) & 1u;
      const int slot = h % p.n_slot;
      if (p.tight && h >= p.tight) {
        // Few statistics slots (large clusters): stay within d = p.tight heads of the local add
        // warps.  A peer then sends for head h only after this CTA's add warps are done with head
        // h - 2d (peer at h => its add warps done with h - d => our pairs of h - d sent => ours
        // done with h - 2d), so 2d slots are enough whatever the number of buffers.
        const int u = h - p.tight;
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tempty[u % p.n_buf]),
                                               static_cast<uint32_t>(u / p.n_buf) & 1u, abort_flag, wait_limit)))
          break;
      }
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tfull[buf]), bph, abort_flag, wait_limit))) break;
      if (threadIdx.x == 0) MD_TRACE(h, 3);
      if (!p.gx && lane == 0 && q == 0) {
        // arm this head's statistics barrier with the bytes all CTAs will send
        mbar_expect_tx(smem_u32(&bars.sfull[slot]), slot_pairs * 8u);
      }
      tc_fence_after();
      const uint32_t tbuf = tmem_base + static_cast<uint32_t>(buf * p.cpl) + lane_addr;
      const uint32_t slot_addr = smem_u32(&stats[slot * slot_pairs + pair_idx]);
      const uint32_t bar_addr = smem_u32(&bars.sfull[slot]);
      // The thread's chunks go through a loop of one chunk per trip whose only taken branch is the
      // loop edge, and whose body is small: with two exp warps per scheduler nobody fills the
      // fetch bubble behind a taken branch (a loop of two chunks per trip with five or six of them
      // per trip - loop edge, jumps around the mask, the first-chunk and the rare-path code - took
      // twice the special-function unit's time), and straight-line code for all chunks of a head
      // misses the instruction cache on every head.  z takes a chunk's logits from tensor memory;
      // once they are turned into exponents in e, the next chunk's load goes out into z and runs
      // under the exponentials, the sum, the check and the store of this one.
      // The stabiliser is the maximum of the thread's FIRST chunk (shared by the two lanes of a
      // row): any value within a few dozen powers of two of the row maximum serves, because every
      // CTA sends the stabiliser it used along with its sum.  Later chunks compute no maximum:
      // should their exponentials push a chunk's sum beyond kSumLimit (extreme logits), that chunk
      // and the ones after it are not stored and not summed (predicates, no branch); after the
      // last chunk one test sends the warp through the careful path for the rest (redo_rest, out
      // of line: a maximum per chunk, stored chunks rescaled whenever the stabiliser moves).
      constexpr float kSumLimit = 1.0995116e12f;   // 2^40
      constexpr float kHidden = -3.0e38f;           // logit of a column the lane must not see (finite: 0 * kHidden = 0)
      float z[kChunk], e[kChunk];
      tc_ld16(tbuf + kChunk * chunk_of(0), z);
      float mx = -INFINITY, sub = 0.0f;
      tc_wait_ld();
      if (mix_lo < mix_hi) {
        // Chunks partly visible to some lane of this warp (the causal triangle, the end of the
        // sequence: one or two per head, and only in the CTA that holds them): the logits of the
        // hidden columns are overwritten in tensor memory with a huge negative number before the
        // loop, so that the loop itself carries no per-column mask.
#pragma unroll 1
        for (int t = 0; t < my_chunks; ++t) {
          const int c = chunk_of(t);
          if (c < mix_lo || c >= mix_hi) continue;
          const int nvis = lim - kChunk * c;
          if (t > 0) {
            tc_ld16(tbuf + kChunk * c, e);
            tc_wait_ld();
          }
#pragma unroll
          for (int j = 0; j < kChunk; ++j) e[j] = (j < nvis) ? (t > 0 ? e[j] : z[j]) : kHidden;
          tc_st16(tbuf + kChunk * c, e);
          if (t == 0) {
#pragma unroll
            for (int j = 0; j < kChunk; ++j) z[j] = e[j];
          }
        }
        tc_wait_st();
      }
      if (my_chunks > 0) {   // stabiliser from the first chunk
        float c4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        const int nvis = lim - kChunk * chunk_of(0);
#pragma unroll
        for (int j = 0; j < kChunk; ++j) c4[j & 3] = fmaxf(c4[j & 3], (j < nvis) ? z[j] : -INFINITY);
        mx = fmaxf(fmaxf(c4[0], c4[1]), fmaxf(c4[2], c4[3])) * p.scale_log2e;   // log2 units; scale > 0 keeps the order
        if (HALVES == 2) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));  // one stabiliser per row
        sub = (mx == -INFINITY) ? 0.0f : mx;   // (first chunk all masked: so are the later ones)
      }
      bool ok = true;   // warp-uniform: no chunk so far left the range
      int stored = 0;   // chunks stored (my_chunks at the end unless a sum left its range)
      float lsum = 0.0f;
#pragma unroll 1
      for (int t = 0; t < my_chunks; ++t) {
        const int c = chunk_of(t);
        const int nvis = lim - kChunk * c;                   // visible columns of this lane in this chunk
        const float sc = nvis > 0 ? p.scale_log2e : 0.0f;    // nothing visible: exponent 0 * z - inf
        const float ns = nvis > 0 ? -sub : -INFINITY;
        tc_wait_ld();
        const uint64_t sc2 = pack2(sc, sc), ns2 = pack2(ns, ns);
#pragma unroll
        for (int j = 0; j < kChunk; j += 2) unpack2(fma2(pack2(z[j], z[j + 1]), sc2, ns2), e[j], e[j + 1]);
        if (t + 1 < my_chunks) tc_ld16(tbuf + kChunk * chunk_of(t + 1), z);
        uint64_t part2[2] = {0ull, 0ull};   // (two packed zeros)
#pragma unroll
        for (int j = 0; j < kChunk; j += 2) {
          e[j] = ex2(e[j]);
          e[j + 1] = ex2(e[j + 1]);
          part2[(j >> 1) & 1] = add2(part2[(j >> 1) & 1], pack2(e[j], e[j + 1]));
        }
        float part[4];
        unpack2(part2[0], part[0], part[1]);
        unpack2(part2[1], part[2], part[3]);
        // (a lane that sees nothing of this chunk: exponent -inf unless the hidden keys hold NaN or
        // inf bits - its sum does not count either way, and what it stores lands in columns nobody reads)
        const float psum = nvis > 0 ? (part[0] + part[1]) + (part[2] + part[3]) : 0.0f;
        ok = ok && !__any_sync(0xffffffffu, !(psum < kSumLimit));   // (the first chunk's sum is at most 16)
        lsum += ok ? psum : 0.0f;
        tc_st16_if(ok, tbuf + kChunk * c, e);
        stored += ok ? 1 : 0;
      }
      if (stored < my_chunks) {   // rare
        const RedoResult r = redo_rest(tbuf, kChunk, stored, my_chunks, lim, kChunk, p.scale_log2e, HALVES == 2, mx, lsum);
        mx = r.mx;
        lsum = r.l;
      }
      if (HALVES == 2) lsum += __shfl_xor_sync(0xffffffffu, lsum, 16);
      if (p.gx) {
        // grid plan: the pair stays in this CTA's shared memory; the publishing warp merges the CTA's
        // pairs of a row and sends one pair per row on its way through global memory
        if (sender) own_pairs[buf * NROWS + row] = make_float2(mx, lsum);
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.gsent[buf]));
      } else if (sender) {
        for (int c = 0; c < p.cluster; ++c)
          st_async_f32x2(map_to_cta(slot_addr, c), mx, lsum, map_to_cta(bar_addr, c));
      }
      // Hand the head's exponentials to the add warps at once.  (The wait for the stores runs under
      // the other group's loop.  Handing over only when the group gets to its next head - two heads
      // on - saves that wait but measured the same, and with two buffers that next head needs the
      // very buffer: its MMAs wait for the add warps, who wait for the hand-over.)
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars.eready[buf]));
      if (threadIdx.x == 0) MD_TRACE(h, 4);
    }
    if constexpr (FILTER) {
      // filter tail, exp warps: selection of this request.  Dynamic shared memory is free by now:
      // all copies have landed, all MMAs have read them and every statistics pair sent to this CTA
      // has been consumed.  Each CTA of the cluster runs the same selection on its own (identical
      // inputs, fixed order: identical lists); rank 0 stores the list.
      __shared__ SelectShared sel_sh;
      common_exit();
      if (cluster_gave_up()) { leave_after_give_up(ft.sel.kept_cnt); return; }
      pdl_wait();   // the outputs written below may still be read by an earlier kernel in the stream
      filter_select(ft.sel, sel_sh, b, threadIdx.x, rank == 0, kept_list, &kept_total_s);
      if (threadIdx.x == 0) MD_TRACE(0, 12);   // selection done
      cta_sync();   // the list is complete: the copy thread may start
      return;
    }
  } else {
    // ---------------- add warps ----------------
    if (kRealloc) asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    const int q = warp & 3;
    const int half = (HALVES == 2) ? (lane >> 4) : 0;
    const int row = (HALVES == 2) ? (16 * q + (lane & 15)) : (32 * q + lane);
    const uint32_t lane_addr = static_cast<uint32_t>(32 * q) << 16;
    const int total_chunks = p.cpl / kChunk;
    const int tid_a = threadIdx.x - kExpThreads;

    uint64_t acc[ACH][kChunk / 2];   // head sums, two columns per register pair
#pragma unroll
    for (int c = 0; c < ACH; ++c)
#pragma unroll
      for (int j = 0; j < kChunk / 2; ++j) acc[c][j] = 0ull;
    // PH: this thread's keys tid_a, tid_a + 128, ... of the CTA: running sum over heads of the per-head maxima
    constexpr int PHK = (ACH * kChunk * HALVES + kAddThreads - 1) / kAddThreads;
    float ph_acc[PHK];
#pragma unroll
    for (int x = 0; x < PHK; ++x) ph_acc[x] = 0.0f;
    const bool real_row = row < p.N;     // lanes beyond the text rows carry padding

    int h = 0;
    for (; h < p.H; ++h) {
      const int buf = h % p.n_buf;
      const uint32_t bph = static_cast<uint32_t>(h / p.n_buf) & 1u;
      const int slot = h % p.n_slot;
      const uint32_t sph = static_cast<uint32_t>(h / p.n_slot) & 1u;
      float f;                                 // factor of this CTA's exponentials of the row
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.sfull[slot]), sph, abort_flag, wait_limit))) break;
      if (tid_a == 0) MD_TRACE(h, 5);
      if (p.gx) {
        // grid plan: one merged pair per CTA in the slot; this CTA's own stabilisers are still in
        // its shared memory (until the buffer is released below)
        const float2* srow = stats + slot * slot_pairs + row;
        float m = -INFINITY;
        for (int c = 0; c < p.cluster; ++c) m = fmaxf(m, srow[c * NROWS].x);
        float l = 0.0f;
        for (int c = 0; c < p.cluster; ++c) {
          const float2 v = srow[c * NROWS];
          l = fmaf(v.y, ex2(v.x - m), l);
        }
        const float inv_l = 1.0f / l;
        f = ex2(own_pairs[buf * NROWS + row].x - m) * inv_l;
      } else {
        // statistics of this row over the whole key range: every CTA's pairs
        const float2* srow = stats + slot * slot_pairs + row;
        float m = -INFINITY;
        for (int c = 0; c < p.cluster; ++c) m = fmaxf(m, srow[c * NROWS].x);
        float l = 0.0f;
        for (int c = 0; c < p.cluster; ++c) {
          const float2 v = srow[c * NROWS];
          l = fmaf(v.y, ex2(v.x - m), l);     // an empty pair is (-inf, 0): contributes 0
        }
        const float inv_l = 1.0f / l;
        f = ex2(srow[rank * NROWS].x - m) * inv_l;
      }
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.eready[buf]), bph, abort_flag, wait_limit))) break;
      if (tid_a == 0) MD_TRACE(h, 6);
      tc_fence_after();
      const uint32_t tbuf = tmem_base + static_cast<uint32_t>(buf * p.cpl) + lane_addr;
#pragma unroll
      for (int c0 = 0; c0 < ACH; c0 += 2) {
        if (c0 < total_chunks) {
          float e[2][kChunk];
          tc_ld16(tbuf + kChunk * c0, e[0]);
          if (c0 + 1 < ACH && c0 + 1 < total_chunks) tc_ld16(tbuf + kChunk * (c0 + 1), e[1]);
          tc_wait_ld();
          const uint64_t f_2 = pack2(f, f);
#pragma unroll
          for (int j = 0; j < kChunk; j += 2) acc[c0][j >> 1] = fma2(pack2(e[0][j], e[0][j + 1]), f_2, acc[c0][j >> 1]);
          if (c0 + 1 < ACH && c0 + 1 < total_chunks) {
#pragma unroll
            for (int j = 0; j < kChunk; j += 2)
              acc[c0 + 1][j >> 1] = fma2(pack2(e[1][j], e[1][j + 1]), f_2, acc[c0 + 1][j >> 1]);
          }
          if constexpr (PH) {
            // Column maxima over this warp's text rows (the lanes): recursive halving - in each of
            // four steps a lane keeps half of its columns and takes its partner's maxima for them,
            // so that lane j of a 16-lane group ends up with column j's maximum over the group.  The
            // probabilities travel as fp16 pairs (two columns per register: half the shuffles,
            // selects and maxima), scaled by 2^14 so that nothing above 4e-9 is subnormal; rounding
            // them costs 2^-11 relative, a quarter of the score tolerance.  With 128 text rows the
            // two 16-lane groups of a warp hold the same columns and are folded first.
            float* const dst = ph_stage + ((h & 1) * kAddWarps + q) * p.tk + half * p.cpl + (lane & 15);
            auto hmax2 = [](uint32_t a, uint32_t b2) {
              uint32_t r;
              asm("max.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b2));
              return r;
            };
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              if (c0 + x < ACH && c0 + x < total_chunks) {
                const float fx = real_row ? f * kPhScale : 0.0f;
                const uint64_t fx2 = pack2(fx, fx);
                uint32_t hv[kChunk / 2];
#pragma unroll
                for (int k = 0; k < kChunk / 2; ++k) {
                  float lo, hi;
                  unpack2(mul2(pack2(e[x][2 * k], e[x][2 * k + 1]), fx2), lo, hi);
                  const __half2 t = __floats2half2_rn(lo, hi);   // (lo, hi) = columns 2k, 2k + 1
                  hv[k] = *reinterpret_cast<const uint32_t*>(&t);
                }
                if (HALVES == 1) {
#pragma unroll
                  for (int k = 0; k < kChunk / 2; ++k) hv[k] = hmax2(hv[k], __shfl_xor_sync(0xffffffffu, hv[k], 16));
                }
#pragma unroll
                for (int step = kChunk / 4; step >= 1; step >>= 1) {   // registers apart: 8, 4, 2 columns
                  const bool upper = (lane & (2 * step)) != 0;
#pragma unroll
                  for (int i = 0; i < step; ++i) {
                    const uint32_t give = upper ? hv[i] : hv[i + step];
                    const uint32_t keep = upper ? hv[i + step] : hv[i];
                    hv[i] = hmax2(keep, __shfl_xor_sync(0xffffffffu, give, 2 * step));
                  }
                }
                // the last step is inside the register: even lanes end with its low half, odd ones with its high half
                const uint32_t r2 = hmax2(hv[0], __shfl_xor_sync(0xffffffffu, hv[0], 1));
                const unsigned short bits = static_cast<unsigned short>((lane & 1) ? (r2 >> 16) : (r2 & 0xffffu));
                if (HALVES == 2 || lane < 16) dst[kChunk * (c0 + x)] = __half2float(__ushort_as_half(bits));
              }
            }
          }
        }
      }
      if constexpr (PH) {
        // the four warps' maxima of this head meet; each thread adds the maximum of its keys
        mbar_arrive(smem_u32(&bars.ph));
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.ph), static_cast<uint32_t>(h) & 1u, abort_flag, wait_limit))) break;
        const float* const src = ph_stage + (h & 1) * kAddWarps * p.tk;
#pragma unroll
        for (int x = 0; x < PHK; ++x) {
          const int key = tid_a + x * kAddThreads;
          if (key < p.tk)
            ph_acc[x] += fmaxf(fmaxf(src[key], src[p.tk + key]), fmaxf(src[2 * p.tk + key], src[3 * p.tk + key]));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars.tempty[buf]));
      if (tid_a == 0) MD_TRACE(h, 7);
    }

    // head mean -> column sum (Eq. 8) and column max (Eq. 10) over the text rows
    mbar_arrive(smem_u32(&bars.fin));
    if (__all_sync(0xffffffffu, h == p.H && mbar_wait(smem_u32(&bars.fin), 0u, abort_flag, wait_limit))) {
      // all TMA copies have landed and all MMAs have read them: the staging area is free
      float* mat = reinterpret_cast<float*>(stage_ptr);
      const int ld = p.tk | 1;
      if (row < p.N) {
#pragma unroll
        for (int c = 0; c < ACH; ++c) {
          if (c < total_chunks) {
            const int key_local = half * p.cpl + kChunk * c;
#pragma unroll
            for (int j = 0; j < kChunk; j += 2) unpack2(acc[c][j >> 1], mat[row * ld + key_local + j], mat[row * ld + key_local + j + 1]);
          }
        }
      }
      mbar_arrive(smem_u32(&bars.fin));
      const bool staged = mbar_wait(smem_u32(&bars.fin), 1u, abort_flag, wait_limit);
      pdl_wait();
      for (int c = tid_a, x = 0; staged && c < p.tk; c += kAddThreads, ++x) {
        const int j = static_cast<int>(rank) * p.tk + c - p.vis_start;   // vision-relative index
        if (j < 0 || j >= p.M) continue;
        float s = 0.0f, mx = -INFINITY;
        for (int r = 0; r < p.N; ++r) {
          const float v = mat[r * ld + c];
          s += v;
          mx = fmaxf(mx, v);
        }
        if constexpr (PH) {
          mx = 0.0f;   // (x < PHK always; a compile-time unrolled pick keeps ph_acc in registers)
#pragma unroll
          for (int y = 0; y < PHK; ++y) mx = (y == x) ? ph_acc[y] : mx;
          mx *= 1.0f / kPhScale;
        }
        const bool present = j < Mb;    // beyond the request's own tokens: zeros
        float gv = present ? s * p.inv_heads : 0.0f, iv = present ? mx * p.inv_heads : 0.0f;
        if (p.combine) {                // the text rows before row0 were scored by the launch before this one
          gv += p.g_out[static_cast<size_t>(b) * p.M + j];
          iv = fmaxf(iv, p.i_out[static_cast<size_t>(b) * p.M + j]);
        }
        p.g_out[static_cast<size_t>(b) * p.M + j] = gv;
        p.i_out[static_cast<size_t>(b) * p.M + j] = iv;
      }
      if (tid_a == 0) MD_TRACE(0, 10);     // scores stored
    }
    if constexpr (FILTER) {
      // filter tail, add warps: row r of the compacted outputs is copied by CTA r mod cluster
      common_exit();
      if (cluster_gave_up()) { leave_after_give_up(ft.sel.kept_cnt); return; }
      pdl_wait();
      cta_sync();   // the exp warps have finished the selection
      if (warp == kExpWarps && lane == 0) {
        filter_gather(ft, gm, bars.gfull, abort_flag, kept_list, kept_total_s, stage_base, static_cast<int>(rank), b, Mb,
                      p.cluster, p.workspace);
        MD_TRACE(0, 13);   // gather done
      }
      return;
    }
  }

  common_exit();   // (score-only kernel; the filter kernel's roles have left above)
  if (cluster_gave_up()) leave_after_give_up(nullptr);
}

// ---- host side ------------------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// bf16 tensor [d3][d2][d1][128] with byte strides s1, s2, s3; box = 64 x rows x 1 x 1, 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* base, uint64_t d1, uint64_t d2, uint64_t d3, uint64_t s1, uint64_t s2,
              uint64_t s3, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[4] = {128, d1, d2, d3};
  const cuuint64_t strides[3] = {s1, s2, s3};
  const cuuint32_t box[4] = {64, box_rows, 1, 1};
  const cuuint32_t elem[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 tensor [d3][d2][d1][128] with byte strides s1, s2, s3, no swizzle; box = 128 x 1 x d2 x 1:
// one token's 256-byte pieces over all heads.
bool make_gather_map(CUtensorMap* map, const void* base, uint64_t d1, uint64_t d2, uint64_t d3, uint64_t s1,
                     uint64_t s2, uint64_t s3) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[4] = {128, d1, d2, d3};
  const cuuint64_t strides[3] = {s1, s2, s3};
  const cuuint32_t box[4] = {128, 1, static_cast<cuuint32_t>(d2), 1};
  const cuuint32_t elem[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Encoded tensor maps of recent calls, kept with the plan: a steady-state call with pointers it
// has seen before (a serving loop cycles through a few buffer sets) encodes nothing.
struct MapCache {
  struct ScoreEntry { const void* q; const void* k; int geo; CUtensorMap q_map, k_map; };
  struct GatherEntry { const void* k; const void* v; const void* k_out; const void* v_out; GatherMaps maps; };
  static constexpr int kEntries = 16;
  std::mutex mu;
  ScoreEntry score[kEntries];
  GatherEntry gather[kEntries];
  int n_score = 0, n_gather = 0, next_score = 0, next_gather = 0;
};

MapCache* map_cache_create() { return new (std::nothrow) MapCache(); }
void map_cache_destroy(MapCache* c) { delete c; }

namespace {

using FusedKernel = void (*)(const CUtensorMap, const CUtensorMap, const FusedParams, const GatherMaps, const FilterTail);

template <bool FILTER, bool PH>
FusedKernel pick_shape(int halves, int ach) {
  if (halves == 2) return ach > 5 ? score_fused_kernel<2, 10, FILTER, PH> : score_fused_kernel<2, 5, FILTER, PH>;
  if (ach > 10) return score_fused_kernel<1, 11, FILTER, PH>;   // 176 columns per lane (one M=128 tile only)
  return ach > 5 ? score_fused_kernel<1, 10, FILTER, PH> : score_fused_kernel<1, 5, FILTER, PH>;
}

FusedKernel pick_kernel(int halves, int ach, bool filter = false, bool per_head = false) {
  if (filter) return per_head ? pick_shape<true, true>(halves, ach) : pick_shape<true, false>(halves, ach);
  return per_head ? pick_shape<false, true>(halves, ach) : pick_shape<false, false>(halves, ach);
}

// Clusters of `cluster` CTAs that can be resident at once (GPC boundaries make this less than
// SMs / cluster); 0 when it cannot be asked (no device) or the shape cannot launch.
int max_resident_clusters(int halves, int ach, int cluster, size_t smem_bytes, bool per_head) {
  FusedKernel kernel = pick_kernel(halves, ach, false, per_head);
  if (ensure_kernel_attributes(reinterpret_cast<const void*>(kernel), true) != cudaSuccess) {
    (void)cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(cluster));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) {
    (void)cudaGetLastError();
    return 0;
  }
  return n;
}

}  // namespace

// Geometry of the fused kernel for a problem; false when the shape is outside what it covers.
// row0 / n_rows: the text rows the launch covers (n_rows = 0: all of them); max_cluster: an upper
// limit on the cluster size (0: none).
bool plan_score_fused(const Resolved& r, int sm_count, int forced_cluster, FusedGeometry* out, int row0, int n_rows,
                      int max_cluster) {
  if (n_rows <= 0) { row0 = 0; n_rows = r.N; }
  const int halves = n_rows <= 64 ? 2 : 1;
  const int nrows = 128 / halves;
  // columns per TMEM lane: 160 (add threads with 10 chunks); 176 with one M=128 tile, where an
  // eleventh chunk per add thread still fits its registers and saves a whole round of clusters
  // for 128 text rows on 704 keys (4 CTAs per request instead of 5)
  const int max_cpl = (halves == 1 ? 11 : 10) * kChunk;
  double best = -1.0;
  FusedGeometry g{};
  for (int c = 1; c <= kMaxCluster; ++c) {
    if (forced_cluster > 0 && c != forced_cluster) continue;
    if (max_cluster > 0 && c > max_cluster) continue;
    const int per_cta = (r.L + c - 1) / c;
    int cpl = (per_cta + halves - 1) / halves;
    cpl = (cpl + kChunk - 1) / kChunk * kChunk;
    if (cpl > max_cpl) continue;
    const int tk = cpl * halves;
    const size_t stage = static_cast<size_t>(nrows + tk) * 256;
    const int ach = cpl <= 5 * kChunk ? 5 : (cpl <= 10 * kChunk ? 10 : 11);   // chunks per add thread (kernel variant)
    // slot size in pairs per row and CTA.  The kernel sends ONE pair per row; wide tiles keep the room for
    // two that they had when the two exp warps of a quadrant shared a head: the cost model's constants and
    // every measured plan choice rest on the stage / buffer / slot counts that this sizing gives.
    const int epr = ach <= 5 ? 1 : kColGroups;
    // Shared memory.  Whole stages first (a head's query tile and keys recycled together): as many
    // tensor-memory buffers as the columns allow (3..8), fewer if their statistics slots (2 x
    // buffers x cluster x rows x pairs x 8 bytes) would leave no room for 2 stages; four stages
    // are preferred over more buffers.  If even three buffers' slots do not fit (large clusters):
    // 2d slots with the exp warps held within d heads of the add warps (d = 2, else 1) - and for
    // those the split layout (two query tiles + a ring of key half-tiles, which needs less
    // memory for the same look-ahead) is tried as well and taken when it allows a wider window.
    const size_t q_tile = static_cast<size_t>(nrows) * 256, k_half = static_cast<size_t>(cpl) * 256;
    // the per-head reading of Eq. 10 stages each add warp's column maxima: 2 heads x 4 warps x tk floats
    const size_t ph_bytes = r.per_head_max ? static_cast<size_t>(2 * kAddWarps) * tk * sizeof(float) : 0;
    const size_t avail = 227 * 1024 - 4096 /* static */ - 1024 /* alignment */ - ph_bytes;
    auto slots_bytes = [&](int n_slot) { return static_cast<size_t>(n_slot) * c * nrows * epr * 8; };
    int n_buf = kTmemCols / cpl;
    if (n_buf > kMaxBufs) n_buf = kMaxBufs;
    const int min_bufs = cpl > 10 * kChunk ? 2 : kMinBufs;   // 176-column tiles: two buffers is all that fits
    if (n_buf < min_bufs) continue;
    const int max_buf = n_buf;
    size_t extra = 0;
    int n_q = 0, n_k = 0, n_slot = 0, split = 0;
    {                                              // whole stages, full set of slots
      // a stage is held for a load latency plus an MMA: as many stages as fit (up to four) first,
      // then as many buffers as still fit (the MMA -> exp -> exchange -> add chain of ~4.6 us
      // per head is spread over them)
      int best_q = 0, best_buf = 0;
      for (int nb = max_buf; nb >= min_bufs; --nb) {
        const size_t e = slots_bytes(2 * nb);
        if (e + 2 * stage > avail) continue;
        int q = static_cast<int>((avail - e) / stage);
        if (q > 4) q = 4;
        if (q > best_q) { best_q = q; best_buf = nb; }
      }
      n_q = best_q;
      if (best_q >= 2) { n_buf = best_buf; n_slot = 2 * n_buf; extra = slots_bytes(n_slot); }
    }
    if (n_q < 2) {                                 // tight windows
      n_buf = max_buf;
      int best_d = 0;
      for (int d = 2; d >= 1 && best_d == 0; --d) {
        const size_t e = slots_bytes(2 * d);
        if (e + 2 * stage <= avail) {              // whole stages
          best_d = d; split = 0; extra = e; n_slot = 2 * d;
          n_q = static_cast<int>((avail - e) / stage);
        } else if (e + 2 * q_tile + (halves + 1) * k_half <= avail) {   // split rings
          best_d = d; split = 1; extra = e; n_slot = 2 * d;
          n_q = 2;
          n_k = static_cast<int>((avail - e - 2 * q_tile) / k_half);
          if (n_k > 4 * halves) n_k = 4 * halves;
        }
      }
      if (best_d == 0) continue;
    }
    if (n_q > 4) n_q = 4;
    // Cost model (microseconds per head and CTA): streaming the stage at ~45 GB/s per SM, or the
    // MMA -> exp -> exchange -> add chain (~4.5 us) spread over the buffers, whichever is longer;
    // times the number of waves of CTAs.
    size_t smem_bytes = (split ? n_q * q_tile + n_k * k_half : n_q * stage) + 1024 + extra + ph_bytes;
    // at least 116 KB, so that two CTAs (each wanting all of tensor memory) never share an SM
    if (smem_bytes < 116 * 1024) smem_bytes = 116 * 1024;
    int resident = max_resident_clusters(halves, ach, c, smem_bytes, r.per_head_max != 0);
    if (resident <= 0 && c <= 8) resident = sm_count / c;    // no device to ask: ignore GPC boundaries
    // (a cluster of more than 8 CTAs is used only where the device says it can hold one)
    if (resident <= 0) continue;
    const long waves = (r.B + resident - 1) / resident;
    const double t_stream = static_cast<double>(stage) / 45.0e3;
    double t_chain = 4.5 / n_buf + 0.02 * c;   // the statistics exchange grows with the cluster
    if (n_slot < 2 * n_buf) {
      // Tight slots: the exchange over the cluster is on the critical path of every head (d = 2)
      // or of every head twice (d = 1).  Measured per head: 2.6 .. 3.3 us at 11 .. 16 CTAs with
      // d = 2, 4.3 us at 10 CTAs with d = 1; a third more with 128 text rows on the lanes.
      t_chain = (n_slot == 4 ? 1.8 + 0.09 * c : 3.0 + 0.13 * c) * (halves == 1 ? 1.3 : 1.0);
    }
    double t_head = t_stream > t_chain ? t_stream : t_chain;
    if (t_head < 1.4) t_head = 1.4;   // the exp stage and its hand-overs take that long per head however narrow the tile
    // among equals: larger clusters while all of them are resident at once (a call by itself gains
    // from spreading its keys over more SMs: measured 62 against 66 us at 16 requests), else smaller ones
    const double tie = (waves == 1) ? 1e-4 * c : -1e-4 * c;
    const double score = 1.0 / (static_cast<double>(waves) * t_head) + tie;
    if (score > best) {
      best = score;
      g.halves = halves; g.cluster = c; g.tk = tk; g.cpl = cpl; g.n_q = n_q; g.n_k = n_k; g.split = split; g.n_buf = n_buf; g.ach = ach;
      g.n_slot = n_slot; g.resident = resident; g.row0 = row0; g.n_rows = n_rows;
      g.est_us = static_cast<float>(waves * r.H * t_head);
      g.smem_bytes = smem_bytes;
    }
  }
  if (best < 0.0) return false;
  *out = g;
  return true;
}

// Grid plan: G CTAs per request with B * G <= SMs, so that every CTA of the batch is resident at
// once (one CTA per SM: each asks for more than half of the shared memory) and no request waits
// for a CTA that has not started.  The statistics of a head cross through global memory (L2).
bool plan_score_grid(const Resolved& r, int sm_count, int forced_ctas, FusedGeometry* out) {
  const int halves = r.N <= 64 ? 2 : 1;
  const int nrows = 128 / halves;
  const int max_g = sm_count / r.B < 32 ? sm_count / r.B : 32;
  double best = -1.0;
  FusedGeometry g{};
  for (int c = 2; c <= max_g; ++c) {
    if (forced_ctas > 0 && c != forced_ctas) continue;
    const int per_cta = (r.L + c - 1) / c;
    int cpl = (per_cta + halves - 1) / halves;
    cpl = (cpl + kChunk - 1) / kChunk * kChunk;
    if (cpl > 10 * kChunk) continue;
    const int tk = cpl * halves;
    if (static_cast<long>(c - 1) * tk >= r.L) continue;       // a CTA without keys
    const size_t stage = static_cast<size_t>(nrows + tk) * 256;
    const int ach = cpl <= 5 * kChunk ? 5 : 10;
    const size_t ph_bytes = r.per_head_max ? static_cast<size_t>(2 * kAddWarps) * tk * sizeof(float) : 0;
    const size_t avail = 227 * 1024 - 4096 - 1024 - ph_bytes;
    int n_buf = kTmemCols / cpl;
    if (n_buf > kMaxBufs) n_buf = kMaxBufs;
    if (n_buf < kMinBufs) continue;
    // shared memory: statistics slots the fetch warp fills (a head's pairs of all the request's
    // CTAs; at least two, so that the next head's are fetched while this one is added) and stages
    const int epr = ach <= 5 ? 1 : kColGroups;   // (room for two pairs per row on wide tiles: see plan_score_fused)
    const size_t slot = static_cast<size_t>(c) * nrows * 8;                 // one merged pair per row and CTA
    const size_t own = static_cast<size_t>(n_buf) * nrows * epr * 8;        // the CTA's own pairs, per buffer
    if (avail < own + 2 * slot + 2 * stage) continue;
    int n_q = static_cast<int>((avail - own - 2 * slot) / stage);
    if (n_q > 3) n_q = 3;
    // (No more slots than buffers: the fetch warp learns that a slot is free from the buffer barrier
    // of the head that used it, by parity; were it n_buf heads behind the add warps, that barrier
    // could complete a second phase unseen.)
    int n_slot = static_cast<int>((avail - own - n_q * stage) / slot);
    if (n_slot > 6) n_slot = 6;
    if (n_slot > n_buf) n_slot = n_buf;
    size_t smem_bytes = n_q * stage + n_slot * slot + own + 1024 + ph_bytes;
    if (smem_bytes < 116 * 1024) smem_bytes = 116 * 1024;
    // Cost per head and CTA (microseconds): streaming the stage at ~45 GB/s per SM; the exp stage
    // (measured: ~0.011 us per column of a lane, two heads at a time on narrow tiles); the
    // MMA -> exp -> exchange through L2 -> add chain (~6 us) spread over the buffers.
    const double t_stream = static_cast<double>(stage) / 45.0e3;
    const double t_exp = (ach <= 5 ? 0.0075 : 0.011) * cpl + 0.2;
    const double t_chain = 6.0 / n_buf;
    double t_head = t_stream > t_exp ? t_stream : t_exp;
    if (t_chain > t_head) t_head = t_chain;
    if (t_head < 1.4) t_head = 1.4;
    const double score = 1.0 / t_head + 1e-4 * c;
    if (score > best) {
      best = score;
      g.halves = halves; g.cluster = c; g.tk = tk; g.cpl = cpl; g.n_q = n_q; g.n_k = 0; g.split = 0; g.n_buf = n_buf;
      g.ach = ach; g.n_slot = n_slot; g.gx = 1; g.resident = sm_count; g.row0 = 0; g.n_rows = r.N;
      g.est_us = static_cast<float>(r.H * t_head + 12.0);    // (+ filling and draining the longer chain)
      g.smem_bytes = smem_bytes;
    }
  }
  if (best < 0.0) return false;
  *out = g;
  return true;
}

size_t grid_plan_stats_bytes(const Resolved& r, const FusedGeometry& g) {
  const int nrows = 128 / g.halves;
  return static_cast<size_t>(r.B) * r.H * g.cluster * nrows * sizeof(float2);   // one merged pair per row, CTA and head
}

namespace {

// Common launch of the score kernel, with (tail != nullptr) or without the selection / gather tail.
cudaError_t launch_fused_common(const mustdrop_plan& plan, const FusedGeometry& geo, bool combine, const void* q_text,
                                const void* k, float* g_out, float* i_out, void* workspace, const GatherMaps* maps,
                                const FilterTail* tail, size_t smem_bytes, cudaStream_t stream,
                                const int32_t* vis_cnt) {
  const Resolved& r = plan.r;
  const int nrows = 128 / geo.halves;
  CUtensorMap q_map, k_map;
  // the launch's text rows: a window of geo.n_rows rows starting at geo.row0 of every head's N rows
  const unsigned char* q_rows = static_cast<const unsigned char*>(q_text) + static_cast<size_t>(geo.row0) * 256;
  const int geo_id = (&geo == &plan.fused_b) ? 1 : 0;
  bool cached = false;
  if (MapCache* mc = plan.map_cache) {
    std::lock_guard<std::mutex> lock(mc->mu);
    for (int x = 0; x < mc->n_score && !cached; ++x)
      if (mc->score[x].q == q_rows && mc->score[x].k == k && mc->score[x].geo == geo_id) {
        q_map = mc->score[x].q_map;
        k_map = mc->score[x].k_map;
        cached = true;
      }
  }
  if (!cached) {
    if (!make_map(&q_map, q_rows, geo.n_rows, r.H, r.B, 256, static_cast<uint64_t>(r.N) * 256,
                  static_cast<uint64_t>(r.H) * r.N * 256, nrows) ||
        !make_map(&k_map, k, r.L, r.H, r.B, static_cast<uint64_t>(r.k_sl) * 2, static_cast<uint64_t>(r.k_sh) * 2,
                  static_cast<uint64_t>(r.k_sb) * 2, geo.cpl))
      return cudaErrorInvalidValue;
    if (MapCache* mc = plan.map_cache) {
      std::lock_guard<std::mutex> lock(mc->mu);
      MapCache::ScoreEntry& en = mc->score[mc->next_score];
      en.q = q_rows; en.k = k; en.geo = geo_id; en.q_map = q_map; en.k_map = k_map;
      mc->next_score = (mc->next_score + 1) % MapCache::kEntries;
      if (mc->n_score < MapCache::kEntries) ++mc->n_score;
    }
  }
  FusedParams p;
  p.g_out = g_out; p.i_out = i_out; p.workspace = workspace;
  p.vis_cnt = vis_cnt;
  p.H = r.H; p.N = geo.n_rows; p.L = r.L; p.M = r.M; p.vis_start = r.vis_start; p.txt_start = r.txt_start;
  p.causal = r.causal;
  p.n_txt = r.N; p.row0 = geo.row0; p.combine = combine ? 1 : 0;
  p.cluster = geo.cluster; p.tk = geo.tk; p.cpl = geo.cpl; p.n_q = geo.n_q; p.n_k = geo.n_k; p.split = geo.split;
  p.n_buf = geo.n_buf; p.n_slot = geo.n_slot; p.tight = (!geo.gx && geo.n_slot < 2 * geo.n_buf) ? geo.n_slot / 2 : 0;
  p.gx = geo.gx;
  p.gx_cnt = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(workspace) + plan.ws_gx_cnt_off);
  p.gx_stats = reinterpret_cast<float2*>(static_cast<unsigned char*>(workspace) + plan.ws_gx_stats_off);
  p.per_head = r.per_head_max;
  p.early_inputs = (r.inputs_ready && vis_cnt == nullptr) ? 1 : 0;
  p.wait_cycles = r.wait_cycles > 0 ? r.wait_cycles : kWaitCycles;
  p.scale_log2e = r.scale_log2e;
  p.inv_heads = 1.0f / static_cast<float>(r.H);

  FusedKernel kernel = pick_kernel(geo.halves, geo.ach, tail != nullptr, r.per_head_max != 0);
  cudaError_t e = ensure_kernel_attributes(reinterpret_cast<const void*>(kernel), true);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(r.B * geo.cluster));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = geo.gx ? 1u : static_cast<unsigned>(geo.cluster);   // grid plans: no cluster
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  static const GatherMaps no_maps = {};
  static const FilterTail no_tail = {};
  return cudaLaunchKernelEx(&cfg, kernel, q_map, k_map, p, maps ? *maps : no_maps, tail ? *tail : no_tail);
}

}  // namespace

cudaError_t launch_score_fused(const mustdrop_plan& plan, const void* q_text, const void* k, float* g_out,
                               float* i_out, void* workspace, cudaStream_t stream, const int32_t* vis_cnt) {
  cudaError_t e = launch_fused_common(plan, plan.fused, false, q_text, k, g_out, i_out, workspace, nullptr, nullptr,
                                      plan.fused.smem_bytes, stream, vis_cnt);
  if (e != cudaSuccess || !plan.row_split) return e;
  // the remaining text rows: same keys again, results combined with the first launch's
  return launch_fused_common(plan, plan.fused_b, true, q_text, k, g_out, i_out, workspace, nullptr, nullptr,
                             plan.fused_b.smem_bytes, stream, vis_cnt);
}

// Shared-memory plan of the gather tail; false when a row does not fit the ring at least three times.
bool plan_filter_single(const Resolved& r, const FusedGeometry& geo, FilterGeometry* out) {
  if (r.H > 256) return false;                                     // box of the per-token K / V copy
  const size_t hidden_pad = (static_cast<size_t>(r.hidden) * 2 + 127) / 128 * 128;
  const size_t slot = hidden_pad + 2 * static_cast<size_t>(r.H) * 256;
  const size_t limit = 227 * 1024 - 4096;                          // dynamic shared memory a CTA may ask for
  const size_t fixed = 1024 + kKeptListBytes;
  size_t want = fixed + kMaxGatherSlots * slot;
  if (want < geo.smem_bytes) want = geo.smem_bytes;
  if (want > limit) want = limit;
  if (want < geo.smem_bytes) return false;
  int n_slot = static_cast<int>((want - fixed) / slot);
  if (n_slot > kMaxGatherSlots) n_slot = kMaxGatherSlots;
  if (n_slot < 3) return false;
  out->smem_bytes = want;
  out->slot_bytes = static_cast<int32_t>(slot);
  out->n_slot = n_slot;
  return true;
}

cudaError_t launch_filter_fused(const mustdrop_plan& plan, const void* q_text, const void* k, const void* v,
                                const void* hidden, const int32_t* key_idx, const int32_t* key_cnt, float* g_out,
                                float* i_out, float* s_out, int32_t* kept_idx, int32_t* kept_cnt, void* hidden_out,
                                void* k_out, void* v_out, void* workspace, cudaStream_t stream, const LayerArgs& la) {
  const Resolved& r = plan.r;
  GatherMaps maps = {};
  const uint64_t out_s1 = 256, out_s2 = static_cast<uint64_t>(r.out_rows) * 256, out_s3 = static_cast<uint64_t>(r.H) * out_s2;
  const void* const gk = k_out != nullptr ? k : nullptr;   // the sources matter only where their output is given
  const void* const gv = v_out != nullptr ? v : nullptr;
  bool cached = false;
  if (MapCache* mc = plan.map_cache) {
    std::lock_guard<std::mutex> lock(mc->mu);
    for (int x = 0; x < mc->n_gather && !cached; ++x) {
      const MapCache::GatherEntry& en = mc->gather[x];
      if (en.k == gk && en.v == gv && en.k_out == k_out && en.v_out == v_out) {
        maps = en.maps;
        cached = true;
      }
    }
  }
  if (!cached) {
    if (k_out != nullptr &&
        (!make_gather_map(&maps.k_src, k, r.L, r.H, r.B, static_cast<uint64_t>(r.k_sl) * 2,
                          static_cast<uint64_t>(r.k_sh) * 2, static_cast<uint64_t>(r.k_sb) * 2) ||
         !make_gather_map(&maps.k_dst, k_out, r.out_rows, r.H, r.B, out_s1, out_s2, out_s3)))
      return cudaErrorInvalidValue;
    if (v_out != nullptr &&
        (!make_gather_map(&maps.v_src, v, r.L, r.H, r.B, static_cast<uint64_t>(r.v_sl) * 2,
                          static_cast<uint64_t>(r.v_sh) * 2, static_cast<uint64_t>(r.v_sb) * 2) ||
         !make_gather_map(&maps.v_dst, v_out, r.out_rows, r.H, r.B, out_s1, out_s2, out_s3)))
      return cudaErrorInvalidValue;
    if (MapCache* mc = plan.map_cache) {
      std::lock_guard<std::mutex> lock(mc->mu);
      MapCache::GatherEntry& en = mc->gather[mc->next_gather];
      en.k = gk; en.v = gv; en.k_out = k_out; en.v_out = v_out; en.maps = maps;
      mc->next_gather = (mc->next_gather + 1) % MapCache::kEntries;
      if (mc->n_gather < MapCache::kEntries) ++mc->n_gather;
    }
  }
  FilterTail t = {};
  t.sel.g = g_out; t.sel.i = i_out; t.sel.key_idx = key_idx; t.sel.key_cnt = key_cnt;
  t.sel.kept_idx = kept_idx; t.sel.kept_cnt = kept_cnt; t.sel.s_out = s_out; t.sel.workspace = workspace;
  t.sel.M = r.M; t.sel.key_max = r.key_max; t.sel.mode = r.mode; t.sel.criteria = r.criteria;
  t.sel.budget = r.budget; t.sel.cap = r.cap; t.sel.gamma = r.gamma; t.sel.alpha = r.alpha;
  t.sel.vis_cnt = la.vis_cnt; t.sel.orig_in = la.orig_in; t.sel.orig_out = la.orig_out;
  t.sel.key_idx_out = la.key_idx_out; t.sel.key_cnt_out = la.key_cnt_out;
  t.sel.vis_start = r.vis_start; t.sel.N = r.N;
  t.sel.gamma_default = r.gamma_default; t.sel.alpha_default = r.alpha_default;
  t.rebuild = r.rebuild; t.N = r.N; t.out_rows = r.out_rows;
  t.hidden = static_cast<const unsigned char*>(hidden);
  t.hidden_out = static_cast<unsigned char*>(hidden_out);
  t.hid_sb = r.hid_sb * 2; t.hid_sl = r.hid_sl * 2;
  t.hidden_bytes = hidden_out != nullptr ? r.hidden * 2 : 0;
  t.hidden_pad = (t.hidden_bytes + 127) / 128 * 128;
  t.kv_bytes = r.H * 256;
  t.has_k = k_out != nullptr; t.has_v = v_out != nullptr;
  t.slot_bytes = plan.filter.slot_bytes; t.n_slot = plan.filter.n_slot;
  t.vis_start = r.vis_start;
  if (plan.row_split) {   // first the score of text rows 0..63 alone, then the rest with the tail
    cudaError_t e = launch_fused_common(plan, plan.fused, false, q_text, k, g_out, i_out, workspace, nullptr, nullptr,
                                        plan.fused.smem_bytes, stream, la.vis_cnt);
    if (e != cudaSuccess) return e;
    return launch_fused_common(plan, plan.fused_b, true, q_text, k, g_out, i_out, workspace, &maps, &t,
                               plan.filter.smem_bytes, stream, la.vis_cnt);
  }
  return launch_fused_common(plan, plan.fused, false, q_text, k, g_out, i_out, workspace, &maps, &t,
                             plan.filter.smem_bytes, stream, la.vis_cnt);
}

}  // namespace mustdrop
