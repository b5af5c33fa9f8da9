// Vision-encoding stage of the method (Sec. 3.3), upstream of the prefill filter:
//   Local Spatial Merging (Eq. 5): non-overlapping 2 x 2 windows of the token grid whose mean
//     pairwise cosine similarity exceeds tau collapse into one averaged token at the window's
//     first slot; the survivors are packed in raster order;
//   Key Retaining (Eq. 6-7): head-averaged [CLS] attention over the patch tokens, and the tokens
//     above an adaptive threshold form the key set O.  The paper names no threshold rule; here it
//     is Tukey's upper fence Q3 + 1.5 (Q3 - Q1) with linearly interpolated quartiles.
// A thread-block cluster of up to eight CTAs of 256 threads works on one image (windows, rows and
// heads are dealt out over the cluster's CTAs; flags and partial attention sums cross through
// distributed shared memory, in a fixed order); both kernels are bound by reading their input
// once (1.2 MB per image at 576 tokens x 1024 channels).
#include <cuda_bf16.h>

#include "mustdrop_internal.h"

namespace mustdrop {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxSlots = 4096;            // tokens per image
constexpr int kOwn = kMaxSlots / kThreads; // consecutive slots per thread in the scans

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of the barrier.  Shared memory of another CTA may only be touched once that CTA
// is known to have started: every kernel arrives in its prologue and waits before its first
// remote store, so the wait costs nothing unless a peer really is late.
__device__ __forceinline__ void cluster_arrive() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of a shared-memory object of this CTA, as seen in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t peer_addr(const void* local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
               : "=r"(r)
               : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(local))), "r"(rank));
  return r;
}

// Exclusive prefix sum of one int per thread over the CTA (fixed order); returns the total too.
__device__ __forceinline__ int cta_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, d);
    if (lane >= d) inc += t;
  }
  __syncthreads();
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    const int s = warp_sums[w];
    if (w < warp) base += s;
    tot += s;
  }
  *total = tot;
  return base + inc - v;
}

// ---- Local Spatial Merging ----------------------------------------------------------------------
struct MergeParams {
  const uint4* tokens;   // [B, g*g, C/8]
  uint4* merged;         // [B, g*g, C/8]
  int32_t* slots;        // [B, g*g]
  int32_t* merged_cnt;   // [B]
  float* window_sim;     // [B, (g/2)^2] or null
  int32_t grid, vecs;    // vecs = C / 8
  float tau;
};

__global__ void __launch_bounds__(kThreads) spatial_merge_kernel(MergeParams p) {
  __shared__ unsigned char merged_flag[kMaxSlots / 4];
  __shared__ int warp_sums[kWarps];
  const int C = static_cast<int>(cluster_size()), rank = static_cast<int>(cluster_rank());
  const int b = blockIdx.x / C, g = p.grid, gw = g / 2, n_win = gw * gw, n_slot = g * g;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  cluster_arrive();          // "this CTA runs": peers wait for it before their first remote store
  bool peers_started = false;
  pdl_launch_dependents();
  pdl_wait();
  const uint4* in = p.tokens + static_cast<size_t>(b) * n_slot * p.vecs;

  // 1. per window: the four norms and six dot products, fp32 accumulation.  The cluster's warps
  //    share the windows; a window's flag is stored into every CTA's copy of the flag array.
  for (int w = rank * kWarps + warp; w < n_win; w += C * kWarps) {
    const int wy = w / gw, wx = w % gw;
    const int s0 = (2 * wy) * g + 2 * wx;
    const uint4* r0 = in + static_cast<size_t>(s0) * p.vecs;
    const uint4* r1 = r0 + p.vecs;                          // (y, x+1)
    const uint4* r2 = r0 + static_cast<size_t>(g) * p.vecs; // (y+1, x)
    const uint4* r3 = r2 + p.vecs;
    float n0 = 0, n1 = 0, n2 = 0, n3 = 0, d01 = 0, d02 = 0, d03 = 0, d12 = 0, d13 = 0, d23 = 0;
#pragma unroll 2
    for (int x = lane; x < p.vecs; x += 32) {
      const uint4 a = r0[x], c = r1[x], e = r2[x], f = r3[x];
      const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, cw[4] = {c.x, c.y, c.z, c.w};
      const uint32_t ew[4] = {e.x, e.y, e.z, e.w}, fw[4] = {f.x, f.y, f.z, f.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
#pragma unroll
        for (int hsel = 0; hsel < 2; ++hsel) {
          const float v0 = hsel ? bf16_hi(aw[q]) : bf16_lo(aw[q]);
          const float v1 = hsel ? bf16_hi(cw[q]) : bf16_lo(cw[q]);
          const float v2 = hsel ? bf16_hi(ew[q]) : bf16_lo(ew[q]);
          const float v3 = hsel ? bf16_hi(fw[q]) : bf16_lo(fw[q]);
          n0 = fmaf(v0, v0, n0); n1 = fmaf(v1, v1, n1); n2 = fmaf(v2, v2, n2); n3 = fmaf(v3, v3, n3);
          d01 = fmaf(v0, v1, d01); d02 = fmaf(v0, v2, d02); d03 = fmaf(v0, v3, d03);
          d12 = fmaf(v1, v2, d12); d13 = fmaf(v1, v3, d13); d23 = fmaf(v2, v3, d23);
        }
      }
    }
    n0 = warp_sum(n0); n1 = warp_sum(n1); n2 = warp_sum(n2); n3 = warp_sum(n3);
    d01 = warp_sum(d01); d02 = warp_sum(d02); d03 = warp_sum(d03);
    d12 = warp_sum(d12); d13 = warp_sum(d13); d23 = warp_sum(d23);
    if (!peers_started) {   // (warp-uniform) every CTA of the cluster has started: its shared memory exists
      cluster_wait();
      peers_started = true;
    }
    if (lane == 0) {
      const float tiny = 1e-30f;
      const float l0 = fmaxf(sqrtf(n0), tiny), l1 = fmaxf(sqrtf(n1), tiny), l2 = fmaxf(sqrtf(n2), tiny),
                  l3 = fmaxf(sqrtf(n3), tiny);
      const float sim = (d01 / (l0 * l1) + d02 / (l0 * l2) + d03 / (l0 * l3) + d12 / (l1 * l2) + d13 / (l1 * l3) +
                         d23 / (l2 * l3)) * (1.0f / 6.0f);
      const uint32_t flag = sim > p.tau ? 1u : 0u;
      for (int c = 0; c < C; ++c)
        asm volatile("st.shared::cluster.u8 [%0], %1;" ::"r"(peer_addr(&merged_flag[w], c)), "r"(flag) : "memory");
      if (p.window_sim != nullptr) p.window_sim[static_cast<size_t>(b) * n_win + w] = sim;
    }
  }
  if (!peers_started) cluster_wait();   // a warp without a window: complete the prologue's barrier
  cluster_barrier();   // every flag has arrived in every CTA; no remote store after this point

  // 2. which slots emit a token (all slots of an unmerged window, the first slot of a merged
  //    one) and where: exclusive scan in raster order, by every CTA for itself; CTA 0 stores it
  const int j0 = threadIdx.x * kOwn;
  uint32_t emit = 0;
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    const int s = j0 + e;
    if (s < n_slot) {
      const int y = s / g, x = s % g;
      const bool m = merged_flag[(y >> 1) * gw + (x >> 1)] != 0;
      if (!m || (((y | x) & 1) == 0)) emit |= 1u << e;
    }
  }
  int total;
  int pos = cta_exclusive_scan(__popc(emit), warp_sums, &total);
  __shared__ int16_t out_pos[kMaxSlots];     // output row of each emitting slot, -1 otherwise
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    const int s = j0 + e;
    if (s < n_slot) {
      if ((emit >> e) & 1u) {
        out_pos[s] = static_cast<int16_t>(pos);
        if (rank == 0) p.slots[static_cast<size_t>(b) * n_slot + pos] = s;
        ++pos;
      } else {
        out_pos[s] = -1;
      }
    }
  }
  if (threadIdx.x == 0 && rank == 0) p.merged_cnt[b] = total;
  __syncthreads();

  // 3. write the surviving rows: a copy, or the plain average of the window in fp32, rounded once
  uint4* out = p.merged + static_cast<size_t>(b) * n_slot * p.vecs;
  for (int s = rank * kWarps + warp; s < n_slot; s += C * kWarps) {
    const int o = out_pos[s];
    if (o < 0) continue;
    const int y = s / g, x = s % g;
    const bool m = merged_flag[(y >> 1) * gw + (x >> 1)] != 0;
    const uint4* r0 = in + static_cast<size_t>(s) * p.vecs;
    uint4* dst = out + static_cast<size_t>(o) * p.vecs;
    if (!m) {
      // a copy: four independent 16-byte loads in flight per lane, then the stores
      for (int v0 = lane; v0 < p.vecs; v0 += 4 * 32) {
        uint4 t[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (v0 + 32 * u < p.vecs) t[u] = r0[v0 + 32 * u];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (v0 + 32 * u < p.vecs) dst[v0 + 32 * u] = t[u];
      }
    } else {
      const uint4* r1 = r0 + p.vecs;
      const uint4* r2 = r0 + static_cast<size_t>(g) * p.vecs;
      const uint4* r3 = r2 + p.vecs;
      for (int v = lane; v < p.vecs; v += 32) {
        const uint4 a = r0[v], c = r1[v], e = r2[v], f = r3[v];
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, cw[4] = {c.x, c.y, c.z, c.w};
        const uint32_t ew[4] = {e.x, e.y, e.z, e.w}, fw[4] = {f.x, f.y, f.z, f.w};
        uint32_t ow[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float lo = ((bf16_lo(aw[q]) + bf16_lo(cw[q])) + (bf16_lo(ew[q]) + bf16_lo(fw[q]))) * 0.25f;
          const float hi = ((bf16_hi(aw[q]) + bf16_hi(cw[q])) + (bf16_hi(ew[q]) + bf16_hi(fw[q]))) * 0.25f;
          const __nv_bfloat16 bl = __float2bfloat16_rn(lo), bh = __float2bfloat16_rn(hi);
          ow[q] = static_cast<uint32_t>(__bfloat16_as_ushort(bl)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bh)) << 16);
        }
        dst[v] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
      }
    }
  }
}

// ---- Key Retaining ------------------------------------------------------------------------------
struct KeySetParams {
  const __nv_bfloat16* q_cls;   // [B, H, D]
  const uint4* k;               // [B, H, M, D/8]
  float* a_cls;                 // [B, M] or null
  float* mu_out;                // [B] or null
  int32_t* key_idx;             // [B, key_max]
  int32_t* key_cnt;             // [B]
  int32_t H, D, M, key_max;
  float scale_log2e;
};

__global__ void __launch_bounds__(kThreads) key_set_kernel(KeySetParams p) {
  __shared__ __align__(16) float a[kMaxSlots];      // head-mean attention
  __shared__ float z[kMaxSlots];      // one head's logits (log2 units)
  __shared__ __align__(16) float q_s[256];
  __shared__ float red[kWarps];
  __shared__ float order[4];          // the four order statistics the quartiles interpolate
  __shared__ int warp_sums[kWarps];
  extern __shared__ float slab[];     // [cluster size][M] partial sums of the cluster's CTAs
  const int C = static_cast<int>(cluster_size()), rank = static_cast<int>(cluster_rank());
  const int b = blockIdx.x / C, M = p.M, dv = p.D / 8;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  cluster_arrive();          // "this CTA runs": peers wait for it before their first remote store
  pdl_launch_dependents();
  pdl_wait();
  for (int j = threadIdx.x; j < M; j += kThreads) a[j] = 0.0f;
  const float inv_h = 1.0f / static_cast<float>(p.H);

  for (int h = rank; h < p.H; h += C) {   // the cluster's CTAs share the heads
    __syncthreads();   // q_s, z and red are free again
    for (int d = threadIdx.x; d < p.D; d += kThreads)
      q_s[d] = __bfloat162float(p.q_cls[(static_cast<size_t>(b) * p.H + h) * p.D + d]);
    __syncthreads();
    const uint4* kh = p.k + (static_cast<size_t>(b) * p.H + h) * M * dv;
    // Coalesced rows: a group of `grp` lanes (the power of two >= D/8) reads one token's row as
    // 16-byte vectors; a warp takes 32/grp consecutive tokens per step, four steps in flight.  Each
    // lane keeps its eight query values in registers for the whole head.
    int grp = 1;
    while (grp < dv) grp <<= 1;
    const int sub = lane % grp, tok_in_warp = lane / grp, per_warp = 32 / grp;
    float qv[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) qv[e] = sub < dv ? q_s[sub * 8 + e] : 0.0f;
    float mx = -INFINITY;
    const int step = kWarps * per_warp;
    constexpr int kFly = 4;   // key rows in flight per lane
    for (int base = warp * per_warp; base < M; base += kFly * step) {   // warp-uniform trip count
      int jt[kFly];
      uint4 kv[kFly];
#pragma unroll
      for (int u = 0; u < kFly; ++u) {
        jt[u] = base + u * step + tok_in_warp;
        kv[u] = make_uint4(0, 0, 0, 0);
        if (jt[u] < M && sub < dv) kv[u] = kh[static_cast<size_t>(jt[u]) * dv + sub];
      }
#pragma unroll
      for (int u = 0; u < kFly; ++u) {
        float da = bf16_lo(kv[u].x) * qv[0];
        da = fmaf(bf16_hi(kv[u].x), qv[1], da);
        da = fmaf(bf16_lo(kv[u].y), qv[2], da);
        da = fmaf(bf16_hi(kv[u].y), qv[3], da);
        da = fmaf(bf16_lo(kv[u].z), qv[4], da);
        da = fmaf(bf16_hi(kv[u].z), qv[5], da);
        da = fmaf(bf16_lo(kv[u].w), qv[6], da);
        da = fmaf(bf16_hi(kv[u].w), qv[7], da);
        for (int d = grp >> 1; d >= 1; d >>= 1) da += __shfl_xor_sync(0xffffffffu, da, d);   // sum over the group's lanes (fixed tree)
        if (sub == 0 && jt[u] < M) {
          const float zz = da * p.scale_log2e;
          z[jt[u]] = zz;
          mx = fmaxf(mx, zz);
        }
      }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    if (lane == 0) red[warp] = mx;
    __syncthreads();
    mx = red[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) mx = fmaxf(mx, red[w]);
    float sum = 0.0f;
    for (int j = threadIdx.x; j < M; j += kThreads) {
      const float e = exp2f(z[j] - mx);
      z[j] = e;
      sum += e;
    }
    sum = warp_sum(sum);
    __syncthreads();   // everyone has read red
    if (lane == 0) red[warp] = sum;
    __syncthreads();
    sum = 0.0f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) sum += red[w];   // fixed order
    const float f = inv_h / sum;
    for (int j = threadIdx.x; j < M; j += kThreads) a[j] = fmaf(z[j], f, a[j]);
  }
  // every CTA hands its partial sums to every CTA; each adds them in rank order (same result everywhere)
  cluster_wait();            // every CTA of the cluster has started: its shared memory exists
  for (int c = 0; c < C; ++c)
    for (int j = threadIdx.x; j < M; j += kThreads)
      asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(peer_addr(&slab[static_cast<size_t>(rank) * M + j], c)), "f"(a[j])
                   : "memory");
  cluster_barrier();
  for (int j = threadIdx.x; j < M; j += kThreads) {
    float sum = 0.0f;
    for (int c = 0; c < C; ++c) sum += slab[static_cast<size_t>(c) * M + j];
    a[j] = sum;
  }
  const int M4 = (M + 3) & ~3;
  if (threadIdx.x < M4 - M) a[M + threadIdx.x] = INFINITY;   // padding that is never counted
  __syncthreads();

  // quartiles by rank counting: the element with r smaller ones (ties by index) is order statistic r.
  // The cluster's CTAs share the tokens; whoever finds one of the four needed statistics stores it in CTA 0.
  const float p1 = 0.25f * static_cast<float>(M - 1), p3 = 0.75f * static_cast<float>(M - 1);
  const int r1 = static_cast<int>(floorf(p1)), r3 = static_cast<int>(floorf(p3));
  const int r1h = min(r1 + 1, M - 1), r3h = min(r3 + 1, M - 1);
  for (int j = threadIdx.x * C + rank; j < M; j += kThreads * C) {
    const float aj = a[j];
    int rk = 0;
    for (int i = 0; i < M4; i += 4) {                          // four candidates per shared load
      const float4 v = *reinterpret_cast<const float4*>(&a[i]);
      rk += (v.x < aj || (v.x == aj && i < j)) ? 1 : 0;
      rk += (v.y < aj || (v.y == aj && i + 1 < j)) ? 1 : 0;
      rk += (v.z < aj || (v.z == aj && i + 2 < j)) ? 1 : 0;
      rk += (v.w < aj || (v.w == aj && i + 3 < j)) ? 1 : 0;
    }
    if (rk == r1) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(peer_addr(&order[0], 0)), "f"(aj) : "memory");
    if (rk == r1h) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(peer_addr(&order[1], 0)), "f"(aj) : "memory");
    if (rk == r3) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(peer_addr(&order[2], 0)), "f"(aj) : "memory");
    if (rk == r3h) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(peer_addr(&order[3], 0)), "f"(aj) : "memory");
  }
  cluster_barrier();
  if (rank != 0) return;   // CTA 0 finishes alone; no store into another CTA's memory after this point
  const float q1 = order[0] + (order[1] - order[0]) * (p1 - static_cast<float>(r1));
  const float q3 = order[2] + (order[3] - order[2]) * (p3 - static_cast<float>(r3));
  const float mu = q3 + 1.5f * (q3 - q1);
  if (threadIdx.x == 0 && p.mu_out != nullptr) p.mu_out[b] = mu;

  // O = { j : a[j] > mu }, ascending; at most key_max of them are stored (the lowest indices)
  const int j0 = threadIdx.x * kOwn;
  uint32_t is_key = 0;
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    const int j = j0 + e;
    if (j < M) {
      if (p.a_cls != nullptr) p.a_cls[static_cast<size_t>(b) * M + j] = a[j];
      if (a[j] > mu) is_key |= 1u << e;
    }
  }
  int total;
  int pos = cta_exclusive_scan(__popc(is_key), warp_sums, &total);
#pragma unroll
  for (int e = 0; e < kOwn; ++e) {
    if ((is_key >> e) & 1u) {
      if (pos < p.key_max) p.key_idx[static_cast<size_t>(b) * p.key_max + pos] = j0 + e;
      ++pos;
    }
  }
  if (threadIdx.x == 0) p.key_cnt[b] = total < p.key_max ? total : p.key_max;
}

inline bool aligned16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; }

template <typename Kernel, typename Params>
cudaError_t launch_cluster(Kernel kernel, int batch, int cluster, size_t smem, cudaStream_t stream, const Params& p) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(batch * cluster));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

inline mustdrop_status_t finish(cudaError_t e) {
  if (e == cudaSuccess) return MUSTDROP_OK;
  set_last_cuda_error(e);
  return MUSTDROP_ERR_CUDA;
}

}  // namespace
}  // namespace mustdrop

extern "C" mustdrop_status_t mustdrop_spatial_merge(int32_t batch, int32_t grid, int32_t window, int32_t channels,
                                                    float tau, const void* tokens, void* merged, int32_t* slots,
                                                    int32_t* merged_cnt, float* window_sim, void* cuda_stream) {
  using namespace mustdrop;
  if (batch <= 0 || grid <= 0 || channels <= 0 || tokens == nullptr || merged == nullptr || slots == nullptr ||
      merged_cnt == nullptr || !(tau == tau))
    return MUSTDROP_ERR_INVALID_ARG;
  if (window != 2 || (grid % 2) != 0 || grid * grid > kMaxSlots || (channels % 8) != 0 || batch > 65535)
    return MUSTDROP_ERR_UNSUPPORTED;
  const void* ptrs[] = {tokens, merged, slots, merged_cnt, window_sim};
  for (const void* q : ptrs)
    if (q != nullptr && !aligned16(q)) return MUSTDROP_ERR_INVALID_ARG;
  MergeParams p;
  p.tokens = static_cast<const uint4*>(tokens);
  p.merged = static_cast<uint4*>(merged);
  p.slots = slots; p.merged_cnt = merged_cnt; p.window_sim = window_sim;
  p.grid = grid; p.vecs = channels / 8; p.tau = tau;
  const int n_win = (grid / 2) * (grid / 2);
  int cluster = 8;                                   // no more CTAs than there are rounds of windows for them
  while (cluster > 1 && (cluster - 1) * kWarps >= n_win) cluster >>= 1;
  return finish(launch_cluster(spatial_merge_kernel, batch, cluster, 0, static_cast<cudaStream_t>(cuda_stream), p));
}

extern "C" mustdrop_status_t mustdrop_key_set(int32_t batch, int32_t n_heads, int32_t head_dim, int32_t n_tokens,
                                              int32_t key_max, const void* q_cls, const void* k, float* a_cls,
                                              float* mu_out, int32_t* key_idx, int32_t* key_cnt, void* cuda_stream) {
  using namespace mustdrop;
  if (batch <= 0 || n_heads <= 0 || head_dim <= 0 || n_tokens <= 0 || key_max <= 0 || q_cls == nullptr ||
      k == nullptr || key_idx == nullptr || key_cnt == nullptr)
    return MUSTDROP_ERR_INVALID_ARG;
  if ((head_dim % 8) != 0 || head_dim > 256 || n_tokens > kMaxSlots || batch > 65535) return MUSTDROP_ERR_UNSUPPORTED;
  const void* ptrs[] = {q_cls, k, a_cls, mu_out, key_idx, key_cnt};
  for (const void* q : ptrs)
    if (q != nullptr && !aligned16(q)) return MUSTDROP_ERR_INVALID_ARG;
  KeySetParams p;
  p.q_cls = static_cast<const __nv_bfloat16*>(q_cls);
  p.k = static_cast<const uint4*>(k);
  p.a_cls = a_cls; p.mu_out = mu_out; p.key_idx = key_idx; p.key_cnt = key_cnt;
  p.H = n_heads; p.D = head_dim; p.M = n_tokens; p.key_max = key_max;
  p.scale_log2e = 1.4426950408889634f / sqrtf(static_cast<float>(head_dim));
  int cluster = 8;
  while (cluster > n_heads) cluster >>= 1;           // 1, 2, 4 or 8 CTAs, at most one per head
  const size_t smem = static_cast<size_t>(cluster) * n_tokens * sizeof(float);
  cudaError_t e = ensure_kernel_attributes(reinterpret_cast<const void*>(key_set_kernel), false);
  if (e != cudaSuccess) return finish(e);
  return finish(launch_cluster(key_set_kernel, batch, cluster, smem, static_cast<cudaStream_t>(cuda_stream), p));
}
