// Importance scores, two-pass form (Eq. 1, Eq. 8, Eq. 10).
//
// Pass 1 (row statistics): one CTA per (request, head) walks all L keys in tiles of 64 and
// keeps, for each text query, the running maximum and the running sum of exponentials of its
// visible logits -> (m, 1/l) in scratch memory, m in log2 units.
// Pass 2 (accumulate): one CTA per (request, tile of 64 vision keys) loops over the heads,
// recomputes the tile's logits, turns them into probabilities with pass 1's statistics and
// adds them up over heads in registers; then column sum (Eq. 8) and column max (Eq. 10) over
// the text rows of the head mean.
//
// Both passes use warp-level bf16 MMA (m16n8k16, fp32 accumulate): a warp owns 16 text rows,
// keys are the n dimension.  The key tensor is read twice; this is the general-shape path.
#include <cuda_bf16.h>

#include "mustdrop_internal.h"

namespace mustdrop {
namespace {

constexpr int kTileKeys = 64;
constexpr int kRowStride = kHeadDim + 8;  // bf16 elements per staged row: 272 bytes, conflict-free fragments

struct ScoreParams {
  const __nv_bfloat16* q;   // [B,H,N,D]
  const __nv_bfloat16* k;   // strided [B,H,L,D]
  float2* rowstats;         // [B,H,N]
  float* g_out;             // [B,M]
  float* i_out;             // [B,M]
  const int32_t* vis_cnt;   // [B] or null: vision tokens the request holds; its text keys follow them
  int32_t H, N, L, M, vis_start, txt_start, causal, n_warps;
  int32_t per_head_max;     // 1: i_out = head mean of the per-head column maxima
  float scale_log2e, inv_heads;
  int64_t k_sb, k_sh, k_sl;
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool valid) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const int bytes = valid ? 16 : 0;  // 0 source bytes => the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Stage `rows` rows of 128 bf16 (row r from gmem_row0 + r*stride) into padded shared rows;
// rows at or beyond `valid_rows` are zero-filled.
__device__ __forceinline__ void stage_rows(__nv_bfloat16* smem, const __nv_bfloat16* gmem_row0, int64_t stride,
                                           int rows, int valid_rows, int n_threads) {
  for (int x = threadIdx.x; x < rows * 16; x += n_threads) {
    const int r = x >> 4, c = x & 15;
    const bool ok = r < valid_rows;
    cp_async16(smem + r * kRowStride + c * 8, gmem_row0 + (ok ? r : 0) * stride + c * 8, ok);
  }
}

// A fragments (16 text rows x 128) of this warp from staged Q.
__device__ __forceinline__ void load_a_frags(uint32_t (&a)[8][4], const __nv_bfloat16* q_s, int warp, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const __nv_bfloat16* r0 = q_s + (warp * 16 + g) * kRowStride + 2 * t;
  const __nv_bfloat16* r1 = r0 + 8 * kRowStride;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    a[ks][0] = *reinterpret_cast<const uint32_t*>(r0 + ks * 16);
    a[ks][1] = *reinterpret_cast<const uint32_t*>(r1 + ks * 16);
    a[ks][2] = *reinterpret_cast<const uint32_t*>(r0 + ks * 16 + 8);
    a[ks][3] = *reinterpret_cast<const uint32_t*>(r1 + ks * 16 + 8);
  }
}

// Logits of the warp's 16 rows against 8 staged keys (block nb of the tile).
__device__ __forceinline__ void tile_block_logits(float (&c)[4], const uint32_t (&a)[8][4],
                                                  const __nv_bfloat16* k_s, int nb, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const __nv_bfloat16* kr = k_s + (nb * 8 + g) * kRowStride + 2 * t;
  c[0] = c[1] = c[2] = c[3] = 0.0f;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint32_t b0 = *reinterpret_cast<const uint32_t*>(kr + ks * 16);
    const uint32_t b1 = *reinterpret_cast<const uint32_t*>(kr + ks * 16 + 8);
    mma_bf16(c, a[ks], b0, b1);
  }
}

// ---- pass 1 ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rowstats_kernel(ScoreParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n_rows = p.n_warps * 16;
  __nv_bfloat16* q_s = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  __nv_bfloat16* k_s0 = q_s + n_rows * kRowStride;
  __nv_bfloat16* k_s1 = k_s0 + kTileKeys * kRowStride;
  const int h = blockIdx.x, b = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int n_threads = blockDim.x;
  pdl_wait();   // the row-statistics scratch may still be read by an earlier launch
  // this request's own sequence: its text keys follow its vision tokens
  const int txt_start = p.vis_cnt ? p.vis_start + clamp_vis_cnt(p.vis_cnt[b], p.M) : p.txt_start;
  const int L = p.vis_cnt ? txt_start + p.N : p.L;
  const __nv_bfloat16* qg = p.q + (static_cast<int64_t>(b) * p.H + h) * p.N * kHeadDim;
  const __nv_bfloat16* kg = p.k + b * p.k_sb + h * p.k_sh;
  const int n_tiles = (L + kTileKeys - 1) / kTileKeys;

  stage_rows(q_s, qg, kHeadDim, n_rows, p.N, n_threads);
  stage_rows(k_s0, kg, p.k_sl, kTileKeys, L, n_threads);
  cp_async_commit();

  const int row0 = warp * 16 + g, row1 = row0 + 8;
  // last visible key of each of this thread's two text rows
  const int last0 = p.causal ? txt_start + row0 : L - 1;
  const int last1 = p.causal ? txt_start + row1 : L - 1;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.0f, l1 = 0.0f;
  uint32_t a[8][4];

  for (int tile = 0; tile < n_tiles; ++tile) {
    __nv_bfloat16* cur = (tile & 1) ? k_s1 : k_s0;
    __nv_bfloat16* nxt = (tile & 1) ? k_s0 : k_s1;
    if (tile + 1 < n_tiles) {
      const int base = (tile + 1) * kTileKeys;
      stage_rows(nxt, kg + static_cast<int64_t>(base) * p.k_sl, p.k_sl, kTileKeys, L - base, n_threads);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (tile == 0) load_a_frags(a, q_s, warp, lane);
    const int key_base = tile * kTileKeys;
    float z[8][4];
    float tmax0 = -INFINITY, tmax1 = -INFINITY;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      tile_block_logits(z[nb], a, cur, nb, lane);
      const int key = key_base + nb * 8 + 2 * t;
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        z[nb][e] = (key + e <= last0 && key + e < L) ? z[nb][e] * p.scale_log2e : -INFINITY;
        z[nb][2 + e] = (key + e <= last1 && key + e < L) ? z[nb][2 + e] * p.scale_log2e : -INFINITY;
        tmax0 = fmaxf(tmax0, z[nb][e]);
        tmax1 = fmaxf(tmax1, z[nb][2 + e]);
      }
    }
    if (tmax0 > -INFINITY) {
      const float mn = fmaxf(m0, tmax0);
      float s = 0.0f;
#pragma unroll
      for (int nb = 0; nb < 8; ++nb) s += exp2f(z[nb][0] - mn) + exp2f(z[nb][1] - mn);
      l0 = l0 * exp2f(m0 - mn) + s;
      m0 = mn;
    }
    if (tmax1 > -INFINITY) {
      const float mn = fmaxf(m1, tmax1);
      float s = 0.0f;
#pragma unroll
      for (int nb = 0; nb < 8; ++nb) s += exp2f(z[nb][2] - mn) + exp2f(z[nb][3] - mn);
      l1 = l1 * exp2f(m1 - mn) + s;
      m1 = mn;
    }
    __syncthreads();  // everyone is done with `cur` before it is refilled
  }
  // combine the four threads that share a row (key 0 is visible to every row, so the max is finite)
#pragma unroll
  for (int d = 1; d <= 2; d <<= 1) {
    const float om0 = __shfl_xor_sync(0xffffffffu, m0, d), ol0 = __shfl_xor_sync(0xffffffffu, l0, d);
    const float om1 = __shfl_xor_sync(0xffffffffu, m1, d), ol1 = __shfl_xor_sync(0xffffffffu, l1, d);
    const float n0 = fmaxf(m0, om0), n1 = fmaxf(m1, om1);
    l0 = (m0 > -INFINITY ? l0 * exp2f(m0 - n0) : 0.0f) + (om0 > -INFINITY ? ol0 * exp2f(om0 - n0) : 0.0f);
    l1 = (m1 > -INFINITY ? l1 * exp2f(m1 - n1) : 0.0f) + (om1 > -INFINITY ? ol1 * exp2f(om1 - n1) : 0.0f);
    m0 = n0;
    m1 = n1;
  }
  if (t == 0) {
    float2* out = p.rowstats + (static_cast<int64_t>(b) * p.H + h) * p.N;
    if (row0 < p.N) out[row0] = make_float2(m0, 1.0f / l0);
    if (row1 < p.N) out[row1] = make_float2(m1, 1.0f / l1);
  }
}

// ---- pass 2 ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) accumulate_kernel(ScoreParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n_rows = p.n_warps * 16;
  const int stage_elems = (n_rows + kTileKeys) * kRowStride;
  __nv_bfloat16* stage0 = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  __nv_bfloat16* stage1 = stage0 + stage_elems;
  float* red = reinterpret_cast<float*>(stage1 + stage_elems);  // [2][n_warps][64]
  float* imax_s = red + 2 * p.n_warps * kTileKeys;              // [64] sum over heads of the per-head column maxima
  const int vt = blockIdx.x, b = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int n_threads = blockDim.x;
  pdl_wait();
  const int j_base = vt * kTileKeys;            // first vision token of this tile
  const int Mb = p.vis_cnt ? clamp_vis_cnt(p.vis_cnt[b], p.M) : p.M;
  const int valid_keys = Mb - j_base;           // rows of the tile that exist (<= 0: none, zeros are stored)
  const __nv_bfloat16* qg = p.q + static_cast<int64_t>(b) * p.H * p.N * kHeadDim;
  const __nv_bfloat16* kg = p.k + b * p.k_sb + static_cast<int64_t>(p.vis_start + j_base) * p.k_sl;
  const float2* stats = p.rowstats + static_cast<int64_t>(b) * p.H * p.N;

  auto stage_head = [&](__nv_bfloat16* st, int h) {
    stage_rows(st, qg + static_cast<int64_t>(h) * p.N * kHeadDim, kHeadDim, n_rows, p.N, n_threads);
    stage_rows(st + n_rows * kRowStride, kg + h * p.k_sh, p.k_sl, kTileKeys, valid_keys, n_threads);
    cp_async_commit();
  };
  stage_head(stage0, 0);
  for (int col = threadIdx.x; col < kTileKeys; col += n_threads) imax_s[col] = 0.0f;

  const int row0 = warp * 16 + g, row1 = row0 + 8;
  float acc[8][4];
#pragma unroll
  for (int nb = 0; nb < 8; ++nb) acc[nb][0] = acc[nb][1] = acc[nb][2] = acc[nb][3] = 0.0f;

  for (int h = 0; h < p.H; ++h) {
    __nv_bfloat16* cur = (h & 1) ? stage1 : stage0;
    __nv_bfloat16* nxt = (h & 1) ? stage0 : stage1;
    if (h + 1 < p.H) {
      stage_head(nxt, h + 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const float2 st0 = row0 < p.N ? stats[h * p.N + row0] : make_float2(0.0f, 0.0f);
    const float2 st1 = row1 < p.N ? stats[h * p.N + row1] : make_float2(0.0f, 0.0f);
    uint32_t a[8][4];
    load_a_frags(a, cur, warp, lane);
    const __nv_bfloat16* k_s = cur + n_rows * kRowStride;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      float c[4];
      tile_block_logits(c, a, k_s, nb, lane);
      const float p0 = exp2f(c[0] * p.scale_log2e - st0.x) * st0.y, p1 = exp2f(c[1] * p.scale_log2e - st0.x) * st0.y;
      const float p2 = exp2f(c[2] * p.scale_log2e - st1.x) * st1.y, p3 = exp2f(c[3] * p.scale_log2e - st1.x) * st1.y;
      acc[nb][0] += p0; acc[nb][1] += p1; acc[nb][2] += p2; acc[nb][3] += p3;
      if (p.per_head_max) {
        // this head's column maxima over the warp's 16 rows (rows at or beyond N do not take part)
        float m0 = fmaxf(row0 < p.N ? p0 : -INFINITY, row1 < p.N ? p2 : -INFINITY);
        float m1 = fmaxf(row0 < p.N ? p1 : -INFINITY, row1 < p.N ? p3 : -INFINITY);
#pragma unroll
        for (int d = 4; d <= 16; d <<= 1) {
          m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, d));
          m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, d));
        }
        if (g == 0) {
          red[warp * kTileKeys + nb * 8 + 2 * t] = m0;
          red[warp * kTileKeys + nb * 8 + 2 * t + 1] = m1;
        }
      }
    }
    if (p.per_head_max) {   // over the warps, then onto the running head sum
      __syncthreads();
      for (int col = threadIdx.x; col < kTileKeys; col += n_threads) {
        float mx = -INFINITY;
        for (int w = 0; w < p.n_warps; ++w) mx = fmaxf(mx, red[w * kTileKeys + col]);
        imax_s[col] += mx;
      }
    }
    __syncthreads();
  }

  // column sum and column max over the text rows; rows at or beyond N do not take part
  const bool ok0 = row0 < p.N, ok1 = row1 < p.N;
#pragma unroll
  for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const float v0 = acc[nb][e], v1 = acc[nb][2 + e];
      float s = (ok0 ? v0 : 0.0f) + (ok1 ? v1 : 0.0f);
      float mx = fmaxf(ok0 ? v0 : -INFINITY, ok1 ? v1 : -INFINITY);
#pragma unroll
      for (int d = 4; d <= 16; d <<= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, d);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
      }
      if (g == 0) {
        const int col = nb * 8 + 2 * t + e;
        red[warp * kTileKeys + col] = s;
        red[(p.n_warps + warp) * kTileKeys + col] = mx;
      }
    }
  }
  __syncthreads();
  for (int col = threadIdx.x; col < kTileKeys; col += n_threads) {
    if (j_base + col >= p.M) continue;
    float s = 0.0f, mx = -INFINITY;
    for (int w = 0; w < p.n_warps; ++w) {
      s += red[w * kTileKeys + col];
      mx = fmaxf(mx, red[(p.n_warps + w) * kTileKeys + col]);
    }
    if (p.per_head_max) mx = imax_s[col];
    if (col >= valid_keys) s = mx = 0.0f;   // beyond the request's own tokens
    p.g_out[static_cast<int64_t>(b) * p.M + j_base + col] = s * p.inv_heads;
    p.i_out[static_cast<int64_t>(b) * p.M + j_base + col] = mx * p.inv_heads;
  }
}

}  // namespace

cudaError_t launch_score_two_pass(const mustdrop_plan& plan, const void* q_text, const void* k, float* g_out,
                                  float* i_out, void* rowstats, cudaStream_t stream, const int32_t* vis_cnt) {
  const Resolved& r = plan.r;
  ScoreParams p;
  p.q = static_cast<const __nv_bfloat16*>(q_text);
  p.k = static_cast<const __nv_bfloat16*>(k);
  p.rowstats = static_cast<float2*>(rowstats);
  p.g_out = g_out; p.i_out = i_out;
  p.vis_cnt = vis_cnt;
  p.per_head_max = r.per_head_max;
  p.H = r.H; p.N = r.N; p.L = r.L; p.M = r.M; p.vis_start = r.vis_start; p.txt_start = r.txt_start;
  p.causal = r.causal;
  p.n_warps = (r.N + 15) / 16;
  p.scale_log2e = r.scale_log2e;
  p.inv_heads = 1.0f / static_cast<float>(r.H);
  p.k_sb = r.k_sb; p.k_sh = r.k_sh; p.k_sl = r.k_sl;
  const int n_rows = p.n_warps * 16;
  const int threads = p.n_warps * 32;
  const size_t smem1 = sizeof(__nv_bfloat16) * static_cast<size_t>(n_rows + 2 * kTileKeys) * kRowStride;
  const size_t smem2 = sizeof(__nv_bfloat16) * 2 * static_cast<size_t>(n_rows + kTileKeys) * kRowStride +
                       sizeof(float) * (2 * p.n_warps + 1) * kTileKeys;
  cudaError_t e = ensure_kernel_attributes(reinterpret_cast<const void*>(rowstats_kernel), false);
  if (e != cudaSuccess) return e;
  e = ensure_kernel_attributes(reinterpret_cast<const void*>(accumulate_kernel), false);
  if (e != cudaSuccess) return e;
  rowstats_kernel<<<dim3(r.H, r.B), threads, smem1, stream>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  accumulate_kernel<<<dim3((r.M + kTileKeys - 1) / kTileKeys, r.B), threads, smem2, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace mustdrop
