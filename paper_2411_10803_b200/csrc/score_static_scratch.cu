// mustdrop_score_static: the importance-score call for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving engine that
// has handed the whole device heap to its own pool allocator, in a plug-in that must not touch
// the allocator of the host application, or late in a process that has already locked its
// memory budget.  mustdrop_score needs a caller-provided workspace for the per-row softmax
// statistics; this entry point keeps that scratch in a fixed array that is part of the
// library image instead, so the caller passes only inputs and outputs.
#include <mutex>

#include "mustdrop_internal.h"

namespace {

// Row statistics (row maximum in log2 units, 1 / row sum) for up to kStaticRows text rows,
// i.e. batch * n_heads * n_txt <= 524288: 4 MiB, resident on every GPU that loads the library
// until the process exits.
constexpr size_t kStaticRows = 512 * 1024;
static __device__ __align__(256) float2 g_static_rowstats[kStaticRows];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {nullptr};   // device address of the array, per device

// The array's name is only a handle on the host side; its device address has to be asked for,
// once per device, while that device is current.
cudaError_t scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_rowstats);
    if (e != cudaSuccess) return e;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" mustdrop_status_t mustdrop_score_static(const mustdrop_plan_t* plan, const void* q_text, const void* k,
                                                   float* g_out, float* i_out, void* cuda_stream) {
  if (plan == nullptr || plan->magic != mustdrop::kPlanMagic || q_text == nullptr || k == nullptr ||
      g_out == nullptr || i_out == nullptr)
    return MUSTDROP_ERR_INVALID_ARG;
  const void* ptrs[] = {q_text, k, g_out, i_out};
  for (const void* p : ptrs)
    if ((reinterpret_cast<uintptr_t>(p) & 15u) != 0) return MUSTDROP_ERR_INVALID_ARG;
  const size_t rows = static_cast<size_t>(plan->r.B) * plan->r.H * plan->r.N;
  if (rows > kStaticRows) return MUSTDROP_ERR_SCRATCH_LIMIT;
  void* scratch = nullptr;
  cudaError_t e = scratch_address(&scratch);
  if (e == cudaSuccess)
    e = mustdrop::launch_score_two_pass(*plan, q_text, k, g_out, i_out, scratch,
                                        static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) {
    mustdrop::set_last_cuda_error(e);
    return MUSTDROP_ERR_CUDA;
  }
  return MUSTDROP_OK;
}

extern "C" size_t mustdrop_score_static_max_rows(void) { return kStaticRows; }
