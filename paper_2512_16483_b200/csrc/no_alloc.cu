// Row selection without any caller-provided scratch buffer.
//
// fvar_row_scores + fvar_select_topr need a scores array between them, which the caller has to
// allocate.  Some callers cannot: code running under a memory planner that hands out every device
// byte up front, plugins living inside another runtime's allocator, or a service whose latency
// budget forbids cudaMalloc's implicit device synchronisation.  For them the scores live in a
// fixed array that is part of the library image.
#include <mutex>
#include <string>

#include "../../include/fvar.h"
#include "internal.h"

namespace fvar {

// The scratch: one fp32 score per (batch element, row).  256 KiB on every GPU that loads the
// library, held until the process exits.
constexpr int kStaticScoreCapacity = FVAR_STATIC_SELECT_MAX_ROWS;
static __device__ __align__(256) float g_static_scores[kStaticScoreCapacity];

constexpr int kMaxDevices = 64;
static float *g_scores_ptr[kMaxDevices];   // device address of g_static_scores, per device ordinal
static std::mutex g_scores_mutex;

// In host code `g_static_scores` is only a handle for the runtime; the address a kernel can use
// comes from cudaGetSymbolAddress, resolved once per device with that device current.
static cudaError_t static_scores_address(float **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scores_mutex);
  if (g_scores_ptr[dev] == nullptr) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scores);
    if (e != cudaSuccess) return e;
    g_scores_ptr[dev] = static_cast<float *>(p);
  }
  *out = g_scores_ptr[dev];
  return cudaSuccess;
}

}  // namespace fvar

using namespace fvar;

extern "C" fvar_status fvar_select_rows_static(const float *x, int B, int M, int C, int r, int *idx, int *inv,
                                               void *stream) {
  if (!x || !idx || !inv || B <= 0 || M <= 0 || C <= 0 || C % 4 || r <= 0 || r > M) {
    set_global_error("select_rows_static: bad arguments");
    return FVAR_EINVAL;
  }
  if (static_cast<long long>(B) * M > kStaticScoreCapacity) {
    set_global_error(("select_rows_static: B * M = " + std::to_string(static_cast<long long>(B) * M) +
                      " exceeds the built-in scratch of " + std::to_string(kStaticScoreCapacity) +
                      " rows; use fvar_row_scores + fvar_select_topr with your own buffer").c_str());
    return FVAR_EUNSUPPORTED;
  }
  float *scores = nullptr;
  cudaError_t e = static_scores_address(&scores);
  if (e == cudaSuccess) e = launch_row_scores(x, RowMap{1, 0, M}, B, M, C, nullptr, scores, static_cast<cudaStream_t>(stream));
  if (e == cudaSuccess) e = launch_select_topr(scores, B, M, r, idx, inv, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    set_global_error((std::string("select_rows_static: ") + cudaGetErrorString(e)).c_str());
    return FVAR_ECUDA;
  }
  return FVAR_OK;
}
