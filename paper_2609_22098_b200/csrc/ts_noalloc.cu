// ts_score_parents_static: the scoring call for callers that cannot hand the library a workspace.
// Its scratch (the per-tile records that the scoring kernel writes and the merge kernel reads)
// lives in a fixed array in the library's own device image instead of caller memory.
#include <stdio.h>

#include <mutex>

#include "ts_internal.h"

// One copy per GPU that loads the library, resident until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[TS_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
// Device address of g_static_scratch on each device.  In host code the symbol's name is only a
// stand-in; the real address has to be asked for, with the device in question current.
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_mutex;

}  // namespace

extern "C" int32_t ts_score_parents_static(ts_ctx* ctx, const void* U, const void* A, const void* W, int32_t P,
                                           const int32_t* parent_req, const int32_t* parent_depth,
                                           const int32_t* parent_token, const uint64_t* parent_hash, float T,
                                           uint64_t seed, float* lse0, float* lseT, int32_t* top_tok,
                                           float* top_logit, int32_t* draw_tok, float* draw_logit, void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_score_parents_static: null context");
  const void* ptrs[] = {U, A, W, parent_req, parent_depth, parent_token, parent_hash, lse0, lseT,
                        top_tok, top_logit, draw_tok, draw_logit};
  for (const void* p : ptrs)
    if (bad_ptr(p)) return set_error(TS_ERR_INVALID, "ts_score_parents_static: null or misaligned pointer");
  if (P < 0) return set_error(TS_ERR_INVALID, "ts_score_parents_static: P must be >= 0");
  if (!(T >= 0.f)) return set_error(TS_ERR_INVALID, "ts_score_parents_static: T must be >= 0");
  if (P == 0) return TS_OK;

  // records of P parents over all vocabulary tiles, plus the scoring kernel's error word
  int cap = 0;
  const size_t rec_bytes = align_up(score_scratch_bytes(ctx, P, &cap), 256);
  const size_t need = rec_bytes + 256;
  if (need > (size_t)TS_STATIC_SCRATCH_BYTES) {
    int cap1 = 0;
    const size_t unit = score_scratch_bytes(ctx, 1, &cap1);  // bytes for the smallest slot block
    char msg[256];
    snprintf(msg, sizeof(msg),
             "ts_score_parents_static: %d parents need %zu bytes of scratch, the built-in array holds %u "
             "(%zu bytes per block of %d parents for this configuration); use ts_score_parents with a workspace instead",
             P, need, (unsigned)TS_STATIC_SCRATCH_BYTES, unit, cap1);
    return set_error(TS_ERR_WORKSPACE, msg);
  }

  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_cuda_error("ts_score_parents_static(device)", e);
  if (dev != ctx->device || dev < 0 || dev >= kMaxDevices)
    return set_error(TS_ERR_INVALID, "ts_score_parents_static: the context's device must be the current device");
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {  // first call on this device: resolve the array's device address
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_static_scratch);
      if (e != cudaSuccess || !p) return set_cuda_error("ts_score_parents_static(symbol address)", e);
      g_scratch_addr[dev] = p;
    }
    scratch = g_scratch_addr[dev];
  }
  // The records need no clearing: the scoring kernel writes every record of (piece, parent < P) before
  // the merge kernel, next on the same stream, reads exactly those.  The error word and the pruning
  // state behind the records must start at zero.
  int* err = (int*)((char*)scratch + rec_bytes);
  e = cudaMemsetAsync(err, 0, 16, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(thr_base(ctx, (float*)scratch, cap), 0, thr_bytes(ctx, cap), (cudaStream_t)stream);
  if (e != cudaSuccess) return set_cuda_error("ts_score_parents_static(memset)", e);
  e = launch_score(ctx, (float*)scratch, cap, err, U, A, W, P, nullptr, parent_req, parent_depth, parent_token,
                   parent_hash, T, seed, lse0, lseT, top_tok, top_logit, draw_tok, draw_logit, (cudaStream_t)stream);
  if (e != cudaSuccess) return set_cuda_error("ts_score_parents_static", e);
  return TS_OK;
}
