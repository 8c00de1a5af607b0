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

  // records of P parents over all vocabulary tiles, laid out like the workspace version's
  WsLayout L{};
  L.Pcap = (P + 7) / 8 * 8;
  L.ntiles = ctx->tile.ntiles;
  L.K = ctx->cfg.K;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t np = (size_t)L.ntiles * L.Pcap, npk = np * (size_t)L.K;
  L.part_m = take(np * 4); L.part_s0 = take(np * 4); L.part_sT = take(np * 4);
  L.part_topv = take(npk * 4); L.part_topi = take(npk * 4);
  L.part_keyv = take(npk * 4); L.part_keyi = take(npk * 4); L.part_keyl = take(npk * 4);
  if (off > (size_t)TS_STATIC_SCRATCH_BYTES) {
    const size_t per_parent = (size_t)L.ntiles * (3 + 5 * (size_t)L.K) * 4;
    char msg[256];
    snprintf(msg, sizeof(msg),
             "ts_score_parents_static: %d parents need %zu bytes of scratch, the built-in array holds %u "
             "(about %zu parents for this configuration); use ts_score_parents with a workspace instead",
             P, off, (unsigned)TS_STATIC_SCRATCH_BYTES, (size_t)TS_STATIC_SCRATCH_BYTES / per_parent);
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
  // Nothing in the array has to start at zero: the scoring kernel writes every record of
  // (tile, parent < P) before the merge kernel, next on the same stream, reads exactly those.
  e = launch_score(ctx, L, (char*)scratch, U, A, W, P, nullptr, parent_req, parent_depth, parent_token, parent_hash,
                   T, seed, lse0, lseT, top_tok, top_logit, draw_tok, draw_logit, (cudaStream_t)stream);
  if (e != cudaSuccess) return set_cuda_error("ts_score_parents_static", e);
  return TS_OK;
}
