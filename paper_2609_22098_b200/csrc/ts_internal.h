// Host-side declarations shared by the translation units of the library.
#pragma once

#include <vector>

#include "ts_common.cuh"

namespace ts {

int32_t set_error(int32_t code, const char* msg);
int32_t set_cuda_error(const char* where, cudaError_t e);

cudaError_t score_setup(ts_ctx* ctx);
cudaError_t verify_setup(ts_ctx* ctx);

// Scoring pass + merge for a parent list whose length is P (host) or *P_dev (device) when P_dev is set.
cudaError_t launch_score(const ts_ctx* ctx, const WsLayout& L, char* ws, const void* U, const void* A, const void* W,
                         int P, const int* P_dev, const int* p_req, const int* p_depth, const int* p_token,
                         const uint64_t* p_hash, float T, uint64_t seed, float* lse0, float* lseT, int* top_tok,
                         float* top_logit, int* draw_tok, float* draw_logit, cudaStream_t st);

enum KernelId { K_INIT, K_SCORE, K_MERGE, K_LEVEL, K_FINAL, K_ZROWS, K_GREEDY, K_WALK, K_CHECK, K_COUNT };

struct Prof {
  bool on = false;
  std::vector<cudaEvent_t> ev;  // pairs: start, stop
  std::vector<int> ids;
  size_t used = 0;
  int64_t launches[K_COUNT] = {};
};

// Brackets one kernel launch with an event pair when instrumentation is on; always counts it.
struct ProfScope {
  Prof* p; cudaStream_t st; size_t slot; bool rec;
  ProfScope(const ts_ctx* ctx, int id, cudaStream_t s) : p((Prof*)ctx->prof), st(s), slot(0), rec(false) {
    if (!p) return;
    p->launches[id]++;
    if (p->on && p->used < p->ids.size()) {
      slot = p->used++; p->ids[slot] = id; rec = true;
      cudaEventRecord(p->ev[2 * slot], st);
    }
  }
  ~ProfScope() { if (rec) cudaEventRecord(p->ev[2 * slot + 1], st); }
};

inline bool bad_ptr(const void* p) { return !p || ((uintptr_t)p & 15u); }

}  // namespace ts
