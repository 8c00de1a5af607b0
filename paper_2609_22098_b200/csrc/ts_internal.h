// Host-side declarations shared by the translation units of the library.
#pragma once

#include <vector>

#include "ts_common.cuh"

namespace ts {

int32_t set_error(int32_t code, const char* msg);
int32_t set_cuda_error(const char* where, cudaError_t e);

cudaError_t score_setup(ts_ctx* ctx);
cudaError_t verify_setup(ts_ctx* ctx);
cudaError_t expand_setup(ts_ctx* ctx);
size_t level_smem_bytes(const ts_config& c);

struct ScoreArgs {
  const void *U, *A, *W;
  int V, D, r, K;
  int P; const int* P_dev;
  const int* P_prev_dev;   // parent count of the previous level (nullptr: none); 0 there means 0 here
  int w_ring;              // tensor-core kernel: 0 = resident W tile, > 0 = slabs of the W ring (streaming form)
  int seed_root_B;         // seed kernel: > 0 = the parents are the roots of that many requests (parent p = request p at depth 0)
  int pdl;                 // host side: launch with programmatic stream serialization
  int few;                 // host side: this launch runs on the few-parents kernel
  const int *p_req, *p_depth, *p_token; const uint64_t* p_hash;
  float T; uint64_t seed;
  int TV, ntiles, cap, S;
  float* rec; int* err;
  unsigned* thr;    // [2][cap]: launch-wide lower bounds (logit, key) per parent, order-preserving encoding
  unsigned* slots;  // [2][cap][K]
  // Scouting for the next level (expansion only; utop == nullptr: none): while its first MMAs are on their
  // way, the tensor-core kernel finds the best base logit of its vocabulary tile in row U[b][scout_depth] of
  // every request b < scout_B that has parents in this launch (scout_live[b] > 0), and leaves (value, token)
  // at utop[(b * D + scout_depth) * ntiles + tile]: the next level's seed bounds are made from those.
  const int* scout_live; int scout_B, scout_depth; uint2* utop;
  // Base logits through the tensor cores (expansion only, at most UMMA_REQ requests): all parents of the launch
  // sit at depth u_depth (-1: not so; the persistent form takes the level instead), and the base logits of
  // requests 0 .. u_B-1 at that depth enter the MMA as extra rows of the B operand against one-hot columns of
  // the A operand, fetched by bulk-tensor loads: the scanning threads load no base logits at all.
  int u_depth, u_B;
  unsigned* seed_cnt;    // [SEED_SPLIT_PARENTS] arrival counters of the seed kernel (zero between launches)
  unsigned* seed_cand;   // [SEED_SPLIT_PARENTS][SEED_PARTS_MAX][NSEED_MAX][2] candidates (value, token) of the parts
  unsigned* thr0;   // [2][cap]: seed bounds (logit, key) per parent, written ahead of the launch; nullptr: none
  uint32_t wait_limit;   // polls before a bounded device-side wait gives up
  int lost_arrival;      // test switch: the A-tile barrier expects one arrival more than will come
};

struct MergeArgs {
  int P; const int* P_dev; int K, ntiles, cap, S, mma; float T;
  int pdl;   // host side: launch with programmatic stream serialization
  int few_ntiles;   // > 0: the level was scored by the few-parents kernel over this many tiles
  const float* rec; unsigned* thr; unsigned* slots; const unsigned* thr0;
  float *lse0, *lseT; int* top_tok; float* top_logit; int* draw_tok; float* draw_logit;
};

// Bytes of record scratch a scoring pass over up to P parents needs, and the slot capacity it implies.
size_t score_scratch_bytes(const ts_ctx* ctx, int P, int* cap_out);
// The pruning state (thresholds + slots) sits behind the records; it must be zero before a launch and
// the merge kernel leaves it zero again.
unsigned* thr_base(const ts_ctx* ctx, float* rec, int cap);
size_t thr_bytes(const ts_ctx* ctx, int cap);

// Scoring pass + merge for a parent list whose length is P (host) or *P_dev (device) when P_dev is set;
// p_bound: an upper bound of *P_dev the host knows (-1: none).  A list that cannot exceed FEW_MAX parents
// goes to the few-parents kernel where the context has one.
// rec: record scratch of score_scratch_bytes(ctx, max parents) bytes with slot capacity cap.
ScoreArgs make_score_args(const ts_ctx* ctx, float* rec, int cap, int* err, const void* U, const void* A, const void* W, float T,
                          uint64_t seed);
void set_seed_pointers(const ts_ctx* ctx, ScoreArgs& a);
// What the expansion adds to a scoring pass: seed bounds that the level kernel already wrote (no seed launch),
// and scouting of the next level's rows (see ScoreArgs).
struct ScoreExtras {
  bool thr0_ready = false;
  int root_B = 0;   // > 0: the parents are the roots of requests 0 .. root_B-1 (parent p = request p, depth 0)
  const int* scout_live = nullptr; int scout_B = 0, scout_depth = -1; uint2* utop = nullptr;
  int u_depth = -1, u_B = 0;
};
cudaError_t launch_score(const ts_ctx* ctx, float* rec, int cap, int* err, const void* U, const void* A, const void* W,
                         int P, const int* P_dev, const int* p_req, const int* p_depth, const int* p_token,
                         const uint64_t* p_hash, float T, uint64_t seed, float* lse0, float* lseT, int* top_tok,
                         float* top_logit, int* draw_tok, float* draw_logit, cudaStream_t st,
                         bool pdl = false, const int* P_prev_dev = nullptr, int p_bound = -1, const ScoreExtras* extras = nullptr);

// Kernel launch, optionally with programmatic stream serialization: the kernel may then start while the
// kernel before it in the stream is still running, and must execute pdl_wait() before it touches anything
// that kernel (or, transitively, an earlier one) wrote.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                                 Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

bool choose_tile_mma(const ts_config& c, int num_sms, int max_smem, bool allow_stream, TileCfg* out);
cudaError_t score_mma_setup(ts_ctx* ctx);
cudaError_t launch_score_mma(const ts_ctx* ctx, const ScoreArgs& a, cudaStream_t st);
// seed bounds of every parent of the list (ts_seed.cu); runs ahead of the tensor-core scoring kernel
cudaError_t launch_seed(const ts_ctx* ctx, const ScoreArgs& a, cudaStream_t st);
// the few-parents kernel (ts_score_few.cu)
int few_tiles(const ts_config& c);
bool few_supported(const ts_ctx* ctx);
cudaError_t launch_score_few(const ts_ctx* ctx, const ScoreArgs& a, int p_bound, cudaStream_t st);
// encodes (or finds cached in the context) the tensor map of W for 64-token boxes; false: not available
bool w_tensor_map(ts_ctx* ctx, const void* W);

enum KernelId { K_INIT, K_SCORE, K_MERGE, K_LEVEL, K_FINAL, K_ZROWS, K_GREEDY, K_WALK, K_CHECK, K_SCORE_FEW, K_ALLOC_SELECT, K_ALLOC_CUT, K_CALIB_ACC, K_CALIB_FIT, K_ATTN_INPUTS, K_SEED, K_PERSIST, K_COUNT };

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
