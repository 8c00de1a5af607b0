// Best-first tree expansion with the theta stop (Algorithm 1, Section 3.5), level-synchronous.
//
// Why levels give exactly the heap's result: a slot's key never exceeds the key of the slot that
// created it (p_hat <= 1, p_hat monotone in q0, and a re-pushed sibling slot maximises over a smaller
// set), so heap pops are non-increasing and the tree is "the first N slots in sorted key order among
// those with key >= theta" of the lazily generated slot forest.  With ties broken by (depth, sibling
// rank path) that order puts every slot after the slots it depends on.  Per request a pool of at most
// N admitted slots is kept; at level d every pool node of depth d whose survival is >= theta is scored
// in one batched pass, its slots are formed, and the pool is cut back to the best N.  A node outside
// the pool at its own level can never enter the final tree, so nothing else needs scoring.
#include <math.h>

#include "ts_internal.h"
#include "ts_scan.cuh"
#include "ts_level.cuh"

namespace ts {

__global__ void expand_init_kernel(ExpandArgs a) {
  pdl_wait();                // whatever ran before in the stream may still be reading what this kernel resets
  pdl_launch_dependents();   // the first scoring launch may run its preamble beside this kernel
  const int b = blockIdx.x;
  // pruning state of the scoring launches: the threshold words, then one word per slot (the slots sit
  // SLOT_STRIDE words apart; only the first word of each is ever used)
  for (int i = b * blockDim.x + threadIdx.x; i < a.thr_words; i += gridDim.x * blockDim.x)
    a.thr[i < a.thr_head ? i : a.thr_head + (size_t)(i - a.thr_head) * SLOT_STRIDE] = 0u;
  if (b == 0) for (int i = threadIdx.x; i < SEED_SPLIT_PARENTS; i += blockDim.x) a.seed_cnt[i] = 0u;
  if (b == 0 && threadIdx.x < 4) a.ex_barrier[threadIdx.x] = 0u;
  if (b >= a.B) return;
  for (int s = threadIdx.x; s < a.N; s += blockDim.x) a.pl_alive[(size_t)b * a.N + s] = 0;
  if (threadIdx.x == 0) {
    const int tok = a.anchor[b];
    const bool ok = tok >= 0 && tok < a.V && a.theta[b] == a.theta[b];
    a.status[b] = ok ? TS_OK : TS_ERR_INVALID;
    a.lst_req[0][b] = b; a.lst_depth[0][b] = 0; a.lst_token[0][b] = ok ? tok : 0; a.lst_hash[0][b] = 0ull;
    a.lst_slot[0][b] = -1;
    a.req_npar[b] = 1; a.req_base[b] = b; a.req_nscored[b] = 0;
    a.root_lseT[b] = nanf("");
    if (b == 0) {
      a.err[0] = 0;
      a.lvl_count[0] = a.B;
      for (int d = 1; d <= DMAX + 1; ++d) a.lvl_count[d] = 0;
    }
  }
}

// One CTA per request; level d = depth of the parents just scored (body in ts_level.cuh).
__global__ void __launch_bounds__(LEVEL_THREADS) expand_level_kernel(ExpandArgs a, int d, int seed_next) {
  extern __shared__ __align__(16) unsigned char sm_raw[];
  __shared__ LevelSmem sm;
  pdl_wait();               // merged scoring results of this level
  pdl_launch_dependents();
  level_step(a, d, seed_next, (int)blockIdx.x, sm, sm_raw, (int)threadIdx.x, [] { __syncthreads(); });
}

struct FinalArgs {
  int B, N, words;
  const int *pl_alive, *pl_depth, *pl_parent, *pl_sib, *pl_tok;
  const double *pl_logkey, *pl_logS; const float *pl_q0, *pl_logqT, *pl_lseT; const uint64_t *pl_hash, *pl_path;
  const float* root_lseT; const int* req_nscored;
  int *n_nodes, *tok, *parent, *depth, *sib_rank; float *logS, *q0, *logqT, *logkey; int* pop_rank;
  uint64_t* node_hash; float* node_lseT; uint64_t* mask; int* n_scored;
  const int* err; int* status;   // a bounded wait that ran out during the expansion is reported for every request still marked fine
};

// Canonical (BFS) renumbering, outputs and ancestor bitmasks; one CTA per request.
__global__ void __launch_bounds__(256) expand_finalize_kernel(FinalArgs a) {
  // the pool of one request is small: it is ranked, renumbered and masked out of shared memory
  __shared__ int s_canon[256], s_alive[256], s_depth[256], s_par[256], s_cpar[256];
  __shared__ uint64_t s_path[256];
  __shared__ double s_key[256];
  __shared__ uint64_t s_mask[256 * 4];
  __shared__ int s_n;
  const int b = blockIdx.x, tid = threadIdx.x, N = a.N;
  const size_t pb = (size_t)b * N;
  pdl_wait();
  if (tid == 0) s_n = 0;
  for (int s = tid; s < N; s += blockDim.x) {
    s_alive[s] = a.pl_alive[pb + s]; s_depth[s] = a.pl_depth[pb + s]; s_path[s] = a.pl_path[pb + s];
    s_key[s] = a.pl_logkey[pb + s]; s_par[s] = a.pl_parent[pb + s];
  }
  __syncthreads();
  for (int s = tid; s < N; s += blockDim.x) {
    s_canon[s] = -1;
    if (!s_alive[s]) continue;
    const int ds = s_depth[s]; const uint64_t ps = s_path[s]; const double ks = s_key[s];
    int cr = 0, pr = 0;
    for (int t = 0; t < N; ++t) {
      if (t == s || !s_alive[t]) continue;
      const int dt = s_depth[t]; const uint64_t pt = s_path[t];
      if (dt < ds || (dt == ds && pt < ps)) ++cr;
      if (before(s_key[t], dt, pt, ks, ds, ps)) ++pr;
    }
    s_canon[s] = cr;
    atomicAdd(&s_n, 1);
    const size_t o = pb + cr;
    a.tok[o] = a.pl_tok[pb + s]; a.depth[o] = ds; a.sib_rank[o] = a.pl_sib[pb + s];
    a.logS[o] = (float)a.pl_logS[pb + s]; a.q0[o] = a.pl_q0[pb + s]; a.logqT[o] = a.pl_logqT[pb + s];
    if (a.logkey) a.logkey[o] = (float)ks;
    if (a.pop_rank) a.pop_rank[o] = pr;
    a.node_hash[(size_t)b * (N + 1) + cr + 1] = a.pl_hash[pb + s];
    if (a.node_lseT) a.node_lseT[(size_t)b * (N + 1) + cr + 1] = a.pl_lseT[pb + s];
  }
  __syncthreads();
  for (int s = tid; s < N; s += blockDim.x) {
    if (s_canon[s] < 0) continue;
    const int ps = s_par[s];
    const int cp = ps < 0 ? -1 : s_canon[ps];
    s_cpar[s_canon[s]] = cp;
    a.parent[pb + s_canon[s]] = cp;
  }
  if (tid == 0) {
    if (*reinterpret_cast<const volatile int*>(a.err) != 0 && a.status[b] == TS_OK) a.status[b] = TS_ERR_TIMEOUT;
    a.n_nodes[b] = s_n;
    a.node_hash[(size_t)b * (N + 1)] = 0ull;
    if (a.node_lseT) a.node_lseT[(size_t)b * (N + 1)] = a.root_lseT[b];
    if (a.n_scored) a.n_scored[b] = a.req_nscored[b];
  }
  __syncthreads();
  // a node's mask row = its parent's row plus its own bit; parents precede children in canonical order
  const int n = s_n;
  if (tid < a.words) {
    for (int i = 0; i < n; ++i) {
      const int p = s_cpar[i];
      uint64_t m = p >= 0 ? s_mask[p * a.words + tid] : 0ull;
      if (i / 64 == tid) m |= 1ull << (i % 64);
      s_mask[i * a.words + tid] = m;
    }
  }
  __syncthreads();
  for (int i = tid; i < n * a.words; i += blockDim.x) a.mask[pb * a.words + i] = s_mask[i];
}

// the level kernel ranks a request's pool and candidates out of dynamic shared memory: opt in once per context
// dynamic shared memory of the level kernel: the ranking entries of a request's pool and candidates, later
// reused for the seed bounds' staged W columns [2K][r], per-pair results [Nmax][2K][2] and a batch of rows of A
size_t level_smem_bytes(const ts_config& c) {
  const size_t entries = (size_t)(c.Nmax + c.Nmax * c.K) * sizeof(Entry);
  const size_t ns = (size_t)(2 * c.K > NSEED_MAX ? NSEED_MAX : (2 * c.K < 8 ? 8 : 2 * c.K));
  const size_t seeds = ns * (size_t)(c.r + 1) * 4 + (size_t)c.Nmax * ns * 2 * 4 + (size_t)SEED_PBATCH * c.r * 2;
  return entries > seeds ? entries : seeds;
}

cudaError_t expand_setup(ts_ctx* ctx) {
  const size_t level_smem = level_smem_bytes(ctx->cfg);
  if (level_smem <= 48 * 1024) return cudaSuccess;
  return cudaFuncSetAttribute(expand_level_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)level_smem);
}

}  // namespace ts

extern "C" int32_t ts_expand_tree(ts_ctx* ctx, const void* U, const void* A, const void* W, int32_t B,
                                  const int32_t* anchor_tok, const float* theta, float T, uint64_t seed,
                                  int32_t* n_nodes, int32_t* tok, int32_t* parent, int32_t* depth, int32_t* sib_rank,
                                  float* logS, float* q0, float* logqT, float* logkey, int32_t* pop_rank,
                                  uint64_t* node_hash, float* node_lseT, uint64_t* mask, int32_t* n_scored,
                                  int32_t* status, void* ws_v, size_t ws_bytes, void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_expand_tree: null context");
  const void* req[] = {U, A, W, anchor_tok, theta, n_nodes, tok, parent, depth, sib_rank, logS, q0, logqT,
                       node_hash, mask, status, ws_v};
  for (const void* p : req)
    if (bad_ptr(p)) return set_error(TS_ERR_INVALID, "ts_expand_tree: null or misaligned pointer");
  const void* opt[] = {logkey, pop_rank, node_lseT, n_scored};
  for (const void* p : opt)
    if (p && ((uintptr_t)p & 15u)) return set_error(TS_ERR_INVALID, "ts_expand_tree: misaligned optional pointer");
  const ts_config& c = ctx->cfg;
  if (B < 1 || B > c.max_batch) return set_error(TS_ERR_INVALID, "ts_expand_tree: B out of range");
  if (!(T >= 0.f)) return set_error(TS_ERR_INVALID, "ts_expand_tree: T must be >= 0");
  const WsLayout L = make_layout(ctx, B);
  if (ws_bytes < L.total) return set_error(TS_ERR_WORKSPACE, "ts_expand_tree: workspace too small");
  char* ws = (char*)ws_v;
  cudaStream_t st = (cudaStream_t)stream;

  ExpandArgs a{};
  a.B = B; a.D = c.D; a.K = c.K; a.N = c.Nmax; a.V = c.V; a.T = T; a.anchor = anchor_tok; a.theta = theta;
  a.calib = ctx->calib;
  a.calib_qT = (ctx->ablation & TS_ABLATE_CALIB_QT) ? 1 : 0;
  for (int i = 0; i < 2; ++i) {
    a.lst_req[i] = (int*)(ws + L.lst_req[i]); a.lst_depth[i] = (int*)(ws + L.lst_depth[i]);
    a.lst_token[i] = (int*)(ws + L.lst_token[i]); a.lst_hash[i] = (uint64_t*)(ws + L.lst_hash[i]);
    a.lst_slot[i] = (int*)(ws + L.lst_slot[i]);
  }
  a.lvl_count = (int*)(ws + L.lvl_count);
  float* res_lse0 = (float*)(ws + L.res_lse0); float* res_lseT = (float*)(ws + L.res_lseT);
  int* res_top_tok = (int*)(ws + L.res_top_tok); float* res_top_logit = (float*)(ws + L.res_top_logit);
  int* res_draw_tok = (int*)(ws + L.res_draw_tok); float* res_draw_logit = (float*)(ws + L.res_draw_logit);
  a.res_lse0 = res_lse0; a.res_lseT = res_lseT; a.res_top_tok = res_top_tok; a.res_top_logit = res_top_logit;
  a.res_draw_tok = res_draw_tok; a.res_draw_logit = res_draw_logit;
  a.pl_alive = (int*)(ws + L.pl_alive); a.pl_depth = (int*)(ws + L.pl_depth); a.pl_parent = (int*)(ws + L.pl_parent);
  a.pl_sib = (int*)(ws + L.pl_sib); a.pl_tok = (int*)(ws + L.pl_tok);
  a.pl_logkey = (double*)(ws + L.pl_logkey); a.pl_logS = (double*)(ws + L.pl_logS);
  a.pl_q0 = (float*)(ws + L.pl_q0); a.pl_logqT = (float*)(ws + L.pl_logqT); a.pl_lseT = (float*)(ws + L.pl_lseT);
  a.pl_hash = (uint64_t*)(ws + L.pl_hash); a.pl_path = (uint64_t*)(ws + L.pl_path);
  a.root_lseT = (float*)(ws + L.root_lseT);
  a.req_npar = (int*)(ws + L.req_npar); a.req_base = (int*)(ws + L.req_base); a.req_nscored = (int*)(ws + L.req_nscored);
  a.cd_valid = (int*)(ws + L.cd_valid); a.cd_parent = (int*)(ws + L.cd_parent); a.cd_sib = (int*)(ws + L.cd_sib);
  a.cd_tok = (int*)(ws + L.cd_tok); a.cd_logkey = (double*)(ws + L.cd_logkey); a.cd_logS = (double*)(ws + L.cd_logS);
  a.cd_q0 = (float*)(ws + L.cd_q0); a.cd_logqT = (float*)(ws + L.cd_logqT); a.cd_rank = (int*)(ws + L.cd_rank);
  a.status = status; a.err = (int*)(ws + L.err);
  a.thr = thr_base(ctx, (float*)(ws + L.rec), L.rec_cap);
  a.thr_head = 2 * L.rec_cap; a.thr_words = a.thr_head + 2 * L.rec_cap * c.K;   // words to clear, not their span
  a.thr0 = a.thr + 2 * (size_t)L.rec_cap + 2 * (size_t)L.rec_cap * c.K * SLOT_STRIDE;
  a.seed_cnt = a.thr0 + 2 * (size_t)L.rec_cap;
  a.U = U; a.A = A; a.W = W; a.r = c.r; a.ntiles = ctx->tile.ntiles; a.cap = L.rec_cap; a.seed = seed;
  a.utop = (const uint2*)(ws + L.utop);
  a.ex_barrier = (unsigned*)(ws + L.ex_barrier);

  cudaError_t e0;
  { ProfScope ps(ctx, K_INIT, st); e0 = launch_kernel(expand_init_kernel, B > 296 ? B : 296, 256, 0, st, true, a); }
  cudaError_t e = e0 != cudaSuccess ? e0 : cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(init)", e);
  const size_t level_smem = level_smem_bytes(c);   // opted into at ts_create when above 48 KB
  const bool seeds_on = ctx->use_mma && !(ctx->test_mode & TS_TEST_NO_SEED);
  // Three forms.  Default: one launch per step of every level (score, merge, level step), chained, for the first
  // TAIL_FROM levels, and one cooperative launch for all levels after those: trees usually end before them, and
  // three launches per empty level (each a hop in the chain of dependent launches) become one that returns at once.
  // TS_TEST_PERSIST: the cooperative launch runs every level.  TS_TEST_NO_TAIL: no cooperative launch at all.
  constexpr int TAIL_FROM = 4;
  int coop_from = c.D;   // first level of the cooperative launch (D: none)
  if (seeds_on && (ctx->test_mode & TS_TEST_PERSIST) && persistent_supported(ctx, B, 0)) coop_from = 0;
  else if (seeds_on && !(ctx->test_mode & TS_TEST_NO_TAIL)) {
    // (a handful of requests rarely has parents at the fourth level either: one level earlier there)
    const int from = (ctx->few_ok && B <= FEW_MAX) ? TAIL_FROM - 1 : TAIL_FROM;
    if (c.D > from + 1 && persistent_supported(ctx, B, from)) coop_from = from;
  }
  long long level_bound = B;   // parents a level can have at most: B at the root, K times more per level, B * Nmax overall
  // Seed bounds of a level on the tensor-core kernel: made by the level kernel before it when that level's scoring
  // launch scouted the rows (it does whenever it runs on the tensor-core kernel itself); by a seed launch otherwise
  // (the root level, and the first tensor-core level after levels on the few-parents kernel).
  bool scouted_prev = false;
  for (int d = 0; d < coop_from; ++d) {
    const int cur = d & 1;
    const bool on_mma = ctx->use_mma && !(ctx->few_ok && level_bound <= FEW_MAX);
    ScoreExtras ex;
    ex.thr0_ready = scouted_prev;
    ex.root_B = d == 0 ? B : 0;
    const bool scout = seeds_on && on_mma && d + 1 < c.D;
    ex.u_depth = d; ex.u_B = B;
    if (scout) { ex.utop = (uint2*)(ws + L.utop); ex.scout_live = a.req_npar; ex.scout_B = B; ex.scout_depth = d + 1; }
    e = launch_score(ctx, (float*)(ws + L.rec), L.rec_cap, (int*)(ws + L.err), U, A, W, 0, a.lvl_count + d,
                     a.lst_req[cur], a.lst_depth[cur], a.lst_token[cur],
                     a.lst_hash[cur], T, seed, res_lse0, res_lseT, res_top_tok, res_top_logit, res_draw_tok,
                     res_draw_logit, st, /*pdl=*/true, d > 0 ? a.lvl_count + d - 1 : nullptr, (int)level_bound, &ex);
    level_bound = level_bound * c.K < (long long)B * c.Nmax ? level_bound * c.K : (long long)B * c.Nmax;
    if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(score)", e);
    { ProfScope ps(ctx, K_LEVEL, st); e = launch_kernel(expand_level_kernel, B, LEVEL_THREADS, level_smem, st, true, a, d, scout ? 1 : 0); }
    scouted_prev = scout;
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(level)", e);
  }
  if (coop_from < c.D) {
    // One cooperative launch runs the remaining levels: scan, merge, level step, separated by grid barriers.  Its
    // first level's seed bounds come from a seed launch (the root level) or from the level kernel before it.
    ScoreArgs sa = make_score_args(ctx, (float*)(ws + L.rec), L.rec_cap, (int*)(ws + L.err), U, A, W, T, seed);
    sa.pdl = 1; sa.P = 0; sa.P_dev = a.lvl_count + coop_from;
    sa.P_prev_dev = coop_from > 0 ? a.lvl_count + coop_from - 1 : nullptr;
    const int cur = coop_from & 1;
    sa.p_req = a.lst_req[cur]; sa.p_depth = a.lst_depth[cur]; sa.p_token = a.lst_token[cur]; sa.p_hash = a.lst_hash[cur];
    set_seed_pointers(ctx, sa);
    if (coop_from == 0) {
      ProfScope ps(ctx, K_SEED, st);
      e = launch_seed(ctx, sa, st);
      if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(seed)", e);
    }
    sa.utop = (uint2*)(ws + L.utop); sa.scout_live = a.req_npar; sa.scout_B = B; sa.scout_depth = coop_from + 1;
    sa.u_depth = coop_from; sa.u_B = B;
    PersistArgs pa{};
    pa.on = 1; pa.first = coop_from; pa.nlevels = c.D; pa.ex = a; pa.barrier = a.ex_barrier;
    pa.lost_arrival = (ctx->test_mode & TS_TEST_LOST_ARRIVAL) ? 1 : 0;
    MergeArgs& m = pa.mg;
    m.pdl = 0; m.few_ntiles = 0; m.P = 0; m.P_dev = nullptr; m.K = c.K; m.ntiles = sa.ntiles; m.cap = L.rec_cap; m.S = 1; m.mma = 1; m.T = T;
    m.rec = sa.rec; m.thr = sa.thr; m.slots = sa.slots; m.thr0 = sa.thr0;
    m.lse0 = res_lse0; m.lseT = res_lseT; m.top_tok = res_top_tok; m.top_logit = res_top_logit; m.draw_tok = res_draw_tok;
    m.draw_logit = res_draw_logit;
    { ProfScope ps(ctx, K_PERSIST, st); e = launch_expand_persistent(ctx, sa, pa, st); }
    if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(cooperative)", e);
  }
  FinalArgs f{};
  f.B = B; f.N = c.Nmax; f.words = L.words;
  f.pl_alive = a.pl_alive; f.pl_depth = a.pl_depth; f.pl_parent = a.pl_parent; f.pl_sib = a.pl_sib; f.pl_tok = a.pl_tok;
  f.pl_logkey = a.pl_logkey; f.pl_logS = a.pl_logS; f.pl_q0 = a.pl_q0; f.pl_logqT = a.pl_logqT; f.pl_lseT = a.pl_lseT;
  f.pl_hash = a.pl_hash; f.pl_path = a.pl_path; f.root_lseT = a.root_lseT; f.req_nscored = a.req_nscored;
  f.n_nodes = n_nodes; f.tok = tok; f.parent = parent; f.depth = depth; f.sib_rank = sib_rank; f.logS = logS; f.q0 = q0;
  f.logqT = logqT; f.logkey = logkey; f.pop_rank = pop_rank; f.node_hash = node_hash; f.node_lseT = node_lseT;
  f.mask = mask; f.n_scored = n_scored; f.err = a.err; f.status = status;
  { ProfScope ps(ctx, K_FINAL, st); e = launch_kernel(expand_finalize_kernel, B, 256, 0, st, true, f); }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(finalize)", e);
  return TS_OK;
}
