// Parent-conditioned scoring (Eq. 1) fused with logsumexp at temperature 1 and T, top-K logits and
// Gumbel top-K sibling draws (Eq. 2), one pass over the vocabulary.
//
// The vocabulary is split into tiles, one CTA per tile with its W tile resident in shared memory for
// all parents of the launch.  Two kernels produce the same per-(piece, parent) records:
//   * score_mma_kernel (ts_score_mma.cu): bf16, the bias [parents x r] . [r x tile] on the tensor
//     cores (tcgen05, accumulators in tensor memory), the scan as its epilogue;
//   * score_tile_kernel (here): fp32 FMA, any dtype / rank / vocabulary size.
// merge_kernel then folds the records of each parent.
#include "ts_internal.h"
#include "ts_scan.cuh"
#include "ts_merge.cuh"

namespace ts {

template <typename TIn, class Lists>
__global__ void __launch_bounds__(SCORE_THREADS, 1) score_tile_kernel(ScoreArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int r = a.r, TV = a.TV, V = a.V;
  TIn* Ws = reinterpret_cast<TIn*>(smem_raw);                              // [r][TV]
  float* as = reinterpret_cast<float*>(smem_raw + (size_t)r * TV * sizeof(TIn));  // [r][SCORE_THREADS]
  float* ghi = as + (size_t)r * SCORE_THREADS;                             // [512]
  const int tid = threadIdx.x;
  const int tile = blockIdx.x;
  const int t0 = tile * TV;
  const int tlen = min(TV, V - t0);
  const TIn* Wg = reinterpret_cast<const TIn*>(a.W);
  const TIn* Ug = reinterpret_cast<const TIn*>(a.U);
  const TIn* Ag = reinterpret_cast<const TIn*>(a.A);
  constexpr int VEC = Elem<TIn>::VEC;
  const bool vec_ok = (V % VEC) == 0;
  pdl_wait();
  pdl_launch_dependents();
  const int P = a.P_dev ? *a.P_dev : a.P;
  if (P <= 0) return;  // an empty level: nothing to stage

  // stage the W tile
  if (vec_ok) {
    const int per_row = TV / VEC;
    for (int i = tid; i < r * per_row; i += SCORE_THREADS) {
      const int k = i / per_row, c = (i % per_row) * VEC;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (c < tlen) v = __ldg(reinterpret_cast<const uint4*>(Wg + (size_t)k * V + t0 + c));
      *reinterpret_cast<uint4*>(Ws + (size_t)k * TV + c) = v;
    }
  } else {
    for (int i = tid; i < r * TV; i += SCORE_THREADS) {
      const int k = i / TV, c = i % TV;
      Ws[(size_t)k * TV + c] = c < tlen ? Wg[(size_t)k * V + t0 + c] : TIn(0.f);
    }
  }
  fill_gumbel_bounds(ghi, tid, SCORE_THREADS);
  __syncthreads();

  const float T = a.T, invT = T > 0.f ? 1.f / T : 1.f;
  const int K = a.K;
  const int rw = rec_words(K);

  for (int pg = 0; pg < P; pg += SCORE_THREADS) {
    const int p = pg + tid;
    if (p >= P) continue;  // no block-wide barrier below
    const int req = a.p_req[p], dep = a.p_depth[p], ptok = a.p_token[p];
    const uint64_t hash = a.p_hash[p];
    for (int k = 0; k < r; ++k) as[k * SCORE_THREADS + tid] = Elem<TIn>::to_f(Ag[(size_t)ptok * r + k]);
    const TIn* Urow = Ug + ((size_t)req * a.D + dep) * V + t0;
    RowScan<Lists> st;
    st.init(K);
    float gL = -INFINITY, gK = -INFINITY;
    const SharedThr gl{a.slots + (size_t)p * K * SLOT_STRIDE, tile % K};
    const SharedThr gk{a.slots + ((size_t)a.cap + p) * K * SLOT_STRIDE, tile % K};
    for (int c0 = 0; c0 < tlen; c0 += CHUNK) {
      const int valid = min(CHUNK, tlen - c0);
      float l[CHUNK];
      load16<TIn>(Urow + c0, vec_ok, valid, l);
      for (int k = 0; k < r; ++k) {
        const float ak = as[k * SCORE_THREADS + tid];
        float w[CHUNK];
        if (sizeof(TIn) == 2) {
          const uint4 w0 = *reinterpret_cast<const uint4*>(Ws + (size_t)k * TV + c0);
          const uint4 w1 = *reinterpret_cast<const uint4*>(Ws + (size_t)k * TV + c0 + 8);
          unpack_bf16x8(w0, w);
          unpack_bf16x8(w1, w + 8);
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(Ws) + (size_t)k * TV + c0 + 4 * i);
            w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
          }
        }
#pragma unroll
        for (int i = 0; i < CHUNK; ++i) l[i] = fmaf(ak, w[i], l[i]);
      }
      if ((c0 & (4 * CHUNK - 1)) == 0) {  // refresh the launch-wide bounds every fourth chunk
        gL = fmaxf(gL, dec_f(slots_min(gl, K)));
        if (T > 0.f) gK = fmaxf(gK, dec_f(slots_min(gk, K)));
      }
      scan_chunk(st, l, t0 + c0, valid, T, invT, a.seed, req, hash, ghi, gL, gK, gl, gk);
    }
    gL = fmaxf(gL, dec_f(slots_min(gl, K)));
    if (T > 0.f) gK = fmaxf(gK, dec_f(slots_min(gk, K)));
    st.store(a.rec + ((size_t)tile * a.cap + p) * rw, gL, gK);  // piece = (tile, 0), slot = p
  }
}

// merge_kernel: one CTA of MERGE_THREADS threads per parent (the body lives in ts_merge.cuh; the persistent
// expansion kernel runs the same body)
template <int KR>
__global__ void __launch_bounds__(MERGE_THREADS) merge_kernel(MergeArgs a) {
  __shared__ MergeSmem sm;
  pdl_wait();               // the scoring launch's records and the level's parent count
  pdl_launch_dependents();
  const int P = a.P_dev ? *a.P_dev : a.P;
  for (int p = blockIdx.x; p < P; p += gridDim.x) merge_parent<KR>(a, p, P, sm, (int)threadIdx.x, [] { __syncthreads(); });
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
size_t score_scratch_bytes(const ts_ctx* ctx, int P, int* cap_out) {
  int cap = (P + 7) / 8 * 8;
  if (ctx->use_mma) { cap = (P + 127) / 128 * 128; if (cap < 128) cap = 128; }
  if (cap_out) *cap_out = cap;
  // records, then the pruning state: 2 threshold words and 2K slot words per slot of capacity
  return record_bytes(ctx, cap) + align_up(((size_t)cap * (4 + 2 * (size_t)ctx->cfg.K * SLOT_STRIDE) + SEED_SPLIT_PARENTS + SEED_CAND_WORDS) * sizeof(unsigned), 256);
}

unsigned* thr_base(const ts_ctx* ctx, float* rec, int cap) {
  return (unsigned*)((char*)rec + record_bytes(ctx, cap));
}

// thresholds [2][cap], slots [2][cap][K] (one 128-byte line each), seed bounds [2][cap], the seed kernel's arrival
// counters [SEED_SPLIT_PARENTS]: the part of the pruning state that must be zero before a launch (the seed
// kernel's candidate scratch follows it and needs no clearing)
size_t thr_bytes(const ts_ctx* ctx, int cap) { return ((size_t)cap * (4 + 2 * (size_t)ctx->cfg.K * SLOT_STRIDE) + SEED_SPLIT_PARENTS) * sizeof(unsigned); }

// the part of the scoring arguments that does not depend on the parent list
ScoreArgs make_score_args(const ts_ctx* ctx, float* rec, int cap, int* err, const void* U, const void* A, const void* W, float T,
                          uint64_t seed) {
  const ts_config& c = ctx->cfg;
  ScoreArgs a{};
  a.U = U; a.A = A; a.W = W; a.V = c.V; a.D = c.D; a.r = c.r; a.K = c.K; a.T = T; a.seed = seed;
  a.TV = ctx->tile.TV; a.ntiles = ctx->tile.ntiles; a.w_ring = ctx->use_mma ? ctx->tile.w_ring : 0; a.cap = cap; a.S = 1; a.rec = rec; a.err = err;
  a.wait_limit = ctx->wait_limit;
  a.lost_arrival = (ctx->test_mode & TS_TEST_LOST_ARRIVAL) ? 1 : 0;
  a.thr = thr_base(ctx, rec, cap); a.slots = a.thr + 2 * (size_t)cap;
  a.thr0 = nullptr;
  a.u_depth = -1; a.u_B = 0;
  return a;
}

// where the seed bounds and the seed kernel's scratch sit behind the slots
void set_seed_pointers(const ts_ctx* ctx, ScoreArgs& a) {
  a.thr0 = a.slots + 2 * (size_t)a.cap * ctx->cfg.K * SLOT_STRIDE;
  a.seed_cnt = a.thr0 + 2 * (size_t)a.cap;
  a.seed_cand = a.seed_cnt + SEED_SPLIT_PARENTS;
}

cudaError_t launch_score(const ts_ctx* ctx, float* rec, int cap, int* err, const void* U, const void* A, const void* W,
                         int P, const int* P_dev, const int* p_req, const int* p_depth, const int* p_token,
                         const uint64_t* p_hash, float T, uint64_t seed, float* lse0, float* lseT, int* top_tok,
                         float* top_logit, int* draw_tok, float* draw_logit, cudaStream_t st, bool pdl, const int* P_prev_dev,
                         int p_bound, const ScoreExtras* extras) {
  const ts_config& c = ctx->cfg;
  ScoreArgs a = make_score_args(ctx, rec, cap, err, U, A, W, T, seed);
  a.pdl = pdl ? 1 : 0; a.P_prev_dev = P_prev_dev;
  a.P = P; a.P_dev = P_dev;
  a.p_req = p_req; a.p_depth = p_depth; a.p_token = p_token; a.p_hash = p_hash;
  cudaError_t e = cudaSuccess;
  // Which kernel scores the level: the few-parents kernel when the host knows that the list cannot hold
  // more than FEW_MAX parents (its own P, or a bound of the device-side count), the tile kernel otherwise.
  const int bound = P_dev ? p_bound : P;
  const bool run_few = ctx->use_mma && ctx->few_ok && bound >= 0 && bound <= FEW_MAX;
  const bool run_tile = !run_few;
  a.few = run_few ? 1 : 0;
  if (run_tile && ctx->use_mma && !(ctx->test_mode & TS_TEST_NO_SEED)) {
    // seed bounds first: exact values of the tokens with the largest base logits of every parent's row
    set_seed_pointers(ctx, a);
    if (!(extras && extras->thr0_ready)) {   // (an expansion's level kernel writes them for the level after it)
      ProfScope ps(ctx, K_SEED, st);
      a.seed_root_B = extras ? extras->root_B : 0;
      e = launch_seed(ctx, a, st);
      a.seed_root_B = 0;
      if (e != cudaSuccess) return e;
    }
    if (extras) { a.u_depth = extras->u_depth; a.u_B = extras->u_B; }
    if (extras && extras->utop) {
      a.utop = extras->utop; a.scout_live = extras->scout_live; a.scout_B = extras->scout_B; a.scout_depth = extras->scout_depth;
    }
  }
  if (run_tile) {
    ProfScope ps(ctx, K_SCORE, st);
    if (ctx->use_mma) {
      e = launch_score_mma(ctx, a, st);
    } else if (c.dt_U == TS_DTYPE_BF16) {
      if (c.K <= 8) e = launch_kernel(score_tile_kernel<__nv_bfloat16, RegLists<8>>, a.ntiles, SCORE_THREADS, ctx->tile.smem, st, pdl, a);
      else e = launch_kernel(score_tile_kernel<__nv_bfloat16, MemLists>, a.ntiles, SCORE_THREADS, ctx->tile.smem, st, pdl, a);
    } else {
      if (c.K <= 8) e = launch_kernel(score_tile_kernel<float, RegLists<8>>, a.ntiles, SCORE_THREADS, ctx->tile.smem, st, pdl, a);
      else e = launch_kernel(score_tile_kernel<float, MemLists>, a.ntiles, SCORE_THREADS, ctx->tile.smem, st, pdl, a);
    }
    if (e != cudaSuccess) return e;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (run_few) {
    ProfScope ps(ctx, K_SCORE_FEW, st);
    e = launch_score_few(ctx, a, bound, st);
    if (e != cudaSuccess) return e;
  }
  MergeArgs m{};
  m.pdl = a.pdl;
  m.few_ntiles = run_few ? few_tiles(c) : 0;
  m.P = P; m.P_dev = P_dev; m.K = c.K; m.ntiles = a.ntiles; m.cap = cap; m.S = a.S; m.mma = ctx->use_mma ? 1 : 0; m.T = T;
  m.rec = rec; m.thr = a.thr; m.slots = a.slots; m.thr0 = a.thr0;
  m.lse0 = lse0; m.lseT = lseT; m.top_tok = top_tok; m.top_logit = top_logit; m.draw_tok = draw_tok; m.draw_logit = draw_logit;
  int blocks = P_dev ? cap : P;
  if (blocks > 2 * ctx->num_sms) blocks = 2 * ctx->num_sms;   // parents beyond that are looped over
  if (blocks < 1) blocks = 1;
  {
    ProfScope ps(ctx, K_MERGE, st);
    if (c.K <= 8) e = launch_kernel(merge_kernel<8>, blocks, MERGE_THREADS, 0, st, pdl, m);
    else e = launch_kernel(merge_kernel<16>, blocks, MERGE_THREADS, 0, st, pdl, m);
  }
  if (e != cudaSuccess) return e;
  return cudaGetLastError();
}

cudaError_t score_setup(ts_ctx* ctx) {
  if (ctx->use_mma) return score_mma_setup(ctx);
  const int sm = (int)ctx->tile.smem;
  cudaError_t e = cudaFuncSetAttribute(score_tile_kernel<__nv_bfloat16, RegLists<8>>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(score_tile_kernel<__nv_bfloat16, MemLists>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(score_tile_kernel<float, RegLists<8>>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(score_tile_kernel<float, MemLists>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  return e;
}

}  // namespace ts

extern "C" int32_t ts_score_parents(ts_ctx* ctx, const void* U, const void* A, const void* W, int32_t P,
                                    const int32_t* parent_req, const int32_t* parent_depth,
                                    const int32_t* parent_token, const uint64_t* parent_hash, float T, uint64_t seed,
                                    float* lse0, float* lseT, int32_t* top_tok, float* top_logit, int32_t* draw_tok,
                                    float* draw_logit, void* ws, size_t ws_bytes, void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_score_parents: null context");
  const void* ptrs[] = {U, A, W, parent_req, parent_depth, parent_token, parent_hash, lse0, lseT,
                        top_tok, top_logit, draw_tok, draw_logit, ws};
  for (const void* p : ptrs)
    if (!p || ((uintptr_t)p & 15u)) return set_error(TS_ERR_INVALID, "ts_score_parents: null or misaligned pointer");
  const WsLayout L = make_layout(ctx, ctx->cfg.max_batch);
  if (P < 0 || P > L.Pcap)
    return set_error(TS_ERR_INVALID, "ts_score_parents: P out of range");
  if (!(T >= 0.f)) return set_error(TS_ERR_INVALID, "ts_score_parents: T must be >= 0");
  if (ws_bytes < L.total) return set_error(TS_ERR_WORKSPACE, "ts_score_parents: workspace too small");
  if (P == 0) return TS_OK;
  cudaError_t e = cudaMemsetAsync((char*)ws + L.err, 0, 16, (cudaStream_t)stream);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(thr_base(ctx, (float*)((char*)ws + L.rec), L.rec_cap), 0, thr_bytes(ctx, L.rec_cap), (cudaStream_t)stream);
  if (e != cudaSuccess) return set_cuda_error("ts_score_parents(memset)", e);
  e = launch_score(ctx, (float*)((char*)ws + L.rec), L.rec_cap, (int*)((char*)ws + L.err), U, A, W, P, nullptr,
                               parent_req, parent_depth, parent_token, parent_hash, T, seed, lse0, lseT, top_tok,
                               top_logit, draw_tok, draw_logit, (cudaStream_t)stream);
  if (e != cudaSuccess) return set_cuda_error("ts_score_parents", e);
  return TS_OK;
}
