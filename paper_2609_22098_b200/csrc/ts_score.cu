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

// ------------------------------------------------------------------------------------------------
// Merge of the per-piece records: one CTA per parent.
// Every thread folds its share of the pieces into a private (max, sums) pair and private top-K
// lists; the block then takes K rounds of arg-max over the list heads (value desc, token asc).
// ------------------------------------------------------------------------------------------------
constexpr int MERGE_THREADS = 512;
constexpr int MERGE_WARPS = MERGE_THREADS / 32;

__device__ __forceinline__ bool better(float va, int ia, float vb, int ib) { return va > vb || (va == vb && ia < ib); }

// Sorted list (value desc, token asc) with compile-time indices only, so it lives in registers.
// The head is always entry 0: taking it shifts the rest up.
template <int KR>
struct MList {
  float v[KR]; int i[KR]; float l[KR];
  __device__ __forceinline__ void init() {
#pragma unroll
    for (int j = 0; j < KR; ++j) { v[j] = -INFINITY; i[j] = 0x7FFFFFFF; l[j] = 0.f; }
  }
  __device__ __forceinline__ void insert(float val, int idx, float lg) {
    if (!better(val, idx, v[KR - 1], i[KR - 1])) return;
#pragma unroll
    for (int j = KR - 1; j >= 0; --j) {
      const bool up = (j > 0) && better(val, idx, v[j > 0 ? j - 1 : 0], i[j > 0 ? j - 1 : 0]);
      if (up) { v[j] = v[j > 0 ? j - 1 : 0]; i[j] = i[j > 0 ? j - 1 : 0]; l[j] = l[j > 0 ? j - 1 : 0]; }
      else if (j == KR - 1 || better(val, idx, v[j], i[j])) { v[j] = val; i[j] = idx; l[j] = lg; }
    }
  }
  __device__ __forceinline__ void pop() {
#pragma unroll
    for (int j = 0; j + 1 < KR; ++j) { v[j] = v[j + 1]; i[j] = i[j + 1]; l[j] = l[j + 1]; }
    v[KR - 1] = -INFINITY; i[KR - 1] = 0x7FFFFFFF; l[KR - 1] = 0.f;
  }
};

// K rounds of block-wide arg-max over the heads of the threads' sorted lists
template <int KR>
__device__ void block_select(MList<KR>& mine, int K, int* out_tok, float* out_val, float* s_v, int* s_i, float* s_l) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int j = 0; j < K; ++j) {
    float wv = mine.v[0]; int wi = mine.i[0]; float wl = mine.l[0];
    for (int off = 16; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, wv, off);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, wi, off);
      const float ol = __shfl_xor_sync(0xFFFFFFFFu, wl, off);
      if (better(ov, oi, wv, wi)) { wv = ov; wi = oi; wl = ol; }
    }
    if (lane == 0) { s_v[warp] = wv; s_i[warp] = wi; s_l[warp] = wl; }
    __syncthreads();
    float gv = s_v[0]; int gi = s_i[0]; float gl = s_l[0];
#pragma unroll
    for (int w = 1; w < MERGE_WARPS; ++w)
      if (better(s_v[w], s_i[w], gv, gi)) { gv = s_v[w]; gi = s_i[w]; gl = s_l[w]; }
    if (gi != 0x7FFFFFFF && mine.i[0] == gi) mine.pop();  // tokens are unique per list
    if (tid == 0) { out_tok[j] = gi == 0x7FFFFFFF ? -1 : gi; out_val[j] = gi == 0x7FFFFFFF ? 0.f : gl; }
    __syncthreads();
  }
}

constexpr int MERGE_CAP = 768;   // candidates per list the fast path can hold

// The K best of a candidate array in shared memory (value desc, token asc), by counting: a candidate's
// place is the number of candidates that beat it (tokens are unique per list, so places are too).  With
// tight bounds a few dozen candidates arrive here, and the whole selection is one short pass.
__device__ void rank_select(const float* cv, const int* ci, const float* cl, int n, int K, int t, int nt, int* out_tok, float* out_val) {
  for (int e = t; e < n; e += nt) {
    const float v = cv[e]; const int idx = ci[e];
    int rank = 0;
    for (int f = 0; f < n; ++f) rank += better(cv[f], ci[f], v, idx) ? 1 : 0;
    if (rank < K) { out_tok[rank] = idx; out_val[rank] = cl[e]; }
  }
  for (int j = n + t; j < K; j += nt) { out_tok[j] = -1; out_val[j] = 0.f; }
}

template <int KR>
__global__ void __launch_bounds__(MERGE_THREADS) merge_kernel(MergeArgs a) {
  __shared__ float s_v[MERGE_WARPS]; __shared__ int s_i[MERGE_WARPS]; __shared__ float s_l[MERGE_WARPS];
  __shared__ float s_m[MERGE_WARPS], s_s0[MERGE_WARPS], s_sT[MERGE_WARPS];
  __shared__ float c_v[2][MERGE_CAP]; __shared__ int c_i[2][MERGE_CAP]; __shared__ float c_l[2][MERGE_CAP];
  __shared__ int c_n[2];
  pdl_wait();               // the scoring launch's records and the level's parent count
  pdl_launch_dependents();
  const int P = a.P_dev ? *a.P_dev : a.P;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float invT = a.T > 0.f ? 1.f / a.T : 1.f;
  const int K = a.K, rw = rec_words(K);
  const bool few = a.few_ntiles > 0;   // the level was scored by the few-parents kernel
  const int R = few ? 1 : (a.mma ? mma_replicas(P) : 1);
  const int npieces = few ? a.few_ntiles : a.ntiles * a.S * R;
  for (int p = blockIdx.x; p < P; p += gridDim.x) {
    // final launch-wide lower bounds of this parent's K-th best logit / key: entries below cannot win
    const SharedThr gl{a.slots + (size_t)p * K * SLOT_STRIDE, 0}, gk{a.slots + ((size_t)a.cap + p) * K * SLOT_STRIDE, 0};
    float bL = dec_f(slots_min(gl, K)), bK = a.T > 0.f ? dec_f(slots_min(gk, K)) : -INFINITY;
    if (a.thr0) {   // never below the parent's seed bounds
      bL = fmaxf(bL, dec_f(__ldcg(a.thr0 + p)));
      if (a.T > 0.f) bK = fmaxf(bK, dec_f(__ldcg(a.thr0 + (size_t)a.cap + p)));
    }
    if (tid < 2) c_n[tid] = 0;
    __syncthreads();
    float m = -INFINITY, s0 = 0.f, sT = 0.f;
    auto rec_of = [&](int q) {
      if (few) return a.rec + ((size_t)q * FEW_MAX + p) * rw;
      const int ts_ = q / R, rho = q % R;
      const int slot = R > 1 ? rho * (128 / R) + p : p;
      return a.rec + ((size_t)ts_ * a.cap + slot) * rw;
    };
    // the header of the next record is requested before this one's entries, so that a thread with
    // several records pays one memory round trip per record, not two
    // ... together with the record's best key: a record whose best logit (its maximum, in the header) and
    // best key are below the final bounds has nothing to offer, and its entries are not read at all
    float4 hn = make_float4(-INFINITY, 0.f, 0.f, 0.f);
    float kn = -INFINITY;
    if (tid < npieces) {
      hn = __ldcg(reinterpret_cast<const float4*>(rec_of(tid)));
      if (a.T > 0.f) kn = __ldcg(rec_of(tid) + 4 + 2 * K);
    }
    for (int q = tid; q < npieces; q += MERGE_THREADS) {
      const float* rec = rec_of(q);
      const float4 h = hn;
      const float kbest = kn;
      if (q + MERGE_THREADS < npieces) {
        hn = __ldcg(reinterpret_cast<const float4*>(rec_of(q + MERGE_THREADS)));
        if (a.T > 0.f) kn = __ldcg(rec_of(q + MERGE_THREADS) + 4 + 2 * K);
      }
      const float* f = rec + 4; const int* ii = reinterpret_cast<const int*>(rec) + 4;
      // all entries of the record are requested at once (independent loads), then filtered
      float tv[KR], kv[KR], kl[KR]; int ti[KR], ki[KR];
      const int cnt = __float_as_int(h.w);
      const int nt = h.x >= bL ? (cnt & 255) : 0, nk = kbest >= bK ? ((cnt >> 8) & 255) : 0;   // entries worth reading
#pragma unroll
      for (int j = 0; j < KR; ++j) {
        ti[j] = j < nt ? __ldcg(ii + K + j) : -1;
        tv[j] = j < nt ? __ldcg(f + j) : 0.f;
        ki[j] = (j < nk && a.T > 0.f) ? __ldcg(ii + 3 * K + j) : -1;
        kv[j] = (j < nk && a.T > 0.f) ? __ldcg(f + 2 * K + j) : 0.f;
        kl[j] = (j < nk && a.T > 0.f) ? __ldcg(f + 4 * K + j) : 0.f;
      }
      if (h.x == -INFINITY) continue;  // a piece that scanned nothing
      if (h.x > m) { const float d = m - h.x; s0 *= __expf(d); sT *= __expf(d * invT); m = h.x; }
      const float d = h.x - m;
      s0 += h.y * __expf(d); sT += h.z * __expf(d * invT);
#pragma unroll
      for (int j = 0; j < KR; ++j) {
        if (ti[j] >= 0 && tv[j] >= bL) {
          const int e = atomicAdd(&c_n[0], 1);
          if (e < MERGE_CAP) { c_v[0][e] = tv[j]; c_i[0][e] = ti[j]; c_l[0][e] = tv[j]; }
        }
        if (ki[j] >= 0 && kv[j] >= bK) {
          const int e = atomicAdd(&c_n[1], 1);
          if (e < MERGE_CAP) { c_v[1][e] = kv[j]; c_i[1][e] = ki[j]; c_l[1][e] = kl[j]; }
        }
      }
    }
    // fold the (max, sums) pairs
    for (int off = 16; off > 0; off >>= 1) {
      const float om = __shfl_xor_sync(0xFFFFFFFFu, m, off);
      const float o0 = __shfl_xor_sync(0xFFFFFFFFu, s0, off);
      const float oT = __shfl_xor_sync(0xFFFFFFFFu, sT, off);
      const float nm = fmaxf(m, om);
      if (nm > -INFINITY) {
        s0 = s0 * __expf(m - nm) + o0 * __expf(om - nm);
        sT = sT * __expf((m - nm) * invT) + oT * __expf((om - nm) * invT);
      }
      m = nm;
    }
    if (lane == 0) { s_m[warp] = m; s_s0[warp] = s0; s_sT[warp] = sT; }
    __syncthreads();
    if (tid == 0) {
      float gm = -INFINITY;
      for (int w = 0; w < MERGE_WARPS; ++w) gm = fmaxf(gm, s_m[w]);
      float g0 = 0.f, gT = 0.f;
      for (int w = 0; w < MERGE_WARPS; ++w)
        if (s_m[w] > -INFINITY) { g0 += s_s0[w] * __expf(s_m[w] - gm); gT += s_sT[w] * __expf((s_m[w] - gm) * invT); }
      a.lse0[p] = gm + logf(g0);
      a.lseT[p] = a.T > 0.f ? gm * invT + logf(gT) : gm + logf(g0);
    }
    // leave the launch-wide pruning state of this parent clean for the next launch
    if (tid < 2 * K) a.slots[(((size_t)(tid / K) * a.cap + p) * K + tid % K) * SLOT_STRIDE] = 0u;
    if (tid < 2) a.thr[(size_t)tid * a.cap + p] = 0u;   // and its condensed copy
    const bool fits = c_n[0] <= MERGE_CAP && c_n[1] <= MERGE_CAP;   // uniform: read after the barrier above
    if (fits) {
      // the usual case: a few dozen candidates survive the bounds; half of the block ranks each list
      const int half = tid / (MERGE_THREADS / 2), t = tid % (MERGE_THREADS / 2);
      if (half == 0) rank_select(c_v[0], c_i[0], c_l[0], c_n[0], K, t, MERGE_THREADS / 2, a.top_tok + (size_t)p * K, a.top_logit + (size_t)p * K);
      else if (a.T > 0.f)
        rank_select(c_v[1], c_i[1], c_l[1], c_n[1], K, t, MERGE_THREADS / 2, a.draw_tok + (size_t)p * K, a.draw_logit + (size_t)p * K);
      __syncthreads();
    } else {
      // too many candidates for the shared arrays (bounds not formed, e.g. tiny vocabularies): every
      // thread rebuilds private sorted lists from its pieces and the block selects over their heads
      MList<KR> top, key;
      top.init(); key.init();
      for (int q = tid; q < npieces; q += MERGE_THREADS) {
        const float* rec = rec_of(q);
        if (__ldcg(rec) == -INFINITY) continue;
        const float* f = rec + 4; const int* ii = reinterpret_cast<const int*>(rec) + 4;
        for (int j = 0; j < K; ++j) {
          const int t = __ldcg(ii + K + j);
          if (t >= 0) top.insert(__ldcg(f + j), t, __ldcg(f + j));
          if (a.T > 0.f) { const int k2 = __ldcg(ii + 3 * K + j); if (k2 >= 0) key.insert(__ldcg(f + 2 * K + j), k2, __ldcg(f + 4 * K + j)); }
        }
      }
      __syncthreads();
      block_select<KR>(top, K, a.top_tok + (size_t)p * K, a.top_logit + (size_t)p * K, s_v, s_i, s_l);
      if (a.T > 0.f) block_select<KR>(key, K, a.draw_tok + (size_t)p * K, a.draw_logit + (size_t)p * K, s_v, s_i, s_l);
    }
    if (!(a.T > 0.f)) {
      if (tid < K) {
        a.draw_tok[(size_t)p * K + tid] = a.top_tok[(size_t)p * K + tid];
        a.draw_logit[(size_t)p * K + tid] = a.top_logit[(size_t)p * K + tid];
      }
    }
    __syncthreads();
  }
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

cudaError_t launch_score(const ts_ctx* ctx, float* rec, int cap, int* err, const void* U, const void* A, const void* W,
                         int P, const int* P_dev, const int* p_req, const int* p_depth, const int* p_token,
                         const uint64_t* p_hash, float T, uint64_t seed, float* lse0, float* lseT, int* top_tok,
                         float* top_logit, int* draw_tok, float* draw_logit, cudaStream_t st, bool pdl, const int* P_prev_dev,
                         int p_bound, const ScoreExtras* extras) {
  const ts_config& c = ctx->cfg;
  ScoreArgs a{};
  a.pdl = pdl ? 1 : 0; a.P_prev_dev = P_prev_dev;
  a.U = U; a.A = A; a.W = W; a.V = c.V; a.D = c.D; a.r = c.r; a.K = c.K; a.P = P; a.P_dev = P_dev;
  a.p_req = p_req; a.p_depth = p_depth; a.p_token = p_token; a.p_hash = p_hash; a.T = T; a.seed = seed;
  a.TV = ctx->tile.TV; a.ntiles = ctx->tile.ntiles; a.cap = cap; a.S = 1; a.rec = rec; a.err = err;
  a.wait_limit = ctx->wait_limit;
  a.lost_arrival = (ctx->test_mode & TS_TEST_LOST_ARRIVAL) ? 1 : 0;
  a.thr = thr_base(ctx, rec, cap); a.slots = a.thr + 2 * (size_t)cap;
  a.thr0 = nullptr;
  cudaError_t e = cudaSuccess;
  // Which kernel scores the level: the few-parents kernel when the host knows that the list cannot hold
  // more than FEW_MAX parents (its own P, or a bound of the device-side count), the tile kernel otherwise.
  const int bound = P_dev ? p_bound : P;
  const bool run_few = ctx->use_mma && ctx->few_ok && bound >= 0 && bound <= FEW_MAX;
  const bool run_tile = !run_few;
  a.few = run_few ? 1 : 0;
  if (run_tile && ctx->use_mma && !(ctx->test_mode & TS_TEST_NO_SEED)) {
    // seed bounds first: exact values of the tokens with the largest base logits of every parent's row
    a.thr0 = a.slots + 2 * (size_t)cap * c.K * SLOT_STRIDE;
    a.seed_cnt = a.thr0 + 2 * (size_t)cap;
    a.seed_cand = a.seed_cnt + SEED_SPLIT_PARENTS;
    if (!(extras && extras->thr0_ready)) {   // (an expansion's level kernel writes them for the level after it)
      ProfScope ps(ctx, K_SEED, st);
      e = launch_seed(ctx, a, st);
      if (e != cudaSuccess) return e;
    }
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
