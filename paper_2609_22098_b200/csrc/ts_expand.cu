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

namespace ts {

struct ExpandArgs {
  int B, D, K, N, V;
  float T;
  const int* anchor; const float* theta;
  DevCalib calib;
  // level lists
  int* lst_req[2]; int* lst_depth[2]; int* lst_token[2]; uint64_t* lst_hash[2]; int* lst_slot[2];
  int* lvl_count;
  // merged scoring results
  const float *res_lse0, *res_lseT; const int* res_top_tok; const float* res_top_logit;
  const int* res_draw_tok; const float* res_draw_logit;
  // pool
  int *pl_alive, *pl_depth, *pl_parent, *pl_sib, *pl_tok;
  double *pl_logkey, *pl_logS; float *pl_q0, *pl_logqT, *pl_lseT; uint64_t *pl_hash, *pl_path;
  float* root_lseT; int *req_npar, *req_base, *req_nscored;
  // candidates
  int *cd_valid, *cd_parent, *cd_sib, *cd_tok; double *cd_logkey, *cd_logS; float *cd_q0, *cd_logqT; int* cd_rank;
  int* status; int* err; unsigned* thr; int thr_head, thr_words;
  unsigned* seed_cnt;   // the seed kernel's arrival counters
  // seed bounds of the next level's parents (made by the level kernel from the scoring kernel's scouting)
  const void *U, *A, *W; int r, ntiles, cap; uint64_t seed; const uint2* utop; unsigned* thr0;
  int calib_qT;   // ablation: the calibrator is fed the tempered conditional when T > 0
};

__device__ __forceinline__ void request_caps(const ExpandArgs& a, int b, int& K_eff, int& N_eff, double& log_theta) {
  const float th = a.theta[b];
  K_eff = a.K < a.V ? a.K : a.V;
  N_eff = a.N;
  if (th >= 1.f) {  // chain member of the price ladder
    K_eff = 1; N_eff = a.D < a.N ? a.D : a.N; log_theta = -INFINITY;
  } else {
    log_theta = th > 0.f ? log((double)th) : -INFINITY;
  }
}

__global__ void expand_init_kernel(ExpandArgs a) {
  pdl_wait();                // whatever ran before in the stream may still be reading what this kernel resets
  pdl_launch_dependents();   // the first scoring launch may run its preamble beside this kernel
  const int b = blockIdx.x;
  // pruning state of the scoring launches: the threshold words, then one word per slot (the slots sit
  // SLOT_STRIDE words apart; only the first word of each is ever used)
  for (int i = b * blockDim.x + threadIdx.x; i < a.thr_words; i += gridDim.x * blockDim.x)
    a.thr[i < a.thr_head ? i : a.thr_head + (size_t)(i - a.thr_head) * SLOT_STRIDE] = 0u;
  if (b == 0) for (int i = threadIdx.x; i < SEED_SPLIT_PARENTS; i += blockDim.x) a.seed_cnt[i] = 0u;
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

struct Entry { double key; uint64_t path; int depth; };

__device__ __forceinline__ bool before(double ka, int da, uint64_t pa, double kb, int db, uint64_t pb) {
  if (ka != kb) return ka > kb;
  if (da != db) return da < db;
  return pa < pb;
}

// One CTA per request; level d = depth of the parents just scored.
__global__ void __launch_bounds__(256) expand_level_kernel(ExpandArgs a, int d, int seed_next) {
  extern __shared__ __align__(16) unsigned char sm_raw[];
  __shared__ int s_cnt[2];
  __shared__ int s_base;
  const int b = blockIdx.x, tid = threadIdx.x;
  const int N = a.N, K = a.K;
  pdl_wait();               // merged scoring results of this level
  pdl_launch_dependents();
  const int npar = a.req_npar[b], base = a.req_base[b];
  const int cur = d & 1, nxt = cur ^ 1;
  int K_eff, N_eff; double log_theta;
  request_caps(a, b, K_eff, N_eff, log_theta);
  const size_t pb = (size_t)b * N, cb = (size_t)b * N * K;
  if (tid == 0) {
    if (a.err[0] != 0 && a.status[b] == TS_OK) a.status[b] = TS_ERR_TIMEOUT;  // a wait in the scoring kernel ran out
    s_base = a.status[b];
  }
  __syncthreads();
  if (npar == 0 || s_base != TS_OK) {  // uniform: read once, before any thread can change the status
    if (tid == 0) a.req_npar[b] = 0;
    return;
  }
  // ---- phase 1: slots of every scored parent, one thread per (parent, sibling rank) -------------
  for (int t = tid; t < npar * K; t += blockDim.x) {
    const int i = t / K, j = t % K;
    const int li = base + i;
    const int slot = a.lst_slot[cur][li];
    const double logS_v = slot < 0 ? 0.0 : a.pl_logS[pb + slot];
    const double lse0 = a.res_lse0[li], lseT = a.res_lseT[li];
    if (j == 0) {
      if (slot < 0) a.root_lseT[b] = (float)lseT; else a.pl_lseT[pb + slot] = (float)lseT;
      if (!(lse0 == lse0) || isinf(lse0)) a.status[b] = TS_ERR_NUMERIC;
    }
    const int* top_tok = a.res_top_tok + (size_t)li * K; const float* top_logit = a.res_top_logit + (size_t)li * K;
    const int* draw_tok = a.res_draw_tok + (size_t)li * K; const float* draw_logit = a.res_draw_logit + (size_t)li * K;
    const size_t ci = cb + (size_t)i * K + j;
    int valid = 0;
    if (j < K_eff) {
      int bi = j;
      if (a.T > 0.f) {  // best token of q0 not among the first j draws: the pre-draw bound
        bi = -1;
        for (int tt = 0; tt < K_eff && bi < 0; ++tt) {
          bool used = false;
          for (int u = 0; u < j; ++u) used |= (draw_tok[u] == top_tok[tt]);
          if (!used) bi = tt;
        }
      }
      const int x = draw_tok[j];
      if (bi >= 0 && top_tok[bi] >= 0 && x >= 0) {
        // the calibrator's input: the untempered conditional, or (ablation) the tempered one
        const bool tempered = a.calib_qT && a.T > 0.f;
        const double lsc = tempered ? 1.0 / (double)a.T : 1.0, lsn = tempered ? lseT : lse0;
        const double key = logS_v + log_phat(a.calib, d, (double)top_logit[bi] * lsc, lsn);
        if (!(key < log_theta)) {
          const double lx = draw_logit[j];
          valid = 1;
          a.cd_parent[ci] = slot; a.cd_sib[ci] = j; a.cd_tok[ci] = x;
          a.cd_logkey[ci] = key;
          a.cd_logS[ci] = logS_v + log_phat(a.calib, d, lx * lsc, lsn);
          a.cd_q0[ci] = (float)exp(lx - lse0);
          a.cd_logqT[ci] = a.T > 0.f ? (float)(lx / (double)a.T - lseT) : (float)(lx - lse0);
        }
      }
    }
    a.cd_valid[ci] = valid;
  }
  __syncthreads();
  // a sibling slot exists only if the one before it was admitted (keys are non-increasing in j)
  for (int i = tid; i < npar; i += blockDim.x) {
    int vals[KMAX];   // all flags of the parent first: independent loads, one round trip
#pragma unroll
    for (int j = 0; j < KMAX; ++j) vals[j] = j < K ? a.cd_valid[cb + (size_t)i * K + j] : 0;
    bool open = true;
#pragma unroll
    for (int j = 0; j < KMAX; ++j) {
      if (j < K) {
        if (!open && vals[j]) a.cd_valid[cb + (size_t)i * K + j] = 0;
        else if (!vals[j]) open = false;
      }
    }
  }
  __syncthreads();
  // ---- phase 2: who survives the cut to N_eff ------------------------------------------------
  const int ncand = npar * K;
  if (tid < 2) s_cnt[tid] = 0;
  __syncthreads();
  {
    int lp = 0, lc = 0;
    for (int s = tid; s < N; s += blockDim.x) lp += a.pl_alive[pb + s] ? 1 : 0;
    for (int c = tid; c < ncand; c += blockDim.x) lc += a.cd_valid[cb + c] ? 1 : 0;
    if (lp) atomicAdd(&s_cnt[0], lp);
    if (lc) atomicAdd(&s_cnt[1], lc);
  }
  __syncthreads();
  const int n_pool = s_cnt[0], n_valid = s_cnt[1];
  const int shift = 60 - 4 * d;
  if (n_pool + n_valid > N_eff) {
    // rank every entry by counting the entries that come before it in (key desc, depth asc, path asc)
    Entry* ent = reinterpret_cast<Entry*>(sm_raw);
    const int M = N + ncand;
    for (int e = tid; e < M; e += blockDim.x) {
      Entry x; x.depth = -1; x.key = 0; x.path = 0;
      if (e < N) {
        if (a.pl_alive[pb + e]) { x.key = a.pl_logkey[pb + e]; x.depth = a.pl_depth[pb + e]; x.path = a.pl_path[pb + e]; }
      } else {
        const size_t ci = cb + (e - N);
        if (a.cd_valid[ci]) {
          const int slot = a.cd_parent[ci];
          x.key = a.cd_logkey[ci]; x.depth = d + 1;
          x.path = (slot < 0 ? 0ull : a.pl_path[pb + slot]) | ((uint64_t)a.cd_sib[ci] << shift);
        }
      }
      ent[e] = x;
    }
    __syncthreads();
    for (int e = tid; e < M; e += blockDim.x) {
      const Entry x = ent[e];
      if (x.depth < 0) continue;
      int rank = 0;
      for (int f = 0; f < M; ++f) {
        const Entry y = ent[f];
        if (y.depth >= 0 && f != e && before(y.key, y.depth, y.path, x.key, x.depth, x.path)) ++rank;
      }
      if (rank >= N_eff) {
        if (e < N) a.pl_alive[pb + e] = 0; else a.cd_valid[cb + (e - N)] = 0;
      }
    }
    __syncthreads();
  }
  // ---- phase 3: place surviving candidates into free pool slots (deterministic order) --------
  // the t-th surviving candidate (in candidate order) takes the t-th free slot (in slot order)
  __shared__ int s_free[256], s_new[256], s_warp[8];
  __shared__ int s_run, s_nb;
  const int lane = tid & 31, warp = tid >> 5;
  {
    const bool fr = tid < N && !a.pl_alive[pb + tid];
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, fr);
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    int off = 0;
    for (int w = 0; w < warp; ++w) off += s_warp[w];
    if (fr) s_free[off + __popc(bal & ((1u << lane) - 1u))] = tid;
    if (tid == 0) s_run = 0;
    __syncthreads();
  }
  int nfree = 0;
  for (int w = 0; w < 8; ++w) nfree += s_warp[w];
  for (int c0 = 0; c0 < ncand; c0 += blockDim.x) {
    const int c = c0 + tid;
    const size_t ci = cb + c;
    const bool v = c < ncand && a.cd_valid[ci];
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, v);
    __syncthreads();  // s_warp is reused
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    int off = s_run;
    for (int w = 0; w < warp; ++w) off += s_warp[w];
    const int t = off + __popc(bal & ((1u << lane) - 1u));
    if (v) {
      if (t >= nfree) { a.status[b] = TS_ERR_OVERFLOW; }
      else {
        const int sl = s_free[t];
        const int slot = a.cd_parent[ci];
        const int x = a.cd_tok[ci];
        a.pl_alive[pb + sl] = 1; a.pl_depth[pb + sl] = d + 1; a.pl_parent[pb + sl] = slot; a.pl_sib[pb + sl] = a.cd_sib[ci];
        a.pl_tok[pb + sl] = x; a.pl_logkey[pb + sl] = a.cd_logkey[ci]; a.pl_logS[pb + sl] = a.cd_logS[ci];
        a.pl_q0[pb + sl] = a.cd_q0[ci]; a.pl_logqT[pb + sl] = a.cd_logqT[ci]; a.pl_lseT[pb + sl] = nanf("");
        a.pl_hash[pb + sl] = path_hash(slot < 0 ? 0ull : a.pl_hash[pb + slot], x);
        a.pl_path[pb + sl] = (slot < 0 ? 0ull : a.pl_path[pb + slot]) | ((uint64_t)a.cd_sib[ci] << shift);
        s_new[t] = sl;
      }
    }
    __syncthreads();
    if (tid == 0) { int tot = 0; for (int w = 0; w < 8; ++w) tot += s_warp[w]; s_run += tot; }
    __syncthreads();
  }
  const int nnew = min(s_run, nfree);
  // ---- phase 4: next level's parents = new nodes that can still have admissible children -----------
  {
    const bool par = (d + 1 < a.D) && tid < nnew && !(a.pl_logS[pb + s_new[tid]] < log_theta);
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, par);
    __syncthreads();
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    int off = 0, cnt = 0;
    for (int w = 0; w < 8; ++w) { if (w < warp) off += s_warp[w]; cnt += s_warp[w]; }
    if (tid == 0) {
      s_nb = cnt > 0 ? atomicAdd(&a.lvl_count[d + 1], cnt) : 0;
      a.req_nscored[b] += npar;
      a.req_npar[b] = cnt;
    }
    __syncthreads();
    if (tid == 0) a.req_base[b] = s_nb;
    int my_li = -1;
    if (par) {
      const int sl = s_new[tid];
      const int li = s_nb + off + __popc(bal & ((1u << lane) - 1u));
      a.lst_req[nxt][li] = b; a.lst_depth[nxt][li] = d + 1; a.lst_token[nxt][li] = a.pl_tok[pb + sl];
      a.lst_hash[nxt][li] = a.pl_hash[pb + sl]; a.lst_slot[nxt][li] = sl;
      my_li = li;
    }
    // ---- phase 5: seed bounds of those parents (bf16 tensor-core path; see ts_seed.cu for what they are) ----
    // The scoring launch of this level left the best base logit of every vocabulary tile of row U[b][d+1]:
    // the warps pick 2K good tokens from those, the tokens' columns of W are staged once for the request,
    // every (parent, token) pair is evaluated exactly by one thread, and one thread per parent takes the
    // K-th best logit and key, less the rounding margin.
    if (seed_next && cnt > 0) {
      __shared__ int s_stok[NSEED_MAX], s_pli[256], s_ptok[256];
      __shared__ float s_sval[NSEED_MAX];
      __shared__ uint64_t s_phash[256];
      const int r = a.r, V = a.V;
      const int npick = max(1, min(2 * K, NSEED_MAX) / 8), NSn = 8 * npick;
      const float invT = a.T > 0.f ? 1.f / a.T : 1.f;
      __syncthreads();   // the Entry array in dynamic shared memory is free now
      float* Wc = reinterpret_cast<float*>(sm_raw);            // [NSn][r]
      float* res = Wc + (size_t)NSn * r;                        // [cnt][NSn][2]: logit, key
      if (par) {
        const int i = off + __popc(bal & ((1u << lane) - 1u));
        s_pli[i] = my_li; s_ptok[i] = a.pl_tok[pb + s_new[tid]]; s_phash[i] = a.pl_hash[pb + s_new[tid]];
      }
      {
        const uint2* ut = a.utop + ((size_t)b * a.D + (d + 1)) * a.ntiles;
        float bv = -INFINITY; int bi = 0x7FFFFFFF;
        for (int t = lane * 8 + warp; t < a.ntiles; t += blockDim.x) {   // consecutive tiles go to different warps
          const uint2 e = __ldcg(ut + t);
          const float v = __uint_as_float(e.x);
          if (v > bv || (v == bv && (int)e.y < bi)) { bv = v; bi = (int)e.y; }
        }
        for (int i = 0; i < npick; ++i) {   // every warp hands over its npick best
          float wv = bv; int wi = bi;
#pragma unroll
          for (int o2 = 16; o2 > 0; o2 >>= 1) {
            const float ov = __shfl_xor_sync(0xFFFFFFFFu, wv, o2);
            const int oi = __shfl_xor_sync(0xFFFFFFFFu, wi, o2);
            if (ov > wv || (ov == wv && oi < wi)) { wv = ov; wi = oi; }
          }
          if (wi == bi && bv > -INFINITY) { bv = -INFINITY; bi = 0x7FFFFFFF; }
          if (lane == 0) { s_stok[warp * npick + i] = (wv > -INFINITY && wi >= 0 && wi < V) ? wi : -1; }
        }
      }
      __syncthreads();
      const __nv_bfloat16* Wg = reinterpret_cast<const __nv_bfloat16*>(a.W);
      const __nv_bfloat16* Ag = reinterpret_cast<const __nv_bfloat16*>(a.A);
      const __nv_bfloat16* Urow = reinterpret_cast<const __nv_bfloat16*>(a.U) + ((size_t)b * a.D + (d + 1)) * V;
      for (int e = tid; e < NSn * r; e += blockDim.x) {
        const int j = e / r, k = e % r;
        Wc[e] = s_stok[j] >= 0 ? __bfloat162float(Wg[(size_t)k * V + s_stok[j]]) : 0.f;
      }
      if (tid < NSn) s_sval[tid] = s_stok[tid] >= 0 ? __bfloat162float(Urow[s_stok[tid]]) : -INFINITY;
      __syncthreads();
      for (int e = tid; e < cnt * NSn; e += blockDim.x) {
        const int i = e / NSn, j = e % NSn;
        float lg = -INFINITY, key = -INFINITY;
        const int tok = s_stok[j];
        if (tok >= 0) {
          const uint4* arow = reinterpret_cast<const uint4*>(Ag + (size_t)s_ptok[i] * r);   // r is a multiple of 8 on this path
          float dot = 0.f;
          for (int k8 = 0; k8 < r / 8; ++k8) {
            float av[8];
            unpack_bf16x8(__ldg(arow + k8), av);
#pragma unroll
            for (int u = 0; u < 8; ++u) dot = fmaf(av[u], Wc[(size_t)j * r + k8 * 8 + u], dot);
          }
          lg = s_sval[j] + dot;
          key = lg;
          if (a.T > 0.f) {
            const uint4 cw = stream_words(a.seed, b, s_phash[i], STREAM_GUMBEL_COARSE, (uint32_t)tok >> 3);
            const uint4 fw = stream_words(a.seed, b, s_phash[i], STREAM_GUMBEL_FINE, (uint32_t)tok >> 3);
            const uint32_t c16 = (word_of(cw, (tok & 7) >> 1) >> (16 * (tok & 1))) & 0xFFFFu;
            const uint32_t f16 = (word_of(fw, (tok & 7) >> 1) >> (16 * (tok & 1))) & 0xFFFFu;
            key = lg * invT + gumbel_from_bits((c16 << 16) | f16);
          }
        }
        res[2 * e] = lg; res[2 * e + 1] = key;
      }
      __syncthreads();
      for (int e = tid; e < 2 * cnt; e += blockDim.x) a.thr0[(size_t)(e & 1) * a.cap + s_pli[e >> 1]] = 0u;   // no bound unless K finite values turn up
      __syncthreads();
      for (int e = tid; e < 2 * cnt * NSn; e += blockDim.x) {
        // one thread per value: the one with exactly K - 1 values before it (ties broken by place) is the K-th best
        const int j = e % NSn, which = (e / NSn) & 1, i = e / (2 * NSn);
        if (which == 1 && !(a.T > 0.f)) continue;
        const float* val = res + (size_t)i * NSn * 2 + which;
        const float mine = val[2 * j];
        int before = 0;
        for (int t = 0; t < NSn; ++t) before += (val[2 * t] > mine || (val[2 * t] == mine && t < j)) ? 1 : 0;
        if (before == K - 1 && mine == mine && fabsf(mine) < INFINITY) {
          const float margin = (2e-4f + 4e-5f * fabsf(mine)) * (which == 0 ? 1.f : fmaxf(invT, 1.f)) + (which == 0 ? 0.f : 2e-4f);
          a.thr0[(size_t)which * a.cap + s_pli[i]] = enc_f(mine - margin);
        }
      }
    }
  }
}

struct FinalArgs {
  int B, N, words;
  const int *pl_alive, *pl_depth, *pl_parent, *pl_sib, *pl_tok;
  const double *pl_logkey, *pl_logS; const float *pl_q0, *pl_logqT, *pl_lseT; const uint64_t *pl_hash, *pl_path;
  const float* root_lseT; const int* req_nscored;
  int *n_nodes, *tok, *parent, *depth, *sib_rank; float *logS, *q0, *logqT, *logkey; int* pop_rank;
  uint64_t* node_hash; float* node_lseT; uint64_t* mask; int* n_scored;
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
// reused for the seed bounds' staged W columns [2K][r] and per-pair results [Nmax][2K][2]
size_t level_smem_bytes(const ts_config& c) {
  const size_t entries = (size_t)(c.Nmax + c.Nmax * c.K) * sizeof(Entry);
  const size_t ns = (size_t)(2 * c.K > NSEED_MAX ? NSEED_MAX : (2 * c.K < 8 ? 8 : 2 * c.K));
  const size_t seeds = ns * (size_t)c.r * 4 + (size_t)c.Nmax * ns * 2 * 4;
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

  cudaError_t e0;
  { ProfScope ps(ctx, K_INIT, st); e0 = launch_kernel(expand_init_kernel, B > 296 ? B : 296, 256, 0, st, true, a); }
  cudaError_t e = e0 != cudaSuccess ? e0 : cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(init)", e);
  const size_t level_smem = level_smem_bytes(c);   // opted into at ts_create when above 48 KB
  long long level_bound = B;   // parents a level can have at most: B at the root, K times more per level, B * Nmax overall
  // Seed bounds of a level on the tensor-core kernel: made by the level kernel before it when that level's scoring
  // launch scouted the rows (it does whenever it runs on the tensor-core kernel itself); by a seed launch otherwise
  // (the root level, and the first tensor-core level after levels on the few-parents kernel).
  const bool seeds_on = ctx->use_mma && !(ctx->test_mode & TS_TEST_NO_SEED);
  bool scouted_prev = false;
  for (int d = 0; d < c.D; ++d) {
    const int cur = d & 1;
    const bool on_mma = ctx->use_mma && !(ctx->few_ok && level_bound <= FEW_MAX);
    ScoreExtras ex;
    ex.thr0_ready = scouted_prev;
    const bool scout = seeds_on && on_mma && d + 1 < c.D;
    if (scout) { ex.utop = (uint2*)(ws + L.utop); ex.scout_live = a.req_npar; ex.scout_B = B; ex.scout_depth = d + 1; }
    e = launch_score(ctx, (float*)(ws + L.rec), L.rec_cap, (int*)(ws + L.err), U, A, W, 0, a.lvl_count + d,
                     a.lst_req[cur], a.lst_depth[cur], a.lst_token[cur],
                     a.lst_hash[cur], T, seed, res_lse0, res_lseT, res_top_tok, res_top_logit, res_draw_tok,
                     res_draw_logit, st, /*pdl=*/true, d > 0 ? a.lvl_count + d - 1 : nullptr, (int)level_bound, &ex);
    level_bound = level_bound * c.K < (long long)B * c.Nmax ? level_bound * c.K : (long long)B * c.Nmax;
    if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(score)", e);
    { ProfScope ps(ctx, K_LEVEL, st); e = launch_kernel(expand_level_kernel, B, 256, level_smem, st, true, a, d, scout ? 1 : 0); }
    scouted_prev = scout;
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(level)", e);
  }
  FinalArgs f{};
  f.B = B; f.N = c.Nmax; f.words = L.words;
  f.pl_alive = a.pl_alive; f.pl_depth = a.pl_depth; f.pl_parent = a.pl_parent; f.pl_sib = a.pl_sib; f.pl_tok = a.pl_tok;
  f.pl_logkey = a.pl_logkey; f.pl_logS = a.pl_logS; f.pl_q0 = a.pl_q0; f.pl_logqT = a.pl_logqT; f.pl_lseT = a.pl_lseT;
  f.pl_hash = a.pl_hash; f.pl_path = a.pl_path; f.root_lseT = a.root_lseT; f.req_nscored = a.req_nscored;
  f.n_nodes = n_nodes; f.tok = tok; f.parent = parent; f.depth = depth; f.sib_rank = sib_rank; f.logS = logS; f.q0 = q0;
  f.logqT = logqT; f.logkey = logkey; f.pop_rank = pop_rank; f.node_hash = node_hash; f.node_lseT = node_lseT;
  f.mask = mask; f.n_scored = n_scored;
  { ProfScope ps(ctx, K_FINAL, st); e = launch_kernel(expand_finalize_kernel, B, 256, 0, st, true, f); }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_expand_tree(finalize)", e);
  return TS_OK;
}
