// One level step of the best-first expansion (Algorithm 1, Section 3.5) for one request: the body shared by
// expand_level_kernel and the persistent expansion kernel.
#pragma once
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
  unsigned* ex_barrier; // grid barrier words of the persistent kernel
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

struct Entry { double key; uint64_t path; int depth; };

__device__ __forceinline__ int warp_of(int tid) { return tid >> 5; }

__device__ __forceinline__ bool before(double ka, int da, uint64_t pa, double kb, int db, uint64_t pb) {
  if (ka != kb) return ka > kb;
  if (da != db) return da < db;
  return pa < pb;
}

// The persistent form of the kernel (one cooperative launch for all levels of an expansion): after the scan of a
// level the grid merges the level's parents (merge_parent, parents dealt to the CTAs), runs the level step of every
// request (level_step, requests dealt to the CTAs), and goes on to the next level while it has parents.  The W
// tile, tensor memory and barriers are set up once; grid barriers (bounded) separate the phases.
struct PersistArgs {
  int on;               // 0: one scan of the parent list in ScoreArgs, nothing else
  int first;            // first level this launch runs (levels before it were run by launches of their own)
  int nlevels;          // D
  ExpandArgs ex;        // level lists, pools, seeds
  MergeArgs mg;         // merged-result arrays
  unsigned* barrier;    // [2] counter and abort word of the grid barrier (zero at launch)
  int lost_arrival;     // test switch: the grid barrier expects one arrival more than will come
};

// host side of the persistent form (ts_score_mma.cu)
bool persistent_supported(const ts_ctx* ctx, int B, int first_level);
cudaError_t launch_expand_persistent(const ts_ctx* ctx, const ScoreArgs& a, const PersistArgs& pa, cudaStream_t st);

constexpr int LEVEL_THREADS = 256;
constexpr int SEED_PBATCH = 64;    // parents whose rows of A the seed phase stages at a time

// shared-memory state of one level step (beside the dynamic array of level_smem_bytes())
struct LevelSmem {
  int s_cnt[2]; int s_base;
  int s_free[256], s_new[256], s_warp[8]; int s_run, s_nb;
  int s_stok[NSEED_MAX], s_pli[256], s_ptok[256]; float s_sval[NSEED_MAX]; uint64_t s_phash[256];
};

// The level step of request b; level d = depth of the parents just scored.  Called by LEVEL_THREADS threads
// (tid = 0 .. LEVEL_THREADS-1) that `sync` synchronises; sm_raw = level_smem_bytes() bytes of shared memory.
template <class Sync>
__device__ __forceinline__ void level_step(const ExpandArgs& a, const int d, const int seed_next, const int b, LevelSmem& sm,
                                           unsigned char* sm_raw, const int tid, Sync sync) {
  int (&s_cnt)[2] = sm.s_cnt; int& s_base = sm.s_base;
  int (&s_free)[256] = sm.s_free; int (&s_new)[256] = sm.s_new; int (&s_warp)[8] = sm.s_warp; int& s_run = sm.s_run; int& s_nb = sm.s_nb;
  int (&s_stok)[NSEED_MAX] = sm.s_stok; int (&s_pli)[256] = sm.s_pli; int (&s_ptok)[256] = sm.s_ptok;
  float (&s_sval)[NSEED_MAX] = sm.s_sval; uint64_t (&s_phash)[256] = sm.s_phash;
  const int N = a.N, K = a.K;
  const int npar = a.req_npar[b], base = a.req_base[b];
  const int cur = d & 1, nxt = cur ^ 1;
  int K_eff, N_eff; double log_theta;
  request_caps(a, b, K_eff, N_eff, log_theta);
  const size_t pb = (size_t)b * N, cb = (size_t)b * N * K;
  if (tid == 0) {
    if (*reinterpret_cast<volatile int*>(a.err) != 0 && a.status[b] == TS_OK) a.status[b] = TS_ERR_TIMEOUT;  // a wait in the scoring kernel ran out
    s_base = a.status[b];
  }
  sync();
  if (npar == 0 || s_base != TS_OK) {  // uniform: read once, before any thread can change the status
    if (tid == 0) a.req_npar[b] = 0;
    return;
  }
  // ---- phase 1: slots of every scored parent, one thread per (parent, sibling rank) -------------
  for (int t = tid; t < npar * K; t += LEVEL_THREADS) {
    const int i = t / K, j = t % K;
    const int li = base + i;
    const int slot = a.lst_slot[cur][li];
    const double logS_v = slot < 0 ? 0.0 : a.pl_logS[pb + slot];
    // (merged results come from other CTAs, which in the persistent kernel wrote them moments ago: read around L1)
    const double lse0 = __ldcg(a.res_lse0 + li), lseT = __ldcg(a.res_lseT + li);
    if (j == 0) {
      if (slot < 0) a.root_lseT[b] = (float)lseT; else a.pl_lseT[pb + slot] = (float)lseT;
      if (!(lse0 == lse0) || isinf(lse0)) a.status[b] = TS_ERR_NUMERIC;
    }
    const int* top_tok = a.res_top_tok + (size_t)li * K; const float* top_logit = a.res_top_logit + (size_t)li * K;
    const int* draw_tok = a.res_draw_tok + (size_t)li * K; const float* draw_logit = a.res_draw_logit + (size_t)li * K;
    const size_t ci = cb + (size_t)i * K + j;
    int valid = 0;
    if (j < K_eff) {
      // the parent's candidate tokens, all requested at once (one memory round trip), then searched in registers
      int tt_[KMAX], dt_[KMAX];
#pragma unroll
      for (int u = 0; u < KMAX; ++u) { tt_[u] = u < K ? __ldcg(top_tok + u) : -1; dt_[u] = u < K ? __ldcg(draw_tok + u) : -1; }
      int bi = j;
      if (a.T > 0.f) {  // best token of q0 not among the first j draws: the pre-draw bound
        bi = -1;
#pragma unroll
        for (int tt = 0; tt < KMAX; ++tt) {
          if (tt < K_eff && bi < 0) {
            bool used = false;
#pragma unroll
            for (int u = 0; u < KMAX; ++u) used |= (u < j && dt_[u] == tt_[tt]);
            if (!used) bi = tt;
          }
        }
      }
      int x = -1, tbi = -1;
#pragma unroll
      for (int u = 0; u < KMAX; ++u) { x = u == j ? dt_[u] : x; tbi = u == bi ? tt_[u] : tbi; }
      if (bi >= 0 && tbi >= 0 && x >= 0) {
        // the calibrator's input: the untempered conditional, or (ablation) the tempered one
        const bool tempered = a.calib_qT && a.T > 0.f;
        const double lsc = tempered ? 1.0 / (double)a.T : 1.0, lsn = tempered ? lseT : lse0;
        const double key = logS_v + log_phat(a.calib, d, (double)__ldcg(top_logit + bi) * lsc, lsn);
        if (!(key < log_theta)) {
          const double lx = __ldcg(draw_logit + j);
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
  sync();
  // a sibling slot exists only if the one before it was admitted (keys are non-increasing in j)
  for (int i = tid; i < npar; i += LEVEL_THREADS) {
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
  sync();
  // ---- phase 2: who survives the cut to N_eff ------------------------------------------------
  const int ncand = npar * K;
  if (tid < 2) s_cnt[tid] = 0;
  sync();
  {
    int lp = 0, lc = 0;
    for (int s = tid; s < N; s += LEVEL_THREADS) lp += a.pl_alive[pb + s] ? 1 : 0;
    for (int c = tid; c < ncand; c += LEVEL_THREADS) lc += a.cd_valid[cb + c] ? 1 : 0;
    if (lp) atomicAdd(&s_cnt[0], lp);
    if (lc) atomicAdd(&s_cnt[1], lc);
  }
  sync();
  const int n_pool = s_cnt[0], n_valid = s_cnt[1];
  const int shift = 60 - 4 * d;
  if (n_pool + n_valid > N_eff) {
    // rank every entry by counting the entries that come before it in (key desc, depth asc, path asc)
    Entry* ent = reinterpret_cast<Entry*>(sm_raw);
    const int M = N + ncand;
    for (int e = tid; e < M; e += LEVEL_THREADS) {
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
    sync();
    // The N_eff-th largest key by radix selection over the keys' order-preserving bit patterns (eight passes of
    // eight bits, a 256-bin histogram each); entries above it stay, entries below it go, and the entries that tie
    // with it are ranked among themselves by (depth asc, path asc) for the places that are left.
    auto skey = [](double k) -> uint64_t {
      if (k == 0.0) k = 0.0;   // -0 and +0 compare equal: one pattern
      const uint64_t b = (uint64_t)__double_as_longlong(k);
      return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
    };
    int* hist = s_free;          // 256 bins (the free-slot list is built in phase 3)
    uint64_t prefix = 0;
    int need = N_eff;            // the entry sought is the need-th largest among those that match the prefix so far
    for (int sh8 = 56; sh8 >= 0; sh8 -= 8) {
      hist[tid] = 0;             // LEVEL_THREADS == 256 bins
      sync();
      for (int e = tid; e < M; e += LEVEL_THREADS) {
        if (ent[e].depth < 0) continue;
        const uint64_t k = skey(ent[e].key);
        if (sh8 == 56 || (k >> (sh8 + 8)) == (prefix >> (sh8 + 8))) atomicAdd(&hist[(int)((k >> sh8) & 255u)], 1);
      }
      sync();
      if (warp_of(tid) == 0) {
        // lane l owns bins 255 - 8l .. 248 - 8l (descending); the bin where the running count reaches `need`
        const int l = tid & 31;
        int mine = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) mine += hist[255 - 8 * l - j];
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (l >= o) incl += v; }
        const unsigned reach = __ballot_sync(0xFFFFFFFFu, incl >= need);
        const int owner = __ffs(reach) - 1;   // reach != 0: at least `need` entries match the prefix
        if (l == owner) {
          int cum = incl - mine, bin = 255 - 8 * l;
          for (int j = 0; j < 8; ++j) {
            const int h = hist[255 - 8 * l - j];
            if (cum + h >= need) { bin = 255 - 8 * l - j; break; }
            cum += h;
          }
          s_warp[0] = bin; s_warp[1] = need - cum;
        }
      }
      sync();
      prefix |= (uint64_t)s_warp[0] << sh8;
      need = s_warp[1];
      sync();
    }
    // the entries that tie with the threshold key (at least the one that defines it), gathered: they are ranked
    // among themselves only, and only when there are more of them than places left
    int* tie_list = s_new;   // (the list of placed slots is built in phase 3)
    if (tid == 0) s_cnt[0] = 0;
    sync();
    for (int e = tid; e < M; e += LEVEL_THREADS) {
      if (ent[e].depth >= 0 && skey(ent[e].key) == prefix) {
        const int idx = atomicAdd(&s_cnt[0], 1);
        if (idx < 256) tie_list[idx] = e;
      }
    }
    sync();
    const int ntie = s_cnt[0];
    for (int e = tid; e < M; e += LEVEL_THREADS) {
      const Entry x = ent[e];
      if (x.depth < 0) continue;
      const uint64_t k = skey(x.key);
      bool drop = k < prefix;
      if (k == prefix && ntie > need) {
        int rank = 0;
        if (ntie <= 256) {
          for (int t = 0; t < ntie; ++t) {
            const int f = tie_list[t];
            const Entry y = ent[f];
            if (f != e && before(y.key, y.depth, y.path, x.key, x.depth, x.path)) ++rank;
          }
        } else {
          for (int f = 0; f < M; ++f) {
            const Entry y = ent[f];
            if (y.depth >= 0 && f != e && skey(y.key) == prefix && before(y.key, y.depth, y.path, x.key, x.depth, x.path)) ++rank;
          }
        }
        drop = rank >= need;
      }
      if (drop) {
        if (e < N) a.pl_alive[pb + e] = 0; else a.cd_valid[cb + (e - N)] = 0;
      }
    }
    sync();
  }
  // ---- phase 3: place surviving candidates into free pool slots (deterministic order) --------
  // the t-th surviving candidate (in candidate order) takes the t-th free slot (in slot order)
  const int lane = tid & 31, warp = tid >> 5;
  {
    const bool fr = tid < N && !a.pl_alive[pb + tid];
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, fr);
    if (lane == 0) s_warp[warp] = __popc(bal);
    sync();
    int off = 0;
    for (int w = 0; w < warp; ++w) off += s_warp[w];
    if (fr) s_free[off + __popc(bal & ((1u << lane) - 1u))] = tid;
    if (tid == 0) s_run = 0;
    sync();
  }
  int nfree = 0;
  for (int w = 0; w < 8; ++w) nfree += s_warp[w];
  // Candidate c = it * LEVEL_THREADS + tid.  Pass 1: every thread notes which of its candidates survive (one bit
  // per trip) and every warp leaves its count per trip; a prefix over (trip, warp) gives every warp's first
  // place; pass 2 places.  (One trip at a time with the running total carried through shared memory cost four
  // block barriers and a chain of loads per trip: 11 trips at the wide configuration, 100 us.)
  const int ntrip = (ncand + LEVEL_THREADS - 1) / LEVEL_THREADS;   // <= Nmax * K / 256 <= 16
  int* trip_cnt = s_pli;    // [ntrip][8] (phase 5 fills these arrays later)
  int* trip_off = s_ptok;
  unsigned vm = 0;
  for (int it = 0; it < ntrip; ++it) {
    const int c = it * LEVEL_THREADS + tid;
    const bool v = c < ncand && a.cd_valid[cb + c];
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, v);
    vm |= (v ? 1u : 0u) << it;
    if (lane == 0) trip_cnt[it * 8 + warp] = __popc(bal);
  }
  sync();
  if (tid < ntrip * 8) {
    int off = 0;
    for (int e = 0; e < tid; ++e) off += trip_cnt[e];
    trip_off[tid] = off;
    if (tid == ntrip * 8 - 1) s_run = off + trip_cnt[tid];
  }
  if (ntrip == 0 && tid == 0) s_run = 0;
  sync();
  for (int it = 0; it < ntrip; ++it) {
    const bool v = (vm >> it) & 1u;
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, v);
    if (!v) continue;
    const size_t ci = cb + (size_t)it * LEVEL_THREADS + tid;
    const int t = trip_off[it * 8 + warp] + __popc(bal & ((1u << lane) - 1u));
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
  sync();
  const int nnew = min(s_run, nfree);
  // ---- phase 4: next level's parents = new nodes that can still have admissible children -----------
  {
    const bool par = (d + 1 < a.D) && tid < nnew && !(a.pl_logS[pb + s_new[tid]] < log_theta);
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, par);
    sync();
    if (lane == 0) s_warp[warp] = __popc(bal);
    sync();
    int off = 0, cnt = 0;
    for (int w = 0; w < 8; ++w) { if (w < warp) off += s_warp[w]; cnt += s_warp[w]; }
    if (tid == 0) {
      s_nb = cnt > 0 ? atomicAdd(&a.lvl_count[d + 1], cnt) : 0;
      a.req_nscored[b] += npar;
      a.req_npar[b] = cnt;
    }
    sync();
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
      const int r = a.r, V = a.V;
      const int npick = max(1, min(2 * K, NSEED_MAX) / 8), NSn = 8 * npick;
      const float invT = a.T > 0.f ? 1.f / a.T : 1.f;
      sync();   // the Entry array in dynamic shared memory is free now
      // (rows of r + 1 words: the threads of a warp read the same k of different picks, which an even row length
      // puts into one bank)
      const int rs = r + 1;
      float* Wc = reinterpret_cast<float*>(sm_raw);            // [NSn][r + 1]
      float* res = Wc + (size_t)NSn * rs;                       // [cnt][NSn][2]: logit, key
      if (par) {
        const int i = off + __popc(bal & ((1u << lane) - 1u));
        s_pli[i] = my_li; s_ptok[i] = a.pl_tok[pb + s_new[tid]]; s_phash[i] = a.pl_hash[pb + s_new[tid]];
      }
      {
        const uint2* ut = a.utop + ((size_t)b * a.D + (d + 1)) * a.ntiles;
        float bv = -INFINITY; int bi = 0x7FFFFFFF;
        for (int t = lane * 8 + warp; t < a.ntiles; t += LEVEL_THREADS) {   // consecutive tiles go to different warps
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
      sync();
      const __nv_bfloat16* Wg = reinterpret_cast<const __nv_bfloat16*>(a.W);
      const __nv_bfloat16* Ag = reinterpret_cast<const __nv_bfloat16*>(a.A);
      const __nv_bfloat16* Urow = reinterpret_cast<const __nv_bfloat16*>(a.U) + ((size_t)b * a.D + (d + 1)) * V;
      for (int e = tid; e < NSn * r; e += LEVEL_THREADS) {
        const int j = e / r, k = e % r;
        Wc[(size_t)j * rs + k] = s_stok[j] >= 0 ? __bfloat162float(Wg[(size_t)k * V + s_stok[j]]) : 0.f;
      }
      if (tid < NSn) s_sval[tid] = s_stok[tid] >= 0 ? __bfloat162float(Urow[s_stok[tid]]) : -INFINITY;
      sync();
      // The parents' rows of A are staged in shared memory a batch of SEED_PBATCH parents at a time (one coalesced
      // sweep per batch): read per pair from global memory they were r / 8 dependent round trips per pair, and a
      // request of the wide configuration has 5,000 pairs.
      uint4* Ast = reinterpret_cast<uint4*>(res + (size_t)a.N * NSn * 2);   // [SEED_PBATCH][r] bf16
      const int cpr = r / 8;                                                  // r is a multiple of 8 on this path
      for (int i0 = 0; i0 < cnt; i0 += SEED_PBATCH) {
        const int nbat = min(SEED_PBATCH, cnt - i0);
        for (int e = tid; e < nbat * cpr; e += LEVEL_THREADS)
          Ast[e] = __ldg(reinterpret_cast<const uint4*>(Ag + (size_t)s_ptok[i0 + e / cpr] * r) + e % cpr);
        sync();
        for (int e = tid; e < nbat * NSn; e += LEVEL_THREADS) {
          const int il = e / NSn, i = i0 + il, j = e % NSn;
          float lg = -INFINITY, key = -INFINITY;
          const int tok = s_stok[j];
          if (tok >= 0) {
            const uint4* arow = Ast + (size_t)il * cpr;
            float dot = 0.f;
            for (int k8 = 0; k8 < cpr; ++k8) {
              float av[8];
              unpack_bf16x8(arow[k8], av);
#pragma unroll
              for (int u = 0; u < 8; ++u) dot = fmaf(av[u], Wc[(size_t)j * rs + k8 * 8 + u], dot);
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
          res[2 * ((size_t)i * NSn + j)] = lg; res[2 * ((size_t)i * NSn + j) + 1] = key;
        }
        sync();
      }
      for (int e = tid; e < 2 * cnt; e += LEVEL_THREADS) a.thr0[(size_t)(e & 1) * a.cap + s_pli[e >> 1]] = 0u;   // no bound unless K finite values turn up
      sync();
      for (int e = tid; e < 2 * cnt * NSn; e += LEVEL_THREADS) {
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


}  // namespace ts
