// Merge of the per-piece scoring records of one parent (Eq. 1 log-normalisers, the K best logits and the K
// best sampling keys of Eq. 2): the body shared by merge_kernel and the persistent expansion kernel.
#pragma once
#include "ts_internal.h"
#include "ts_scan.cuh"

namespace ts {

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
template <int KR, class Sync>
__device__ void block_select(MList<KR>& mine, int K, int* out_tok, float* out_val, float* s_v, int* s_i, float* s_l, const int tid, Sync sync) {
  const int lane = tid & 31, warp = tid >> 5;
  for (int j = 0; j < K; ++j) {
    float wv = mine.v[0]; int wi = mine.i[0]; float wl = mine.l[0];
    for (int off = 16; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, wv, off);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, wi, off);
      const float ol = __shfl_xor_sync(0xFFFFFFFFu, wl, off);
      if (better(ov, oi, wv, wi)) { wv = ov; wi = oi; wl = ol; }
    }
    if (lane == 0) { s_v[warp] = wv; s_i[warp] = wi; s_l[warp] = wl; }
    sync();
    float gv = s_v[0]; int gi = s_i[0]; float gl = s_l[0];
#pragma unroll
    for (int w = 1; w < MERGE_WARPS; ++w)
      if (better(s_v[w], s_i[w], gv, gi)) { gv = s_v[w]; gi = s_i[w]; gl = s_l[w]; }
    if (gi != 0x7FFFFFFF && mine.i[0] == gi) mine.pop();  // tokens are unique per list
    if (tid == 0) { out_tok[j] = gi == 0x7FFFFFFF ? -1 : gi; out_val[j] = gi == 0x7FFFFFFF ? 0.f : gl; }
    sync();
  }
}

constexpr int MERGE_CAP = 768;   // candidates per list the fast path can hold

// The K best of a candidate array in shared memory (value desc, token asc), by counting: a candidate's
// place is the number of candidates that beat it (tokens are unique per list, so places are too).  With
// tight bounds a few dozen candidates arrive here, and the whole selection is one short pass.
__device__ __forceinline__ void rank_select(const float* cv, const int* ci, const float* cl, int n, int K, int t, int nt, int* out_tok, float* out_val) {
  for (int e = t; e < n; e += nt) {
    const float v = cv[e]; const int idx = ci[e];
    int rank = 0;
    for (int f = 0; f < n; ++f) rank += better(cv[f], ci[f], v, idx) ? 1 : 0;
    if (rank < K) { out_tok[rank] = idx; out_val[rank] = cl[e]; }
  }
  for (int j = n + t; j < K; j += nt) { out_tok[j] = -1; out_val[j] = 0.f; }
}

struct MergeSmem {
  float s_v[MERGE_WARPS]; int s_i[MERGE_WARPS]; float s_l[MERGE_WARPS];
  float s_m[MERGE_WARPS], s_s0[MERGE_WARPS], s_sT[MERGE_WARPS];
  float c_v[2][MERGE_CAP]; int c_i[2][MERGE_CAP]; float c_l[2][MERGE_CAP];
  int c_n[2];
};

// Every thread folds its share of the pieces into a private (max, sums) pair and hands the list entries that
// survive the final bounds to shared memory; the block then ranks them (value desc, token asc).  Called by
// MERGE_THREADS threads (tid = 0 .. MERGE_THREADS-1) that `sync` synchronises; P = parents of the launch.
template <int KR, class Sync>
__device__ __forceinline__ void merge_parent(const MergeArgs& a, const int p, const int P, MergeSmem& sm, const int tid, Sync sync) {
  float (&s_v)[MERGE_WARPS] = sm.s_v; int (&s_i)[MERGE_WARPS] = sm.s_i; float (&s_l)[MERGE_WARPS] = sm.s_l;
  float (&s_m)[MERGE_WARPS] = sm.s_m; float (&s_s0)[MERGE_WARPS] = sm.s_s0; float (&s_sT)[MERGE_WARPS] = sm.s_sT;
  float (&c_v)[2][MERGE_CAP] = sm.c_v; int (&c_i)[2][MERGE_CAP] = sm.c_i; float (&c_l)[2][MERGE_CAP] = sm.c_l;
  int (&c_n)[2] = sm.c_n;
  const int lane = tid & 31, warp = tid >> 5;
  const float invT = a.T > 0.f ? 1.f / a.T : 1.f;
  const int K = a.K, rw = rec_words(K);
  const bool few = a.few_ntiles > 0;   // the level was scored by the few-parents kernel
  const int R = few ? 1 : (a.mma ? mma_replicas(P) : 1);
  const int npieces = few ? a.few_ntiles : a.ntiles * a.S * R;
  {
    // final launch-wide lower bounds of this parent's K-th best logit / key: entries below cannot win
    const SharedThr gl{a.slots + (size_t)p * K * SLOT_STRIDE, 0}, gk{a.slots + ((size_t)a.cap + p) * K * SLOT_STRIDE, 0};
    float bL = dec_f(slots_min(gl, K)), bK = a.T > 0.f ? dec_f(slots_min(gk, K)) : -INFINITY;
    if (a.thr0) {   // never below the parent's seed bounds
      bL = fmaxf(bL, dec_f(__ldcg(a.thr0 + p)));
      if (a.T > 0.f) bK = fmaxf(bK, dec_f(__ldcg(a.thr0 + (size_t)a.cap + p)));
    }
    if (tid < 2) c_n[tid] = 0;
    sync();
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
    sync();
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
      sync();
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
      sync();
      block_select<KR>(top, K, a.top_tok + (size_t)p * K, a.top_logit + (size_t)p * K, s_v, s_i, s_l, tid, sync);
      if (a.T > 0.f) block_select<KR>(key, K, a.draw_tok + (size_t)p * K, a.draw_logit + (size_t)p * K, s_v, s_i, s_l, tid, sync);
    }
    if (!(a.T > 0.f)) {
      if (tid < K) {
        a.draw_tok[(size_t)p * K + tid] = a.top_tok[(size_t)p * K + tid];
        a.draw_logit[(size_t)p * K + tid] = a.top_logit[(size_t)p * K + tid];
      }
    }
    sync();
  }
}


}  // namespace ts
