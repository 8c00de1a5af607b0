// Seed bounds for the tensor-core scoring kernel (Eq. 1, Eq. 2: which tokens can be among a parent's K best).
//
// The scoring kernel skips a token whose logit (or whose sampling key, bounded from above) lies below a
// lower bound of the parent's K-th best logit (key).  Any K tokens evaluated exactly give such a bound,
// and the bound is tight when those tokens are good ones.  The low-rank bias moves a logit by far less
// than the base logits spread, so the tokens with the largest base logits U[b][d][v] of the parent's row
// are nearly the parent's best tokens.  Per parent: sweep the row once (every thread keeps the best token of
// its share; with few parents several CTAs take parts of the row and the last one to arrive finishes),
// let every warp pick the best of its lanes' bests (2K tokens in all), evaluate those exactly (bias by fused
// multiply-adds, sampling key with the same generator and noise function as the scoring kernel), and leave
//   thr0[0][p] = K-th best exact logit, thr0[1][p] = K-th best exact key,
// each lowered by a margin that covers the rounding difference between this evaluation and the
// tensor-core one, in the order-preserving encoding of the pruning state (0 = no bound).
#include "ts_internal.h"
#include "ts_scan.cuh"

namespace ts {

constexpr int SEED_THREADS = 256;

// Every warp hands over the `npick` best (value desc, token asc) of its lanes' candidates (one per lane, taken
// away as they are picked): 8 * npick good tokens per CTA without any ranking pass.  Entries land in
// s_tok / s_val at [warp * npick + i]; an exhausted warp leaves token -1.
__device__ __forceinline__ void warp_picks(float v, int idx, int npick, int* s_tok, float* s_val) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i = 0; i < npick; ++i) {
    float bv = v; int bi = idx;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, off);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, off);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (bi == idx && v > -INFINITY) { v = -INFINITY; idx = 0x7FFFFFFF; }   // tokens are distinct: exactly one lane gives its candidate up
    if (lane == 0) { s_tok[warp * npick + i] = bv > -INFINITY ? bi : -1; s_val[warp * npick + i] = bv; }
  }
}

__global__ void __launch_bounds__(SEED_THREADS, 2) seed_parents_kernel(const ScoreArgs a) {
  __shared__ int s_tok[NSEED_MAX];
  __shared__ float s_log[NSEED_MAX], s_key[NSEED_MAX];
  __shared__ float s_a[RMAX];
  __shared__ int s_last;
  static_assert((SEED_THREADS / 32) * (NSEED_MAX / (SEED_THREADS / 32)) <= NSEED_MAX, "picks fit the candidate arrays");
  const int tid = threadIdx.x;
  // The parent list and its length come from the kernel before -- except for the root level of an expansion, where
  // parent p is request p at depth 0: there the sweep of the first row (most of this kernel's time) needs nothing
  // from that kernel and runs beside it; the wait comes before the first thing that does.
  const bool root = a.seed_root_B > 0;
  bool waited = !root;
  if (!root) pdl_wait();
  pdl_launch_dependents();
  const int P = root ? a.seed_root_B : (a.P_dev ? *a.P_dev : a.P);
  if (P <= 0) { if (!waited) pdl_wait(); return; }
  const int V = a.V, r = a.r, K = a.K;
  const int npick = max(1, min(2 * K, NSEED_MAX) / (SEED_THREADS / 32));   // 2K tokens per parent (at least 8)
  const float T = a.T, invT = T > 0.f ? 1.f / T : 1.f;
  const __nv_bfloat16* Wg = reinterpret_cast<const __nv_bfloat16*>(a.W);
  const __nv_bfloat16* Ug = reinterpret_cast<const __nv_bfloat16*>(a.U);
  const __nv_bfloat16* Ag = reinterpret_cast<const __nv_bfloat16*>(a.A);
  // With few parents a row is swept by several CTAs (parts of whole 16-byte vectors), so that the sweep is
  // bound by bandwidth and not by the loads one CTA can keep in flight; the last part to arrive finishes.
  int nparts = (int)gridDim.x / P;
  nparts = nparts < 1 ? 1 : (nparts > SEED_PARTS_MAX ? SEED_PARTS_MAX : nparts);
  if (P > SEED_SPLIT_PARENTS) nparts = 1;
  const int nvec = V / 8;
  for (int item = blockIdx.x; item < P * nparts; item += gridDim.x) {
    const int p = item / nparts, part = item % nparts;
    const int req = root ? p : a.p_req[p], dep = root ? 0 : a.p_depth[p];
    const __nv_bfloat16* Urow = Ug + ((size_t)req * a.D + dep) * V;
    if (tid == 0) s_last = 0;
    // ---- the best base logit of every thread's share of this part of the row ------------------------------
    float bv = -INFINITY; int bi = 0x7FFFFFFF;
    {
      const int v_lo = (int)((long long)nvec * part / nparts), v_hi = (int)((long long)nvec * (part + 1) / nparts);
      constexpr int UNR = 8;
      int c = v_lo + tid;
      for (; c + (UNR - 1) * SEED_THREADS < v_hi; c += UNR * SEED_THREADS) {
        uint4 x[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) x[u] = __ldg(reinterpret_cast<const uint4*>(Urow) + c + u * SEED_THREADS);
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
          float f[8];
          unpack_bf16x8(x[u], f);
#pragma unroll
          for (int i = 0; i < 8; ++i) if (f[i] > bv) { bv = f[i]; bi = (c + u * SEED_THREADS) * 8 + i; }
        }
      }
      for (; c < v_hi; c += SEED_THREADS) {
        float f[8];
        unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(Urow) + c), f);
#pragma unroll
        for (int i = 0; i < 8; ++i) if (f[i] > bv) { bv = f[i]; bi = c * 8 + i; }
      }
    }
    warp_picks(bv, bi, npick, s_tok, s_log);
    __syncthreads();
    if (!waited) { pdl_wait(); waited = true; }   // arrival counters, parent tokens and hashes, the bound words
    const int n = (SEED_THREADS / 32) * npick;   // places; an empty one holds token -1
    if (nparts > 1) {
      // leave this part's candidates for whoever finishes the parent; the last part to arrive does
      unsigned* cand = a.seed_cand + ((size_t)p * SEED_PARTS_MAX + part) * NSEED_MAX * 2;
      if (tid < NSEED_MAX) {
        cand[2 * tid] = (tid < n && s_tok[tid] >= 0) ? __float_as_uint(s_log[tid]) : __float_as_uint(-INFINITY);
        cand[2 * tid + 1] = (tid < n && s_tok[tid] >= 0) ? (unsigned)s_tok[tid] : 0x7FFFFFFFu;
      }
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        const unsigned arrived = atomicAdd(a.seed_cnt + p, 1u);
        s_last = (arrived == (unsigned)nparts - 1u) ? 1 : 0;
        if (s_last) a.seed_cnt[p] = 0u;   // clean for the next launch
      }
      __syncthreads();
      if (!s_last) continue;   // uniform
      __threadfence();
      const unsigned* all = a.seed_cand + (size_t)p * SEED_PARTS_MAX * NSEED_MAX * 2;
      // every thread keeps the better of its (at most two) candidates of all parts, then the warps pick again
      float cv = -INFINITY; int ci = 0x7FFFFFFF;
      // (entry e goes to lane e / 8 of warp e % 8: every warp gets its share however few parts there are)
      for (int e = (tid & 31) * 8 + (tid >> 5); e < nparts * NSEED_MAX; e += SEED_THREADS) {
        const float v = __uint_as_float(__ldcg(all + 2 * e)); const int i2 = (int)__ldcg(all + 2 * e + 1);
        if (v > cv || (v == cv && i2 < ci)) { cv = v; ci = i2; }
      }
      __syncthreads();
      warp_picks(cv, ci, npick, s_tok, s_log);
      __syncthreads();
    }
    // ---- exact logits and keys of those tokens: eight lanes per token ---------------------------------------
    const int ptok = a.p_token[p];
    const uint64_t hash = a.p_hash[p];
    for (int k = tid; k < r; k += SEED_THREADS) s_a[k] = __bfloat162float(Ag[(size_t)ptok * r + k]);
    __syncthreads();
    {
      const int j = tid >> 3, sub = tid & 7;
      float part_sum = 0.f;
      int tok = 0;
      const bool have = j < n && s_tok[j] >= 0;
      if (have) {
        tok = s_tok[j];
        for (int k0 = sub; k0 < r; k0 += 64) {   // eight independent loads at a time
          __nv_bfloat16 w[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) w[u] = (k0 + 8 * u < r) ? Wg[(size_t)(k0 + 8 * u) * V + tok] : __float2bfloat16(0.f);
#pragma unroll
          for (int u = 0; u < 8; ++u) if (k0 + 8 * u < r) part_sum = fmaf(s_a[k0 + 8 * u], __bfloat162float(w[u]), part_sum);
        }
      }
      part_sum += __shfl_xor_sync(0xFFFFFFFFu, part_sum, 1);
      part_sum += __shfl_xor_sync(0xFFFFFFFFu, part_sum, 2);
      part_sum += __shfl_xor_sync(0xFFFFFFFFu, part_sum, 4);
      __syncthreads();   // s_log held the candidates' base logits until here
      if (j < n && sub == 0 && !have) { s_log[j] = -INFINITY; s_key[j] = -INFINITY; }
      if (have && sub == 0) {
        const float lg = __bfloat162float(Urow[tok]) + part_sum;
        s_log[j] = lg;
        float key = lg;
        if (T > 0.f) {
          const uint4 cw = stream_words(a.seed, req, hash, STREAM_GUMBEL_COARSE, (uint32_t)tok >> 3);
          const uint4 fw = stream_words(a.seed, req, hash, STREAM_GUMBEL_FINE, (uint32_t)tok >> 3);
          const uint32_t c16 = (word_of(cw, (tok & 7) >> 1) >> (16 * (tok & 1))) & 0xFFFFu;
          const uint32_t f16 = (word_of(fw, (tok & 7) >> 1) >> (16 * (tok & 1))) & 0xFFFFu;
          key = lg * invT + gumbel_from_bits((c16 << 16) | f16);
        }
        s_key[j] = key;
      }
    }
    __syncthreads();
    // ---- K-th best of each, lowered by the margin ---------------------------------------------------------------
    if (tid < 2) a.thr0[(size_t)tid * a.cap + p] = 0u;   // no bound unless K finite values turn up below
    __syncthreads();
    if (tid < 2 * n && (tid < n || T > 0.f)) {
      // one thread per value: the one with exactly K - 1 values before it (ties broken by place) is the K-th best
      const int which = tid / n, j = tid % n;
      const float* val = which == 0 ? s_log : s_key;
      const float mine = val[j];
      int before = 0;
      for (int t = 0; t < n; ++t) before += (val[t] > mine || (val[t] == mine && t < j)) ? 1 : 0;
      if (before == K - 1 && mine == mine && fabsf(mine) < INFINITY) {
        // rounding of an r-term fp32 sum in another order, of the division by T and of the fast logarithms
        const float margin = (2e-4f + 4e-5f * fabsf(mine)) * (which == 0 ? 1.f : fmaxf(invT, 1.f)) + (which == 0 ? 0.f : 2e-4f);
        a.thr0[(size_t)which * a.cap + p] = enc_f(mine - margin);
      }
    }
    __syncthreads();
  }
  if (!waited) pdl_wait();
}

cudaError_t launch_seed(const ts_ctx* ctx, const ScoreArgs& a, cudaStream_t st) {
  const int blocks = 2 * ctx->num_sms;   // work items (parent, part of its row) are dealt to a fixed grid
  const cudaError_t e = launch_kernel(seed_parents_kernel, blocks, SEED_THREADS, 0, st, a.pdl != 0, a);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ts
