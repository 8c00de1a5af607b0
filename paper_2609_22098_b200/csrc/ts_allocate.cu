// Per-request budget allocation under one node budget for the batch (Section 4, second component of
// the controller): greedy water-filling over the admission keys of all trees, then the cut.
//
// Because a request's keys never increase along its admission order, handing the budget out one node at
// a time to the request with the largest next key is the same as taking the `budget` largest candidates
// of the whole batch under the order (key descending, request ascending, admission rank ascending).  So
// the allocation is one selection: find the key of the budget-th candidate (a most-significant-digit
// radix select over the order-preserving integer image of the fp32 keys, four passes of eight bits),
// count per request the candidates above it, and hand the candidates equal to it out in request order
// until the budget is gone.  One CTA does this; the keys' images stay in shared memory between the passes
// when they fit (11k candidates), else the keys are re-read from L2 (a few hundred KB at most).  A second kernel, one CTA per request and one thread per node, compacts the per-node
// arrays in place: all reads, a barrier, all writes.
#include "ts_internal.h"

namespace ts {

constexpr int SEL_THREADS = 1024;
constexpr int CUT_THREADS = 256;   // >= Nmax

struct AllocArgs {
  int B, N, words, budget;
  int* n_nodes; int* tok; int* parent; int* depth; int* sib;
  float* logS; float* q0; float* logqT; float* logkey; int* pop;
  uint64_t* hash; float* lseT; uint64_t* mask;
  float* log_price;
  int* keep;   // workspace, [B]
};

// order-preserving image of a float (-0 counts as +0); every finite or infinite value maps above 0
__device__ __forceinline__ unsigned key_image(float f) {
  const unsigned u = __float_as_uint(f + 0.f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_of_image(unsigned e) {
  return __uint_as_float((e & 0x80000000u) ? (e & 0x7FFFFFFFu) : ~e);
}

__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int o = __shfl_up_sync(0xFFFFFFFFu, v, off);
    if (lane >= off) v += o;
  }
  return v;
}

// exclusive prefix sums of s[0..n) in place, whole block; *total gets the sum.  tmp: 33 ints of shared memory
__device__ void block_excl_scan(int* s, int n, int* tmp, int* total) {
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5, nw = blockDim.x >> 5;
  const int per = (n + blockDim.x - 1) / blockDim.x;
  const int lo = min(t * per, n), hi = min(lo + per, n);
  int sum = 0;
  for (int i = lo; i < hi; ++i) sum += s[i];
  const int incl = warp_incl_scan(sum, lane);
  if (lane == 31) tmp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < nw ? tmp[lane] : 0;
    const int wi = warp_incl_scan(w, lane);
    tmp[lane] = wi - w;
    if (lane == 31) tmp[32] = wi;
  }
  __syncthreads();
  int run = tmp[warp] + incl - sum;
  for (int i = lo; i < hi; ++i) { const int v = s[i]; s[i] = run; run += v; }
  if (t == 0) *total = tmp[32];
  __syncthreads();
}

__global__ void __launch_bounds__(SEL_THREADS) allocate_select_kernel(const AllocArgs a, const int cached) {
  extern __shared__ int s_dyn[];   // n[B], counts[B], then (cached) the key images [B * N]
  __shared__ int s_hist[256];
  __shared__ int s_tmp[33];
  __shared__ int s_total;
  __shared__ unsigned s_prefix;
  __shared__ int s_remaining;
  int* s_n = s_dyn; int* s_cnt = s_dyn + a.B;
  unsigned* s_img = reinterpret_cast<unsigned*>(s_dyn + 2 * a.B);
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  pdl_wait();                 // the trees come from the kernels before this one
  pdl_launch_dependents();
  const int B = a.B, N = a.N, M = B * N;

  for (int b = t; b < B; b += SEL_THREADS) { s_n[b] = min(max(a.n_nodes[b], 0), N); s_cnt[b] = 0; }
  __syncthreads();
  // image of candidate e, 0 (below every key) where the tree has no node e
  auto image = [&](int e) -> unsigned {
    if (cached) return s_img[e];
    const int b = e / N;
    return e - b * N < s_n[b] ? key_image(a.logkey[e]) : 0u;
  };
  {
    int sum = 0;   // how many candidates there are at all
    for (int b = t; b < B; b += SEL_THREADS) sum += s_n[b];
    if (cached)
      for (int e = t; e < M; e += SEL_THREADS) {
        const int b = e / N;
        s_img[e] = e - b * N < s_n[b] ? key_image(a.logkey[e]) : 0u;
      }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, off);
    if (lane == 0) s_tmp[warp] = sum;
    __syncthreads();
    if (warp == 0) {
      int tot = s_tmp[lane];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) tot += __shfl_xor_sync(0xFFFFFFFFu, tot, off);
      if (lane == 0) s_total = tot;
    }
    __syncthreads();
  }
  const int total = s_total;
  const int want = min(max(a.budget, 0), total);
  if (want == 0 || want == total) {   // nothing to hand out, or enough for everybody: no selection
    for (int b = t; b < B; b += SEL_THREADS) a.keep[b] = want ? s_n[b] : 0;
    if (a.log_price) {
      // the smallest key of the batch is the price when every candidate is taken
      unsigned mn = 0xFFFFFFFFu;
      if (want)
        for (int e = t; e < M; e += SEL_THREADS) { const unsigned img = image(e); if (img) mn = min(mn, img); }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) mn = min(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, off));
      __syncthreads();
      if (lane == 0) s_tmp[warp] = (int)mn;
      __syncthreads();
      if (t == 0) {
        unsigned m = 0xFFFFFFFFu;
        for (int w = 0; w < SEL_THREADS / 32; ++w) m = min(m, (unsigned)s_tmp[w]);
        *a.log_price = want ? key_of_image(m) : -INFINITY;
      }
    }
    return;
  }

  // ---- radix select: the image of the want-th largest key, and how many candidates equal to it are taken ----
  if (t == 0) { s_prefix = 0u; s_remaining = want; }
  unsigned fixed = 0u;   // mask of the digits already decided
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (t < 256) s_hist[t] = 0;
    __syncthreads();
    const unsigned prefix = s_prefix;
    for (int e = t; e < M; e += SEL_THREADS) {
      const unsigned img = image(e);
      if (img && (img & fixed) == prefix) atomicAdd(&s_hist[(img >> shift) & 255u], 1);
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns the digits 255 - 8l .. 248 - 8l, highest first
      int h[8], sum = 0;
#pragma unroll
      for (int k = 0; k < 8; ++k) { h[k] = s_hist[255 - 8 * lane - k]; sum += h[k]; }
      const int incl = warp_incl_scan(sum, lane);
      const int rem = s_remaining;
      const unsigned hit = __ballot_sync(0xFFFFFFFFu, incl >= rem);
      const int owner = __ffs(hit) - 1;   // hit is never empty: the matching candidates number >= rem
      if (lane == owner) {
        int before = incl - sum, d = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          if (before + h[k] >= rem) { d = 255 - 8 * lane - k; break; }
          before += h[k];
        }
        s_prefix = prefix | ((unsigned)d << shift);
        s_remaining = rem - before;
      }
    }
    fixed |= 255u << shift;
    __syncthreads();
  }
  const unsigned thr = s_prefix;
  const int ties_taken = s_remaining;   // 1 .. number of candidates equal to the price

  // ---- per request: candidates above the price (low half), candidates at the price (high half) -----------------
  for (int e = t; e < M; e += SEL_THREADS) {
    const unsigned img = image(e);
    if (img > thr) atomicAdd(&s_cnt[e / N], 1);
    else if (img == thr) atomicAdd(&s_cnt[e / N], 1 << 16);
  }
  __syncthreads();
  // the candidates at the price are handed out in request order: exclusive prefix sums of their counts
  int my_gt[4], my_tie[4];   // requests b = t, t + 1024, ... (max_batch <= 4096)
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int b = t + k * SEL_THREADS;
    const int w = b < B ? s_cnt[b] : 0;
    my_gt[k] = w & 0xFFFF; my_tie[k] = w >> 16;
    if (b < B) s_n[b] = my_tie[k];
  }
  __syncthreads();
  block_excl_scan(s_n, B, s_tmp, &s_total);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int b = t + k * SEL_THREADS;
    if (b < B) a.keep[b] = my_gt[k] + min(max(ties_taken - s_n[b], 0), my_tie[k]);
  }
  if (t == 0 && a.log_price) *a.log_price = key_of_image(thr);
}

__global__ void __launch_bounds__(CUT_THREADS) allocate_cut_kernel(const AllocArgs a) {
  __shared__ int s_new[CUT_THREADS];
  __shared__ int s_warp[CUT_THREADS / 32];
  const int b = blockIdx.x, i = threadIdx.x, lane = i & 31, warp = i >> 5;
  pdl_wait();
  pdl_launch_dependents();
  const int N = a.N, n = min(max(a.n_nodes[b], 0), N), keep = a.keep[b];
  if (keep >= n) return;   // the whole tree stays (uniform over the CTA)
  const size_t base = (size_t)b * N, hbase = (size_t)b * (N + 1);
  const bool valid = i < n;
  const int pop = valid ? a.pop[base + i] : 0x7FFFFFFF;
  const bool kept = valid && pop < keep;

  // new index = number of kept nodes before this one
  const unsigned bal = __ballot_sync(0xFFFFFFFFu, kept);
  if (lane == 0) s_warp[warp] = __popc(bal);
  __syncthreads();
  int before = __popc(bal & ((1u << lane) - 1u));
  for (int w = 0; w < warp; ++w) before += s_warp[w];
  s_new[i] = kept ? before : -1;

  // ---- all reads ----
  int v_tok = 0, v_par = -1, v_dep = 0, v_sib = 0;
  float v_logS = 0.f, v_q0 = 0.f, v_lq = 0.f, v_key = 0.f, v_lse = 0.f;
  uint64_t v_hash = 0, v_mask[4] = {0, 0, 0, 0};
  if (kept) {
    if (a.tok) v_tok = a.tok[base + i];
    if (a.parent) v_par = a.parent[base + i];
    if (a.depth) v_dep = a.depth[base + i];
    if (a.sib) v_sib = a.sib[base + i];
    if (a.logS) v_logS = a.logS[base + i];
    if (a.q0) v_q0 = a.q0[base + i];
    if (a.logqT) v_lq = a.logqT[base + i];
    v_key = a.logkey[base + i];
    if (a.hash) v_hash = a.hash[hbase + 1 + i];
    if (a.lseT) v_lse = a.lseT[hbase + 1 + i];
    if (a.mask) {
#pragma unroll
      for (int w = 0; w < 4; ++w)
        if (w < a.words) v_mask[w] = a.mask[(base + i) * a.words + w];
    }
  }
  __syncthreads();   // every read of the old numbering is done, s_new is complete

  // ---- all writes ----
  if (kept) {
    const size_t o = base + before;
    if (a.tok) a.tok[o] = v_tok;
    if (a.parent) a.parent[o] = v_par < 0 ? -1 : s_new[v_par];
    if (a.depth) a.depth[o] = v_dep;
    if (a.sib) a.sib[o] = v_sib;
    if (a.logS) a.logS[o] = v_logS;
    if (a.q0) a.q0[o] = v_q0;
    if (a.logqT) a.logqT[o] = v_lq;
    a.logkey[o] = v_key;
    a.pop[o] = pop;
    if (a.hash) a.hash[hbase + 1 + before] = v_hash;
    if (a.lseT) a.lseT[hbase + 1 + before] = v_lse;
    if (a.mask) {
      // an ancestor of a kept node is kept: every set bit moves to its node's new index
      uint64_t m[4] = {0, 0, 0, 0};
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        uint64_t bits = v_mask[w];   // words past the row's length are zero
        while (bits) {
          const int j = w * 64 + __ffsll((long long)bits) - 1;
          bits &= bits - 1;
          const int nj = s_new[j];
          const uint64_t bit = nj >= 0 ? 1ull << (nj & 63) : 0ull;
#pragma unroll
          for (int x = 0; x < 4; ++x) m[x] |= (nj >> 6) == x ? bit : 0ull;
        }
      }
#pragma unroll
      for (int w = 0; w < 4; ++w)
        if (w < a.words) a.mask[o * a.words + w] = m[w];
    }
  }
  if (i == 0) a.n_nodes[b] = keep;
}

}  // namespace ts

extern "C" int32_t ts_allocate_budget(ts_ctx* ctx, int32_t B, int32_t budget, int32_t* n_nodes, int32_t* tok,
                                      int32_t* parent, int32_t* depth, int32_t* sib_rank, float* logS, float* q0,
                                      float* logqT, float* logkey, int32_t* pop_rank, uint64_t* node_hash,
                                      float* node_lseT, uint64_t* mask, float* log_price, void* ws_v, size_t ws_bytes,
                                      void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_allocate_budget: null context");
  const void* req[] = {n_nodes, logkey, pop_rank, ws_v};
  for (const void* p : req)
    if (bad_ptr(p)) return set_error(TS_ERR_INVALID, "ts_allocate_budget: null or misaligned pointer");
  const void* opt[] = {tok, parent, depth, sib_rank, logS, q0, logqT, node_hash, node_lseT, mask};
  for (const void* p : opt)
    if (p && ((uintptr_t)p & 15u)) return set_error(TS_ERR_INVALID, "ts_allocate_budget: misaligned optional pointer");
  if (log_price && ((uintptr_t)log_price & 3u)) return set_error(TS_ERR_INVALID, "ts_allocate_budget: misaligned log_price");
  const ts_config& c = ctx->cfg;
  if (B < 1 || B > c.max_batch) return set_error(TS_ERR_INVALID, "ts_allocate_budget: B out of range");
  if (budget < 0) return set_error(TS_ERR_INVALID, "ts_allocate_budget: budget must be >= 0");
  if (c.Nmax > CUT_THREADS) return set_error(TS_ERR_UNSUPPORTED, "ts_allocate_budget: Nmax <= 256 required");
  const WsLayout L = make_layout(ctx, B);
  if (ws_bytes < L.total) return set_error(TS_ERR_WORKSPACE, "ts_allocate_budget: workspace too small");
  cudaStream_t st = (cudaStream_t)stream;

  AllocArgs a{};
  a.B = B; a.N = c.Nmax; a.words = L.words; a.budget = budget;
  a.n_nodes = n_nodes; a.tok = tok; a.parent = parent; a.depth = depth; a.sib = sib_rank;
  a.logS = logS; a.q0 = q0; a.logqT = logqT; a.logkey = logkey; a.pop = pop_rank;
  a.hash = node_hash; a.lseT = node_lseT; a.mask = mask; a.log_price = log_price;
  a.keep = (int*)((char*)ws_v + L.req_npar);
  cudaError_t e;
  {
    ProfScope ps(ctx, K_ALLOC_SELECT, st);
    // the key images stay in shared memory between the passes when they fit the default 48 KB
    const size_t small = (size_t)2 * B * sizeof(int), all = small + (size_t)B * c.Nmax * sizeof(unsigned);
    const int cached = all <= 48 * 1024 - 2048 ? 1 : 0;
    e = launch_kernel(allocate_select_kernel, dim3(1), dim3(SEL_THREADS), cached ? all : small, st, true, a, cached);
  }
  if (e == cudaSuccess) {
    ProfScope ps(ctx, K_ALLOC_CUT, st);
    e = launch_kernel(allocate_cut_kernel, dim3(B), dim3(CUT_THREADS), 0, st, true, a);
  }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_allocate_budget", e);
  return TS_OK;
}
