// Calibration statistics from verified trees and the refit of the edge-acceptance map (Section 3.4).
//
// Accumulation: one CTA per request, one thread per node.  The committed path marks its nodes in shared
// memory; an edge belongs to the ancestors-accepted population when its parent is the root or marked.
// Every edge adds (1, label, logit) as integers to the cell (population, parent depth, nearest knot) of
// a histogram in shared memory, and the CTA's non-empty cells go to the caller's array with one atomic
// each.  Integer sums: the array does not depend on the order in which CTAs, rounds or streams add.
//
// Refit: one CTA, one thread per cell (depth row, knot).  The two scalars of Eq. 3 by Newton's method with
// step halving on the cell-weighted logistic likelihood (block-wide sums, every thread takes the same
// step), the table by pool-adjacent-violators over the sixteen cells of a depth row (one thread per row).
#include "ts_internal.h"

namespace ts {

constexpr int CAL_THREADS = 256;           // >= Nmax, and >= D * KNOTS cells
constexpr int CAL_WORDS = 3;
constexpr double CAL_UNIT = 16777216.0;    // 2^24
constexpr double CAL_SHIFT = 32.0;

struct CalAccArgs {
  int B, N, D;
  double lo, hi;
  const int* n_nodes; const int* parent; const int* depth; const float* q0;
  const int* acc_len; const int* acc_node; const float* edge_stat;
  unsigned long long* stats;   // [2][D][KNOTS][3]
};

__global__ void __launch_bounds__(CAL_THREADS) calib_accumulate_kernel(const CalAccArgs a) {
  __shared__ unsigned long long s_hist[2 * DMAX * KNOTS * CAL_WORDS];
  __shared__ unsigned char s_on_path[CAL_THREADS];
  const int b = blockIdx.x, i = threadIdx.x;
  const int cells = 2 * a.D * KNOTS * CAL_WORDS;
  pdl_wait();                 // trees and verdicts come from the kernels before this one
  pdl_launch_dependents();
  for (int c = i; c < cells; c += CAL_THREADS) s_hist[c] = 0ull;
  s_on_path[i] = 0;
  __syncthreads();
  const int n = min(max(a.n_nodes[b], 0), a.N);
  const int L = min(max(a.acc_len[b], 0), a.D);
  if (i < L) {
    const int node = a.acc_node[(size_t)b * a.D + i];
    if (node >= 0 && node < n) s_on_path[node] = 1;
  }
  __syncthreads();
  if (i < n) {
    const size_t e = (size_t)b * a.N + i;
    const int p = a.parent[e];
    const bool anc = p < 0 || (p < n && s_on_path[p]);
    double q = (double)a.q0[e];
    if (q > 1.0 - 1e-12) q = 1.0 - 1e-12;
    double t = q > 0.0 ? log(q) - log1p(-q) : -30.0;
    t = t > 30.0 ? 30.0 : (t < -30.0 ? -30.0 : t);
    const double pos = (t - a.lo) / (a.hi - a.lo) * (KNOTS - 1);
    int j = (int)floor(pos + 0.5);
    j = j < 0 ? 0 : (j > KNOTS - 1 ? KNOTS - 1 : j);
    int d = a.depth[e] - 1;
    d = d < 0 ? 0 : (d > a.D - 1 ? a.D - 1 : d);
    const unsigned long long y = (unsigned long long)__double2ll_rn((double)a.edge_stat[e] * CAL_UNIT);
    const unsigned long long x = (unsigned long long)__double2ll_rn((t + CAL_SHIFT) * CAL_UNIT);
    for (int pop = 0; pop < (anc ? 2 : 1); ++pop) {
      unsigned long long* cell = s_hist + ((size_t)(pop * a.D + d) * KNOTS + j) * CAL_WORDS;
      atomicAdd(cell, 1ull);
      atomicAdd(cell + 1, y);
      atomicAdd(cell + 2, x);
    }
  }
  __syncthreads();
  for (int c = i; c < cells; c += CAL_THREADS)
    if (s_hist[c]) atomicAdd(a.stats + c, s_hist[c]);
}

struct CalFitArgs {
  int D, pop, min_count;
  DevCalib calib;
  const unsigned long long* stats;
  const float* fallback; float* table; double* platt;
};

// sum over the block; every thread gets the same value (fixed order: lanes, then warps)
__device__ __forceinline__ double block_sum(double v, double* s_part) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  __syncthreads();   // the previous use of s_part is over
  if (lane == 0) s_part[warp] = v;
  __syncthreads();
  double tot = 0.0;
#pragma unroll
  for (int w = 0; w < CAL_THREADS / 32; ++w) tot += s_part[w];
  return tot;
}

__global__ void __launch_bounds__(CAL_THREADS) calib_refit_kernel(const CalFitArgs a) {
  __shared__ double s_part[CAL_THREADS / 32];
  const int t = threadIdx.x;
  pdl_wait();
  pdl_launch_dependents();
  const int d = t / KNOTS, j = t % KNOTS;
  const bool live = d < a.D;
  double n = 0.0, ysum = 0.0, xsum = 0.0;
  if (live) {
    const unsigned long long* cell = a.stats + ((size_t)(a.pop * a.D + d) * KNOTS + j) * CAL_WORDS;
    n = (double)cell[0]; ysum = (double)cell[1]; xsum = (double)cell[2];
  }
  const bool has = n > 0.0;
  const double x = has ? xsum / CAL_UNIT / n - CAL_SHIFT : 0.0;
  const double y = has ? ysum / CAL_UNIT / n : 0.0;

  // ---- the two scalars of Eq. 3 -------------------------------------------------------------------
  if (a.platt) {
    // negative log-likelihood of the cells under (qa, qb); the same value in every thread
    auto nll = [&](double qa, double qb) -> double {
      double f = 0.0;
      if (has) {
        const double z = qa * x + qb;
        f = n * (fmax(z, 0.0) + log1p(exp(-fabs(z))) - y * z);
      }
      return block_sum(f, s_part);
    };
    double pa = 0.0, pb = 0.0;
    double f = nll(pa, pb);
    int it = 0;
    for (it = 1; it <= 100; ++it) {
      double r = 0.0, w = 0.0;
      if (has) {
        const double p = 1.0 / (1.0 + exp(-(pa * x + pb)));
        r = n * (y - p);
        w = n * p * (1.0 - p);
      }
      const double ga = block_sum(r * x, s_part), gb = block_sum(r, s_part);
      const double haa = block_sum(w * x * x, s_part) + 1e-12, hab = block_sum(w * x, s_part);
      const double hbb = block_sum(w, s_part) + 1e-12;
      const double det = haa * hbb - hab * hab;
      if (!(det > 1e-300)) break;
      const double da = (hbb * ga - hab * gb) / det, db = (haa * gb - hab * ga) / det;
      // halve the step until the likelihood does not get worse (every thread takes the same decisions)
      double step = 1.0, na = pa, nb = pb, nf = f;
      bool ok = false;
      for (int h = 0; h < 30; ++h) {
        na = pa + step * da; nb = pb + step * db;
        nf = nll(na, nb);
        if (nf <= f) { ok = true; break; }
        step *= 0.5;
      }
      if (!ok) break;
      const double moved = fmax(fabs(na - pa), fabs(nb - pb));
      pa = na; pb = nb; f = nf;
      if (moved < 1e-12) break;
    }
    if (it > 100) it = 100;
    const double used = block_sum(n, s_part);
    if (t == 0) { a.platt[0] = pa; a.platt[1] = pb; a.platt[2] = (double)it; a.platt[3] = used; }
  }

  // ---- the per-depth table ---------------------------------------------------------------------------
  if (a.table && live && j == 0) {
    const unsigned long long* row = a.stats + (size_t)(a.pop * a.D + d) * KNOTS * CAL_WORDS;
    const double need = (double)(a.min_count > 1 ? a.min_count : 1);
    // blocks of pool-adjacent-violators over the knots that have data
    double bm[KNOTS], bw[KNOTS]; int bl[KNOTS], have[KNOTS];
    int nb = 0, nh = 0;
    for (int k = 0; k < KNOTS; ++k) {
      const double cn = (double)row[k * CAL_WORDS];
      if (!(cn >= need)) continue;
      have[nh++] = k;
      bm[nb] = ((double)row[k * CAL_WORDS + 1] / CAL_UNIT + 1.0) / (cn + 2.0);   // rule of succession
      bw[nb] = cn; bl[nb] = 1; ++nb;
      while (nb > 1 && bm[nb - 2] > bm[nb - 1]) {
        const double w = bw[nb - 2] + bw[nb - 1];
        bm[nb - 2] = (bm[nb - 2] * bw[nb - 2] + bm[nb - 1] * bw[nb - 1]) / w;
        bw[nb - 2] = w; bl[nb - 2] += bl[nb - 1]; --nb;
      }
    }
    float* out = a.table + (size_t)d * KNOTS;
    if (nh == 0) {
      // no data at this depth: the caller's fallback row, else the context's own map at the knots
      for (int k = 0; k < KNOTS; ++k) {
        float v;
        if (a.fallback) v = a.fallback[d * KNOTS + k];
        else if (a.calib.mode == 1) v = a.calib.table[d * KNOTS + k];
        else {
          const double tk = a.calib.lo + (a.calib.hi - a.calib.lo) * k / (KNOTS - 1);
          v = (float)(1.0 / (1.0 + exp(-(a.calib.a * tk + a.calib.b))));
        }
        out[k] = v;
      }
    } else {
      double iso[KNOTS];   // value at the i-th knot with data
      for (int blk = 0, i = 0; blk < nb; ++blk)
        for (int c = 0; c < bl[blk]; ++c) iso[i++] = bm[blk];
      int seg = 0;         // largest index with have[seg] <= k
      for (int k = 0; k < KNOTS; ++k) {
        double v;
        if (k <= have[0]) v = iso[0];
        else if (k >= have[nh - 1]) v = iso[nh - 1];
        else {
          while (seg + 1 < nh && have[seg + 1] <= k) ++seg;
          if (have[seg] == k) v = iso[seg];
          else {
            const double f = (double)(k - have[seg]) / (double)(have[seg + 1] - have[seg]);
            v = iso[seg] + f * (iso[seg + 1] - iso[seg]);
          }
        }
        v = v < 1e-6 ? 1e-6 : (v > 1.0 ? 1.0 : v);
        out[k] = (float)v;
      }
    }
  }
}

}  // namespace ts

extern "C" int32_t ts_calib_accumulate(ts_ctx* ctx, int32_t B, const int32_t* n_nodes, const int32_t* parent,
                                       const int32_t* depth, const float* q0, const int32_t* acc_len,
                                       const int32_t* acc_node, const float* edge_stat, uint64_t* stats, void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_calib_accumulate: null context");
  const void* req[] = {n_nodes, parent, depth, q0, acc_len, acc_node, edge_stat, stats};
  for (const void* p : req)
    if (bad_ptr(p)) return set_error(TS_ERR_INVALID, "ts_calib_accumulate: null or misaligned pointer");
  const ts_config& c = ctx->cfg;
  if (B < 1 || B > c.max_batch) return set_error(TS_ERR_INVALID, "ts_calib_accumulate: B out of range");
  if (c.Nmax > CAL_THREADS) return set_error(TS_ERR_UNSUPPORTED, "ts_calib_accumulate: Nmax <= 256 required");
  CalAccArgs a{};
  a.B = B; a.N = c.Nmax; a.D = c.D; a.lo = ctx->calib.lo; a.hi = ctx->calib.hi;
  a.n_nodes = n_nodes; a.parent = parent; a.depth = depth; a.q0 = q0;
  a.acc_len = acc_len; a.acc_node = acc_node; a.edge_stat = edge_stat;
  a.stats = reinterpret_cast<unsigned long long*>(stats);
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  {
    ProfScope ps(ctx, K_CALIB_ACC, st);
    e = launch_kernel(calib_accumulate_kernel, dim3(B), dim3(CAL_THREADS), 0, st, true, a);
  }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_calib_accumulate", e);
  return TS_OK;
}

extern "C" int32_t ts_calib_refit(ts_ctx* ctx, const uint64_t* stats, int32_t population, int32_t min_count,
                                  const float* fallback, float* table, double* platt, void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_calib_refit: null context");
  if (bad_ptr(stats)) return set_error(TS_ERR_INVALID, "ts_calib_refit: null or misaligned stats");
  const void* opt[] = {fallback, table, platt};
  for (const void* p : opt)
    if (p && ((uintptr_t)p & 15u)) return set_error(TS_ERR_INVALID, "ts_calib_refit: misaligned pointer");
  if (!table && !platt) return set_error(TS_ERR_INVALID, "ts_calib_refit: neither table nor platt requested");
  if (population != 0 && population != 1) return set_error(TS_ERR_INVALID, "ts_calib_refit: population must be 0 or 1");
  if (min_count < 0) return set_error(TS_ERR_INVALID, "ts_calib_refit: min_count must be >= 0");
  CalFitArgs a{};
  a.D = ctx->cfg.D; a.pop = population; a.min_count = min_count; a.calib = ctx->calib;
  a.stats = reinterpret_cast<const unsigned long long*>(stats);
  a.fallback = fallback; a.table = table; a.platt = platt;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  {
    ProfScope ps(ctx, K_CALIB_FIT, st);
    e = launch_kernel(calib_refit_kernel, dim3(1), dim3(CAL_THREADS), 0, st, true, a);
  }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_calib_refit", e);
  return TS_OK;
}

extern "C" int32_t ts_calib_load_table(ts_ctx* ctx, const float* table, void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_calib_load_table: null context");
  if (bad_ptr(table)) return set_error(TS_ERR_INVALID, "ts_calib_load_table: null or misaligned table");
  if (ctx->cfg.calib_mode != 1 || !ctx->d_table)
    return set_error(TS_ERR_INVALID, "ts_calib_load_table: the context was not created in table mode");
  const size_t bytes = (size_t)ctx->cfg.D * KNOTS * sizeof(float);
  const cudaError_t e = cudaMemcpyAsync(ctx->d_table, table, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e != cudaSuccess) return set_cuda_error("ts_calib_load_table", e);
  return TS_OK;
}
