// Lossless tree verification (Section 3.2 item 3, Section 3.3).
//
// Stage 1 (all rows, fully parallel): max, arg-max and log-sum-exp at temperature T of every target
//   row, one CTA per row.  With these, the first-sibling accept ratio of every edge is a scalar
//   expression, so per-edge statistics and greedy walks need no further vocabulary pass.
// Stage 2, T == 0: pointer chase along arg-max matches.
// Stage 2, T > 0: one persistent cooperative kernel.  The recursive-rejection walk is run as a
//   scalar sequence: with R(w) = max(p(w) - C q(w), 0) the unnormalised residual after rejections,
//   sibling j is accepted with probability min(1, max(p(x)/q(x) - C, 0) / c_j), c_j = Z_j / (1 - Q),
//   and a rejection moves C to C + c_j and needs Z_{j+1} = sum_w R(w), one reduction over the
//   vocabulary (tokens already tested keep the residual they had when tested).  Every grid step
//   runs that reduction for all requests that just rejected, each CTA owning a vocabulary range;
//   q is recomputed from U, A, W, no per-node vocabulary vector is stored.  The bonus token is the
//   inverse CDF of the final residual in token order: range sums locate the range, one CTA rescans it.
#include <cooperative_groups.h>
#include <math.h>

#include "ts_internal.h"
#include "ts_scan.cuh"
#include "ts_tc.cuh"

namespace ts {

// 2^x by the hardware approximation (the library exp2f costs several times more in the hot loops here)
__device__ __forceinline__ float fast_ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

// maximum that returns NaN when either operand is NaN (fmaxf drops NaNs)
__device__ __forceinline__ float max_nan(float a, float b) { float y; asm("max.NaN.f32 %0, %1, %2;" : "=f"(y) : "f"(a), "f"(b)); return y; }

constexpr int ZT = 512;  // threads per target row in the row-statistics kernel

// ------------------------------------------------------------------------------------------------
// Stage 1: row statistics
// ------------------------------------------------------------------------------------------------
template <typename TIn>
__global__ void __launch_bounds__(ZT) zrow_stats_kernel(const TIn* Z, const int64_t* z_row_off, int B, int V, float T,
                                                       float* z_max, int* z_arg, float* z_logs, unsigned* walk_barrier) {
  // One CTA per target row, one sweep: every thread keeps a running (max, arg-max, sum of exp((z-max)/T))
  // over its share of the row, four 16-byte loads in flight, and the block folds the triples.
  __shared__ float s_v[ZT / 32]; __shared__ int s_i[ZT / 32]; __shared__ float s_s[ZT / 32];
  pdl_wait();   // the target logits (and the tree) may come from the kernel just before this one
  pdl_launch_dependents();
  // the walk's barrier words start at zero (done here rather than by a memset, which would sit between
  // this kernel and the walk in the stream and keep the walk from starting its preamble early)
  if (walk_barrier && blockIdx.x == 0 && threadIdx.x < 16) walk_barrier[threadIdx.x] = 0u;
  const int64_t rows = z_row_off[B];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int VEC = Elem<TIn>::VEC;
  constexpr int UNR = 4;
  const bool vec_ok = (V % VEC) == 0;
  const float invT = T > 0.f ? 1.f / T : 1.f;
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const TIn* z = Z + row * V;
    float bv = -INFINITY, sum = 0.f; int bi = 0x7FFFFFFF;
    // per vector: the maximum by a compare tree (its position is looked for only when it beats the running
    // maximum, which is rare), then one fused multiply-add and one ex2 per element
    const float sc = invT * 1.4426950408889634f;
    float boff = 0.f;   // -bv * sc while bv is finite
    bool has_nan = false;
    auto take = [&](const float* x, int c, int n) {
      float vm = x[0];
#pragma unroll
      for (int i = 1; i < VEC; ++i) if (i < n) vm = max_nan(vm, x[i]);
      has_nan |= vm != vm;   // one test per vector: a NaN anywhere in it survives the maximum
      if (vm > bv) {   // first maximum wins: indices increase
        int vi = 0;
#pragma unroll
        for (int i = VEC - 1; i >= 0; --i) if (i < n && x[i] == vm) vi = i;
        sum *= fast_ex2((bv - vm) * sc);
        bv = vm; bi = c + vi; boff = -vm * sc;
      }
      if (T > 0.f) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) if (i < n) sum += fast_ex2(fmaf(x[i], sc, boff));
      }
    };
    if (vec_ok) {
      int c = tid * VEC;
      for (; c + (UNR - 1) * ZT * VEC < V; c += UNR * ZT * VEC) {
        float x[UNR][8];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
          const TIn* pz = z + c + u * ZT * VEC;
          if (sizeof(TIn) == 2) unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(pz)), x[u]);
          else { const float4 v = __ldg(reinterpret_cast<const float4*>(pz)); x[u][0] = v.x; x[u][1] = v.y; x[u][2] = v.z; x[u][3] = v.w; }
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) take(x[u], c + u * ZT * VEC, VEC);
      }
      for (; c < V; c += ZT * VEC) {
        float x[8];
        if (sizeof(TIn) == 2) unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(z + c)), x);
        else { const float4 v = __ldg(reinterpret_cast<const float4*>(z + c)); x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
        take(x, c, VEC);
      }
    } else {
      for (int c = tid; c < V; c += ZT) { float x[8]; x[0] = Elem<TIn>::to_f(z[c]); take(x, c, 1); }
    }
    // fold (max, arg-max, sum): value descending, ties to the lowest token
    for (int off = 16; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, off); const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, off);
      const float os = __shfl_xor_sync(0xFFFFFFFFu, sum, off);
      const float nm = fmaxf(bv, ov);
      const float ns = (nm > -INFINITY) ? sum * __expf((bv - nm) * invT) + os * __expf((ov - nm) * invT) : 0.f;
      if (ov > bv || (ov == bv && oi < bi)) { bi = oi; }
      bv = nm; sum = ns;
    }
    if (lane == 0) { s_v[warp] = bv; s_i[warp] = bi; s_s[warp] = sum; }
    const int row_nan = __syncthreads_or(has_nan ? 1 : 0);
    if (tid == 0) {
      float gv = s_v[0]; int gi = s_i[0];
      for (int w = 1; w < ZT / 32; ++w) if (s_v[w] > gv || (s_v[w] == gv && s_i[w] < gi)) { gv = s_v[w]; gi = s_i[w]; }
      float gs = 0.f;
      for (int w = 0; w < ZT / 32; ++w) if (s_v[w] > -INFINITY) gs += s_s[w] * __expf((s_v[w] - gv) * invT);
      z_max[row] = row_nan ? nanf("") : gv; z_arg[row] = gi;   // a NaN maximum marks a row that holds a NaN
      if (T > 0.f) z_logs[row] = logf(gs);
    }
    __syncthreads();
  }
}

struct VerifyArgs {
  const void *U, *A, *W, *Z; const int64_t* z_row_off;
  int B, V, D, r, K, N; float T; uint64_t seed;
  const int *anchor, *n_nodes, *tok, *parent, *depth, *sib; const uint64_t* node_hash;
  const float *logqT, *node_lseT;
  const float* z_max; const int* z_arg; const float* z_logs;
  int *acc_len, *acc_node, *acc_tok, *bonus; float* edge_stat; uint32_t* flags; int* status;
  double *edge_px, *edge_qx, *edge_u;   // per edge: target and draft probability of its token, its accept uniform
  VerifyState* state; float* part; unsigned* barrier;
  int* child_first; int* child_cnt;   // [B][N+1], slot 0 = root
  int* wk_list; int* sc_list;         // [2][B] requests that asked for a reduction / a range rescan, by step parity
  int* ctr;                           // [0..1] reduction counts, [2..3] rescan counts (by parity), [4] unfinished requests
  int vt_TV, vt_n, max_steps;
  uint32_t wait_limit;   // polls before a bounded wait (grid barrier, mbarrier) gives up
  int lost_arrival;      // test switch: grid barriers expect one arrival more than will come
  int w_smem;   // 1: the kernel keeps its range of W in dynamic shared memory
  int w_stream; // 1 (tensor-core form only): the range does not fit; blocks of W stream through a ring instead
};

// ------------------------------------------------------------------------------------------------
// Stage 2, T == 0
// ------------------------------------------------------------------------------------------------
__global__ void verify_greedy_kernel(VerifyArgs a) {
  const int b = blockIdx.x, N = a.N;
  const int n_in = a.n_nodes[b];
  const bool okn = n_in >= 0 && n_in <= N;
  const int n = okn ? n_in : 0;
  const int64_t row0 = a.z_row_off[b];
  const size_t nb = (size_t)b * N;
  // a target row that holds a NaN (its maximum is NaN) or nothing finite has no arg-max
  int bad = 0;
  for (int i = threadIdx.x; i <= n; i += blockDim.x) {
    const float zm = a.z_max[row0 + i];
    bad |= (zm != zm || zm == -INFINITY) ? 1 : 0;
  }
  bad = __syncthreads_or(okn ? bad : 0);
  if (a.edge_stat)
    for (int i = threadIdx.x; i < n; i += blockDim.x)
      a.edge_stat[nb + i] = (!bad && a.tok[nb + i] == a.z_arg[row0 + a.parent[nb + i] + 1]) ? 1.f : 0.f;
  if (threadIdx.x == 0) {
    int cur = -1, acc = 0;
    if (!okn || bad) a.bonus[b] = -1;
    else
      for (;;) {
        const int g = a.z_arg[row0 + cur + 1];
        int hit = -1;
        for (int i = cur + 1; i < n; ++i)  // children come after their parent in canonical order
          if (a.parent[nb + i] == cur && a.tok[nb + i] == g) { hit = i; break; }
        if (hit < 0 || acc >= a.D) { a.bonus[b] = g; break; }
        a.acc_node[(size_t)b * a.D + acc] = hit; a.acc_tok[(size_t)b * a.D + acc] = g; ++acc; cur = hit;
      }
    for (int i = acc; i < a.D; ++i) { a.acc_node[(size_t)b * a.D + i] = -1; a.acc_tok[(size_t)b * a.D + i] = -1; }
    a.acc_len[b] = acc; a.flags[b] = 0u; a.status[b] = !okn ? TS_ERR_INVALID : (bad ? TS_ERR_NUMERIC : TS_OK);
  }
}

// ------------------------------------------------------------------------------------------------
// Stage 2, T > 0
// ------------------------------------------------------------------------------------------------
template <typename TIn>
__device__ __forceinline__ float z_elem(const VerifyArgs& a, int64_t row, int w) {
  return Elem<TIn>::to_f(reinterpret_cast<const TIn*>(a.Z)[row * a.V + w]);
}

// probability of token w under softmax(Z[row]/T), double
template <typename TIn>
__device__ __forceinline__ double p_of(const VerifyArgs& a, int64_t row, int w) {
  return exp(((double)z_elem<TIn>(a, row, w) - (double)a.z_max[row]) / (double)a.T - (double)a.z_logs[row]);
}

// Scalar state machine of one request, run by one warp of the request's owner CTA.
// need: 0 walking, 1 reduction after a rejection, 4 reduction for the bonus draw, 5 walk over (bonus token
// still to be drawn), 2 range rescan, 3 finished.  The bonus draws of all requests are left to the end of
// the kernel (closing == true): locating the range and rescanning it would otherwise hold up, at every
// step, the requests that are still walking.
// Lane 0 decides; at every visited node the lanes fetch the accept-test inputs of all its children at
// once (one memory round trip per node), and the warp folds range sums together.
template <typename TIn>
__device__ void advance(const VerifyArgs& a, int b, int lane, int parity, bool closing) {
  VerifyState* gst = a.state + b;
  const int N = a.N;
  const size_t nb = (size_t)b * N;
  const int need_in = gst->need;
  const int cur0 = gst->cur, cf0 = gst->cfirst, cc0 = gst->ccnt;
  if (need_in == 3 || (need_in == 5 && !closing)) return;
  // accept-test inputs of the current node's children, requested together with everything else this step
  // needs (the range sums, the state): one memory round trip instead of a chain of three
  int x0 = -1; double px0 = 0.0, qx0 = 1.0, ux0 = 0.0;
  if ((need_in == 0 || need_in == 1 || need_in == 4) && lane < cc0) {
    x0 = a.tok[nb + cf0 + lane];
    px0 = a.edge_px[nb + cf0 + lane]; qx0 = a.edge_qx[nb + cf0 + lane]; ux0 = a.edge_u[nb + cf0 + lane];
  }
  // ---- fold in the reduction that just ran -------------------------------------------------
  double fsum = 0.0;
  if (need_in == 1 || need_in == 4) {
    float pv[8];   // the first 256 range sums in one memory round trip
#pragma unroll
    for (int k = 0; k < 8; ++k) pv[k] = (k * 32 + lane < a.vt_n) ? __ldcg(a.part + (size_t)b * a.vt_n + k * 32 + lane) : 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) if (k * 32 + lane < a.vt_n) fsum += (double)pv[k];
    for (int t = 256 + lane; t < a.vt_n; t += 32) fsum += (double)__ldcg(a.part + (size_t)b * a.vt_n + t);
    for (int off = 16; off > 0; off >>= 1) fsum += __shfl_xor_sync(0xFFFFFFFFu, fsum, off);
  }
  VerifyState st;   // working copy (written back once at the end)
  if (lane == 0) st = *gst;
  int go_scan = 0;
  if (lane == 0) {
    if (need_in == 1 || need_in == 4) {
      double zn = fsum;  // the pass used passC for every token; tested siblings keep their own C_i
      for (int i = 0; i < st.nf; ++i)
        zn += fmax(st.fp[i] - st.fC[i] * st.fq[i], 0.0) - fmax(st.fp[i] - st.passC * st.fq[i], 0.0);
      if (need_in == 1) {
        if (zn <= 1e-30 * st.Zj) {  // residual lost its mass: keep the previous one
          a.flags[b] |= TS_FLAG_ZERO_MASS;
          st.fC[st.nf - 1] = st.C;
          st.partsC = -1.0;
        } else { st.C = st.passC; st.Zj = zn; st.partsC = st.passC; }
      } else { st.Zj = zn; st.partsC = st.passC; }
      st.need = 0;
    }
    if (st.need == 2) {  // the rescan wrote its token
      a.bonus[b] = st.result;
      a.acc_len[b] = st.acc;
      a.flags[b] |= (uint32_t)min(st.npass, 0xFFFF) << 8;   // bits 8..23: reductions this walk needed
      st.need = 3;
    }
    if (st.need == 5) go_scan = 1;   // closing: draw the bonus token now
  }
  int walking = __shfl_sync(0xFFFFFFFFu, lane == 0 ? (st.need == 0) : 0, 0);
  bool at_start = true;   // still at the node the step began at: its children were fetched above
  while (walking) {
    // inputs of every child's accept test at the current node, one child per lane
    const int v = __shfl_sync(0xFFFFFFFFu, st.cur, 0);
    int first = cf0, m = cc0;
    double px = px0, qx = qx0; int x = x0;
    double ux = ux0;
    if (!at_start || v != cur0) {
      first = a.child_first[(size_t)b * (N + 1) + v + 1]; m = a.child_cnt[(size_t)b * (N + 1) + v + 1];
      px = 0.0; qx = 1.0; x = -1; ux = 0.0;
      if (lane < m) {   // computed for every edge when the walk was set up
        x = a.tok[nb + first + lane];
        px = a.edge_px[nb + first + lane]; qx = a.edge_qx[nb + first + lane]; ux = a.edge_u[nb + first + lane];
      }
      if (lane == 0) { st.cfirst = first; st.ccnt = m; }
    }
    at_start = false;
    // lane 0 runs the sibling chain at this node until it accepts, needs a reduction, or runs out
    int again = 0;
    for (int j = __shfl_sync(0xFFFFFFFFu, st.j, 0); j < 32; ++j) {   // m <= K <= 16; earlier siblings were tested in earlier steps
      const double pxj = __shfl_sync(0xFFFFFFFFu, px, j), qxj = __shfl_sync(0xFFFFFFFFu, qx, j);
      const int xj = __shfl_sync(0xFFFFFFFFu, x, j);
      const double uj = __shfl_sync(0xFFFFFFFFu, ux, j);
      int stop = 0;
      if (lane == 0) {
        if (st.j != j) { }   // siblings before st.j were tested in an earlier step
        else if (st.j < m && st.acc < a.D) {
          const double cj = st.Zj / (1.0 - st.Qused);
          const double num = fmax(pxj / qxj - st.C, 0.0);
          const double rho = fmin(1.0, num / cj);
          if (uj < rho) {
            a.acc_node[(size_t)b * a.D + st.acc] = first + j; a.acc_tok[(size_t)b * a.D + st.acc] = xj;
            st.acc++; st.cur = first + j; st.j = 0; st.C = 0.0; st.Zj = 1.0; st.Qused = 0.0; st.nf = 0; st.partsC = -1.0;
            stop = 1; again = 1;          // descend: next node
          } else {
            st.fx[st.nf] = xj; st.fp[st.nf] = pxj; st.fq[st.nf] = qxj; st.fC[st.nf] = st.C + cj; st.nf++;
            st.Qused += qxj; st.j++;
            st.passC = st.C + cj; st.row_node = v; st.need = 1;
            stop = 1;                      // wait for the reduction
          }
        } else {
          if (st.partsC != st.C) { st.passC = st.C; st.row_node = v; st.need = 4; }
          else go_scan = 1;
          stop = 1;
        }
      }
      stop = __shfl_sync(0xFFFFFFFFu, stop, 0);
      if (stop) break;
    }
    walking = __shfl_sync(0xFFFFFFFFu, again, 0);
  }
  go_scan = __shfl_sync(0xFFFFFFFFu, go_scan, 0);
  if (go_scan && !closing) {
    if (lane == 0) { st.need = 5; atomicSub(a.ctr + 4, 1); }   // one walker fewer
  } else if (go_scan) {
    // locate the vocabulary range holding the bonus token: cumulative corrected range sums
    const int cur = __shfl_sync(0xFFFFFFFFu, st.cur, 0), nf = __shfl_sync(0xFFFFFFFFu, st.nf, 0);
    const double C = __shfl_sync(0xFFFFFFFFu, st.C, 0), Zj = __shfl_sync(0xFFFFFFFFu, st.Zj, 0);
    const uint64_t hv = a.node_hash[(size_t)b * (N + 1) + cur + 1];
    const double u = u01(stream_words(a.seed, b, hv, STREAM_BONUS, 0u).x);
    const double target = u * Zj;
    double carry = 0.0; int found = -1; double before = 0.0; int last_pos = -1;
    // correction of tested sibling i (lane i): its range, and the difference between the residual it kept
    // and the one the last reduction gave it (the state in global memory is current: this runs in a later
    // step than the one that wrote it)
    int f_tile = -1; double f_delta = 0.0;
    if (lane < nf) {
      const int fxi = gst->fx[lane];
      const double fpi = gst->fp[lane], fqi = gst->fq[lane], fCi = gst->fC[lane];
      f_tile = fxi / a.vt_TV;
      f_delta = fmax(fpi - fCi * fqi, 0.0) - fmax(fpi - C * fqi, 0.0);
    }
    // the first 256 range sums are requested together (one memory round trip for the usual grid sizes)
    float pre[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) pre[k] = (k * 32 + lane < a.vt_n) ? __ldcg(a.part + (size_t)b * a.vt_n + k * 32 + lane) : 0.f;
    for (int t0 = 0; t0 < a.vt_n && found < 0; t0 += 32) {
      const int t = t0 + lane;
      double pt = 0.0;
      if (t0 < 256) {
        float pv = pre[0];
#pragma unroll
        for (int k = 1; k < 8; ++k) pv = (t0 >> 5) == k ? pre[k] : pv;
        pt = (double)pv;
      } else if (t < a.vt_n) pt = (double)__ldcg(a.part + (size_t)b * a.vt_n + t);
      for (int i = 0; i < nf; ++i) {   // tested siblings keep the residual they had when tested
        const int ti = __shfl_sync(0xFFFFFFFFu, f_tile, i);
        const double di = __shfl_sync(0xFFFFFFFFu, f_delta, i);
        if (t == ti) pt += di;
      }
      if (pt < 0.0) pt = 0.0;
      double inc = pt;
      for (int off = 1; off < 32; off <<= 1) { const double o = __shfl_up_sync(0xFFFFFFFFu, inc, off); if (lane >= off) inc += o; }
      const bool cross = (t < a.vt_n) && (carry + inc > target);
      const unsigned bal = __ballot_sync(0xFFFFFFFFu, cross);
      const unsigned pos = __ballot_sync(0xFFFFFFFFu, pt > 0.0);
      if (pos) last_pos = t0 + 31 - __clz(pos);
      if (bal) {
        const int src = __ffs(bal) - 1;
        found = t0 + src;
        before = carry + __shfl_sync(0xFFFFFFFFu, inc - pt, src);
      }
      carry += __shfl_sync(0xFFFFFFFFu, inc, 31);
    }
    if (lane == 0) {
      if (found < 0) { found = last_pos >= 0 ? last_pos : 0; before = -1.0; }  // rounding: take the last range with mass
      st.scan_tile = found; st.target = target; st.before = before; st.need = 2;
    }
  }
  if (lane == 0) {
    *gst = st;   // made visible to the other CTAs by the fence of the grid barrier that follows
    if (st.need == 1 || st.need == 4) a.wk_list[parity * a.B + atomicAdd(a.ctr + parity, 1)] = b;
    if (st.need == 1 || st.need == 4) gst->npass = st.npass + 1;
    else if (st.need == 2) a.sc_list[parity * a.B + atomicAdd(a.ctr + 2 + parity, 1)] = b;
  }
  __syncwarp();
}

// logits of up to G parents for the VEC tokens at v (global W, coalesced 16-byte loads)
template <typename TIn, int G>
__device__ __forceinline__ void logits_group(const VerifyArgs& a, const float* as, int ng, const int* rq_req,
                                             const int* rq_dep, int v, float (*acc)[8], const TIn* Wsrc, size_t wstride,
                                             int woff) {
  constexpr int VEC = Elem<TIn>::VEC;
  const TIn* Ug = reinterpret_cast<const TIn*>(a.U);
  for (int g = 0; g < G; ++g) {
    if (g < ng) {
      const TIn* u = Ug + ((size_t)rq_req[g] * a.D + rq_dep[g]) * a.V + v;
      if (sizeof(TIn) == 2) { const uint4 x = __ldg(reinterpret_cast<const uint4*>(u)); unpack_bf16x8(x, acc[g]); }
      else { const float4 x = __ldg(reinterpret_cast<const float4*>(u)); acc[g][0] = x.x; acc[g][1] = x.y; acc[g][2] = x.z; acc[g][3] = x.w; }
    }
  }
  for (int k = 0; k < a.r; ++k) {
    float w[8];
    // W comes from the CTA's shared-memory copy of its vocabulary range when that fits, else from global
    if (sizeof(TIn) == 2) { const uint4 x = *reinterpret_cast<const uint4*>(Wsrc + (size_t)k * wstride + woff); unpack_bf16x8(x, w); }
    else { const float4 x = *reinterpret_cast<const float4*>(Wsrc + (size_t)k * wstride + woff); w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w; }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float ak = as[g * RMAX + k];
#pragma unroll
      for (int i = 0; i < VEC; ++i) acc[g][i] = fmaf(ak, w[i], acc[g][i]);
    }
  }
}

template <typename TIn>
__device__ __forceinline__ float logit_scalar(const VerifyArgs& a, int req, int dep, int ptok, int w) {
  const TIn* Wg = reinterpret_cast<const TIn*>(a.W);
  const TIn* Ug = reinterpret_cast<const TIn*>(a.U);
  const TIn* Ag = reinterpret_cast<const TIn*>(a.A);
  float acc = Elem<TIn>::to_f(Ug[((size_t)req * a.D + dep) * a.V + w]);
  for (int k = 0; k < a.r; ++k)
    acc = fmaf(Elem<TIn>::to_f(Ag[(size_t)ptok * a.r + k]), Elem<TIn>::to_f(Wg[(size_t)k * a.V + w]), acc);
  return acc;
}

constexpr int VG = 4;  // requests sharing one sweep over the W columns

// One work item of a reduction step: NG requests of one group over tokens [c_lo, c_hi) of the CTA's range.
template <typename TIn>
struct SweepCtx {
  const TIn *Z, *U, *Wsrc; size_t wstride; int wshift; int V, D, r; float invT;
  const float* a; const int *req, *dep; const long long* row; const float *C, *zmax, *zlogs, *lseT;
};

template <typename TIn, int NG>
__device__ __forceinline__ void sweep_item(const SweepCtx<TIn>& c, int g0, int c_lo, int c_hi, int lane, float* out) {
  constexpr int VEC = Elem<TIn>::VEC;
  float sum[NG];
  bool need_q = false;
#pragma unroll
  for (int g = 0; g < NG; ++g) { sum[g] = 0.f; need_q |= (c.C[g0 + g] != 0.f); }
  for (int v = c_lo + lane * VEC; v < c_hi; v += 32 * VEC) {
    float z[NG][8], acc[NG][8];
#pragma unroll
    for (int g = 0; g < NG; ++g) {   // every load of the step first: target rows, base rows
      const TIn* zp = c.Z + c.row[g0 + g] * c.V + v;
      const TIn* up = c.U + ((size_t)c.req[g0 + g] * c.D + c.dep[g0 + g]) * c.V + v;
      const bool ldq = need_q && c.C[g0 + g] != 0.f;   // a member with C = 0 needs no proposal: its base row is not touched
      if (sizeof(TIn) == 2) {
        unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(zp)), z[g]);
        if (ldq) unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(up)), acc[g]);
      } else {
        const float4 x = __ldg(reinterpret_cast<const float4*>(zp)); z[g][0] = x.x; z[g][1] = x.y; z[g][2] = x.z; z[g][3] = x.w;
        if (ldq) { const float4 y = __ldg(reinterpret_cast<const float4*>(up)); acc[g][0] = y.x; acc[g][1] = y.y; acc[g][2] = y.z; acc[g][3] = y.w; }
      }
      if (need_q && !ldq) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[g][i] = 0.f;
      }
    }
    if (need_q) {
      const TIn* wp = c.Wsrc + (v + c.wshift);
#pragma unroll 4
      for (int k = 0; k < c.r; ++k) {
        float w[8];
        if (sizeof(TIn) == 2) unpack_bf16x8(*reinterpret_cast<const uint4*>(wp + (size_t)k * c.wstride), w);
        else { const float4 x = *reinterpret_cast<const float4*>(wp + (size_t)k * c.wstride); w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w; }
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          const float ak = c.a[(g0 + g) * RMAX + k];
#pragma unroll
          for (int i = 0; i < VEC; ++i) acc[g][i] = fmaf(ak, w[i], acc[g][i]);
        }
      }
    }
#pragma unroll
    for (int g = 0; g < NG; ++g) {
      const float Cg = c.C[g0 + g], zm = c.zmax[g0 + g], zl = c.zlogs[g0 + g], lt = c.lseT[g0 + g];
#pragma unroll
      for (int i = 0; i < VEC; ++i) {
        const float p = __expf((z[g][i] - zm) * c.invT - zl);
        const float q = Cg != 0.f ? __expf(acc[g][i] * c.invT - lt) : 0.f;
        sum[g] += fmaxf(p - Cg * q, 0.f);
      }
    }
  }
#pragma unroll
  for (int g = 0; g < NG; ++g) {
    float sg = sum[g];
    for (int off = 16; off > 0; off >>= 1) sg += __shfl_xor_sync(0xFFFFFFFFu, sg, off);
    if (lane == 0) out[(size_t)g * 16] = sg;
  }
}


constexpr int SB = 32; // requests whose head rows are staged together
constexpr int WT = 288;       // threads of the walk kernel: eight worker warps and the warp that issues the MMAs
constexpr int WALK_EPI = 8;   // worker warps that read the accumulators of a tensor-core reduction
constexpr int WALK_BLK = 256;  // tokens per MMA block (one accumulator buffer)
constexpr int WALK_NBUF = 2;  // accumulator buffers in tensor memory
constexpr int WALK_MAX_BLK = 32;

// Tensor-core state of one walk CTA: shared-memory operands, barriers, tensor-memory base and the running
// count of 128-token blocks issued so far (it selects the accumulator buffer and the barrier parity).
struct WalkTc {
  unsigned char* Ws; unsigned char* As; uint64_t* t_full; uint64_t* t_empty; volatile int* s_abort;
  uint32_t tmem_base, slab_bytes; int rp; uint32_t it;
  // Streaming form (ranks at which the range of W does not fit shared memory): Ws is a ring of WALK_RING blocks
  // of WALK_SBLK tokens, refilled by bulk-tensor loads for every block of every reduction.
  int stream; const CUtensorMap* tm; uint64_t* w_full; uint64_t* w_free; uint32_t wit;
};
constexpr int WALK_SBLK = 128;   // tokens per block of the streaming form (two 64-token slabs of W)
constexpr int WALK_RING = 2;     // blocks of W in flight or in use

// One reduction step on the tensor cores: sum over this CTA's tokens [t0, t0 + tlen) of
// max(p(w) - C q(w), 0) for up to 128 requests at once.  The low-rank part of the draft logits,
// [requests x r] . [r x tokens], is one MMA tile per 128 tokens (requests on the rows, replicated when
// there are few); worker warp w reads the rows of quarter w % 4 and the 16-token chunks of column split
// w / 4, adds the base logits, and accumulates the residual with the target row.  Partial sums are
// combined in a fixed order.  Returns false when a bounded wait ran out.
template <typename TIn, int BLK>
__device__ bool mma_pass(const VerifyArgs& a, WalkTc& tc, int nreq, int t0, int tlen, float invT,
                         const int* sb_req, const int* sb_dep, const int* sb_tok, const long long* sb_row,
                         const float* sb_C, const float* sb_zmax, const float* sb_zlogs, const float* sb_lseT, float* s_part) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = a.r, rp = tc.rp, V = a.V;
  const int R = mma_replicas(nreq), per = 128 / R, rsh = R == 4 ? 2 : (R == 2 ? 1 : 0), psh = 7 - rsh;
  const int cpr = rp / 8;                      // 16-byte chunks per A row
  const uint32_t a_slab_bytes = 128u * 128u;
  const __nv_bfloat16* Ag = reinterpret_cast<const __nv_bfloat16*>(a.A);
  {
    // ask L2 for this CTA's share of every request's target row and base-logit row now; the worker warps
    // come for them a few microseconds later, after the MMAs
    const int lines = (tlen * 2 + 127) / 128;
    const __nv_bfloat16* Zg = reinterpret_cast<const __nv_bfloat16*>(a.Z);
    const __nv_bfloat16* Ug = reinterpret_cast<const __nv_bfloat16*>(a.U);
    for (int i = tid; i < nreq * lines * 2; i += WT) {
      const int g = i / (lines * 2), rem = i % (lines * 2), which = rem / lines, ln = rem % lines;
      const __nv_bfloat16* base = which == 0 ? Zg + (size_t)sb_row[g] * V : Ug + ((size_t)sb_req[g] * a.D + sb_dep[g]) * V;
      if (which == 0 || sb_C[g] != 0.f) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + t0 + ln * 64));
    }
  }
  // head rows A[x] of the requests' current nodes, K-major with the 128-byte swizzle
  for (int idx = tid; idx < 128 * cpr; idx += WT) {
    const int rr = idx / cpr, ck = idx % cpr;
    const int g = rr % per;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (g < nreq && ck * 8 < r) v = __ldg(reinterpret_cast<const uint4*>(Ag + (size_t)sb_tok[g] * r + ck * 8));
    *reinterpret_cast<uint4*>(tc.As + (size_t)(ck >> 3) * a_slab_bytes + rr * 128 + (((ck & 7) ^ (rr & 7)) << 4)) = v;
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const int nblk = (tlen + BLK - 1) / BLK;
  if (warp < WALK_EPI) {
    const int q = warp & 3, s = warp >> 2;
    const int row = q * 32 + lane;
    const int g = row & (per - 1), rho = row >> psh;   // rho is uniform within a warp
    const bool active = g < nreq;
    const __nv_bfloat16* Zrow = reinterpret_cast<const __nv_bfloat16*>(a.Z);
    const __nv_bfloat16* Urow = reinterpret_cast<const __nv_bfloat16*>(a.U);
    float C = 0.f, zs = 0.f, zoff = 0.f, qoff = 0.f;
    if (active) {
      Zrow += (size_t)sb_row[g] * V;
      Urow += ((size_t)sb_req[g] * a.D + sb_dep[g]) * V;
      C = sb_C[g];
      zs = invT * 1.4426950408889634f;                         // exponentials as powers of two
      zoff = (-sb_zmax[g] * invT - sb_zlogs[g]) * 1.4426950408889634f;
      qoff = C != 0.f ? -sb_lseT[g] * 1.4426950408889634f : -1e30f;   // lseT may be NaN where it is not needed
    }
    float sum = 0.f, sum2 = 0.f;
    bool alive = true;
    const bool need_q = C != 0.f;
    // Owned chunks of a block: c = c0 + 2R j (2R divides the 16 chunks of a block).  They are taken two
    // at a time so that the two chunks' loads and exponentials overlap; the target and base-logit rows
    // of the next pair are requested while this pair is worked on.
    const int c0 = rho + R * s, cstep = 2 * R;
    uint4 nz[2][2], nu[2][2];
    auto request = [&](int cg, int h) {
      const int vn = t0 + cg * 16;
      const uint4 zero = make_uint4(0, 0, 0, 0);
      const bool in = active && cg * 16 < tlen;
      // target logits outside the vocabulary are -inf (eight bf16 -inf): p = 0 there and the residual term vanishes
      const uint4 ninf = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
      nz[h][0] = in ? __ldg(reinterpret_cast<const uint4*>(Zrow + vn)) : ninf;
      nz[h][1] = (in && V - vn > 8) ? __ldg(reinterpret_cast<const uint4*>(Zrow + vn + 8)) : ninf;
      nu[h][0] = (in && need_q) ? __ldg(reinterpret_cast<const uint4*>(Urow + vn)) : zero;
      nu[h][1] = (in && need_q && V - vn > 8) ? __ldg(reinterpret_cast<const uint4*>(Urow + vn + 8)) : zero;
    };
    auto residual = [&](const uint32_t* racc, const uint4& z0, const uint4& z1, const uint4& u0, const uint4& u1, float& acc_sum) {
      float zz[16], ub[16];
      unpack_bf16x8(z0, zz); unpack_bf16x8(z1, zz + 8);
      unpack_bf16x8(u0, ub); unpack_bf16x8(u1, ub + 8);
      // one path for every lane: a request with C == 0 has qoff = -huge, so its q term vanishes
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float p = fast_ex2(fmaf(zz[i], zs, zoff));
        const float qq = fast_ex2(fmaf(__uint_as_float(racc[i]) + ub[i], zs, qoff));
        acc_sum += fmaxf(fmaf(-C, qq, p), 0.f);   // tokens past the vocabulary: p = 0, C >= 0, term 0
      }
    };
    request(c0, 0);
    request(c0 + cstep, 1);
    for (int nb = 0; nb < nblk && alive; ++nb) {
      const uint32_t it = tc.it + (uint32_t)nb, tb = it % WALK_NBUF, u = it / WALK_NBUF;
      int ok = 1;
      if (lane == 0) ok = mbar_wait(tc.t_full + tb, u & 1, tc.s_abort, nullptr, a.wait_limit) ? 1 : 0;
      ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
      if (!ok) { alive = false; break; }
      tc_fence_after();
      const int nch = min(BLK / 16, (tlen - nb * BLK + 15) / 16);
      for (int ca = c0; ca < nch; ca += 2 * cstep) {
        const int cb = ca + cstep;
        const bool hb = cb < nch;   // warp-uniform
        const int cga = nb * (BLK / 16) + ca;
        uint32_t ra[16], rb[16];
        const uint32_t tbase = tc.tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(tb * WALK_BLK);
        tmem_ld16_issue(tbase + (uint32_t)(ca * 16), ra);
        if (hb) tmem_ld16_issue(tbase + (uint32_t)(cb * 16), rb);
        tmem_ld_wait();
        const uint4 za0 = nz[0][0], za1 = nz[0][1], ua0 = nu[0][0], ua1 = nu[0][1];
        const uint4 zb0 = nz[1][0], zb1 = nz[1][1], ub0 = nu[1][0], ub1 = nu[1][1];
        // next pair: the rest of this block, else the first pair of the next block
        {
          int na = cga + 2 * cstep;
          if (ca + 2 * cstep >= BLK / 16) na = (nb + 1) * (BLK / 16) + c0;
          request(na, 0);
          request(na + cstep, 1);
        }
        if (active) {
          residual(ra, za0, za1, ua0, ua1, sum);
          if (hb) residual(rb, zb0, zb1, ub0, ub1, sum2);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tc.t_empty + tb);
    }
    sum += sum2;
    s_part[row * 2 + s] = active ? sum : 0.f;
  } else if (warp == WALK_EPI && lane == 0) {
    const uint32_t ws_addr = smem_u32(tc.Ws), as_addr = smem_u32(tc.As);
    // streaming form: block nb of this pass goes to ring slot (wit + nb) % WALK_RING, once the MMAs that read the
    // slot's previous block are done; the next block is requested before this one is waited for
    int requested = 0, consumed = 0;   // blocks whose loads were issued / whose loads were waited for
    auto w_request = [&](int nb) -> bool {
      const uint32_t wi = tc.wit + (uint32_t)nb, slot = wi % WALK_RING, use = wi / WALK_RING;
      if (use >= 1 && !mbar_wait(tc.w_free + slot, (use - 1) & 1, tc.s_abort, nullptr, a.wait_limit)) return false;
      const int ns = (tlen - nb * BLK > 64) ? 2 : 1;
      mbar_expect_tx(tc.w_full + slot, (uint32_t)ns * tc.slab_bytes);
      for (int h = 0; h < ns; ++h)
        tma_load_box(tc.Ws + (size_t)(slot * (BLK / 64) + h) * tc.slab_bytes, tc.tm, t0 + nb * BLK + h * 64, 0, tc.w_full + slot);
      ++requested;
      return true;
    };
    bool live = true;
    if (tc.stream) live = w_request(0);
    for (int nb = 0; nb < nblk && live; ++nb) {
      const uint32_t it = tc.it + (uint32_t)nb, tb = it % WALK_NBUF, u = it / WALK_NBUF;
      uint32_t wslab = (uint32_t)(BLK / 64 * nb);   // first slab of the block's W (resident form)
      if (tc.stream) {
        if (nb + 1 < nblk && !w_request(nb + 1)) break;
        const uint32_t wi = tc.wit + (uint32_t)nb, slot = wi % WALK_RING;
        if (!mbar_wait(tc.w_full + slot, (wi / WALK_RING) & 1, tc.s_abort, nullptr, a.wait_limit)) break;
        ++consumed;
        wslab = slot * (uint32_t)(BLK / 64);
      }
      if (u >= 1) {
        if (!mbar_wait(tc.t_empty + tb, (u - 1) & 1, tc.s_abort, nullptr, a.wait_limit)) break;
        tc_fence_after();
      }
      const int n = min(BLK, (tlen - nb * BLK + 63) / 64 * 64);   // whole 64-token slabs
      const uint32_t idesc = instr_desc(n);
      const uint32_t d_tmem = tc.tmem_base + tb * (uint32_t)WALK_BLK;
      for (int ks = 0; ks < rp / 16; ++ks) {
        const uint64_t adesc = smem_desc(as_addr + (uint32_t)(ks >> 2) * a_slab_bytes + (uint32_t)(ks & 3) * 32u, 16u, 1024u);
        const uint64_t bdesc = smem_desc(ws_addr + wslab * tc.slab_bytes + (uint32_t)ks * 2048u, tc.slab_bytes, 1024u);
        mma_bf16(d_tmem, adesc, bdesc, idesc, ks > 0 ? 1u : 0u);
      }
      mma_commit(tc.t_full + tb);
      if (tc.stream) mma_commit(tc.w_free + ((tc.wit + (uint32_t)nb) % WALK_RING));
    }
    if (tc.stream && requested > consumed) {
      // gave up with a block of W on its way: it writes this CTA's shared memory, so wait for it (bounded)
      const uint32_t wi = tc.wit + (uint32_t)consumed, slot = wi % WALK_RING;
      bool landed = false;
      for (uint32_t i = 0; i < WAIT_LIMIT && !landed; ++i) { landed = mbar_try_wait(tc.w_full + slot, (wi / WALK_RING) & 1); if (!landed) __nanosleep(100); }
    }
  }
  if (tc.stream) tc.wit += (uint32_t)nblk;
  tc.it += (uint32_t)nblk;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (*tc.s_abort) return false;
  if (tid < nreq) {
    float t = 0.f;
    for (int rho = 0; rho < R; ++rho) { t += s_part[(rho * per + tid) * 2]; t += s_part[(rho * per + tid) * 2 + 1]; }
    a.part[(size_t)sb_req[tid] * a.vt_n + blockIdx.x] = t;
  }
  __syncthreads();
  return true;
}


// The walk proper.  Returns false when a bounded wait ran out (every thread of the CTA returns the same).
template <typename TIn, bool MMA>
__device__ __forceinline__ bool walk_body(const VerifyArgs& a, WalkTc& tc, unsigned char* w_raw) {
  constexpr int SBX = MMA ? 128 : SB;   // requests per reduction pass
  __shared__ float s_a[VG * RMAX];
  __shared__ int s_req[VG], s_dep[VG], s_node[VG];
  __shared__ float s_C[VG], s_zmax[VG], s_zlogs[VG], s_lseT[VG];
  __shared__ float s_red[VG][WT / 32];
  __shared__ double s_scan[WT];
  __shared__ int s_found, s_last;
  __shared__ float sb_a[MMA ? 256 : SB * RMAX];
  __shared__ int sb_req[SBX], sb_dep[SBX], sb_tok[SBX];
  __shared__ long long sb_row[SBX];
  __shared__ float sb_C[SBX], sb_zmax[SBX], sb_zlogs[SBX], sb_lseT[SBX], sb_part[MMA ? 256 : SB * 16];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned nblocks = gridDim.x;
  const unsigned nexpect = nblocks + (a.lost_arrival ? 1u : 0u);   // arrivals a grid barrier waits for
  unsigned gen = 0;
  constexpr int VEC = Elem<TIn>::VEC;
  const bool vec_ok = (a.V % VEC) == 0;
  const float invT = 1.f / a.T;
  const int v_lo = blockIdx.x * a.vt_TV, v_hi = min(a.V, v_lo + a.vt_TV);
  const TIn* Zg = reinterpret_cast<const TIn*>(a.Z);
  const TIn* Ag = reinterpret_cast<const TIn*>(a.A);
  const TIn* Wg = reinterpret_cast<const TIn*>(a.W);
  const int N = a.N;
  TIn* Ws = reinterpret_cast<TIn*>(w_raw);   // [r][vt_TV] when a.w_smem
  if (!MMA && a.w_smem && vec_ok) {
    const int per_row = a.vt_TV / VEC;
    for (int i = tid; i < a.r * per_row; i += WT) {
      const int k = i / per_row, c = (i % per_row) * VEC;
      uint4 x = make_uint4(0, 0, 0, 0);
      if (v_lo + c < a.V) x = __ldg(reinterpret_cast<const uint4*>(Wg + (size_t)k * a.V + v_lo + c));
      *reinterpret_cast<uint4*>(Ws + (size_t)k * a.vt_TV + c) = x;
    }
  }
  const bool ws_ok = !MMA && a.w_smem && vec_ok;

  // ---- per-edge statistics, child ranges and state initialisation (owner CTA of each request) ------
  if (blockIdx.x == 0 && tid < 5) a.ctr[tid] = tid == 4 ? a.B : 0;
  for (int b = blockIdx.x; b < a.B; b += nblocks) {
    const int n = a.n_nodes[b];
    const bool okn = n >= 0 && n <= N;
    const size_t nb = (size_t)b * N, cbase = (size_t)b * (N + 1);
    const int64_t row0 = a.z_row_off[b];
    for (int i = tid; i <= N; i += WT) { a.child_first[cbase + i] = -1; a.child_cnt[cbase + i] = 0; }
    // non-finite inputs: a target row with a NaN (its maximum is NaN), without finite mass, or a node whose
    // proposal log-probability is NaN (its expansion was reported TS_ERR_NUMERIC) -- the request is not walked
    int bad = 0;
    if (okn) {
      for (int i = tid; i <= n; i += WT) {
        const float zm = a.z_max[row0 + i], zl = a.z_logs[row0 + i];
        bad |= (zm != zm || isinf(zm) || zl != zl || isinf(zl)) ? 1 : 0;
      }
      for (int i = tid; i < n; i += WT) { const float lq = a.logqT[nb + i]; bad |= (lq != lq) ? 1 : 0; }
    }
    bad = __syncthreads_or(bad);
    if (bad && a.edge_stat)
      for (int i = tid; i < n; i += WT) a.edge_stat[nb + i] = 0.f;
    if (okn && !bad)
      for (int i = tid; i < n; i += WT) {
        const int par = a.parent[nb + i];
        if (i == 0 || a.parent[nb + i - 1] != par) a.child_first[cbase + par + 1] = i;   // siblings are contiguous
        atomicAdd(&a.child_cnt[cbase + par + 1], 1);
        {
          // what the accept test of this edge needs, off the walk's critical path: p(x), q(x) and the uniform
          // of sibling j at its parent (j = place among the contiguous siblings)
          const int64_t row = row0 + par + 1;
          int j = 0;
          while (i - j - 1 >= 0 && a.parent[nb + i - j - 1] == par) ++j;
          a.edge_px[nb + i] = exp(((double)z_elem<TIn>(a, row, a.tok[nb + i]) - (double)a.z_max[row]) / (double)a.T - (double)a.z_logs[row]);
          a.edge_qx[nb + i] = exp((double)a.logqT[nb + i]);
          a.edge_u[nb + i] = u01(stream_words(a.seed, b, a.node_hash[(size_t)b * (N + 1) + par + 1], STREAM_ACCEPT, (uint32_t)j).x);
        }
        if (a.edge_stat) {
          const int64_t row = row0 + par + 1;
          const double lr = ((double)z_elem<TIn>(a, row, a.tok[nb + i]) - (double)a.z_max[row]) / (double)a.T -
                            (double)a.z_logs[row] - (double)a.logqT[nb + i];
          a.edge_stat[nb + i] = (float)exp(fmin(lr, 0.0));
        }
      }
    __syncthreads();   // the root's child range is read below
    if (tid == 0) {
      VerifyState& st = a.state[b];
      st.cur = -1; st.j = 0; st.acc = 0; st.need = 0; st.nf = 0; st.scan_tile = -1; st.row_node = -1; st.result = -1;
      st.C = 0.0; st.Zj = 1.0; st.Qused = 0.0; st.target = 0.0; st.before = 0.0; st.passC = 0.0; st.partsC = -1.0;
      st.npass = 0; st.pad_ = 0;
      st.cfirst = a.child_first[cbase]; st.ccnt = a.child_cnt[cbase];   // children of the root
      a.flags[b] = 0u;
      a.status[b] = !okn ? TS_ERR_INVALID : (bad ? TS_ERR_NUMERIC : TS_OK);
      if (!okn || bad) { st.need = 3; a.acc_len[b] = 0; a.bonus[b] = -1; }
      for (int i = 0; i < a.D; ++i) { a.acc_node[(size_t)b * a.D + i] = -1; a.acc_tok[(size_t)b * a.D + i] = -1; }
    }
    __syncthreads();
  }
  __threadfence();
  if (!grid_barrier(a.barrier, nexpect, gen, a.wait_limit)) return false;
  // requests rejected at set-up leave the count of unfinished ones
  for (int b = blockIdx.x; b < a.B; b += nblocks)
    if (tid == 0 && a.state[b].need == 3) atomicSub(a.ctr + 4, 1);

  // stage 0: walk steps until every request's walk is over; stage 1: one step that locates and rescans the
  // range of every bonus token; stage 2: the owners commit the results
  int stage = 0;
  for (int step = 0; step < a.max_steps; ++step) {
    const int par = step & 1;
    // ---- phase A: scalar walks of the requests this CTA owns, one warp each ----------------------
    for (int b = blockIdx.x + warp * (int)nblocks; b < a.B; b += (WT / 32) * (int)nblocks) advance<TIn>(a, b, lane, par, stage > 0);
    if (stage == 2) return true;
    if (!grid_barrier(a.barrier, nexpect, gen, a.wait_limit)) return false;
    // ---- phase B: vocabulary work requested by the walks -----------------------------------------
    const int nwk = __ldcg(a.ctr + par), nsc = __ldcg(a.ctr + 2 + par), left = __ldcg(a.ctr + 4);
    if (blockIdx.x == 0 && tid < 2) a.ctr[2 * tid + (par ^ 1)] = 0;   // next step's counters
    if (MMA) {
      for (int sb0 = 0; sb0 < nwk; sb0 += SBX) {
        const int nreq = min(SBX, nwk - sb0);
        if (tid < nreq) {
          const int b = __ldcg(a.wk_list + par * a.B + sb0 + tid);
          const VerifyState* st = a.state + b;
          const int v = st->row_node;
          const int64_t row = a.z_row_off[b] + v + 1;
          sb_req[tid] = b; sb_row[tid] = row; sb_dep[tid] = v < 0 ? 0 : min(a.depth[(size_t)b * N + v], a.D - 1);   // a leaf at depth D asks only for its target row (C = 0): keep the base-row index inside U
          sb_tok[tid] = v < 0 ? a.anchor[b] : a.tok[(size_t)b * N + v];
          sb_C[tid] = (float)st->passC; sb_zmax[tid] = a.z_max[row]; sb_zlogs[tid] = a.z_logs[row];
          sb_lseT[tid] = a.node_lseT[(size_t)b * (N + 1) + v + 1];
        }
        __syncthreads();
        const bool pass_ok = tc.stream ? mma_pass<TIn, WALK_SBLK>(a, tc, nreq, v_lo, v_hi - v_lo, invT, sb_req, sb_dep, sb_tok, sb_row, sb_C,
                                                                  sb_zmax, sb_zlogs, sb_lseT, sb_part)
                                       : mma_pass<TIn, WALK_BLK>(a, tc, nreq, v_lo, v_hi - v_lo, invT, sb_req, sb_dep, sb_tok, sb_row, sb_C,
                                                                 sb_zmax, sb_zlogs, sb_lseT, sb_part);
        if (!pass_ok) {
          if (tid == 0) atomicExch(a.barrier + 1, 1u);   // the word the follow-up kernel checks
          return false;
        }
      }
    } else if (vec_ok) {
      // Reductions sum_w max(p(w) - C q(w), 0) over this CTA's vocabulary range, for up to SB requests
      // at a time.  Work item = (group of VG requests, chunk of the range); items are dealt to the warps,
      // so a single request still uses several warps and many requests run side by side.  Partial sums
      // are combined in a fixed order.
      const int len = v_hi - v_lo;
      const int chunk = max(256, ((len + 15) / 16 + 255) / 256 * 256);   // at most 16 chunks
      const int nchunk = (len + chunk - 1) / chunk;
      for (int sb0 = 0; sb0 < nwk; sb0 += SB) {
        const int nreq = min(SB, nwk - sb0);
        if (tid < nreq) {
          const int b = __ldcg(a.wk_list + par * a.B + sb0 + tid);
          const VerifyState* st = a.state + b;
          const int v = st->row_node;
          const int64_t row = a.z_row_off[b] + v + 1;
          sb_req[tid] = b; sb_row[tid] = row; sb_dep[tid] = v < 0 ? 0 : min(a.depth[(size_t)b * N + v], a.D - 1);   // a leaf at depth D asks only for its target row (C = 0): keep the base-row index inside U
          sb_tok[tid] = v < 0 ? a.anchor[b] : a.tok[(size_t)b * N + v];
          sb_C[tid] = (float)st->passC; sb_zmax[tid] = a.z_max[row]; sb_zlogs[tid] = a.z_logs[row];
          sb_lseT[tid] = a.node_lseT[(size_t)b * (N + 1) + v + 1];
        }
        __syncthreads();
        for (int i = tid; i < nreq * a.r; i += WT) {
          const int g = i / a.r, k = i % a.r;
          sb_a[g * RMAX + k] = Elem<TIn>::to_f(Ag[(size_t)sb_tok[g] * a.r + k]);
        }
        __syncthreads();
        const int ngrp = (nreq + VG - 1) / VG;
        for (int item = warp; item < ngrp * nchunk; item += WT / 32) {
          const int grp = item / nchunk, ch = item % nchunk;
          const int g0 = grp * VG, ng = min(VG, nreq - g0);
          const int c_lo = v_lo + ch * chunk, c_hi = min(v_hi, c_lo + chunk);
          const SweepCtx<TIn> sc{Zg, reinterpret_cast<const TIn*>(a.U), ws_ok ? Ws : Wg, ws_ok ? (size_t)a.vt_TV : (size_t)a.V,
                                 ws_ok ? -v_lo : 0, a.V, a.D, a.r, invT, sb_a, sb_req, sb_dep, sb_row, sb_C, sb_zmax, sb_zlogs, sb_lseT};
          float* out = sb_part + (size_t)g0 * 16 + ch;
          switch (ng) {
            case 1: sweep_item<TIn, 1>(sc, g0, c_lo, c_hi, lane, out); break;
            case 2: sweep_item<TIn, 2>(sc, g0, c_lo, c_hi, lane, out); break;
            case 3: sweep_item<TIn, 3>(sc, g0, c_lo, c_hi, lane, out); break;
            default: sweep_item<TIn, 4>(sc, g0, c_lo, c_hi, lane, out); break;
          }
        }
        __syncthreads();
        if (tid < nreq) {
          float t = 0.f;
          for (int ch = 0; ch < nchunk; ++ch) t += sb_part[tid * 16 + ch];
          a.part[(size_t)sb_req[tid] * a.vt_n + blockIdx.x] = t;
        }
        __syncthreads();
      }
    } else
    for (int w0 = 0; w0 < nwk; w0 += VG) {
      const int ng = min(VG, nwk - w0);
      if (tid < ng) {
        const int b = __ldcg(a.wk_list + par * a.B + w0 + tid);
        const VerifyState* st = a.state + b;
        const int v = st->row_node;
        const int64_t row = a.z_row_off[b] + v + 1;
        s_req[tid] = b; s_node[tid] = v; s_dep[tid] = v < 0 ? 0 : min(a.depth[(size_t)b * N + v], a.D - 1);
        s_C[tid] = (float)st->passC; s_zmax[tid] = a.z_max[row]; s_zlogs[tid] = a.z_logs[row];
        s_lseT[tid] = a.node_lseT[(size_t)b * (N + 1) + v + 1];
      }
      __syncthreads();
      for (int i = tid; i < ng * a.r; i += WT) {
        const int g = i / a.r, k = i % a.r;
        const int v = s_node[g];
        const int ptok = v < 0 ? a.anchor[s_req[g]] : a.tok[(size_t)s_req[g] * N + v];
        s_a[g * RMAX + k] = Elem<TIn>::to_f(Ag[(size_t)ptok * a.r + k]);
      }
      __syncthreads();
      float sum[VG];
#pragma unroll
      for (int g = 0; g < VG; ++g) sum[g] = 0.f;
      bool need_q = false;
      for (int g = 0; g < ng; ++g) need_q |= (s_C[g] != 0.f);
      if (vec_ok) {
        for (int v = v_lo + tid * VEC; v < v_hi; v += WT * VEC) {
          float acc[VG][8];
          if (need_q) logits_group<TIn, VG>(a, s_a, ng, s_req, s_dep, v, acc, ws_ok ? Ws : Wg,
                                            ws_ok ? (size_t)a.vt_TV : (size_t)a.V, ws_ok ? v - v_lo : v);
#pragma unroll
          for (int g = 0; g < VG; ++g) {
            if (g < ng) {
              const int64_t row = a.z_row_off[s_req[g]] + s_node[g] + 1;
              float z[8];
              if (sizeof(TIn) == 2) { const uint4 x = __ldg(reinterpret_cast<const uint4*>(Zg + row * a.V + v)); unpack_bf16x8(x, z); }
              else { const float4 x = __ldg(reinterpret_cast<const float4*>(Zg + row * a.V + v)); z[0] = x.x; z[1] = x.y; z[2] = x.z; z[3] = x.w; }
#pragma unroll
              for (int i = 0; i < VEC; ++i) {
                const float p = __expf((z[i] - s_zmax[g]) * invT - s_zlogs[g]);
                const float q = s_C[g] != 0.f ? __expf(acc[g][i] * invT - s_lseT[g]) : 0.f;
                sum[g] += fmaxf(p - s_C[g] * q, 0.f);
              }
            }
          }
        }
      } else {
        for (int v = v_lo + tid; v < v_hi; v += WT) {
          for (int g = 0; g < ng; ++g) {
            const int b = s_req[g];
            const int64_t row = a.z_row_off[b] + s_node[g] + 1;
            const float p = __expf((z_elem<TIn>(a, row, v) - s_zmax[g]) * invT - s_zlogs[g]);
            float q = 0.f;
            if (s_C[g] != 0.f) {
              const int ptok = s_node[g] < 0 ? a.anchor[b] : a.tok[(size_t)b * N + s_node[g]];
              q = __expf(logit_scalar<TIn>(a, b, s_dep[g], ptok, v) * invT - s_lseT[g]);
            }
            sum[g] += fmaxf(p - s_C[g] * q, 0.f);
          }
        }
      }
#pragma unroll
      for (int g = 0; g < VG; ++g) {
        float sg = sum[g];
        for (int off = 16; off > 0; off >>= 1) sg += __shfl_xor_sync(0xFFFFFFFFu, sg, off);
        if (lane == 0) s_red[g][warp] = sg;
      }
      __syncthreads();
      if (tid < ng) {
        float t = 0.f;
        for (int w = 0; w < WT / 32; ++w) t += s_red[tid][w];
        a.part[(size_t)s_req[tid] * a.vt_n + blockIdx.x] = t;
      }
      __syncthreads();
    }
    // range rescans for bonus tokens that fall into this CTA's range: the residual of every token of
    // the range is evaluated once (tokens dealt round-robin to the threads: row i of the range holds
    // tokens i*WT .. i*WT+WT-1), then prefix sums in token order locate the crossing
    // Rescans are dealt round-robin to the CTAs (several bonus tokens often fall into one range, and a
    // rescan needs nothing of the CTA that owns the range except its columns of W, which any CTA can read
    // from global memory).
    for (int si = blockIdx.x; si < nsc; si += (int)nblocks) {
      const int b = __ldcg(a.sc_list + par * a.B + si);
      const VerifyState& st = a.state[b];
      const int s_lo = st.scan_tile * a.vt_TV, s_hi = min(a.V, s_lo + a.vt_TV);
      const bool own = st.scan_tile == (int)blockIdx.x;   // this CTA's own range: W is in shared memory
      const int v = st.cur;
      const int64_t row = a.z_row_off[b] + v + 1;
      const int dep = v < 0 ? 0 : a.depth[(size_t)b * N + v];
      const int ptok = v < 0 ? a.anchor[b] : a.tok[(size_t)b * N + v];
      const double C = st.C;
      const double zmax = a.z_max[row], zlogs = a.z_logs[row];
      const double lseT = C != 0.0 ? (double)a.node_lseT[(size_t)b * (N + 1) + v + 1] : 0.0;
      const int nf = st.nf;
      const double want = st.before >= 0.0 ? st.target - st.before : 1e300;
      for (int k = tid; k < a.r; k += WT) sb_a[k] = Elem<TIn>::to_f(Ag[(size_t)ptok * a.r + k]);
      if (tid == 0) { s_found = 0x7FFFFFFF; s_last = -1; }
      __syncthreads();
      const int len = s_hi - s_lo;
      const int nrow = (len + WT - 1) / WT;
      double carry = 0.0;
      for (int i = 0; i < nrow; ++i) {
        const int o = i * WT + tid, w = s_lo + o;
        double rw = 0.0;
        if (o < len) {
          double Cw = C;
          for (int f = 0; f < nf; ++f) if (st.fx[f] == w) Cw = st.fC[f];
          const double p = exp(((double)z_elem<TIn>(a, row, w) - zmax) / (double)a.T - zlogs);
          double q = 0.0;
          if (Cw != 0.0) {
            float acc = Elem<TIn>::to_f(reinterpret_cast<const TIn*>(a.U)[((size_t)b * a.D + dep) * a.V + w]);
            if (MMA && own && !tc.stream) {
              // the range's W columns sit in the tensor-core operand layout: 64-token slabs of [rp][128 B],
              // 16-byte chunk j of row k at chunk j ^ (k & 7)
              const unsigned char* wsl = tc.Ws + (size_t)(o >> 6) * tc.slab_bytes + (o & 7) * 2;
              const int j = (o & 63) >> 3;
              for (int k = 0; k < a.r; ++k)
                acc = fmaf(sb_a[k], __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(wsl + k * 128 + ((j ^ (k & 7)) << 4))), acc);
            } else if (ws_ok && own) { for (int k = 0; k < a.r; ++k) acc = fmaf(sb_a[k], Elem<TIn>::to_f(Ws[(size_t)k * a.vt_TV + o]), acc); }
            else {
              // another CTA's range: the column of W comes from global memory, eight rows requested at a time
              // (same order of the multiply-adds as above, so the same bits)
              int k = 0;
              for (; k + 8 <= a.r; k += 8) {
                TIn wv[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) wv[u] = Wg[(size_t)(k + u) * a.V + w];
#pragma unroll
                for (int u = 0; u < 8; ++u) acc = fmaf(sb_a[k + u], Elem<TIn>::to_f(wv[u]), acc);
              }
              for (; k < a.r; ++k) acc = fmaf(sb_a[k], Elem<TIn>::to_f(Wg[(size_t)k * a.V + w]), acc);
            }
            q = exp((double)acc / (double)a.T - lseT);
          }
          rw = fmax(p - Cw * q, 0.0);
        }
        // inclusive prefix over the row in thread (= token) order
        double inc = rw;
        for (int off = 1; off < 32; off <<= 1) { const double t = __shfl_up_sync(0xFFFFFFFFu, inc, off); if (lane >= off) inc += t; }
        if (lane == 31) s_scan[warp] = inc;
        __syncthreads();
        double wbase = 0.0, rowsum = 0.0;
        for (int w2 = 0; w2 < WT / 32; ++w2) { if (w2 < warp) wbase += s_scan[w2]; rowsum += s_scan[w2]; }
        const double cum = carry + wbase + inc;
        if (o < len && rw > 0.0) atomicMax(&s_last, o);
        if (o < len && cum > want) atomicMin(&s_found, o);
        carry += rowsum;
        __syncthreads();
        if (s_found != 0x7FFFFFFF) break;   // uniform: read after the barrier
      }
      if (tid == 0) {
        int o = s_found;
        if (o == 0x7FFFFFFF) o = s_last >= 0 ? s_last : len - 1;   // rounding pushed the crossing past the range
        a.state[b].result = s_lo + o;
      }
      __syncthreads();
    }
    __threadfence();
    if (!grid_barrier(a.barrier, nexpect, gen, a.wait_limit)) return false;
    if (stage == 1) stage = 2;
    else if (left == 0 && nwk == 0) stage = 1;   // uniform over the grid: both were read after the step's first barrier
  }
  // steps ran out
  for (int b = blockIdx.x; b < a.B; b += nblocks)
    if (tid == 0 && a.state[b].need != 3) a.status[b] = TS_ERR_TIMEOUT;
  return true;
}

// Kernel wrapper.  MMA = true (bf16 inputs on sm_100): the CTA's range of W is loaded once in the tensor-core
// operand layout (bulk-tensor loads when a tensor map is available, plain loads otherwise), tensor memory is
// allocated for the accumulators, and both are released on every way out.
template <typename TIn, bool MMA>
__global__ void __launch_bounds__(WT, 1) verify_walk_kernel(const VerifyArgs a, const __grid_constant__ CUtensorMap tmW, const int use_tma) {
  extern __shared__ __align__(16) unsigned char w_raw[];
  WalkTc tc{};
  if (!MMA) { pdl_wait(); walk_body<TIn, false>(a, tc, w_raw); return; }
  const int tid = threadIdx.x, warp = tid >> 5;
  const int r = a.r, rp = (r + 63) / 64 * 64;
  const int t0 = blockIdx.x * a.vt_TV, tlen = min(a.vt_TV, a.V - t0);
  const bool stream = a.w_stream != 0;   // (needs the tensor map: the host selects it only then)
  const int nslab = stream ? WALK_RING * (WALK_SBLK / 64) : a.vt_TV / 64, nblk = stream ? 0 : (tlen + 127) / 128;
  unsigned char* sm = w_raw + ((1024u - (smem_u32(w_raw) & 1023u)) & 1023u);
  tc.rp = rp; tc.slab_bytes = (uint32_t)rp * 128u; tc.it = 0;
  tc.stream = stream ? 1 : 0; tc.tm = &tmW; tc.wit = 0;
  tc.Ws = sm;
  tc.As = tc.Ws + (size_t)nslab * tc.slab_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tc.As + (size_t)(rp / 64) * 128 * 128);
  tc.t_full = bars; tc.t_empty = bars + WALK_NBUF;
  uint64_t* w_full = bars + 2 * WALK_NBUF;
  tc.w_full = w_full; tc.w_free = w_full + WALK_RING;   // (streaming form: the first 2 * WALK_RING of these barriers)
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(w_full + WALK_MAX_BLK);
  tc.s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  constexpr uint32_t TMEM_COLS = WALK_NBUF * WALK_BLK;
  if (warp == WALK_EPI) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < WALK_NBUF; ++i) { mbar_init(tc.t_full + i, 1); mbar_init(tc.t_empty + i, WALK_EPI); }
    *tc.s_abort = 0;
    if (use_tma) for (int i = 0; i < (stream ? 2 * WALK_RING : nblk); ++i) mbar_init(w_full + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (use_tma) {
      for (int nb = 0; nb < nblk; ++nb) {
        const int ns = (tlen - nb * 128 > 64) ? 2 : 1;
        mbar_expect_tx(w_full + nb, (uint32_t)ns * tc.slab_bytes);
        for (int h = 0; h < ns; ++h) tma_load_box(tc.Ws + (size_t)(2 * nb + h) * tc.slab_bytes, &tmW, t0 + (2 * nb + h) * 64, 0, w_full + nb);
      }
    }
  }
  if (!use_tma) {
    const __nv_bfloat16* Wg = reinterpret_cast<const __nv_bfloat16*>(a.W);
    const int per_slab = rp * 8;
    for (int idx = tid; idx < nslab * per_slab; idx += WT) {
      const int slab = idx / per_slab, rem = idx % per_slab, k = rem >> 3, j = rem & 7;
      const int tok = t0 + slab * 64 + j * 8;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (k < r && tok < a.V) v = __ldg(reinterpret_cast<const uint4*>(Wg + (size_t)k * a.V + tok));
      *reinterpret_cast<uint4*>(tc.Ws + (size_t)slab * tc.slab_bytes + k * 128 + ((j ^ (k & 7)) << 4)) = v;
    }
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  tc.tmem_base = *s_tmem;
  pdl_wait();   // row statistics and the tree come from earlier kernels; W (loaded above) does not
  bool ok = true;
  if (use_tma) {
    // the whole range must have landed before anything reads it (the rescans read it with plain loads)
    if (tid == 0)
      for (int nb = 0; nb < nblk; ++nb) if (!mbar_wait(w_full + nb, 0, tc.s_abort, nullptr, a.wait_limit)) break;
    __syncthreads();
    ok = *tc.s_abort == 0;
    if (!ok && tid == 0) atomicExch(a.barrier + 1, 1u);
  }
  if (ok) walk_body<TIn, true>(a, tc, w_raw);
  if (use_tma && !ok && tid == 0) {
    // gave up on a load: do not leave while it may still be writing this CTA's shared memory
    for (int nb = 0; nb < nblk; ++nb) {
      bool done = false;
      for (uint32_t i = 0; i < WAIT_LIMIT && !done; ++i) { done = mbar_try_wait(w_full + nb, 0); if (!done) __nanosleep(100); }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == WALK_EPI) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tc.tmem_base), "r"(TMEM_COLS) : "memory");
  }
}



// after a barrier timeout the kernel returns early; this marks every unfinished request
__global__ void verify_check_kernel(VerifyArgs a) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= a.B) return;
  if (a.barrier[1] != 0u && a.state[b].need != 3) a.status[b] = TS_ERR_TIMEOUT;
}

cudaError_t verify_setup(ts_ctx* ctx) {
  // the walk kernel may keep its range of W in shared memory: allow the full opt-in size
  cudaError_t e = cudaFuncSetAttribute(verify_walk_kernel<__nv_bfloat16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       ctx->max_smem - 40 * 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(verify_walk_kernel<__nv_bfloat16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem - 12 * 1024);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(verify_walk_kernel<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem - 40 * 1024);
}

}  // namespace ts

extern "C" int32_t ts_verify_tree(ts_ctx* ctx, const void* U, const void* A, const void* W, const void* Z,
                                  const int64_t* z_row_off, int32_t B, const int32_t* anchor_tok,
                                  const int32_t* n_nodes, const int32_t* tok, const int32_t* parent,
                                  const int32_t* depth, const int32_t* sib_rank, const uint64_t* node_hash,
                                  const float* logqT, const float* node_lseT, float T, uint64_t seed,
                                  int32_t* acc_len, int32_t* acc_node, int32_t* acc_tok, int32_t* bonus_tok,
                                  float* edge_stat, uint32_t* flags, int32_t* status, void* ws_v, size_t ws_bytes,
                                  void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_verify_tree: null context");
  const void* req[] = {U, A, W, Z, z_row_off, anchor_tok, n_nodes, tok, parent, depth, sib_rank, node_hash,
                       acc_len, acc_node, acc_tok, bonus_tok, flags, status, ws_v};
  for (const void* p : req)
    if (bad_ptr(p)) return set_error(TS_ERR_INVALID, "ts_verify_tree: null or misaligned pointer");
  if (edge_stat && ((uintptr_t)edge_stat & 15u)) return set_error(TS_ERR_INVALID, "ts_verify_tree: misaligned edge_stat");
  const ts_config& c = ctx->cfg;
  if (B < 1 || B > c.max_batch) return set_error(TS_ERR_INVALID, "ts_verify_tree: B out of range");
  if (!(T >= 0.f)) return set_error(TS_ERR_INVALID, "ts_verify_tree: T must be >= 0");
  if (T > 0.f && (bad_ptr(logqT) || bad_ptr(node_lseT)))
    return set_error(TS_ERR_INVALID, "ts_verify_tree: logqT and node_lseT are required when T > 0");
  const WsLayout L = make_layout(ctx, B);
  if (ws_bytes < L.total) return set_error(TS_ERR_WORKSPACE, "ts_verify_tree: workspace too small");
  char* ws = (char*)ws_v;
  cudaStream_t st = (cudaStream_t)stream;

  VerifyArgs a{};
  a.U = U; a.A = A; a.W = W; a.Z = Z; a.z_row_off = z_row_off; a.B = B; a.V = c.V; a.D = c.D; a.r = c.r; a.K = c.K;
  a.N = c.Nmax; a.T = T; a.seed = seed; a.anchor = anchor_tok; a.n_nodes = n_nodes; a.tok = tok; a.parent = parent;
  a.depth = depth; a.sib = sib_rank; a.node_hash = node_hash; a.logqT = logqT; a.node_lseT = node_lseT;
  float* z_max = (float*)(ws + L.z_max); int* z_arg = (int*)(ws + L.z_arg); float* z_logs = (float*)(ws + L.z_lse);
  a.z_max = z_max; a.z_arg = z_arg; a.z_logs = z_logs;
  a.acc_len = acc_len; a.acc_node = acc_node; a.acc_tok = acc_tok; a.bonus = bonus_tok; a.edge_stat = edge_stat;
  a.flags = flags; a.status = status;
  a.state = (VerifyState*)(ws + L.vf_state); a.part = (float*)(ws + L.vf_part); a.barrier = (unsigned*)(ws + L.vf_barrier);
  a.child_first = (int*)(ws + L.vf_child); a.child_cnt = a.child_first + (size_t)B * (c.Nmax + 1);
  a.edge_px = (double*)(ws + L.vf_edge); a.edge_qx = a.edge_px + (size_t)B * c.Nmax; a.edge_u = a.edge_qx + (size_t)B * c.Nmax;
  a.wk_list = (int*)(ws + L.vf_lists); a.sc_list = a.wk_list + 2 * (size_t)B; a.ctr = a.sc_list + 2 * (size_t)B;
  a.vt_TV = ctx->vt_TV; a.vt_n = ctx->vt_n; a.max_steps = 2 * (c.Nmax + c.D) + 10;
  a.wait_limit = ctx->wait_limit; a.lost_arrival = (ctx->test_mode & TS_TEST_LOST_ARRIVAL) ? 1 : 0;

  const int max_rows = B * (c.Nmax + 1);
  int grid_rows = max_rows < 8 * ctx->num_sms ? max_rows : 8 * ctx->num_sms;
  cudaError_t ez;
  {
    ProfScope ps(ctx, K_ZROWS, st);
    if (c.dt_Z == TS_DTYPE_BF16)
      ez = launch_kernel(zrow_stats_kernel<__nv_bfloat16>, grid_rows, ZT, 0, st, true, (const __nv_bfloat16*)Z, z_row_off, B, c.V, T, z_max, z_arg, z_logs, T > 0.f ? a.barrier : (unsigned*)nullptr);
    else
      ez = launch_kernel(zrow_stats_kernel<float>, grid_rows, ZT, 0, st, true, (const float*)Z, z_row_off, B, c.V, T, z_max, z_arg, z_logs, T > 0.f ? a.barrier : (unsigned*)nullptr);
  }
  cudaError_t e = ez != cudaSuccess ? ez : cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_verify_tree(rows)", e);
  if (T == 0.f) {
    { ProfScope ps(ctx, K_GREEDY, st); verify_greedy_kernel<<<B, 128, 0, st>>>(a); }
    e = cudaGetLastError();
    if (e != cudaSuccess) return set_cuda_error("ts_verify_tree(greedy)", e);
    return TS_OK;
  }
  size_t w_bytes = (size_t)c.r * ctx->vt_TV * (c.dt_W == TS_DTYPE_BF16 ? 2 : 4);
  a.w_smem = (w_bytes + 40 * 1024 <= (size_t)ctx->max_smem) ? 1 : 0;
  // tensor-core reductions: bf16 everywhere, the range of W in operand layout plus the A tile within shared memory
  const size_t rp = (size_t)(c.r + 63) / 64 * 64;
  const size_t mma_bytes = (size_t)(ctx->vt_TV / 64) * rp * 128 + (rp / 64) * 128 * 128 + (2 * WALK_NBUF + WALK_MAX_BLK) * 8 + 64 + 1024;
  const bool mma_shape = ctx->use_mma && c.dt_Z == TS_DTYPE_BF16 && c.dt_U == TS_DTYPE_BF16 && c.dt_W == TS_DTYPE_BF16 &&
                         c.dt_A == TS_DTYPE_BF16 && ctx->vt_TV % 64 == 0 && ctx->vt_TV / 128 < WALK_MAX_BLK;
  const bool resident = mma_shape && mma_bytes + 32 * 1024 <= (size_t)ctx->max_smem;
  // The range of W does not fit (large ranks): blocks of 128 tokens stream through a ring of two, by bulk-tensor
  // loads, for every reduction.  Needs the tensor map; the kernel's static shared memory is about 9 KB.
  const size_t stream_bytes = (size_t)WALK_RING * (WALK_SBLK / 64) * rp * 128 + (rp / 64) * 128 * 128 + (2 * WALK_NBUF + WALK_MAX_BLK) * 8 + 64 + 1024;
  int use_tma = 0;
  CUtensorMap tm;
  memset(&tm, 0, sizeof(tm));
  if (mma_shape && w_tensor_map(ctx, W)) { memcpy(&tm, ctx->tmapW, sizeof(tm)); use_tma = 1; }
  const bool streaming = mma_shape && !resident && use_tma && stream_bytes + 12 * 1024 <= (size_t)ctx->max_smem;
  const bool mma = resident || streaming;
  a.w_stream = streaming ? 1 : 0;
  if (!mma) use_tma = 0;
  void* kargs[] = {(void*)&a, (void*)&tm, (void*)&use_tma};
  const void* fn = mma ? (const void*)verify_walk_kernel<__nv_bfloat16, true>
                       : (c.dt_Z == TS_DTYPE_BF16 ? (const void*)verify_walk_kernel<__nv_bfloat16, false>
                                                  : (const void*)verify_walk_kernel<float, false>);
  if (mma) w_bytes = streaming ? stream_bytes : mma_bytes;
  {
    ProfScope ps(ctx, K_WALK, st);
    // cooperative (the grid barriers need every CTA resident) and, where the driver takes both attributes,
    // chained to the row statistics so that the W load and the tensor-memory allocation run beside them
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.vt_n); cfg.blockDim = dim3(WT); cfg.dynamicSmemBytes = (mma || a.w_smem) ? w_bytes : 0; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative; attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization; attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = ctx->walk_pdl >= 0 ? 2 : 1;
    e = cudaLaunchKernelExC(&cfg, fn, kargs);
    if (e != cudaSuccess && cfg.numAttrs == 2) {   // not accepted together: remember, and launch cooperative only
      (void)cudaGetLastError();
      ctx->walk_pdl = -1;
      cfg.numAttrs = 1;
      e = cudaLaunchKernelExC(&cfg, fn, kargs);
    }
  }
  if (e != cudaSuccess) return set_cuda_error("ts_verify_tree(walk)", e);
  { ProfScope ps(ctx, K_CHECK, st); verify_check_kernel<<<(B + 127) / 128, 128, 0, st>>>(a); }
  e = cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_verify_tree(check)", e);
  return TS_OK;
}
