// Scoring kernel for levels with few parents (single-request decoding, the last levels of a batch).
//
// With a handful of parents the low-rank bias [parents x r] . [r x V] is no dense contraction: a
// 128-row tensor-core tile would carry one to sixteen useful rows, and the epilogue of the tensor-core
// kernel -- one parent per lane -- would leave most lanes idle while it walks the vocabulary.  Here the
// mapping is turned round: one warp = one (parent, 256-token tile), one lane = eight consecutive tokens.
// The lane forms its eight logits with fused multiply-adds (U + sum_k A[x_p][k] W[k][v], k ascending),
// every token gets its exact Gumbel key (no bounds: a tile is over before any could arrive), and the
// warp's K best logits and K best keys come out of K rounds of a shuffle arg-max.  The whole grid works
// on every parent at once: the launch takes a few microseconds instead of the tens the tile kernel needs
// to get going.  W is read through L1 (the eight warps of a CTA share a tile and its lines).
//
// Records have the layout of the other scoring kernels (header (max, sum0, sumT, counts), then K logits,
// K tokens, K keys, K tokens, K logits), one per (tile, parent) at rec[(tile * FEW_MAX + p) * rec_words];
// the merge kernel is told which kernel ran.  The host sends a level here when it knows that the level
// cannot have more than FEW_MAX parents (B * K^depth and B * Nmax bound it).
#include "ts_internal.h"
#include "ts_scan.cuh"

namespace ts {

constexpr int FEW_THREADS = 256;
constexpr int FEW_WARPS = FEW_THREADS / 32;
constexpr int FEW_TILE = 256;   // tokens per tile: eight per lane

// (value desc, token asc) arg-max over the warp; every lane gets the winner
__device__ __forceinline__ void warp_best(float& v, int& tok) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float ov = __shfl_xor_sync(0xFFFFFFFFu, v, off);
    const int ot = __shfl_xor_sync(0xFFFFFFFFu, tok, off);
    if (ov > v || (ov == v && ot < tok)) { v = ov; tok = ot; }
  }
}

__global__ void __launch_bounds__(FEW_THREADS) score_few_kernel(const ScoreArgs a) {
  __shared__ float s_a[FEW_WARPS][256];   // head row A[x_p] of each warp's parent (r <= 256)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  pdl_wait();                // the parent list and its length come from the kernel before
  pdl_launch_dependents();
  const int P = a.P_dev ? *a.P_dev : a.P;
  if (P <= 0 || P > FEW_MAX) return;   // an empty level (the host never sends a longer list here)
  const int p = blockIdx.y * FEW_WARPS + warp;
  if (p >= P) return;                  // no block-wide barrier below
  const int V = a.V, r = a.r, K = a.K;
  const int tile = blockIdx.x, v = tile * FEW_TILE + lane * 8;
  const bool in = v < V;               // V is a multiple of 8: a lane's eight tokens are all inside or all outside
  const __nv_bfloat16* Wg = reinterpret_cast<const __nv_bfloat16*>(a.W);
  const __nv_bfloat16* Ug = reinterpret_cast<const __nv_bfloat16*>(a.U);
  const __nv_bfloat16* Ag = reinterpret_cast<const __nv_bfloat16*>(a.A);
  const int req = a.p_req[p], dep = a.p_depth[p], ptok = a.p_token[p];
  const uint64_t hash = a.p_hash[p];
  for (int k = lane; k < r; k += 32) s_a[warp][k] = __bfloat162float(Ag[(size_t)ptok * r + k]);
  __syncwarp();

  // ---- logits of the lane's eight tokens -------------------------------------------------------------
  float l[8];
  if (in) {
    unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(Ug + ((size_t)req * a.D + dep) * V + v)), l);
#pragma unroll 16
    for (int k = 0; k < r; ++k) {
      float w[8];
      unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(Wg + (size_t)k * V + v)), w);
      const float ak = s_a[warp][k];
#pragma unroll
      for (int i = 0; i < 8; ++i) l[i] = fmaf(ak, w[i], l[i]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) l[i] = -INFINITY;
  }

  // ---- max and sums of exponentials over the tile -----------------------------------------------------
  const float T = a.T, invT = T > 0.f ? 1.f / T : 1.f;
  const bool two = (T > 0.f) && (T != 1.f);
  float m = l[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) m = fmaxf(m, l[i]);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
  float s0 = 0.f, sT = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float d = l[i] - m;   // -inf for tokens outside V: contributes 0
    s0 += __expf(d);
    if (two) sT += __expf(d * invT);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    s0 += __shfl_xor_sync(0xFFFFFFFFu, s0, off);
    sT += __shfl_xor_sync(0xFFFFFFFFu, sT, off);
  }
  if (!two) sT = s0;

  // ---- K best logits: K rounds of arg-max, lane j keeps the j-th ---------------------------------------
  float topv = -INFINITY; int topi = -1;
  {
    uint32_t taken = 0;
    for (int j = 0; j < K; ++j) {
      float bv = -INFINITY; int bi = 0x7FFFFFFF;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (!((taken >> i) & 1u) && l[i] > bv) { bv = l[i]; bi = v + i; }   // first maximum: lowest token
      warp_best(bv, bi);
      if (bv > -INFINITY && bi >= v && bi < v + 8) taken |= 1u << (bi - v);
      if (lane == j) { topv = bv; topi = bv > -INFINITY ? bi : -1; }
    }
  }

  // ---- K best Gumbel keys (without-replacement draws in order) -----------------------------------------
  float keyv = -INFINITY, keyl = 0.f; int keyi = -1;
  if (T > 0.f) {
    float key[8];
    if (in) {
      const uint4 cw = stream_words(a.seed, req, hash, STREAM_GUMBEL_COARSE, (uint32_t)v >> 3);
      const uint4 fw = stream_words(a.seed, req, hash, STREAM_GUMBEL_FINE, (uint32_t)v >> 3);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t c16 = (word_of(cw, i >> 1) >> (16 * (i & 1))) & 0xFFFFu;
        const uint32_t f16 = (word_of(fw, i >> 1) >> (16 * (i & 1))) & 0xFFFFu;
        key[i] = l[i] * invT + gumbel_from_bits((c16 << 16) | f16);
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) key[i] = -INFINITY;
    }
    uint32_t taken = 0;
    for (int j = 0; j < K; ++j) {
      float bv = -INFINITY; int bi = 0x7FFFFFFF;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (!((taken >> i) & 1u) && key[i] > bv) { bv = key[i]; bi = v + i; }
      warp_best(bv, bi);
      const bool mine = bv > -INFINITY && bi >= v && bi < v + 8;
      float lg = 0.f;
      if (mine) {
        taken |= 1u << (bi - v);
#pragma unroll
        for (int i = 0; i < 8; ++i) lg = (bi - v == i) ? l[i] : lg;
      }
      // the winner's logit travels to lane j (exactly one lane holds it)
      const unsigned who = __ballot_sync(0xFFFFFFFFu, mine);
      const float wl = who ? __shfl_sync(0xFFFFFFFFu, lg, __ffs(who) - 1) : 0.f;
      if (lane == j) { keyv = bv; keyi = bv > -INFINITY ? bi : -1; keyl = wl; }
    }
  }

  // ---- publish the piece's best values (the merge filters the records with the resulting bounds) -----
  {
    const float bestL = __shfl_sync(0xFFFFFFFFu, topv, 0), bestK = __shfl_sync(0xFFFFFFFFu, keyv, 0);
    if (lane == 0) {
      const SharedThr gl{a.slots + (size_t)p * K * SLOT_STRIDE, tile % K};
      const SharedThr gk{a.slots + ((size_t)a.cap + p) * K * SLOT_STRIDE, tile % K};
      if (bestL > -INFINITY) publish(gl, bestL);
      if (T > 0.f && bestK > -INFINITY) publish(gk, bestK);
    }
  }

  // ---- record ----------------------------------------------------------------------------------------------
  const int rw = rec_words(K);
  float* rec = a.rec + ((size_t)tile * FEW_MAX + p) * rw;
  const int nt = __popc(__ballot_sync(0xFFFFFFFFu, lane < K && topi >= 0));
  const int nk = __popc(__ballot_sync(0xFFFFFFFFu, lane < K && keyi >= 0));
  if (lane == 0) *reinterpret_cast<float4*>(rec) = make_float4(m, s0, sT, __int_as_float(nt | (nk << 8)));
  if (lane < K) {
    float* f = rec + 4; int* ii = reinterpret_cast<int*>(rec) + 4;
    f[lane] = topv; ii[K + lane] = topi; f[2 * K + lane] = keyv; ii[3 * K + lane] = keyi; f[4 * K + lane] = keyl;
  }
}

int few_tiles(const ts_config& c) { return (c.V + FEW_TILE - 1) / FEW_TILE; }

// bf16 inputs with 16-byte rows; the records of the largest level this kernel takes must fit the scratch
bool few_supported(const ts_ctx* ctx) {
  const ts_config& c = ctx->cfg;
  return ctx->use_mma && c.dt_U == TS_DTYPE_BF16 && c.V % 8 == 0 && c.r <= 256 && c.K <= 32;
}

cudaError_t launch_score_few(const ts_ctx* ctx, const ScoreArgs& a, int p_bound, cudaStream_t st) {
  const dim3 grid(few_tiles(ctx->cfg), (p_bound + FEW_WARPS - 1) / FEW_WARPS > 0 ? (p_bound + FEW_WARPS - 1) / FEW_WARPS : 1);
  const cudaError_t e = launch_kernel(score_few_kernel, grid, dim3(FEW_THREADS), 0, st, a.pdl != 0, a);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ts
