// Parent-conditioned scoring (Eq. 1) fused with logsumexp at temperature 1 and T, top-K logits and
// Gumbel top-K sibling draws (Eq. 2), one pass over the vocabulary.
//
// Decomposition: the vocabulary is split into tiles, one CTA per tile with its W tile resident in
// shared memory for all parents; every thread owns one parent and scans the tile's tokens in
// order, so the running max / sums / candidate lists are thread-private.  A second kernel merges
// the per-tile records of each parent.
#include "ts_internal.h"

namespace ts {

// Thread-private running state of one parent over the tokens scanned so far.
struct RowScan {
  float m, s0, sT;
  float thrL, thrK;
  int K;
  float topv[KMAX]; int topi[KMAX];
  float keyv[KMAX]; int keyi[KMAX]; float keyl[KMAX];

  __device__ __forceinline__ void init(int K_) {
    K = K_; m = -INFINITY; s0 = 0.f; sT = 0.f; thrL = -INFINITY; thrK = -INFINITY;
    for (int i = 0; i < KMAX; ++i) { topv[i] = -INFINITY; topi[i] = -1; keyv[i] = -INFINITY; keyi[i] = -1; keyl[i] = 0.f; }
  }
  // tokens arrive in increasing order, so an equal value never displaces an earlier entry
  __device__ __forceinline__ void insert_top(float v, int tok) {
    int pos = K - 1;
    while (pos > 0 && v > topv[pos - 1]) { topv[pos] = topv[pos - 1]; topi[pos] = topi[pos - 1]; --pos; }
    topv[pos] = v; topi[pos] = tok;
    thrL = topv[K - 1];
  }
  __device__ __forceinline__ void insert_key(float key, int tok, float logit) {
    int pos = K - 1;
    while (pos > 0 && key > keyv[pos - 1]) {
      keyv[pos] = keyv[pos - 1]; keyi[pos] = keyi[pos - 1]; keyl[pos] = keyl[pos - 1]; --pos;
    }
    keyv[pos] = key; keyi[pos] = tok; keyl[pos] = logit;
    thrK = keyv[K - 1];
  }
};

struct ScoreArgs {
  const void *U, *A, *W;
  int V, D, r, K;
  int P; const int* P_dev;
  const int *p_req, *p_depth, *p_token; const uint64_t* p_hash;
  float T; uint64_t seed;
  int TV, ntiles, Pcap;
  float *part_m, *part_s0, *part_sT, *part_topv, *part_keyv, *part_keyl;
  int *part_topi, *part_keyi;
};

// One 16-token chunk of one parent: logits l[0..16) for tokens v0.., `valid` of them inside V.
__device__ __forceinline__ void scan_chunk(RowScan& st, const float* l, int v0, int valid, float T, float invT,
                                           uint64_t seed, int req, uint64_t hash, const float* ghi) {
  float cm = -INFINITY;
#pragma unroll
  for (int i = 0; i < CHUNK; ++i) if (i < valid) cm = fmaxf(cm, l[i]);
  if (cm > st.m) {
    const float d = st.m - cm;  // -inf on the first chunk: both factors become 0
    st.s0 *= __expf(d);
    st.sT *= __expf(d * invT);
    st.m = cm;
  }
  float a0 = 0.f, aT = 0.f;
  const bool two = (T > 0.f) && (T != 1.f);
#pragma unroll
  for (int i = 0; i < CHUNK; ++i) {
    if (i < valid) {
      const float d = l[i] - st.m;
      a0 += __expf(d);
      if (two) aT += __expf(d * invT);
    }
  }
  st.s0 += a0;
  st.sT += two ? aT : a0;
  if (cm > st.thrL || st.topi[st.K - 1] < 0) {
#pragma unroll
    for (int i = 0; i < CHUNK; ++i)
      if (i < valid && (l[i] > st.thrL || st.topi[st.K - 1] < 0)) st.insert_top(l[i], v0 + i);
  }
  if (T > 0.f) {
    // top byte of each token's uniform: one generator call for the chunk
    const uint4 cw = stream_words(seed, req, hash, STREAM_GUMBEL_COARSE, (uint32_t)v0 >> 4);
    uint4 fw = make_uint4(0, 0, 0, 0);
    int fine_call = -1;
#pragma unroll
    for (int i = 0; i < CHUNK; ++i) {
      if (i < valid) {
        const uint32_t c8 = (word_of(cw, i >> 2) >> (8 * (i & 3))) & 0xFFu;
        const float base = l[i] * invT;
        // ghi[c8] bounds the noise from above given only the top byte; most tokens stop here
        if (base + ghi[c8] > st.thrK || st.keyi[st.K - 1] < 0) {
          if (fine_call != (i >> 2)) {
            fw = stream_words(seed, req, hash, STREAM_GUMBEL_FINE, ((uint32_t)(v0 + i)) >> 2);
            fine_call = i >> 2;
          }
          const uint32_t X = (c8 << 24) | (word_of(fw, i & 3) >> 8);
          const float key = base + gumbel_from_bits(X);
          if (key > st.thrK || st.keyi[st.K - 1] < 0) st.insert_key(key, v0 + i, l[i]);
        }
      }
    }
  }
}

template <typename TIn>
__global__ void __launch_bounds__(SCORE_THREADS, 1) score_tile_kernel(ScoreArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int r = a.r, TV = a.TV, V = a.V;
  TIn* Ws = reinterpret_cast<TIn*>(smem_raw);                              // [r][TV]
  float* as = reinterpret_cast<float*>(smem_raw + (size_t)r * TV * sizeof(TIn));  // [r][SCORE_THREADS]
  float* ghi = as + (size_t)r * SCORE_THREADS;                             // [256]
  const int tid = threadIdx.x;
  const int tile = blockIdx.x;
  const int t0 = tile * TV;
  const int tlen = min(TV, V - t0);
  const TIn* Wg = reinterpret_cast<const TIn*>(a.W);
  const TIn* Ug = reinterpret_cast<const TIn*>(a.U);
  const TIn* Ag = reinterpret_cast<const TIn*>(a.A);
  constexpr int VEC = Elem<TIn>::VEC;
  const bool vec_ok = (V % VEC) == 0;
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
  // upper bound of the Gumbel noise given the top byte of the uniform, with a safety margin
  for (int c = tid; c < 256; c += SCORE_THREADS) {
    const double u = ((double)(((uint32_t)c << 24) | 0xFFFFFFu) + 0.5) * (1.0 / 4294967296.0);
    const double g = -log(-log(u));
    ghi[c] = (float)(g + 1e-4 * fabs(g) + 1e-4);
  }
  __syncthreads();

  const float T = a.T, invT = T > 0.f ? 1.f / T : 1.f;
  const int K = a.K;

  for (int pg = 0; pg < P; pg += SCORE_THREADS) {
    const int p = pg + tid;
    if (p >= P) continue;  // no block-wide barrier below
    const int req = a.p_req[p], dep = a.p_depth[p], ptok = a.p_token[p];
    const uint64_t hash = a.p_hash[p];
    for (int k = 0; k < r; ++k) as[k * SCORE_THREADS + tid] = Elem<TIn>::to_f(Ag[(size_t)ptok * r + k]);
    const TIn* Urow = Ug + ((size_t)req * a.D + dep) * V + t0;
    RowScan st;
    st.init(K);
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
      scan_chunk(st, l, t0 + c0, valid, T, invT, a.seed, req, hash, ghi);
    }
    // record of (parent, tile)
    const size_t o = (size_t)tile * a.Pcap + p;
    a.part_m[o] = st.m; a.part_s0[o] = st.s0; a.part_sT[o] = st.sT;
    for (int j = 0; j < K; ++j) {
      const size_t oj = ((size_t)tile * K + j) * a.Pcap + p;
      a.part_topv[oj] = st.topv[j]; a.part_topi[oj] = st.topi[j];
      a.part_keyv[oj] = st.keyv[j]; a.part_keyi[oj] = st.keyi[j]; a.part_keyl[oj] = st.keyl[j];
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Merge of the per-tile records: one warp per parent
// ------------------------------------------------------------------------------------------------
struct MergeArgs {
  int P; const int* P_dev; int K, ntiles, Pcap; float T;
  const float *part_m, *part_s0, *part_sT, *part_topv, *part_keyv, *part_keyl;
  const int *part_topi, *part_keyi;
  float *lse0, *lseT; int* top_tok; float* top_logit; int* draw_tok; float* draw_logit;
};

constexpr int MERGE_MAX_TILES_PER_LANE = 16;

// K rounds of warp-wide arg-max over the heads of the per-tile sorted lists
__device__ void merge_lists(const float* pv, const int* pi, const float* pl, int p, int K, int ntiles, int Pcap,
                            int lane, int* out_tok, float* out_val) {
  unsigned char cur[MERGE_MAX_TILES_PER_LANE];
  for (int i = 0; i < MERGE_MAX_TILES_PER_LANE; ++i) cur[i] = 0;
  for (int j = 0; j < K; ++j) {
    float bv = -INFINITY; int bi = 0x7FFFFFFF, bt = -1; float bl = 0.f;
    for (int s = 0, t = lane; t < ntiles; t += 32, ++s) {
      if (cur[s] >= K) continue;
      const size_t o = ((size_t)t * K + cur[s]) * Pcap + p;
      const int idx = pi[o];
      if (idx < 0) continue;
      const float v = pv[o];
      if (v > bv || (v == bv && idx < bi)) { bv = v; bi = idx; bt = s; bl = pl ? pl[o] : v; }
    }
    float wv = bv; int wi = bi;
    for (int off = 16; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, wv, off);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, wi, off);
      if (ov > wv || (ov == wv && oi < wi)) { wv = ov; wi = oi; }
    }
    const bool mine = (bt >= 0) && (wi == bi) && (wv == bv);
    if (mine) cur[bt]++;
    const unsigned who = __ballot_sync(0xFFFFFFFFu, mine);
    if (who == 0u) { if (lane == 0) { out_tok[j] = -1; out_val[j] = 0.f; } continue; }
    const int src = __ffs(who) - 1;
    const float lv = __shfl_sync(0xFFFFFFFFu, bl, src);
    if (lane == 0) { out_tok[j] = wi; out_val[j] = lv; }
  }
}

__global__ void merge_kernel(MergeArgs a) {
  const int P = a.P_dev ? *a.P_dev : a.P;
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const int nwarps = (gridDim.x * blockDim.x) >> 5;
  const float invT = a.T > 0.f ? 1.f / a.T : 1.f;
  for (int p = warp; p < P; p += nwarps) {
    float m = -INFINITY;
    for (int t = lane; t < a.ntiles; t += 32) m = fmaxf(m, a.part_m[(size_t)t * a.Pcap + p]);
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
    float s0 = 0.f, sT = 0.f;
    for (int t = lane; t < a.ntiles; t += 32) {
      const size_t o = (size_t)t * a.Pcap + p;
      const float d = a.part_m[o] - m;
      if (d > -INFINITY) { s0 += a.part_s0[o] * __expf(d); sT += a.part_sT[o] * __expf(d * invT); }
    }
    for (int off = 16; off > 0; off >>= 1) {
      s0 += __shfl_xor_sync(0xFFFFFFFFu, s0, off);
      sT += __shfl_xor_sync(0xFFFFFFFFu, sT, off);
    }
    if (lane == 0) {
      a.lse0[p] = m + logf(s0);
      a.lseT[p] = a.T > 0.f ? m * invT + logf(sT) : m + logf(s0);
    }
    merge_lists(a.part_topv, a.part_topi, nullptr, p, a.K, a.ntiles, a.Pcap, lane, a.top_tok + (size_t)p * a.K,
                a.top_logit + (size_t)p * a.K);
    if (a.T > 0.f) {
      merge_lists(a.part_keyv, a.part_keyi, a.part_keyl, p, a.K, a.ntiles, a.Pcap, lane,
                  a.draw_tok + (size_t)p * a.K, a.draw_logit + (size_t)p * a.K);
    } else {
      __syncwarp();
      for (int j = lane; j < a.K; j += 32) {
        a.draw_tok[(size_t)p * a.K + j] = a.top_tok[(size_t)p * a.K + j];
        a.draw_logit[(size_t)p * a.K + j] = a.top_logit[(size_t)p * a.K + j];
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
cudaError_t launch_score(const ts_ctx* ctx, const WsLayout& L, char* ws, const void* U, const void* A, const void* W,
                         int P, const int* P_dev, const int* p_req, const int* p_depth, const int* p_token,
                         const uint64_t* p_hash, float T, uint64_t seed, float* lse0, float* lseT, int* top_tok,
                         float* top_logit, int* draw_tok, float* draw_logit, cudaStream_t st) {
  const ts_config& c = ctx->cfg;
  ScoreArgs a{};
  a.U = U; a.A = A; a.W = W; a.V = c.V; a.D = c.D; a.r = c.r; a.K = c.K; a.P = P; a.P_dev = P_dev;
  a.p_req = p_req; a.p_depth = p_depth; a.p_token = p_token; a.p_hash = p_hash; a.T = T; a.seed = seed;
  a.TV = ctx->tile.TV; a.ntiles = ctx->tile.ntiles; a.Pcap = L.Pcap;
  a.part_m = (float*)(ws + L.part_m); a.part_s0 = (float*)(ws + L.part_s0); a.part_sT = (float*)(ws + L.part_sT);
  a.part_topv = (float*)(ws + L.part_topv); a.part_topi = (int*)(ws + L.part_topi);
  a.part_keyv = (float*)(ws + L.part_keyv); a.part_keyi = (int*)(ws + L.part_keyi); a.part_keyl = (float*)(ws + L.part_keyl);
  {
    ProfScope ps(ctx, K_SCORE, st);
    if (c.dt_U == TS_DTYPE_BF16)
      score_tile_kernel<__nv_bfloat16><<<a.ntiles, SCORE_THREADS, ctx->tile.smem, st>>>(a);
    else
      score_tile_kernel<float><<<a.ntiles, SCORE_THREADS, ctx->tile.smem, st>>>(a);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  MergeArgs m{};
  m.P = P; m.P_dev = P_dev; m.K = c.K; m.ntiles = a.ntiles; m.Pcap = L.Pcap; m.T = T;
  m.part_m = a.part_m; m.part_s0 = a.part_s0; m.part_sT = a.part_sT; m.part_topv = a.part_topv;
  m.part_keyv = a.part_keyv; m.part_keyl = a.part_keyl; m.part_topi = a.part_topi; m.part_keyi = a.part_keyi;
  m.lse0 = lse0; m.lseT = lseT; m.top_tok = top_tok; m.top_logit = top_logit; m.draw_tok = draw_tok; m.draw_logit = draw_logit;
  const int pmax = P_dev ? L.Pcap : P;
  int blocks = (pmax + 7) / 8;
  if (blocks > 4 * ctx->num_sms) blocks = 4 * ctx->num_sms;
  if (blocks < 1) blocks = 1;
  {
    ProfScope ps(ctx, K_MERGE, st);
    merge_kernel<<<blocks, 256, 0, st>>>(m);
  }
  return cudaGetLastError();
}

cudaError_t score_setup(ts_ctx* ctx) {
  cudaError_t e = cudaFuncSetAttribute(score_tile_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)ctx->tile.smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(score_tile_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->tile.smem);
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
  cudaError_t e = launch_score(ctx, L, (char*)ws, U, A, W, P, nullptr, parent_req, parent_depth, parent_token,
                               parent_hash, T, seed, lse0, lseT, top_tok, top_logit, draw_tok, draw_logit,
                               (cudaStream_t)stream);
  if (e != cudaSuccess) return set_cuda_error("ts_score_parents", e);
  return TS_OK;
}
