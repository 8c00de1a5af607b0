// The thread-private vocabulary scan shared by both scoring kernels, and the record it leaves per
// (vocabulary piece, parent).  A piece is the set of tokens one thread scanned for one parent: a whole
// tile in the FMA kernel, an interleaved subset of a tile's 16-token chunks in the tensor-core kernel.
#pragma once

#include "ts_common.cuh"

namespace ts {

// Record layout in 32-bit words: [m, s0, sT, pad, topv[K], topi[K], keyv[K], keyi[K], keyl[K]]
__host__ __device__ __forceinline__ int rec_words(int K) { return (4 + 5 * K + 3) & ~3; }  // 16-byte multiple

// Candidate lists of one (piece, parent): K best logits and K best sampling keys seen so far, both
// sorted descending.  They are indexed dynamically, so they live in local memory; everything that
// touches them sits in the out-of-line functions below, which keeps the hot loop small.
struct RowLists {
  int K;
  float topv[KMAX]; int topi[KMAX];
  float keyv[KMAX]; int keyi[KMAX]; float keyl[KMAX];
};

// Thread-private running state of one parent over the tokens scanned so far.
struct RowScan {
  float m, s0, sT;
  float thrL, thrK;      // K-th best of this thread's own lists (-inf until they are full)
  float gL, gK;          // launch-wide lower bounds of the parent's K-th best logit / key, as last read
  float bestL, bestK;    // best logit / key this thread has published
  RowLists L;

  __device__ __forceinline__ void init(int K_) {
    L.K = K_; m = -INFINITY; s0 = 0.f; sT = 0.f; thrL = -INFINITY; thrK = -INFINITY;
    gL = -INFINITY; gK = -INFINITY; bestL = -INFINITY; bestK = -INFINITY;
    for (int i = 0; i < KMAX; ++i) { L.topv[i] = -INFINITY; L.topi[i] = -1; L.keyv[i] = -INFINITY; L.keyi[i] = -1; L.keyl[i] = 0.f; }
  }
  // one record, 16-byte aligned
  __device__ __forceinline__ void store(float* rec) const {
    float4* r4 = reinterpret_cast<float4*>(rec);
    r4[0] = make_float4(m, s0, sT, 0.f);
    float* f = rec + 4;
    int* ii = reinterpret_cast<int*>(rec) + 4;
    const int K = L.K;
    for (int j = 0; j < K; ++j) {
      f[j] = L.topv[j]; ii[K + j] = L.topi[j]; f[2 * K + j] = L.keyv[j]; ii[3 * K + j] = L.keyi[j]; f[4 * K + j] = L.keyl[j];
    }
  }
};

// Insert into the logit list; returns the list's new K-th value.  Tokens arrive in increasing order
// within a piece, so an equal value never displaces an earlier entry.
static __device__ __noinline__ float insert_top(RowLists* L, float v, int tok) {
  const int K = L->K;
  int pos = K - 1;
  while (pos > 0 && v > L->topv[pos - 1]) { L->topv[pos] = L->topv[pos - 1]; L->topi[pos] = L->topi[pos - 1]; --pos; }
  L->topv[pos] = v; L->topi[pos] = tok;
  return L->topv[K - 1];
}

// Upper bound of the Gumbel noise -log(-log u) given only the leading bits of the 32-bit uniform, with
// a safety margin so that the bound never prunes a token the exact key would keep.  Table 0 is indexed
// by the top byte; for the top bucket (byte 255, where the noise is unbounded as u -> 1) table 1 is
// indexed by the second byte.
__device__ __forceinline__ float gumbel_bound_for_byte(int c, int level) {
  const uint32_t hi = level == 0 ? (((uint32_t)c << 24) | 0xFFFFFFu) : (0xFF000000u | ((uint32_t)c << 16) | 0xFFFFu);
  const double u = ((double)hi + 0.5) * (1.0 / 4294967296.0);
  const double g = -log(-log(u));
  return (float)(g + 1e-4 * fabs(g) + 1e-4);
}
// both tables, 512 floats: ghi[0..256) by top byte, ghi[256..512) by second byte within the top bucket
__device__ __forceinline__ void fill_gumbel_bounds(float* ghi, int tid, int nthreads) {
  for (int c = tid; c < 512; c += nthreads) ghi[c] = gumbel_bound_for_byte(c & 255, c >> 8);
}

// Order-preserving map float -> unsigned (0 is below every float), so that atomicMax works on floats.
__device__ __forceinline__ unsigned enc_f(float f) {
  const unsigned b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float dec_f(unsigned e) {
  if (e == 0u) return -INFINITY;
  return __uint_as_float((e & 0x80000000u) ? (e & 0x7FFFFFFFu) : ~e);
}

// Launch-wide pruning state of one parent: K slots, slot j holding the best value published by the
// pieces whose id is j modulo K.  Different slots therefore hold values of different tokens, and the
// minimum over the slots is a lower bound of the parent's K-th best value; a token strictly below it
// cannot be among the K best.  Publishing is one atomicMax, reading is K words.
struct SharedThr {
  unsigned* slot;   // [K], order-preserving encoding, 0 = nothing published
  int mine;         // this piece's slot
};

__device__ __forceinline__ void publish(const SharedThr& g, float x) { atomicMax(g.slot + g.mine, enc_f(x)); }

__device__ __forceinline__ unsigned slots_min(const SharedThr& g, int K) {
  unsigned m = __ldcg(g.slot);
  for (int j = 1; j < K; ++j) m = min(m, __ldcg(g.slot + j));
  return m;
}

// Exact sampling key of one token (low half of its uniform from the second generator stream) and, if
// it beats both bounds, insertion into the key list.  Returns (new K-th key of the list, the key if
// inserted else -inf).  Out of line: it runs for a few tokens per thousand once the bounds are warm.
static __device__ __noinline__ float2 key_exact(RowLists* L, float base, float logit, uint32_t c16, int v, uint64_t seed,
                                         int req, uint64_t hash, float thrK, float gK) {
  const uint4 fw = stream_words(seed, req, hash, STREAM_GUMBEL_FINE, (uint32_t)v >> 3);
  const uint32_t f16 = (word_of(fw, (v & 7) >> 1) >> (16 * (v & 1))) & 0xFFFFu;
  const float key = base + gumbel_from_bits((c16 << 16) | f16);
  if (!(key > thrK && key >= gK)) return make_float2(thrK, -INFINITY);
  const int K = L->K;
  int pos = K - 1;
  while (pos > 0 && key > L->keyv[pos - 1]) {
    L->keyv[pos] = L->keyv[pos - 1]; L->keyi[pos] = L->keyi[pos - 1]; L->keyl[pos] = L->keyl[pos - 1]; --pos;
  }
  L->keyv[pos] = key; L->keyi[pos] = v; L->keyl[pos] = logit;
  return make_float2(L->keyv[K - 1], key);
}

// One 16-token chunk of one parent: logits l[0..16) for tokens v0.., `valid` of them inside V.
__device__ __forceinline__ void scan_chunk(RowScan& st, const float* l, int v0, int valid, float T, float invT,
                                           uint64_t seed, int req, uint64_t hash, const float* ghi,
                                           const SharedThr& gl, const SharedThr& gk) {
  const int K = st.L.K;
  // launch-wide bounds: loads issued first, consumed after the sums below
  const unsigned rdL = slots_min(gl, K);
  const unsigned rdK = T > 0.f ? slots_min(gk, K) : 0u;
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
  st.gL = fmaxf(st.gL, dec_f(rdL));
  st.gK = fmaxf(st.gK, dec_f(rdK));
  // top-K logits: a token below the launch-wide bound cannot be among the parent's K best
  if (cm > st.thrL && cm >= st.gL) {
#pragma unroll
    for (int i = 0; i < CHUNK; ++i)
      if (i < valid && l[i] > st.thrL && l[i] >= st.gL) st.thrL = insert_top(&st.L, l[i], v0 + i);
    if (cm > st.bestL) { st.bestL = cm; publish(gl, cm); }
  }
  if (T > 0.f) {
    // high half of each token's uniform: one generator call per eight tokens
    const uint4 cw0 = stream_words(seed, req, hash, STREAM_GUMBEL_COARSE, (uint32_t)v0 >> 3);
    const uint4 cw1 = stream_words(seed, req, hash, STREAM_GUMBEL_COARSE, ((uint32_t)v0 >> 3) + 1u);
    float kmax = -INFINITY;
#pragma unroll
    for (int i = 0; i < CHUNK; ++i) {
      if (i < valid) {
        const uint32_t word = word_of(i < 8 ? cw0 : cw1, (i & 7) >> 1);
        const uint32_t c16 = (word >> (16 * (i & 1))) & 0xFFFFu;
        const float base = l[i] * invT;
        // the leading bits bound the noise from above; almost every token stops here
        const float bnd = base + ((c16 >> 8) != 255u ? ghi[c16 >> 8] : ghi[256 + (c16 & 255u)]);
        if (bnd > st.thrK && bnd >= st.gK) {
          const float2 r = key_exact(&st.L, base, l[i], c16, v0 + i, seed, req, hash, st.thrK, st.gK);
          st.thrK = r.x;
          kmax = fmaxf(kmax, r.y);
        }
      }
    }
    if (kmax > st.bestK) { st.bestK = kmax; publish(gk, kmax); }
  }
}

// Replication of parents over the 128 rows of a tensor-core tile when a level has few parents:
// with P <= 32 every parent occupies one row in each of the four 32-row quarters (R = 4), with
// P <= 64 one row in each half (R = 2); the copies split the tile's chunks between them.
__host__ __device__ __forceinline__ int mma_replicas(int P) { return P <= 32 ? 4 : (P <= 64 ? 2 : 1); }

}  // namespace ts
