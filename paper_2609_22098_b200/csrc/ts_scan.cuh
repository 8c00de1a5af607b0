// The thread-private vocabulary scan shared by both scoring kernels, and the record it leaves per
// (vocabulary piece, parent).  A piece is the set of tokens one thread scanned for one parent: a whole
// tile in the FMA kernel, an interleaved subset of a tile's 16-token chunks in the tensor-core kernel.
#pragma once

#include "ts_common.cuh"

namespace ts {

// Record layout in 32-bit words: [m, s0, sT, counts, topv[K], topi[K], keyv[K], keyi[K], keyl[K]]
// counts = (#logit entries >= launch-wide bound at store time) | (#key entries >= bound) << 8
__host__ __device__ __forceinline__ int rec_words(int K) { return (4 + 5 * K + 3) & ~3; }  // 16-byte multiple

// Candidate lists of one (piece, parent): K best logits and K best sampling keys seen so far, both
// sorted descending.  Two holders with the same interface:
//   RegLists<8>  for K <= 8: fixed-size arrays that only ever see compile-time indices, so they stay in
//                registers and an insertion is a short predicated shift network;
//   MemLists     for K <= 16: dynamically indexed (local memory), insertion out of line.
template <int KR>
struct RegLists {
  // The lists always hold KR >= K entries (every index below is a compile-time constant, which is what
  // keeps them in registers); the pruning threshold is the KR-th entry, a little looser than the K-th
  // when K < KR, and the record keeps the first K.
  int K;
  float topv[KR]; int topi[KR];
  float keyv[KR]; int keyi[KR]; float keyl[KR];
  __device__ __forceinline__ void init(int K_) {
    K = K_;
#pragma unroll
    for (int i = 0; i < KR; ++i) { topv[i] = -INFINITY; topi[i] = -1; keyv[i] = -INFINITY; keyi[i] = -1; keyl[i] = 0.f; }
  }
  // Callers offer a value only when it beats the last entry.  Tokens arrive in increasing order within
  // a piece, so an equal value never displaces an earlier one.
  __device__ __forceinline__ float insert_top(float v, int tok) {
#pragma unroll
    for (int j = KR - 1; j >= 0; --j) {
      const bool up = (j > 0) && (v > topv[j > 0 ? j - 1 : 0]);   // entry j-1 moves down into j
      const bool here = !up && (j == KR - 1 || v > topv[j]);      // v lands in j
      if (up) { topv[j] = topv[j > 0 ? j - 1 : 0]; topi[j] = topi[j > 0 ? j - 1 : 0]; }
      else if (here) { topv[j] = v; topi[j] = tok; }
    }
    return topv[KR - 1];
  }
  __device__ __forceinline__ float insert_key(float key, int tok, float logit) {
#pragma unroll
    for (int j = KR - 1; j >= 0; --j) {
      const bool up = (j > 0) && (key > keyv[j > 0 ? j - 1 : 0]);
      const bool here = !up && (j == KR - 1 || key > keyv[j]);
      if (up) { keyv[j] = keyv[j > 0 ? j - 1 : 0]; keyi[j] = keyi[j > 0 ? j - 1 : 0]; keyl[j] = keyl[j > 0 ? j - 1 : 0]; }
      else if (here) { keyv[j] = key; keyi[j] = tok; keyl[j] = logit; }
    }
    return keyv[KR - 1];
  }
  // writes the first K entries; returns how many logit / key entries can still matter given the
  // launch-wide bounds (the lists are sorted, so those are prefixes)
  __device__ __forceinline__ int store(float* f, int* ii, float gL, float gK) const {
    int nt = 0, nk = 0;
#pragma unroll
    for (int j = 0; j < KR; ++j)
      if (j < K) {
        f[j] = topv[j]; ii[K + j] = topi[j]; f[2 * K + j] = keyv[j]; ii[3 * K + j] = keyi[j]; f[4 * K + j] = keyl[j];
        nt += (topi[j] >= 0 && topv[j] >= gL); nk += (keyi[j] >= 0 && keyv[j] >= gK);
      }
    return nt | (nk << 8);
  }
};

struct MemListsData {
  int K;
  float topv[KMAX]; int topi[KMAX];
  float keyv[KMAX]; int keyi[KMAX]; float keyl[KMAX];
};
static __device__ __noinline__ float mem_insert_top(MemListsData* L, float v, int tok) {
  const int K = L->K;
  int pos = K - 1;
  while (pos > 0 && v > L->topv[pos - 1]) { L->topv[pos] = L->topv[pos - 1]; L->topi[pos] = L->topi[pos - 1]; --pos; }
  L->topv[pos] = v; L->topi[pos] = tok;
  return L->topv[K - 1];
}
static __device__ __noinline__ float mem_insert_key(MemListsData* L, float key, int tok, float logit) {
  const int K = L->K;
  int pos = K - 1;
  while (pos > 0 && key > L->keyv[pos - 1]) {
    L->keyv[pos] = L->keyv[pos - 1]; L->keyi[pos] = L->keyi[pos - 1]; L->keyl[pos] = L->keyl[pos - 1]; --pos;
  }
  L->keyv[pos] = key; L->keyi[pos] = tok; L->keyl[pos] = logit;
  return L->keyv[K - 1];
}
struct MemLists {
  MemListsData d;
  __device__ __forceinline__ void init(int K_) {
    d.K = K_;
    for (int i = 0; i < KMAX; ++i) { d.topv[i] = -INFINITY; d.topi[i] = -1; d.keyv[i] = -INFINITY; d.keyi[i] = -1; d.keyl[i] = 0.f; }
  }
  __device__ __forceinline__ float insert_top(float v, int tok) { return mem_insert_top(&d, v, tok); }
  __device__ __forceinline__ float insert_key(float key, int tok, float logit) { return mem_insert_key(&d, key, tok, logit); }
  __device__ __forceinline__ int store(float* f, int* ii, float gL, float gK) const {
    const int K = d.K;
    int nt = 0, nk = 0;
    for (int j = 0; j < K; ++j) {
      f[j] = d.topv[j]; ii[K + j] = d.topi[j]; f[2 * K + j] = d.keyv[j]; ii[3 * K + j] = d.keyi[j]; f[4 * K + j] = d.keyl[j];
      nt += (d.topi[j] >= 0 && d.topv[j] >= gL); nk += (d.keyi[j] >= 0 && d.keyv[j] >= gK);
    }
    return nt | (nk << 8);
  }
};

// Thread-private running state of one parent over the tokens scanned so far.
template <class Lists>
struct RowScan {
  float m, s0, sT;
  float thrL, thrK;      // K-th best of this thread's own lists (-inf until they are full)
  float bestL, bestK;    // best logit / key this thread has published
  int K;
  Lists L;

  __device__ __forceinline__ void init(int K_) {
    K = K_; L.init(K_); m = -INFINITY; s0 = 0.f; sT = 0.f; thrL = -INFINITY; thrK = -INFINITY;
    bestL = -INFINITY; bestK = -INFINITY;
  }
  // one record, 16-byte aligned; the header's fourth word says how many list entries are worth reading
  __device__ __forceinline__ void store(float* rec, float gL, float gK) const {
    const int cnt = L.store(rec + 4, reinterpret_cast<int*>(rec) + 4, gL, gK);
    *reinterpret_cast<float4*>(rec) = make_float4(m, s0, sT, __int_as_float(cnt));
  }
};

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

__device__ __forceinline__ void publish(const SharedThr& g, float x) { atomicMax(g.slot + g.mine * SLOT_STRIDE, enc_f(x)); }

__device__ __forceinline__ unsigned slots_min(const SharedThr& g, int K) {
  unsigned m = __ldcg(g.slot);
  for (int j = 1; j < K; ++j) m = min(m, __ldcg(g.slot + j * SLOT_STRIDE));
  return m;
}

// low halves of the uniforms of the eight tokens around v: second generator stream, out of line because
// it runs for a few tokens per thousand once the bounds are warm
static __device__ __noinline__ uint4 fine_words(int v, uint64_t seed, int req, uint64_t hash) {
  return stream_words(seed, req, hash, STREAM_GUMBEL_FINE, (uint32_t)v >> 3);
}

// register-array element by run-time index (a select chain: the array stays in registers)
__device__ __forceinline__ float pick16(const float* a, int i) {
  float r = a[0];
#pragma unroll
  for (int j = 1; j < 16; ++j) r = (i == j) ? a[j] : r;
  return r;
}
__device__ __forceinline__ uint32_t pick8(const uint4& a, const uint4& b, int i) {
  uint32_t r = a.x;
  r = i == 1 ? a.y : r; r = i == 2 ? a.z : r; r = i == 3 ? a.w : r;
  r = i == 4 ? b.x : r; r = i == 5 ? b.y : r; r = i == 6 ? b.z : r; r = i == 7 ? b.w : r;
  return r;
}

// 2^x by the hardware approximation
__device__ __forceinline__ float ex2_approx(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
// index into the two noise-bound tables for the leading 16 bits of a uniform: by top byte, or, inside the top
// bucket, by the second byte
__device__ __forceinline__ uint32_t noise_bound_index(uint32_t c16) { return (c16 >> 8) != 255u ? (c16 >> 8) : 256u + (c16 & 255u); }

// One 16-token chunk of one parent: logits l[0..16) for tokens v0.., `valid` of them inside V.
// gL / gK: launch-wide lower bounds of the parent's K-th best logit / key as the caller last read them.
// The common case is branch-free: sums, then one bit per token saying whether it can still be a
// candidate; the few tokens whose bit is set are handled one at a time by a single copy of the code.
// Padded == true: the caller guarantees that l[i] is -infinity for every i >= valid (the tensor-core kernel
// does); the per-token range tests then fall away: -infinity loses every comparison and adds exp(-inf) = 0.
template <class Lists, bool Padded = false>
__device__ __forceinline__ void scan_chunk(RowScan<Lists>& st, const float* l, int v0, int valid, float T, float invT,
                                           uint64_t seed, int req, uint64_t hash, const float* ghi,
                                           float gL, float gK, const SharedThr& gl, const SharedThr& gk,
                                           const volatile unsigned* liveL = nullptr, const volatile unsigned* liveK = nullptr) {
  // High half of each token's uniform, one generator call per eight tokens.  Issued first and in the same
  // straight-line block as the sums below: the generator's long dependent chains and the exponentials'
  // latencies then overlap instead of following each other.
  uint4 cw0 = make_uint4(0, 0, 0, 0), cw1 = cw0;
  if (T > 0.f) {
    cw0 = stream_words(seed, req, hash, STREAM_GUMBEL_COARSE, (uint32_t)v0 >> 3);
    cw1 = stream_words(seed, req, hash, STREAM_GUMBEL_COARSE, ((uint32_t)v0 >> 3) + 1u);
  }
  float cm = -INFINITY;
  float gmax[4];   // best logit of each group of four tokens (the key gate below uses them again)
  if constexpr (Padded) {
#pragma unroll
    for (int sg = 0; sg < 4; ++sg) {
      gmax[sg] = fmaxf(fmaxf(l[4 * sg], l[4 * sg + 1]), fmaxf(l[4 * sg + 2], l[4 * sg + 3]));
      cm = fmaxf(cm, gmax[sg]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < CHUNK; ++i) if (i < valid) cm = fmaxf(cm, l[i]);
  }
  {
    // rescale to the new running maximum without a branch (no change: factor 1; first chunk: factor 0)
    const float nm = fmaxf(st.m, cm);
    const float d = (st.m == nm) ? 0.f : st.m - nm;
    st.s0 *= __expf(d);
    st.sT *= __expf(d * invT);
    st.m = nm;
  }
  float a0 = 0.f, aT = 0.f;
  const bool two = (T > 0.f) && (T != 1.f);
  if constexpr (Padded) {
    // exp(l - m) as ex2(l * log2(e) - m * log2(e)): one fused multiply-add and one ex2 per token.  While
    // nothing finite has been seen (m = -inf) the offset is 0: every l is -inf then and contributes 0.
    constexpr float LOG2E = 1.4426950408889634f;
    const float mref = st.m == -INFINITY ? 0.f : st.m;
    const float off0 = -mref * LOG2E, scT = LOG2E * invT, offT = off0 * invT;
#pragma unroll
    for (int i = 0; i < CHUNK; ++i) {
      a0 += ex2_approx(fmaf(l[i], LOG2E, off0));
      if (two) aT += ex2_approx(fmaf(l[i], scT, offT));
    }
  } else {
#pragma unroll
    for (int i = 0; i < CHUNK; ++i) {
      if (i < valid) {
        const float d = l[i] - st.m;
        a0 += __expf(d);
        if (two) aT += __expf(d * invT);
      }
    }
  }
  st.s0 += a0;
  st.sT += two ? aT : a0;
  // the chunk's best logit is a candidate for the top-K list (it is inserted further down): publishing it
  // right away costs nothing and gives the other pieces of the launch their first logit bounds early
  if (cm > st.bestL && cm > st.thrL && cm >= gL) { st.bestL = cm; publish(gl, cm); }
  if (T > 0.f) {
    const float thr = fmaxf(st.thrK, gK);
    uint32_t mk = 0;
    // The whole chunk first (padded chunks): its best logit plus the noise bound of the largest leading bits
    // among its sixteen tokens bounds every key in it.
    bool chunk_may = true;
    if constexpr (Padded) {
      const uint32_t m8 = __vmaxu2(__vmaxu2(__vmaxu2(cw0.x, cw0.y), __vmaxu2(cw0.z, cw0.w)),
                                   __vmaxu2(__vmaxu2(cw1.x, cw1.y), __vmaxu2(cw1.z, cw1.w)));
      const uint32_t c16all = max(m8 & 0xFFFFu, m8 >> 16);
      chunk_may = cm * invT + ghi[noise_bound_index(c16all)] >= thr && cm > -INFINITY;
    }
    // Four tokens at a time: their best logit plus the noise bound of their largest leading bits bounds
    // all four keys.  Only when that passes (a few groups per thousand) are the four looked at singly.
    if (chunk_may)
#pragma unroll
    for (int sg = 0; sg < 4; ++sg) {
      const uint4& cw = sg < 2 ? cw0 : cw1;
      const uint32_t wa = (sg & 1) ? cw.z : cw.x, wb = (sg & 1) ? cw.w : cw.y;
      const uint32_t m2 = __vmaxu2(wa, wb);
      const uint32_t c16m = max(m2 & 0xFFFFu, m2 >> 16);
      if constexpr (Padded) {
        const float gb = gmax[sg] * invT + ghi[noise_bound_index(c16m)];
        if (gb >= thr && gmax[sg] > -INFINITY) {   // (while no bound exists thr is -inf, and so is a padded group's gb)
#pragma unroll
          for (int i = 4 * sg; i < 4 * sg + 4; ++i) {
            const uint32_t word = word_of(i < 8 ? cw0 : cw1, (i & 7) >> 1);
            const uint32_t c16 = (word >> (16 * (i & 1))) & 0xFFFFu;
            const float bnd = l[i] * invT + ghi[noise_bound_index(c16)];
            mk |= (uint32_t)(bnd >= thr && l[i] > -INFINITY) << i;
          }
        }
      } else {
        const float lm = fmaxf(fmaxf(l[4 * sg], l[4 * sg + 1]), fmaxf(l[4 * sg + 2], l[4 * sg + 3]));
        const float gb = lm * invT + ((c16m >> 8) != 255u ? ghi[c16m >> 8] : ghi[256 + (c16m & 255u)]);
        if (4 * sg < valid && gb >= thr) {
#pragma unroll
          for (int i = 4 * sg; i < 4 * sg + 4; ++i) {
            const uint32_t word = word_of(i < 8 ? cw0 : cw1, (i & 7) >> 1);
            const uint32_t c16 = (word >> (16 * (i & 1))) & 0xFFFFu;
            const float bnd = l[i] * invT + ((c16 >> 8) != 255u ? ghi[c16 >> 8] : ghi[256 + (c16 & 255u)]);
            mk |= (uint32_t)(i < valid && bnd >= thr) << i;
          }
        }
      }
    }
    uint4 fw = make_uint4(0, 0, 0, 0);
    int fine_call = -1;
#pragma unroll 1
    while (mk) {
      const int i = __ffs(mk) - 1;
      mk &= mk - 1;
      const float li = pick16(l, i);
      const uint32_t c16 = (pick8(cw0, cw1, i >> 1) >> (16 * (i & 1))) & 0xFFFFu;
      if (liveK) {
        // the bounds may have risen since the mask was built (they do, steeply, while a launch warms up)
        gK = fmaxf(gK, dec_f(*liveK));
        const float bnd = li * invT + ((c16 >> 8) != 255u ? ghi[c16 >> 8] : ghi[256 + (c16 & 255u)]);
        if (bnd < fmaxf(st.thrK, gK)) continue;
      }
      if (fine_call != (i >> 3)) { fw = fine_words(v0 + i, seed, req, hash); fine_call = i >> 3; }
      const uint32_t fword = ((i & 7) >> 1) == 0 ? fw.x : (((i & 7) >> 1) == 1 ? fw.y : (((i & 7) >> 1) == 2 ? fw.z : fw.w));
      const float key = li * invT + gumbel_from_bits((c16 << 16) | ((fword >> (16 * (i & 1))) & 0xFFFFu));
      if (key > st.thrK && key >= gK) {
        st.thrK = st.L.insert_key(key, v0 + i, li);
        if (key > st.bestK) { st.bestK = key; publish(gk, key); }
      }
    }
  }
  // top-K logits, after the keys: in the first chunks of a launch the key section is the longer one and
  // the one whose published values the other pieces wait for.  A token below the launch-wide bound cannot
  // be among the parent's K best.
  if (liveL) gL = fmaxf(gL, dec_f(*liveL));
  if (cm > st.thrL && cm >= gL) {
    uint32_t mk = 0;
#pragma unroll
    for (int i = 0; i < CHUNK; ++i) mk |= (uint32_t)((Padded || i < valid) && l[i] > st.thrL && l[i] >= gL) << i;
#pragma unroll 1
    while (mk) {
      const int i = __ffs(mk) - 1;
      mk &= mk - 1;
      const float li = pick16(l, i);
      if (liveL) gL = fmaxf(gL, dec_f(*liveL));
      if (li > st.thrL && li >= gL) {
        st.thrL = st.L.insert_top(li, v0 + i);
        // publish at once: early in a launch every piece is waiting for the first bounds
        if (li > st.bestL) { st.bestL = li; publish(gl, li); }
      }
    }
  }
}

// Replication of parents over the 128 rows of a tensor-core tile when a level has few parents:
// with P <= 32 every parent occupies one row in each of the four 32-row quarters (R = 4), with
// P <= 64 one row in each half (R = 2); the copies split the tile's chunks between them.
__host__ __device__ __forceinline__ int mma_replicas(int P) { return P <= 32 ? 4 : (P <= 64 ? 2 : 1); }

}  // namespace ts
