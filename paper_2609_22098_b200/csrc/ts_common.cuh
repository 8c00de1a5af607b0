// Shared device/host pieces of the TreeSpark CUDA library: context, workspace layout, the
// counter-based generator, input loads and the per-thread vocabulary scan.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/treespark.h"

namespace ts {

constexpr int KMAX = TS_KMAX;
constexpr int DMAX = TS_DMAX;
constexpr int KNOTS = TS_CALIB_KNOTS;
constexpr int RMAX = 256;   // largest Markov rank r (the paper's head has r = 256)
// Programmatic dependent launch (the kernels of one expansion are chained with it).  pdl_wait(): everything
// the kernels before this one in the stream wrote is visible afterwards; a kernel launched without the
// attribute passes straight through.  pdl_launch_dependents(): the next kernel in the stream may start its
// own preamble now.  Every chained kernel waits before it lets its dependents go and before it exits, so
// a kernel that has passed its wait knows that ALL earlier kernels of the chain have completed.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Words between two pruning-bound slots: one 128-byte line each.  Every piece of a launch publishes into
// these words with atomicMax in the launch's first microseconds; packed together they queue up on a
// handful of L2 lines (measured: a third of the scoring launch at stride 1).
constexpr int SLOT_STRIDE = 32;
// Seed kernel: a parent's base-logit row is swept by up to SEED_PARTS_MAX CTAs when there are few parents;
// the parts of at most SEED_SPLIT_PARENTS parents meet in a scratch of NSEED_MAX candidates per part.
constexpr int SEED_PARTS_MAX = 16, SEED_SPLIT_PARENTS = 256, NSEED_MAX = 32;
constexpr size_t SEED_CAND_WORDS = (size_t)SEED_SPLIT_PARENTS * SEED_PARTS_MAX * NSEED_MAX * 2;
constexpr int UMMA_REQ = 32;         // requests whose base logits can ride through the tensor cores (rows of one extra B-operand slab)
constexpr int FEW_MAX = 8;           // levels with at most this many parents go to the few-parents scoring kernel
constexpr int SCORE_THREADS = 128;   // one parent per thread; every thread scans the CTA's whole tile
constexpr int CHUNK = 16;            // tokens per coarse generator call
constexpr int MMA_S = 4;             // column splits per tile in the tensor-core scoring kernel (scanning warps per row quarter)

enum Stream : uint32_t { STREAM_GUMBEL_COARSE = 1, STREAM_GUMBEL_FINE = 2, STREAM_ACCEPT = 3, STREAM_BONUS = 4 };

// ------------------------------------------------------------------------------------------------
// Context (host) and the device-visible part of it
// ------------------------------------------------------------------------------------------------
struct DevCalib {
  int mode;
  double a, b, lo, hi;
  const float* table;  // device [D][16]
};

struct TileCfg {
  int TV;       // tokens per vocabulary tile (multiple of 64)
  int ntiles;   // tiles covering V
  size_t smem;  // dynamic shared memory of the scoring kernel
  int umma;     // the tiling leaves room for the one-hot slab and the base-logit slab ring (base logits through the MMA)
  int w_ring;   // 0: the W tile is resident; > 0: that many 64-token slabs of W stream through a ring (large ranks)
};

}  // namespace ts

struct ts_ctx {
  ts_config cfg;
  float* d_table;
  int device;
  int num_sms;
  int cc_major;
  int max_smem;
  ts::TileCfg tile;
  int vt_TV, vt_n;  // vocabulary ranges of the verification walk, one per CTA
  int use_mma;      // 1: scoring runs on the tensor-core kernel, 0: on the fp32 FMA kernel
  int few_ok;       // 1: levels with <= FEW_MAX parents run on the few-parents kernel instead
  ts::DevCalib calib;
  void* prof;  // ts::Prof*, instrumentation state
  // tensor-map descriptor of the W matrix last scored with (bulk-tensor loads of the W tile); -1: the
  // driver's encoder is not available, the kernel stages W with plain loads
  alignas(64) unsigned char tmapW[128];
  const void* tmapW_ptr;
  alignas(64) unsigned char tmapU[128];   // tensor map of the base logits last expanded with ([request][depth][token] boxes)
  const void* tmapU_ptr; int tmapU_B;
  int tma_state;   // 0 not tried yet, 1 encoder found, -1 unavailable
  int walk_pdl;    // -1: the driver refused a cooperative launch with programmatic serialization
  int persist_pdl; // the same for the persistent expansion kernel
  unsigned ablation;   // TS_ABLATE_* switches (0 = the method)
  unsigned test_mode;  // TS_TEST_* switches (0 = the product's kernel selection and wait limits)
  uint32_t wait_limit; // polls before a bounded device-side wait gives up
};

namespace ts {

// ------------------------------------------------------------------------------------------------
// Workspace layout (bytes offsets into the caller's workspace), a function of (config, batch)
// ------------------------------------------------------------------------------------------------
struct WsLayout {
  int B, N, K, Pcap, ntiles, words;
  // scoring records, [ntiles * S][rec_cap][rec_words]
  size_t rec; int rec_cap;
  size_t err;            // int[4]: error word raised by a bounded wait inside the scoring kernel
  // merged per-parent results of the level being expanded, [Pcap] / [Pcap][K]
  size_t res_lse0, res_lseT, res_top_tok, res_top_logit, res_draw_tok, res_draw_logit;
  // level parent lists (two, alternating) [Pcap]
  size_t lst_req[2], lst_depth[2], lst_token[2], lst_hash[2], lst_slot[2];
  size_t lvl_count;      // int[DMAX + 2]
  size_t ex_barrier;     // unsigned[4]: grid barrier of the persistent expansion kernel
  size_t utop;           // uint2[B][D][ntiles]: best base logit (value, token) of every vocabulary tile of every row
  // per-request pool, [B][N]
  size_t pl_alive, pl_depth, pl_parent, pl_sib, pl_tok, pl_lidx, pl_new, pl_logkey, pl_logS, pl_q0, pl_logqT,
      pl_lseT, pl_hash, pl_path;
  size_t root_lseT;      // float[B]
  size_t req_npar, req_base;  // int[B]: parents of the request in the current level list and their base index
  size_t req_nscored;    // int[B]
  // candidates of one level, [B][N*K]
  size_t cd_valid, cd_parent, cd_sib, cd_tok, cd_logkey, cd_logS, cd_q0, cd_logqT, cd_rank;
  // verification
  size_t z_max, z_arg, z_lse;            // per Z row, [B*(N+1)]
  size_t vf_state;                       // VerifyState[B]
  size_t vf_part;                        // float[B][ntiles]
  size_t vf_barrier;                     // unsigned[4]
  size_t vf_child;                       // int[2][B][N+1]: first child and child count of every node
  size_t vf_lists;                       // int[2][B] reduction list, int[2][B] rescan list, int[8] counters
  size_t vf_edge;                        // double[3][B][N]: per edge p(x), q(x) and the accept uniform
  size_t total;
};

__host__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct VerifyState {
  int cur;        // current node (-1 = root)
  int j;          // next sibling to test
  int acc;        // accepted so far
  int need;       // 0 none, 1 residual pass, 2 in-tile CDF scan, 3 finished
  int nf;         // tested (frozen) siblings at the current node
  int scan_tile;  // tile holding the bonus token
  int row_node;   // node whose rows the pass reads
  int result;     // token found by the range rescan
  int npass;      // vocabulary reductions this request has asked for
  int cfirst, ccnt;  // first child and child count of the current node (saves the walk a dependent load)
  int pad_;
  double C, Zj, Qused, target, before;
  double passC;   // C of the requested pass
  double partsC;  // C the stored range sums were computed for (-1 = none)
  int fx[KMAX];
  double fC[KMAX];
  double fp[KMAX], fq[KMAX];
};

// Bytes of the scoring records for `cap` parent slots: one record per (tile, slot) of the tile kernels,
// and room for the few-parents kernel's records (one per 256-token tile and parent, at most FEW_MAX
// parents), whichever is larger.
__host__ inline size_t record_bytes(const ts_ctx* ctx, int cap) {
  const size_t rw = (4 + 5 * (size_t)ctx->cfg.K + 3) & ~(size_t)3;
  const size_t tile = (size_t)ctx->tile.ntiles * (size_t)cap;
  const size_t few = (size_t)((ctx->cfg.V + 255) / 256) * FEW_MAX;
  return align_up((tile > few ? tile : few) * rw * sizeof(float), 256);
}

__host__ inline WsLayout make_layout(const ts_ctx* ctx, int B) {
  WsLayout L{};
  const ts_config& c = ctx->cfg;
  L.B = B; L.N = c.Nmax; L.K = c.K; L.Pcap = B * c.Nmax > B ? B * c.Nmax : B; L.ntiles = ctx->tile.ntiles;
  L.words = (c.Nmax + 63) / 64;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t P = (size_t)L.Pcap, K = (size_t)c.K, N = (size_t)c.Nmax, b = (size_t)B;
  {
    int cap = (L.Pcap + 7) / 8 * 8;
    if (ctx->use_mma) cap = (L.Pcap + 127) / 128 * 128;
    L.rec_cap = cap;
    L.rec = take(record_bytes(ctx, cap) + ((size_t)cap * (4 + 2 * K * SLOT_STRIDE) + SEED_SPLIT_PARENTS + SEED_CAND_WORDS) * 4);
    L.err = take(16);
  }
  L.res_lse0 = take(P * 4); L.res_lseT = take(P * 4);
  L.res_top_tok = take(P * K * 4); L.res_top_logit = take(P * K * 4);
  L.res_draw_tok = take(P * K * 4); L.res_draw_logit = take(P * K * 4);
  for (int i = 0; i < 2; ++i) {
    L.lst_req[i] = take(P * 4); L.lst_depth[i] = take(P * 4); L.lst_token[i] = take(P * 4);
    L.lst_hash[i] = take(P * 8); L.lst_slot[i] = take(P * 4);
  }
  L.lvl_count = take((DMAX + 2) * 4);
  L.ex_barrier = take(64);
  L.utop = take(b * (size_t)c.D * (size_t)ctx->tile.ntiles * 8);
  L.pl_alive = take(b * N * 4); L.pl_depth = take(b * N * 4); L.pl_parent = take(b * N * 4);
  L.pl_sib = take(b * N * 4); L.pl_tok = take(b * N * 4); L.pl_lidx = take(b * N * 4); L.pl_new = take(b * N * 4);
  L.pl_logkey = take(b * N * 8); L.pl_logS = take(b * N * 8); L.pl_q0 = take(b * N * 4);
  L.pl_logqT = take(b * N * 4); L.pl_lseT = take(b * N * 4); L.pl_hash = take(b * N * 8); L.pl_path = take(b * N * 8);
  L.root_lseT = take(b * 4);
  L.req_npar = take(b * 4); L.req_base = take(b * 4); L.req_nscored = take(b * 4);
  const size_t NK = N * K;
  L.cd_valid = take(b * NK * 4); L.cd_parent = take(b * NK * 4); L.cd_sib = take(b * NK * 4);
  L.cd_tok = take(b * NK * 4); L.cd_logkey = take(b * NK * 8); L.cd_logS = take(b * NK * 8);
  L.cd_q0 = take(b * NK * 4); L.cd_logqT = take(b * NK * 4); L.cd_rank = take(b * NK * 4);
  const size_t rows = b * (N + 1);
  L.z_max = take(rows * 4); L.z_arg = take(rows * 4); L.z_lse = take(rows * 4);
  L.vf_state = take(b * sizeof(VerifyState));
  L.vf_part = take(b * (size_t)ctx->vt_n * 4);
  L.vf_barrier = take(64);
  L.vf_child = take(2 * b * (N + 1) * 4);
  L.vf_lists = take((4 * b + 8) * 4);
  L.vf_edge = take(3 * b * N * 8);
  L.total = off;
  return L;
}

// ------------------------------------------------------------------------------------------------
// Counter-based random numbers (Philox4x32-10) and the path hash
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                               uint32_t k1) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint4 stream_words(uint64_t seed, int req, uint64_t hash, uint32_t stream, uint32_t index) {
  return philox4x32_10(index, (uint32_t)hash, (uint32_t)(hash >> 32), ((uint32_t)req & 0xFFFFFFu) | (stream << 24),
                       (uint32_t)seed, (uint32_t)(seed >> 32));
}

__host__ __device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__host__ __device__ __forceinline__ uint64_t path_hash(uint64_t parent_hash, int token) {
  return splitmix64(parent_hash ^ (((uint64_t)(uint32_t)token + 1ull) * 0x9E3779B97F4A7C15ull));
}

__device__ __forceinline__ uint32_t word_of(const uint4& w, int i) {
  return i == 0 ? w.x : (i == 1 ? w.y : (i == 2 ? w.z : w.w));
}

// uniform in (0,1) from a 32-bit word, in double (scalar uses only)
__device__ __forceinline__ double u01(uint32_t x) { return ((double)x + 0.5) * (1.0 / 4294967296.0); }

// Gumbel noise -log(-log u) for u = (X + 0.5) / 2^32, accurate in fp32 over the whole range: near
// u = 1 the complement 1-u is formed exactly from the integer.
__device__ __forceinline__ float gumbel_from_bits(uint32_t X) {
  // absolute error of the fast logarithm is ~1e-7 * |log2 x|: a few 1e-6 on the key at most, far
  // inside the near-tie margin the parity tests use; log1pf keeps the u -> 1 end exact
  float a;
  if (X >= 0x80000000u) {
    const float t = ((float)(0xFFFFFFFFu - X) + 0.5f) * 2.3283064365386963e-10f;
    a = -log1pf(-t);
  } else {
    const float u = ((float)X + 0.5f) * 2.3283064365386963e-10f;
    a = -__logf(u);
  }
  return -__logf(a);
}

// ------------------------------------------------------------------------------------------------
// Input element loads
// ------------------------------------------------------------------------------------------------
template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int VEC = 4;  // elements per 16-byte load
  __device__ static __forceinline__ float to_f(float x) { return x; }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int VEC = 8;
  __device__ static __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
};

// 16 consecutive elements starting at p (p 16-byte aligned when `vec`), as floats
template <typename T>
__device__ __forceinline__ void load16(const T* p, bool vec, int valid, float* out);

template <>
__device__ __forceinline__ void load16<float>(const float* p, bool vec, int valid, float* out) {
  if (vec && valid >= 16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(p) + i);
      out[4 * i] = v.x; out[4 * i + 1] = v.y; out[4 * i + 2] = v.z; out[4 * i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) out[i] = i < valid ? __ldg(p + i) : 0.f;
  }
}

__device__ __forceinline__ void unpack_bf16x8(const uint4& v, float* out) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

template <>
__device__ __forceinline__ void load16<__nv_bfloat16>(const __nv_bfloat16* p, bool vec, int valid, float* out) {
  if (vec && valid >= 16) {
    const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(p));
    const uint4 v1 = __ldg(reinterpret_cast<const uint4*>(p) + 1);
    unpack_bf16x8(v0, out);
    unpack_bf16x8(v1, out + 8);
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) out[i] = i < valid ? __bfloat162float(p[i]) : 0.f;
  }
}

// ------------------------------------------------------------------------------------------------
// Calibrated edge estimate (Eq. 3 or the per-depth table), scalar, in double
// ------------------------------------------------------------------------------------------------
// log p_hat for a child with logit lx under a parent with log-normaliser lse0 (depth d = parent depth)
__device__ __forceinline__ double log_phat(const DevCalib& c, int d, double lx, double lse0) {
  const double lq = lx - lse0;
  double q = exp(lq);
  if (q > 1.0 - 1e-12) q = 1.0 - 1e-12;
  double t = lq - log1p(-q);
  // non-finite logits (reported per request as TS_ERR_NUMERIC) must not reach the table lookup below: a NaN
  // position passes both range tests and its integer part is not a usable index
  if (!(t == t)) return t;
  t = t > 30.0 ? 30.0 : (t < -30.0 ? -30.0 : t);
  if (c.mode == 0) {
    const double x = c.a * t + c.b;
    return x >= 0 ? -log1p(exp(-x)) : x - log1p(exp(x));
  }
  const float* y = c.table + d * KNOTS;
  const double pos = (t - c.lo) / (c.hi - c.lo) * (KNOTS - 1);
  double v;
  if (pos <= 0.0) v = y[0];
  else if (pos >= KNOTS - 1) v = y[KNOTS - 1];
  else {
    int i = (int)floor(pos);
    i = i < 0 ? 0 : (i > KNOTS - 2 ? KNOTS - 2 : i);
    const double f = pos - i;
    v = (double)y[i] + f * ((double)y[i + 1] - (double)y[i]);
  }
  return log(v);
}

// ------------------------------------------------------------------------------------------------
// Bounded grid barrier for cooperative (co-resident) launches: counter + generation in global memory.
// Returns false when the wait ran out; the caller must then stop using the barrier and exit.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool grid_barrier(unsigned* bar, unsigned nblocks, unsigned& gen, unsigned limit = 1u << 22) {
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned target = (gen + 1) * nblocks;
    atomicAdd(&bar[0], 1u);
    unsigned spins = 0;
    while (*((volatile unsigned*)&bar[0]) < target) {
      if (*((volatile unsigned*)&bar[1]) != 0u) { ok = false; break; }
      if (++spins > limit) { atomicExch(&bar[1], 1u); ok = false; break; }
      if (spins > 256u) __nanosleep(32);
    }
    __threadfence();
  }
  gen++;
  ok = __syncthreads_and((int)ok) != 0;
  return ok;
}

}  // namespace ts
