// Tensor-core scoring kernel for sm_100a: the low-rank bias [parents x r] . [r x tile] runs on the
// 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory), and the vocabulary scan
// (add base logits, online max / sum-exp, top-K, Gumbel top-K) is its epilogue, one tensor-memory
// lane = one parent row per thread.
//
// CTA = one vocabulary tile, resident for the whole launch.  Shared memory holds
//   W tile  : B operand, MN-major, 128-byte swizzle: slabs of 64 tokens, slab = [rp rows][128 B];
//             loaded by bulk-tensor copies (one mbarrier per 128-token block), or by plain loads when
//             no tensor map could be encoded
//   A tile  : A operand, K-major, 128-byte swizzle: [rp/64 slabs][128 rows][128 B] (gathered rows A[x_p])
// (rp = r rounded up to 64, padding zero-filled).  Warps 0..7 are epilogue warps: warp w reads the
// tensor-memory lanes 32*(w%4).. (its quarter of the 128 parent rows).  When a level has few parents the
// rows are replicated R = 2 or 4 times over the quarters; of the tile's 16-token chunks, chunk cg belongs
// to replica cg % R and column split (cg / R) % 2 (= w / 4).  Warp 8 allocates tensor memory and its
// lane 0 issues the MMAs: per block of 128 tokens rp/16 instructions of M=128, N=128 (64 at a ragged
// end), K=16 into one of four 128-column accumulator buffers, then a commit that arrives on that
// buffer's "full" barrier; epilogue warps arrive on its "empty" barrier when they have drained it.
// Warp 9 keeps shared-memory copies of the launch-wide pruning bounds of every row current.
// Every wait is bounded: when one runs out the kernel raises an error word, skips the remaining work,
// waits (again bounded) for bulk loads still in flight, frees its tensor memory and returns.
#include "ts_tc.cuh"
#include "ts_internal.h"
namespace ts {
#ifdef TS_DEBUG_TIMING
// developer aid: per-CTA timestamps (globaltimer ns) of the phases of one launch
__device__ unsigned long long g_dbg[148 * 64];
__device__ __forceinline__ unsigned long long gtime() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define DBG(slot) do { if ((threadIdx.x & 31) == 0 && blockIdx.x < 148) g_dbg[blockIdx.x * 64 + (slot)] = gtime(); } while (0)
#define TS_SCAN_MARK(n) do { if (threadIdx.x == 0 && blockIdx.x < 148 && g_dbg[blockIdx.x * 64 + 56 + (n)] == 0ull) g_dbg[blockIdx.x * 64 + 56 + (n)] = gtime(); } while (0)
#else
#define DBG(slot) do { } while (0)
#endif

}  // namespace ts
#include "ts_scan.cuh"

namespace ts {

constexpr int EPI_WARPS = 4 * MMA_S;
constexpr int MMA_THREADS = (EPI_WARPS + 2) * 32;   // epilogue warps, the MMA warp, the bounds-refresh warp
constexpr int BLK_N = 128;
constexpr int NBUF = 4;                 // accumulator buffers of BLK_N columns in tensor memory
constexpr uint32_t TMEM_COLS = NBUF * BLK_N;
constexpr int MAX_BLK = 32;             // blocks of BLK_N tokens in the largest tile (4096 tokens)

template <class Lists>
__global__ void __launch_bounds__(MMA_THREADS, 1) score_mma_kernel(const ScoreArgs a, const __grid_constant__ CUtensorMap tmW, const int use_tma) {
  extern __shared__ unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // The preamble below (shared-memory carve-up, tensor-memory allocation, barriers, bulk loads of W, noise
  // table) reads nothing an earlier kernel of the stream wrote, so in a chained launch it runs while the
  // previous kernel is still finishing.  When the level before this one was empty, this one is too.
  if (a.P_prev_dev && *a.P_prev_dev <= 0) { pdl_wait(); return; }

  const int r = a.r, rp = (r + 63) / 64 * 64, V = a.V, TV = a.TV, K = a.K;
  const int tile = blockIdx.x, t0 = tile * TV, tlen = min(TV, V - t0);
  const int nslab = TV / 64;
  const int nblk_w = (tlen + BLK_N - 1) / BLK_N;
  const uint32_t slab_bytes = (uint32_t)rp * 128u;       // one 64-token slab of W
  const uint32_t a_slab_bytes = 128u * 128u;             // 128 rows x 128 B
  unsigned char* sm = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* Ws = sm;
  unsigned char* As = Ws + (size_t)nslab * slab_bytes;
  float* ghi = reinterpret_cast<float*>(As + (size_t)(rp / 64) * a_slab_bytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(ghi + 512);
  uint64_t* a_full = bars;            // epilogue threads -> MMA: the A tile of this group is in place
  uint64_t* t_full = bars + 1;             // [NBUF] MMA -> epilogue: accumulator buffer written
  uint64_t* t_empty = bars + 1 + NBUF;     // [NBUF] epilogue -> MMA: accumulator buffer drained
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 + 2 * NBUF);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  // per-row copies of the launch-wide pruning bounds (logit, key), refreshed once per block of tokens
  volatile unsigned* s_thr = reinterpret_cast<volatile unsigned*>(s_tmem + 4);   // [group parity][2][128]
  volatile int* s_done = reinterpret_cast<volatile int*>(s_tmem + 2);             // epilogue warps finished
  uint64_t* w_full = reinterpret_cast<uint64_t*>(const_cast<unsigned*>(s_thr) + 512);   // [MAX_BLK] W slabs of block nb landed

  const __nv_bfloat16* Wg = reinterpret_cast<const __nv_bfloat16*>(a.W);
  const __nv_bfloat16* Ug = reinterpret_cast<const __nv_bfloat16*>(a.U);
  const __nv_bfloat16* Ag = reinterpret_cast<const __nv_bfloat16*>(a.A);

  // ---- set-up ------------------------------------------------------------------------------------
  if (warp == 0) DBG(0);
  if (warp == EPI_WARPS) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const bool early_w = !a.P_prev_dev || *a.P_prev_dev >= 16;
  auto issue_w = [&]() {   // one thread
    for (int nb = 0; nb < nblk_w; ++nb) {
      const int ns = (tlen - nb * BLK_N > 64) ? 2 : 1;
      mbar_expect_tx(w_full + nb, (uint32_t)ns * slab_bytes);
      for (int h = 0; h < ns; ++h)
        tma_load_box(Ws + (size_t)(2 * nb + h) * slab_bytes, &tmW, t0 + (2 * nb + h) * 64, 0, w_full + nb);
    }
  };
  if (tid == 0) {
    mbar_init(a_full, EPI_WARPS * 32);
    for (int i = 0; i < NBUF; ++i) { mbar_init(t_full + i, 1); mbar_init(t_empty + i, EPI_WARPS); }
    *s_abort = 0;
    *s_done = 0;
    if (use_tma) for (int i = 0; i < nblk_w; ++i) mbar_init(w_full + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // W tile by bulk-tensor loads, one barrier per block of 128 tokens so that the first MMAs start while
    // the rest of the tile is still in flight; tokens past V and rows past r arrive as zeros.  Issued here,
    // before the kernel may look at its own parent count, when the level before was large enough for this
    // one to be populated almost surely; after the count is known otherwise (a level that turns out empty then
    // fetches nothing).
    if (use_tma && early_w) issue_w();
  }
  if (!use_tma) {  // W tile: 16-byte chunks (8 tokens of one row), swizzled: chunk j of row k lands at chunk j ^ (k & 7)
    const int per_slab = rp * 8;
    for (int idx = tid; idx < nslab * per_slab; idx += MMA_THREADS) {
      const int slab = idx / per_slab, rem = idx % per_slab, k = rem >> 3, j = rem & 7;
      const int tok = t0 + slab * 64 + j * 8;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (k < r && tok < V) v = __ldg(reinterpret_cast<const uint4*>(Wg + (size_t)k * V + tok));
      *reinterpret_cast<uint4*>(Ws + (size_t)slab * slab_bytes + k * 128 + ((j ^ (k & 7)) << 4)) = v;
    }
  }
  if (warp == 0) DBG(1);
  fill_gumbel_bounds(ghi, tid, MMA_THREADS);
  for (int i = tid; i < 512; i += MMA_THREADS) s_thr[i] = 0u;
  if (warp == 0) DBG(2);
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  if (warp == 0) DBG(3);
  pdl_wait();                // parent lists and the level's parent count come from the previous kernel
  pdl_launch_dependents();
  const int P = a.P_dev ? *a.P_dev : a.P;   // may be 0: an empty level only tears down
  if (use_tma && !early_w && P > 0 && tid == 0) issue_w();

  const int R = mma_replicas(P), rsh = R == 4 ? 2 : (R == 2 ? 1 : 0);
  const int ngroups = P <= 0 ? 0 : (R > 1 ? 1 : (P + 127) / 128);
  const int nblk = (tlen + BLK_N - 1) / BLK_N;
  const float T = a.T, invT = T > 0.f ? 1.f / T : 1.f;
  const int rw = rec_words(K);

  if (warp < EPI_WARPS) {
    // ======================= epilogue warps =======================================================
    const int q = warp & 3, s = warp >> 2;
    const int row = q * 32 + lane;
    const int e = warp * 32 + lane;  // 0..255
    const int cpr = rp / 8;          // 16-byte chunks per A row
    bool alive = true;
    for (int g = 0; g < ngroups && alive; ++g) {
      // gather this group's parent rows A[x_p] into the swizzled A tile
      for (int idx = e; idx < 128 * cpr; idx += EPI_WARPS * 32) {
        const int rr = idx / cpr, ck = idx % cpr;
        const int p = R > 1 ? rr % (128 / R) : g * 128 + rr;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (p < P && ck * 8 < r) v = __ldg(reinterpret_cast<const uint4*>(Ag + (size_t)a.p_token[p] * r + ck * 8));
        *reinterpret_cast<uint4*>(As + (size_t)(ck >> 3) * a_slab_bytes + rr * 128 + (((ck & 7) ^ (rr & 7)) << 4)) = v;
      }
      fence_async_smem();
      mbar_arrive(a_full);
      if (warp == 0) DBG(4);

      const int p = R > 1 ? row % (128 / R) : g * 128 + row;
      const int rho = R > 1 ? row / (128 / R) : 0;   // uniform within a warp (128/R is a multiple of 32)
      const bool active = p < P;
      int req = 0; uint64_t hash = 0; const __nv_bfloat16* Urow = Ug;
      if (active) {
        req = a.p_req[p]; hash = a.p_hash[p];
        Urow = Ug + ((size_t)req * a.D + a.p_depth[p]) * V;
      }
      RowScan<Lists> st;
      st.init(K);
      // where this parent's cached bounds live: rows of group g use the buffer of parity g & 1.  That
      // buffer last served group g-2; the refresh warp is at group g-1 or g by now (every warp has
      // passed the A-tile barrier of g-1), so clearing it here cannot be overwritten with stale values.
      const int prow = (g & 1) * 256 + (R > 1 ? row % (128 / R) : row);
      if (s == 0) { s_thr[(g & 1) * 256 + row] = 0u; s_thr[(g & 1) * 256 + 128 + row] = 0u; }
      uint4 nx0 = make_uint4(0, 0, 0, 0), nx1 = nx0;    // prefetched base logits of the next owned chunk
      bool have_next = false;
      const int pc = active ? p : 0;
      const int pid = ((tile * MMA_S + s) * R + rho) % K;   // which of the parent's K slots this piece feeds
      const SharedThr gl{a.slots + (size_t)pc * K * SLOT_STRIDE, pid};
      const SharedThr gk{a.slots + ((size_t)a.cap + pc) * K * SLOT_STRIDE, pid};
      // Pass nb = -1 is a dry run of the scan on an empty chunk while the first MMAs are still on their
      // way: it changes nothing in `st`, but it brings the scan's instructions into the instruction cache
      // and requests the base logits of the first chunk this warp owns.
      for (int nb = -1; nb < nblk; ++nb) {
        const bool dry = nb < 0;
        const int it = g * nblk + (dry ? 0 : nb), tb = it % NBUF, u = it / NBUF;
        if (!dry) {
          int ok = 1;
          if (lane == 0) ok = mbar_wait(t_full + tb, u & 1, s_abort, a.err) ? 1 : 0;
          ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
          if (!ok) { alive = false; break; }
          tc_fence_after();
          if (nb < 10 && g == 0) DBG(8 + warp * 6 + 0 + (nb >= 1 ? 2 : 0) + (nb >= 8 ? 2 : 0));
        }
        const int nch = dry ? 1 : min(8, (tlen - nb * BLK_N + 15) / 16);
        for (int c = 0; c < nch; ++c) {
          // owned chunks: cg = rho + R * (s + MMA_S * j); the dry pass sits one step before the first
          const int cg = dry ? rho + R * s - R * MMA_S : nb * 8 + c;
          if (!dry && ((cg & (R - 1)) != rho || ((cg >> rsh) % MMA_S) != s)) continue;   // warp-uniform; R is 1, 2 or 4
          float acc[16];
          if (!dry) {
            tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(tb * BLK_N + c * 16), acc);
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = 0.f;
          }
          if (active) {
            const int v0 = dry ? t0 : t0 + cg * 16;
            const int valid = dry ? 0 : min(16, V - v0);   // 8 or 16: V and v0 are multiples of 8
            // this chunk's base logits were requested one chunk ago; request the next owned chunk's now
            const uint4 u0 = have_next ? nx0 : (dry ? make_uint4(0, 0, 0, 0) : __ldg(reinterpret_cast<const uint4*>(Urow + v0)));
            const uint4 u1 = have_next ? nx1 : (valid > 8 ? __ldg(reinterpret_cast<const uint4*>(Urow + v0 + 8)) : make_uint4(0, 0, 0, 0));
            {
              const int cgn = cg + R * MMA_S;           // the next chunk this warp owns
              const int vn = t0 + cgn * 16;
              have_next = (cgn * 16 < tlen);
              if (have_next) {
                nx0 = __ldg(reinterpret_cast<const uint4*>(Urow + vn));
                nx1 = (V - vn > 8) ? __ldg(reinterpret_cast<const uint4*>(Urow + vn + 8)) : make_uint4(0, 0, 0, 0);
              }
            }
            float ub[16];
            unpack_bf16x8(u0, ub);
            unpack_bf16x8(u1, ub + 8);
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] += ub[i];
            if (valid < 16) {   // warp-uniform and rare (the vocabulary's last chunk, the dry pass): the scan's padding value
#pragma unroll
              for (int i = 0; i < 16; ++i) acc[i] = (i < valid) ? acc[i] : -INFINITY;
            }
            const float gLc = dec_f(s_thr[prow]), gKc = dec_f(s_thr[128 + prow]);   // kept fresh by the refresh warp
            scan_chunk<Lists, true>(st, acc, v0, valid, T, invT, a.seed, req, hash, ghi, gLc, gKc, gl, gk, s_thr + prow, s_thr + 128 + prow);
          }
        }
        if (dry) continue;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(t_empty + tb);
        if (nb < 10 && g == 0) DBG(8 + warp * 6 + 1 + (nb >= 1 ? 2 : 0) + (nb >= 8 ? 2 : 0));
      }
      if (alive && active) {
        const int gslot = R > 1 ? row : g * 128 + row;
        st.store(a.rec + ((size_t)(tile * MMA_S + s) * a.cap + gslot) * rw, dec_f(s_thr[prow]), dec_f(s_thr[128 + prow]));
      }
      if (lane == 0) atomicAdd((int*)s_done, 1);   // one tick per warp per group
    }
    if (!alive && lane == 0) atomicAdd((int*)s_done, 1 << 20);   // gave up: release the refresh warp
  } else if (warp == EPI_WARPS + 1) {
    // ======================= bounds-refresh warp ====================================================
    // keeps the shared-memory copies of every row's launch-wide pruning bounds current, so that the
    // epilogue threads never wait on those (contended) global words
    for (int g = 0; g < ngroups; ++g) {
      const int per = R > 1 ? 128 / R : 128;
      for (uint32_t spin = 0; spin < WAIT_LIMIT; ++spin) {
        if (*s_done >= (g + 1) * EPI_WARPS || *s_abort) break;
        // (1) This CTA condenses the slots of the parents it is responsible for (parent p belongs to tile
        // p mod ntiles) into two words per parent; (2) every CTA reads the condensed words of its rows.
        // Only one CTA per parent reads the slot lines, which every piece of the launch is hitting with
        // atomics.  The loads of both steps are issued together: one memory round trip per pass.
        const int p_lo = R > 1 ? 0 : g * 128, p_hi = min(P, p_lo + per);
        const int nt = a.ntiles;
        const int p_own = p_lo + ((tile - p_lo % nt + nt) % nt);   // first parent of this group this CTA owns
        const int which = lane >> 4, j = lane & 15;                  // lanes 0..15: logit slots, 16..31: key slots
        unsigned v = 0xFFFFFFFFu;
        if (p_own < p_hi && j < K) v = __ldcg(a.slots + (((size_t)which * a.cap + p_own) * K + j) * SLOT_STRIDE);
        unsigned rL[4], rK[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int rr = lane + 32 * k, p = R > 1 ? rr : g * 128 + rr;
          const bool in = rr < per && p < P;
          rL[k] = in ? __ldcg(a.thr + p) : 0u;
          rK[k] = in ? __ldcg(a.thr + (size_t)a.cap + p) : 0u;
        }
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) v = min(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
        if (p_own < p_hi && j == 0) __stcg(a.thr + (size_t)which * a.cap + p_own, v);
        for (int p = p_own + nt; p < p_hi; p += nt) {   // more parents than tiles: the rest, one at a time
          unsigned w = 0xFFFFFFFFu;
          if (j < K) w = __ldcg(a.slots + (((size_t)which * a.cap + p) * K + j) * SLOT_STRIDE);
#pragma unroll
          for (int off = 8; off > 0; off >>= 1) w = min(w, __shfl_xor_sync(0xFFFFFFFFu, w, off));
          if (j == 0) __stcg(a.thr + (size_t)which * a.cap + p, w);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int rr = lane + 32 * k, p = R > 1 ? rr : g * 128 + rr;
          if (rr < per && p < P) { s_thr[(g & 1) * 256 + rr] = rL[k]; s_thr[(g & 1) * 256 + 128 + rr] = rK[k]; }
        }
        if (spin >= 24u) __nanosleep(500);   // poll flat out while the launch warms up, then back off
      }
      __syncwarp();
    }
  } else if (warp == EPI_WARPS && lane == 0) {
    // ======================= MMA issuer ===========================================================
    const uint32_t ws_addr = smem_u32(Ws), as_addr = smem_u32(As);
    bool alive = true;
    for (int g = 0; g < ngroups && alive; ++g) {
      if (!mbar_wait(a_full, g & 1, s_abort, a.err)) break;
      tc_fence_after();
      for (int nb = 0; nb < nblk; ++nb) {
        const int it = g * nblk + nb, tb = it % NBUF, u = it / NBUF;
        if (u >= 1) {
          if (!mbar_wait(t_empty + tb, (u - 1) & 1, s_abort, a.err)) { alive = false; break; }
          tc_fence_after();
        }
        if (use_tma && g == 0) {
          if (!mbar_wait(w_full + nb, 0, s_abort, a.err)) { alive = false; break; }
        }
        const int n = (tlen - nb * BLK_N > 64) ? 128 : 64;
        const uint32_t idesc = instr_desc(n);
        const uint32_t d_tmem = tmem_base + (uint32_t)(tb * BLK_N);
        for (int ks = 0; ks < rp / 16; ++ks) {
          const uint64_t adesc = smem_desc(as_addr + (uint32_t)(ks >> 2) * a_slab_bytes + (uint32_t)(ks & 3) * 32u, 16u, 1024u);
          const uint64_t bdesc = smem_desc(ws_addr + (uint32_t)(2 * nb) * slab_bytes + (uint32_t)ks * 2048u, slab_bytes, 1024u);
          mma_bf16(d_tmem, adesc, bdesc, idesc, ks > 0 ? 1u : 0u);
        }
        mma_commit(t_full + tb);
      }
    }
  }
  // ---- tear-down -----------------------------------------------------------------------------------
  if (warp == 0) DBG(5);
  if (use_tma && tid == 0 && ((*s_abort && (early_w || P > 0)) || (P <= 0 && early_w))) {
    // gave up somewhere, or nothing to score: do not leave while a bulk load may still be writing this
    // CTA's shared memory
    for (int nb = 0; nb < nblk_w; ++nb) {
      bool done = false;
      for (uint32_t i = 0; i < WAIT_LIMIT && !done; ++i) { done = mbar_try_wait(w_full + nb, 0); if (!done) __nanosleep(100); }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) DBG(6);
  if (warp == EPI_WARPS) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

static size_t mma_smem_bytes(const ts_config& c, int TV) {
  const size_t rp = (size_t)(c.r + 63) / 64 * 64;
  return (size_t)(TV / 64) * rp * 128 + (rp / 64) * 128 * 128 + 512 * 4 + 128 + 512 * 4 + MAX_BLK * 8 + 1024;
}

// tile size for the tensor-core path: W tile + A tile + table + barriers within the shared-memory limit,
// a whole number of waves over the SMs
bool choose_tile_mma(const ts_config& c, int num_sms, int max_smem, TileCfg* out) {
  const size_t rp = (size_t)(c.r + 63) / 64 * 64;
  const size_t fixed = (rp / 64) * 128 * 128 + 512 * 4 + 128 + 512 * 4 + MAX_BLK * 8 + 1024;
  if ((size_t)max_smem < fixed + rp * 128) return false;
  int tv_max = (int)(((size_t)max_smem - fixed) / (rp * 2) / 64) * 64;
  if (tv_max < 64) return false;
  if (tv_max > 4096) tv_max = 4096;
  const int min_tiles = (c.V + tv_max - 1) / tv_max;
  const int waves = (min_tiles + num_sms - 1) / num_sms;
  const int want = waves * num_sms;
  int tv = ((c.V + want - 1) / want + 63) / 64 * 64;
  if (tv > tv_max) tv = tv_max;
  out->TV = tv;
  out->ntiles = (c.V + tv - 1) / tv;
  out->smem = mma_smem_bytes(c, tv);
  return out->ntiles <= 4096;
}

cudaError_t score_mma_setup(ts_ctx* ctx) {
  cudaError_t e = cudaFuncSetAttribute(score_mma_kernel<RegLists<8>>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->tile.smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(score_mma_kernel<RegLists<16>>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->tile.smem);
}

#ifdef TS_DEBUG_TIMING
extern "C" int ts_debug_timing(unsigned long long* out) {
  const int rc = (int)cudaMemcpyFromSymbol(out, g_dbg, sizeof(g_dbg));
  static unsigned long long zeros[148 * 64];
  cudaMemcpyToSymbol(g_dbg, zeros, sizeof(zeros));
  return rc;
}
#endif

// Tensor map of W = [r][V] bf16 for boxes of 64 tokens x rp rows with the 128-byte swizzle the MMA's
// B descriptor expects.  The encoder lives in the driver library; it is looked up through the runtime
// so that this library has no link-time dependency on the driver.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

bool w_tensor_map(ts_ctx* ctx, const void* W) {
  if (ctx->tma_state < 0) return false;
  const int rp = (ctx->cfg.r + 63) / 64 * 64;
  if (rp > 256 || ((uintptr_t)W & 15u) != 0) return false;   // box rows are limited to 256
  if (ctx->tma_state == 1 && ctx->tmapW_ptr == W) return true;
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
        q != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      ctx->tma_state = -1;
      return false;
    }
    g_encode = (EncodeTiledFn)fn;
  }
  const cuuint64_t gdim[2] = {(cuuint64_t)ctx->cfg.V, (cuuint64_t)ctx->cfg.r};
  const cuuint64_t gstride[1] = {(cuuint64_t)ctx->cfg.V * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)rp};
  const cuuint32_t estr[2] = {1u, 1u};
  CUtensorMap tm;
  const CUresult rc = g_encode(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(W), gdim, gstride, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (rc != CUDA_SUCCESS) { ctx->tma_state = -1; return false; }
  memcpy(ctx->tmapW, &tm, sizeof(tm));
  ctx->tmapW_ptr = W;
  ctx->tma_state = 1;
  return true;
}

cudaError_t launch_score_mma(const ts_ctx* ctx, const ScoreArgs& a, cudaStream_t st) {
  ts_ctx* c = const_cast<ts_ctx*>(ctx);
  const int use_tma = w_tensor_map(c, a.W) ? 1 : 0;
  CUtensorMap tm;
  memcpy(&tm, c->tmapW, sizeof(tm));
  cudaError_t e;
  if (a.K <= 8) e = launch_kernel(score_mma_kernel<RegLists<8>>, a.ntiles, MMA_THREADS, ctx->tile.smem, st, a.pdl != 0, a, tm, use_tma);
  else e = launch_kernel(score_mma_kernel<RegLists<16>>, a.ntiles, MMA_THREADS, ctx->tile.smem, st, a.pdl != 0, a, tm, use_tma);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ts
