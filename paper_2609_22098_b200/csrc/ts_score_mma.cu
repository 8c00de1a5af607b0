// Tensor-core scoring kernel for sm_100a: the low-rank bias [parents x r] . [r x tile] runs on the
// 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory), and the vocabulary scan
// (add base logits, online max / sum-exp, candidates for the top-K and Gumbel top-K lists) is its
// epilogue, one tensor-memory lane = one parent row per thread.
//
// CTA = one vocabulary tile, resident for the whole launch.  Shared memory holds
//   W tile  : B operand, MN-major, 128-byte swizzle: slabs of 64 tokens, slab = [rp rows][128 B];
//             loaded by bulk-tensor copies (one mbarrier per 128-token block), or by plain loads when
//             no tensor map could be encoded
//   A tile  : A operand, K-major, 128-byte swizzle: [rp/64 slabs][128 rows][128 B] (gathered rows A[x_p])
//   lists   : per parent row the K best logits and K best sampling keys this CTA has seen
//   queues  : candidates on their way from the scanning warps to the selector warps
// (rp = r rounded up to 64, padding zero-filled).
//
// Warps 0..15 scan: warp w reads the tensor-memory lanes 32*(w%4).. (its quarter of the 128 parent
// rows) and, of the tile's 64-token blocks, those of split w/4 (block nb belongs to split nb % 4).  When
// a level has few parents the rows are replicated R = 2 or 4 times over the quarters and the copies
// split a block's four 16-token chunks: chunk c belongs to replica c % R.  A scanning thread keeps only the running
// (max, sums) of its row; a token that can still be among the row's K best (its logit, or the upper
// bound of its sampling key given the leading 16 bits of its uniform, reaches the row's current bound)
// is appended to a queue with a few instructions, so that the 32 rows of a warp never wait for the
// rare, long evaluation of one of them.  Warps 18 and 19 (rows 0..63 / 64..127) drain the queues, one
// candidate per lane: exact key (second generator call, two logarithms), insertion into the row's
// sorted lists, publication of new bests.  Warp 16 allocates tensor memory and its lane 0 issues the
// MMAs: per block of 64 tokens rp/16 instructions of M=128, N=64, K=16 into one of eight 64-column
// accumulator buffers (two per split), then a commit that arrives on that buffer's "full" barrier;
// scanning warps arrive on its "empty" barrier when they have drained it.  Warp 17 keeps shared-memory
// copies of the launch-wide pruning bounds of every row current.
//
// Launch-wide bounds.  Per parent K slots in global memory; slot j holds the best value published by
// the pieces (tile, split, replica) whose number is j modulo K.  Pieces hold disjoint tokens, so the
// slots hold values of K different tokens and their minimum is a lower bound of the parent's K-th best
// value: a token strictly below it cannot be among the K best.  So that bounds exist before the scan
// begins, a kernel ahead of this one (seed_parents_kernel) evaluates for every parent the tokens with the
// largest base logits exactly and leaves the K-th best logit and key among them, less a rounding margin,
// as the parent's seed bounds; the bounds used here are never below those.
//
// Every wait is bounded: when one runs out the kernel raises an error word, skips the remaining work,
// waits (again bounded) for bulk loads still in flight, frees its tensor memory and returns.
#include "ts_tc.cuh"
#include "ts_internal.h"
#include "ts_scan.cuh"
#include "ts_merge.cuh"
#include "ts_level.cuh"

namespace ts {

constexpr int EPI_S = MMA_S;                // column splits = scanning warps per row quarter
constexpr int EPI_WARPS = 4 * EPI_S;
constexpr int W_MMA = EPI_WARPS;            // warp roles
constexpr int W_REFRESH = EPI_WARPS + 1;
constexpr int W_SEL = EPI_WARPS + 2;
constexpr int NSEL = 2;                     // selector warps (rows 0..63, 64..127)
constexpr int MMA_THREADS = (EPI_WARPS + 2 + NSEL) * 32;
constexpr int BLK_N = 64;               // tokens per block: one MMA tile, one accumulator buffer, one slab of W
constexpr int WBLK = 128;               // tokens per bulk-load barrier of W (two slabs)
constexpr int NBUF = 8;                 // accumulator buffers of BLK_N columns in tensor memory: two per split
constexpr uint32_t TMEM_COLS = NBUF * BLK_N;
constexpr int MAX_BLK = 32;             // W load barriers (WBLK tokens each) of the largest tile (4096 tokens)
constexpr int QCAP = 128;               // entries per candidate queue (power of two)
constexpr int NUB = 4;                  // ring of base-logit slabs (UMMA_REQ rows x 64 tokens) ahead of the MMAs
constexpr uint32_t KIND_TOP = 1u, KIND_KEY = 2u;

template <int ID, int NT>
struct NamedSync {
  __device__ __forceinline__ void operator()() const { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(NT) : "memory"); }
};

// Shared-memory state of the selection side of one CTA.
struct SelShared {
  float* lists;             // [128][5K]: topv, topi, keyv, keyi, keyl of every row, sorted (value desc, token asc)
  volatile float* lthr;     // [2][128]: K-th best logit / key of the row's lists (-inf until they are full)
  volatile float* best;     // [2][EPI_S][128]: best logit / key published so far by the piece (row, split)
  uint4* q;                 // [NSEL][QCAP] entries: token, logit, row | split << 8 | kind << 12 | c16 << 16, tag
  volatile unsigned* q_head;   // [NSEL] entries consumed
  unsigned* q_tail;            // [NSEL] entries claimed
};

// insertion into one sorted list of K entries (value desc, token asc); returns the new K-th value
__device__ __forceinline__ float list_insert(float* v, int* t, float* aux, int K, float val, int tok, float lg) {
  int pos = K - 1;
  if (!(val > v[pos] || (val == v[pos] && (unsigned)tok < (unsigned)t[pos]))) return v[pos];
  while (pos > 0 && (val > v[pos - 1] || (val == v[pos - 1] && (unsigned)tok < (unsigned)t[pos - 1]))) {
    v[pos] = v[pos - 1]; t[pos] = t[pos - 1];
    if (aux) aux[pos] = aux[pos - 1];
    --pos;
  }
  v[pos] = val; t[pos] = tok;
  if (aux) aux[pos] = lg;
  return v[K - 1];
}

// One candidate, handled by one selector lane: exact key, insertion, publication.
__device__ __forceinline__ void select_candidate(const ScoreArgs& a, const SelShared& sh, const uint4 e, const float* ghi,
                                                 float invT, int K, int tile, int R, int g, const volatile unsigned* s_thr,
                                                 int pbase, bool do_insert, const int* lp_req, const uint64_t* lp_hash) {
  const int tok = (int)e.x;
  const float lg = __uint_as_float(e.y);
  const int row = (int)(e.z & 0xFFu), s = (int)((e.z >> 8) & 0xFu);
  const uint32_t kind = (e.z >> 12) & 0xFu, c16 = e.z >> 16;
  const int per = 128 / R;
  const int p = R > 1 ? row % per : g * 128 + row, rho = R > 1 ? row / per : 0;
  const int prow = pbase + (R > 1 ? row % per : row);
  const int pid = ((tile * EPI_S + s) * R + rho) % K;
  float* L = sh.lists + (size_t)row * 5 * K;
  if (kind & KIND_TOP) {
    const float gL = dec_f(s_thr[prow]);
    if (lg >= gL && lg >= sh.lthr[row] && do_insert) {
      sh.lthr[row] = list_insert(L, reinterpret_cast<int*>(L) + K, nullptr, K, lg, tok, 0.f);
      volatile float* b = sh.best + (0 * EPI_S + s) * 128 + row;
      if (lg > *b) { *b = lg; atomicMax(a.slots + ((size_t)p * K + pid) * SLOT_STRIDE, enc_f(lg)); }
    }
  }
  if (kind & KIND_KEY) {
    const float thr = fmaxf(dec_f(s_thr[128 + prow]), sh.lthr[128 + row]);
    const float bnd = lg * invT + ghi[noise_bound_index(c16)];
    if (bnd >= thr && do_insert) {   // the bounds have often risen since the candidate was queued
      const uint4 fw = stream_words(a.seed, __ldcg(lp_req + p), __ldcg(lp_hash + p), STREAM_GUMBEL_FINE, (uint32_t)tok >> 3);
      const uint32_t f16 = (word_of(fw, (tok & 7) >> 1) >> (16 * (tok & 1))) & 0xFFFFu;
      const float key = lg * invT + gumbel_from_bits((c16 << 16) | f16);
      if (key >= thr) {
        sh.lthr[128 + row] = list_insert(L + 2 * K, reinterpret_cast<int*>(L) + 3 * K, L + 4 * K, K, key, tok, lg);
        volatile float* b = sh.best + (1 * EPI_S + s) * 128 + row;
        if (key > *b) { *b = key; atomicMax(a.slots + (((size_t)a.cap + p) * K + pid) * SLOT_STRIDE, enc_f(key)); }
      }
    }
  }
}

// BIGK: the instantiation whose cooperative form merges with 16-entry lists (K > 8); it exists beside the other
// one so that the merge's registers do not weigh on the scan of the launches that never merge.
template <bool UMMA, bool BIGK = false>
__global__ void __launch_bounds__(MMA_THREADS, 1) score_mma_kernel(const ScoreArgs a, const __grid_constant__ CUtensorMap tmW, const int use_tma, const __grid_constant__ PersistArgs pa,
                                                                   const __grid_constant__ CUtensorMap tmU) {
  extern __shared__ unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // The preamble below (shared-memory carve-up, tensor-memory allocation, barriers, bulk loads of W, noise
  // table) reads nothing an earlier kernel of the stream wrote, so in a chained launch it runs while the
  // previous kernel is still finishing.  When the level before this one was empty, this one is too.
  if (a.P_prev_dev && *a.P_prev_dev <= 0) { pdl_wait(); return; }

  const int r = a.r, rp = (r + 63) / 64 * 64, V = a.V, TV = a.TV, K = a.K;
  // This CTA's vocabulary tiles: blockIdx.x, blockIdx.x + gridDim.x, ... (one tile per CTA whenever the tiles fit
  // the SMs; at large ranks, where the W tile is small, a CTA takes several in turn and pays its set-up once)
  int tile = blockIdx.x, t0 = tile * TV, tlen = min(TV, V - t0);
  int tile_it = 0;          // tiles this CTA has finished: the W barriers' phase
  const int wring = UMMA ? 0 : a.w_ring;   // > 0: W streams through a ring of that many 64-token slabs (one tile per CTA)
  const int nslab = wring ? wring : TV / 64;
  int nblk_w = wring ? 0 : (tlen + WBLK - 1) / WBLK;
  const uint32_t slab_bytes = (uint32_t)rp * 128u;       // one 64-token slab of W
  const uint32_t a_slab_bytes = 128u * 128u;             // 128 rows x 128 B
  unsigned char* sm = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* Ws = sm;
  unsigned char* As = Ws + (size_t)nslab * slab_bytes;
  // (one more slab of the A tile holds the one-hot request columns, and a ring of slabs the base logits they select)
  unsigned char* Us = As + (size_t)(rp / 64 + (UMMA ? 1 : 0)) * a_slab_bytes;   // [NUB][UMMA_REQ rows][128 B], 128-byte swizzle
  float* ghi = reinterpret_cast<float*>(Us + (UMMA ? (size_t)NUB * UMMA_REQ * 128 : 0));
  SelShared sh;
  sh.q = reinterpret_cast<uint4*>(ghi + 512);                                   // 16-byte aligned
  sh.lists = reinterpret_cast<float*>(sh.q + NSEL * QCAP);
  sh.lthr = sh.lists + (size_t)128 * 5 * K;
  sh.best = sh.lthr + 2 * 128;
  float* s_part = const_cast<float*>(sh.best) + 2 * EPI_S * 128;                // [3][EPI_S][128]: m, s0, sT of every (split, row)
  volatile unsigned* s_thr = reinterpret_cast<volatile unsigned*>(s_part + 3 * EPI_S * 128);   // [group parity][2][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(const_cast<unsigned*>(s_thr) + 512);
  uint64_t* a_full = bars;            // scanning threads -> MMA: the A tile of this group is in place
  uint64_t* t_full = bars + 1;             // [NBUF] MMA -> scan: accumulator buffer written
  uint64_t* t_empty = bars + 1 + NBUF;     // [NBUF] scan -> MMA: accumulator buffer drained
  uint64_t* w_full = bars + 1 + 2 * NBUF;  // [MAX_BLK] W slabs of block nb landed
  uint64_t* u_full = w_full + MAX_BLK;     // [NUB] base-logit slab landed
  uint64_t* u_free = u_full + NUB;         // [NUB] the MMAs that read the slab are done
  uint64_t* w_free = u_free + NUB;         // [MAX_BLK] streaming form: the MMAs that read the ring slot are done
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(w_free + MAX_BLK);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  volatile int* s_done = reinterpret_cast<volatile int*>(s_tmem + 2);             // scanning warps finished (cumulative)
  sh.q_head = reinterpret_cast<volatile unsigned*>(s_tmem + 4);
  sh.q_tail = s_tmem + 4 + NSEL;

  const __nv_bfloat16* Wg = reinterpret_cast<const __nv_bfloat16*>(a.W);
  const __nv_bfloat16* Ug = reinterpret_cast<const __nv_bfloat16*>(a.U);
  const __nv_bfloat16* Ag = reinterpret_cast<const __nv_bfloat16*>(a.A);
  const uint32_t wait_limit = a.wait_limit;

  // ---- set-up ------------------------------------------------------------------------------------
  if (warp == W_MMA) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const bool early_w = !a.P_prev_dev || *a.P_prev_dev >= 16;
  auto issue_w = [&]() {   // one thread
    for (int nb = 0; nb < nblk_w; ++nb) {
      const int ns = (tlen - nb * WBLK > 64) ? 2 : 1;
      mbar_expect_tx(w_full + nb, (uint32_t)ns * slab_bytes);
      for (int h = 0; h < ns; ++h)
        tma_load_box(Ws + (size_t)(2 * nb + h) * slab_bytes, &tmW, t0 + (2 * nb + h) * 64, 0, w_full + nb);
    }
  };
  if (tid == 0) {
    mbar_init(a_full, EPI_WARPS * 32 + (a.lost_arrival ? 1 : 0));
    for (int i = 0; i < NBUF; ++i) { mbar_init(t_full + i, 1); mbar_init(t_empty + i, 4); }   // a buffer is drained by the four quarter warps of one split
    *s_abort = 0;
    *s_done = 0;
    for (int i = 0; i < NSEL; ++i) { sh.q_head[i] = 0u; sh.q_tail[i] = 0u; }
    if (use_tma) for (int i = 0; i < (wring ? wring : nblk_w); ++i) mbar_init(w_full + i, 1);
    for (int i = 0; i < wring; ++i) mbar_init(w_free + i, 1);
    for (int i = 0; i < NUB; ++i) { mbar_init(u_full + i, 1); mbar_init(u_free + i, 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // W tile by bulk-tensor loads, one barrier per block of 128 tokens so that the first MMAs start while
    // the rest of the tile is still in flight; tokens past V and rows past r arrive as zeros.  Issued here,
    // before the kernel may look at its own parent count, when the level before was large enough for this
    // one to be populated almost surely; after the count is known otherwise (a level that turns out empty then
    // fetches nothing).
    if (use_tma && early_w && !wring) issue_w();
  }
  auto fill_w_plain = [&]() {  // W tile: 16-byte chunks (8 tokens of one row), swizzled: chunk j of row k lands at chunk j ^ (k & 7)
    const int per_slab = rp * 8;
    for (int idx = tid; idx < nslab * per_slab; idx += MMA_THREADS) {
      const int slab = idx / per_slab, rem = idx % per_slab, k = rem >> 3, j = rem & 7;
      const int tok = t0 + slab * 64 + j * 8;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (k < r && tok < V) v = __ldg(reinterpret_cast<const uint4*>(Wg + (size_t)k * V + tok));
      *reinterpret_cast<uint4*>(Ws + (size_t)slab * slab_bytes + k * 128 + ((j ^ (k & 7)) << 4)) = v;
    }
  };
  if (!use_tma && !wring) fill_w_plain();
  fill_gumbel_bounds(ghi, tid, MMA_THREADS);
  for (int i = tid; i < 512; i += MMA_THREADS) s_thr[i] = 0u;
  auto reset_selection = [&]() {   // empty lists, no local thresholds, nothing published
    for (int i = tid; i < 128 * 5 * K; i += MMA_THREADS) {
      const int f = (i / K) % 5;   // fields: topv, topi, keyv, keyi, keyl
      sh.lists[i] = (f == 0 || f == 2) ? -INFINITY : ((f == 1 || f == 3) ? __int_as_float(-1) : 0.f);
    }
    for (int i = tid; i < 2 * 128; i += MMA_THREADS) sh.lthr[i] = -INFINITY;
    for (int i = tid; i < 2 * EPI_S * 128; i += MMA_THREADS) sh.best[i] = -INFINITY;
  };
  reset_selection();   // the first group's, here in the preamble; later groups' when they begin
  for (int i = tid; i < NSEL * QCAP; i += MMA_THREADS) sh.q[i] = make_uint4(0u, 0u, 0u, 0u);   // tag 0 = never written
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  pdl_wait();                // parent lists and the level's parent count come from the previous kernel
  pdl_launch_dependents();
  const bool persist = pa.on != 0;
  int gg = 0;               // groups scanned so far, over all levels (barrier parities and use counts run on)
  uint32_t ul = 0;          // block pairs of all groups before this one (MMA issuer: slot and use of their base-logit slabs)
  unsigned gen = 0;         // grid barriers passed
  bool dead = false;        // a bounded wait ran out somewhere
  bool w_issued = (use_tma && early_w) || wring;   // bulk loads of the W tile are (or were) in flight (streaming form: the issuer's business)
  uint32_t wl = 0;          // streaming form: slabs of all groups before this one (ring slot and use of a block's slab)
  int gg_tile = 0;          // value of gg when the current tile began: its first group waits for the tile's W blocks
  for (;;) {   // this CTA's tiles
  gg_tile = gg;
  for (int lvl = persist ? pa.first : 0; !dead; ++lvl) {
  // the parent list of this level (in the persistent form written by the level step before it: read around L1)
  const int cur = lvl & 1;
  const int* lp_req = persist ? pa.ex.lst_req[cur] : a.p_req;
  const int* lp_depth = persist ? pa.ex.lst_depth[cur] : a.p_depth;
  const int* lp_token = persist ? pa.ex.lst_token[cur] : a.p_token;
  const uint64_t* lp_hash = persist ? pa.ex.lst_hash[cur] : a.p_hash;
  const int scout_depth = persist ? lvl + 1 : a.scout_depth;
  const bool scout = a.utop != nullptr && scout_depth < a.D;
  const int u_depth = persist ? lvl : a.u_depth;   // UMMA: the depth every parent of this level sits at
  const int P = persist ? __ldcg(pa.ex.lvl_count + lvl) : (a.P_dev ? *a.P_dev : a.P);   // may be 0: an empty level only tears down
  if (persist && P <= 0) break;   // (a launch that starts at a later level finds out here that the tree ended before it)
  if (use_tma && !w_issued && P > 0) { if (tid == 0) issue_w(); w_issued = true; }

  const int R = mma_replicas(P);
  const int per = 128 / R;
  const int ngroups = P <= 0 ? 0 : (R > 1 ? 1 : (P + 127) / 128);
  const int nblk = (tlen + BLK_N - 1) / BLK_N;
  const float T = a.T, invT = T > 0.f ? 1.f / T : 1.f;
  const bool keys = T > 0.f;
  const int rw = rec_words(K);

  for (int g = 0; g < ngroups; ++g) {
    const int pbase = (gg & 1) * 256;   // successive groups alternate between two bound buffers
    // ---- per-group reset of the selection state (every thread) ---------------------------------------
    if (gg > 0) reset_selection();
    for (int i = tid; i < 2 * 128; i += MMA_THREADS) {
      // the row's bounds start at its parent's seed bounds (exact values of K tokens, found before the launch)
      const int which = i >> 7, rr = i & 127;
      const int p = R > 1 ? rr % per : g * 128 + rr;
      s_thr[pbase + i] = (a.thr0 && p < P && (R == 1 || rr < per)) ? __ldcg(a.thr0 + (size_t)which * a.cap + p) : 0u;
    }
    __syncthreads();

    if (warp < EPI_WARPS) {
      // ======================= scanning warps =======================================================
      const int q = warp & 3, s = warp >> 2;
      const int row = q * 32 + lane;
      const int e = warp * 32 + lane;
      const int cpr = rp / 8;          // 16-byte chunks per A row
      // gather this group's parent rows A[x_p] into the swizzled A tile (a later tile of a launch with one group
      // finds them in place)
      const bool a_in_place = tile_it > 0 && ngroups == 1;
      for (int idx = e; idx < 128 * cpr && !a_in_place; idx += EPI_WARPS * 32) {
        const int rr = idx / cpr, ck = idx % cpr;
        const int p = R > 1 ? rr % per : g * 128 + rr;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (p < P && ck * 8 < r) v = __ldg(reinterpret_cast<const uint4*>(Ag + (size_t)__ldcg(lp_token + p) * r + ck * 8));
        *reinterpret_cast<uint4*>(As + (size_t)(ck >> 3) * a_slab_bytes + rr * 128 + (((ck & 7) ^ (rr & 7)) << 4)) = v;
      }
      if (UMMA) {
        // one more K-slab of the A tile: column b of row rr is 1 when the row's parent belongs to request b, so the
        // MMA adds that request's base logits (rows of the base-logit slab) to the row's bias
        for (int idx = e; idx < 128 * 8 && !a_in_place; idx += EPI_WARPS * 32) {
          const int rr = idx >> 3, ck = idx & 7;
          const int p = R > 1 ? rr % per : g * 128 + rr;
          uint4 v = make_uint4(0, 0, 0, 0);
          if (p < P) {
            const int b = __ldcg(lp_req + p);
            if ((b >> 3) == ck) {
              const uint32_t one = 0x3F80u << (16 * (b & 1));   // bf16 1.0 in the half-word of column b
              const int w = (b & 7) >> 1;
              v.x = w == 0 ? one : 0u; v.y = w == 1 ? one : 0u; v.z = w == 2 ? one : 0u; v.w = w == 3 ? one : 0u;
            }
          }
          *reinterpret_cast<uint4*>(As + (size_t)(rp / 64) * a_slab_bytes + rr * 128 + ((ck ^ (rr & 7)) << 4)) = v;
        }
      }
      fence_async_smem();
      mbar_arrive(a_full);
      if (scout && g == 0) {
        // scouting (see ScoreArgs): fills the wait for the first accumulators, and brings the rows the next
        // level will score into L2
        const int nvec = tlen / 8;
        for (int b = warp; b < a.scout_B; b += EPI_WARPS) {
          if (__ldcg(a.scout_live + b) <= 0) continue;   // warp-uniform
          const uint4* src = reinterpret_cast<const uint4*>(Ug + ((size_t)b * a.D + scout_depth) * V + t0);
          float bv = -INFINITY; int bi = 0x7FFFFFFF;
          for (int c0 = 0; c0 < nvec; c0 += 5 * 32) {
            uint4 x[5];
#pragma unroll
            for (int u = 0; u < 5; ++u) {
              const int c = c0 + u * 32 + lane;
              x[u] = c < nvec ? __ldg(src + c) : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // -inf
            }
#pragma unroll
            for (int u = 0; u < 5; ++u) {
              float f[8];
              unpack_bf16x8(x[u], f);
#pragma unroll
              for (int i = 0; i < 8; ++i) if (f[i] > bv) { bv = f[i]; bi = t0 + (c0 + u * 32 + lane) * 8 + i; }
            }
          }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, off);
            const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, off);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          if (lane == 0) a.utop[((size_t)b * a.D + scout_depth) * a.ntiles + tile] = make_uint2(__float_as_uint(bv), (unsigned)bi);
        }
      }

      const int p = R > 1 ? row % per : g * 128 + row;
      const int rho = R > 1 ? row / per : 0;   // uniform within a warp (128/R is a multiple of 32)
      const bool active = p < P;
      int req = 0; uint64_t hash = 0; const __nv_bfloat16* Urow = Ug;
      if (active) {
        req = __ldcg(lp_req + p); hash = __ldcg(lp_hash + p);
        Urow = Ug + ((size_t)req * a.D + __ldcg(lp_depth + p)) * V;
      }
      const int prow = pbase + (R > 1 ? row % per : row);
      const int sel = row >> 6;
      const uint32_t ztag = (uint32_t)row | ((uint32_t)s << 8);
      float m = -INFINITY, s0 = 0.f, sT = 0.f;
      uint4 nx0 = make_uint4(0, 0, 0, 0), nx1 = nx0;    // prefetched base logits of the next owned chunk
      bool have_next = false;
      bool alive = true;
      // Blocks of 64 tokens are dealt to the splits round-robin (block nb belongs to split nb % 4), and a split
      // alternates between two accumulator buffers of its own, so its four quarter warps and the MMA issuer form a
      // pipeline of their own: a slow warp holds up three others, not fifteen, and the next block's accumulators
      // are written while this one is scanned.  A row's 128 bytes of base logits per block are one cache line;
      // the line of the split's next block is requested from L2 when a block begins.
      const int nuse = nblk > s ? (nblk - s + EPI_S - 1) / EPI_S : 0;   // blocks of this split per group
      auto prefetch_block = [&](int nb) {
        if (active && nb < nblk) asm volatile("prefetch.global.L2 [%0];" ::"l"(Urow + t0 + nb * BLK_N));
      };
      if (!UMMA) prefetch_block(s);
      for (int nb = s; nb < nblk && alive; nb += EPI_S) {
        const int j = nb / EPI_S, h = j & 1;
        const int tb = s + EPI_S * h, u = gg * ((nuse + 1 - h) >> 1) + (j >> 1);   // buffer, and how often it was used before
        if (!UMMA) prefetch_block(nb + EPI_S);
        {
          int ok = 1;
          if (lane == 0) ok = mbar_wait(t_full + tb, u & 1, s_abort, a.err, wait_limit) ? 1 : 0;
          ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
          if (!ok) { alive = false; break; }
          tc_fence_after();
        }
        const int nch = min(BLK_N / 16, (tlen - nb * BLK_N + 15) / 16);
        for (int c = 0; c < nch; ++c) {
          const int cg = nb * (BLK_N / 16) + c;
          if ((c & (R - 1)) != rho) continue;   // warp-uniform; R is 1, 2 or 4: the replicas split a block's chunks
          float acc[16];
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(tb * BLK_N + c * 16), acc);
          if (!active) continue;
          const int v0 = t0 + cg * 16;
          const int valid = min(16, V - v0);   // 8 or 16: V and v0 are multiples of 8
          if (!UMMA) {
            // this chunk's base logits were requested one chunk ago; request the next owned chunk's now
            const uint4 u0 = have_next ? nx0 : __ldg(reinterpret_cast<const uint4*>(Urow + v0));
            const uint4 u1 = have_next ? nx1 : (valid > 8 ? __ldg(reinterpret_cast<const uint4*>(Urow + v0 + 8)) : make_uint4(0, 0, 0, 0));
            {
              const int cgn = (c + R < BLK_N / 16) ? cg + R : (nb + EPI_S) * (BLK_N / 16) + rho;   // the next chunk this warp owns
              const int vn = t0 + cgn * 16;
              have_next = (cgn * 16 < tlen);
              if (have_next) {
                nx0 = __ldg(reinterpret_cast<const uint4*>(Urow + vn));
                nx1 = (V - vn > 8) ? __ldg(reinterpret_cast<const uint4*>(Urow + vn + 8)) : make_uint4(0, 0, 0, 0);
              }
            }
            {
              float ub[16];
              unpack_bf16x8(u0, ub);
              unpack_bf16x8(u1, ub + 8);
  #pragma unroll
              for (int i = 0; i < 16; ++i) acc[i] += ub[i];
            }
          }
          if (valid < 16) {   // warp-uniform and rare (the vocabulary's last chunk): padding that loses every comparison
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = (i < valid) ? acc[i] : -INFINITY;
          }
          // the row's bounds as the refresh warp last left them (read here: the loads' latency hides under the scan)
          const float thrL = dec_f(s_thr[prow]), thrK = dec_f(s_thr[128 + prow]);
          // ---- the scan of one chunk -------------------------------------------------------------
          // high halves of the sixteen uniforms: two generator calls, issued first so that their long
          // dependent chains overlap the exponentials below
          uint4 cw0 = make_uint4(0, 0, 0, 0), cw1 = cw0;
          if (keys) {
            cw0 = stream_words(a.seed, req, hash, STREAM_GUMBEL_COARSE, (uint32_t)v0 >> 3);
            cw1 = stream_words(a.seed, req, hash, STREAM_GUMBEL_COARSE, ((uint32_t)v0 >> 3) + 1u);
          }
          float gmax[4];
          float cm = -INFINITY;
#pragma unroll
          for (int sg = 0; sg < 4; ++sg) {
            gmax[sg] = fmaxf(fmaxf(acc[4 * sg], acc[4 * sg + 1]), fmaxf(acc[4 * sg + 2], acc[4 * sg + 3]));
            cm = fmaxf(cm, gmax[sg]);
          }
          {
            // rescale to the new running maximum without a branch (no change: factor 1; first chunk: factor 0)
            const float nm = fmaxf(m, cm);
            const float d = (m == nm) ? 0.f : m - nm;
            s0 *= __expf(d);
            sT *= __expf(d * invT);
            m = nm;
          }
          {
            // exp(l - m) as ex2(l * log2(e) - m * log2(e)): one fused multiply-add and one ex2 per token.  While
            // nothing finite has been seen (m = -inf) the offset is 0: every l is -inf then and contributes 0.
            constexpr float LOG2E = 1.4426950408889634f;
            const bool two = keys && (T != 1.f);
            const float mref = m == -INFINITY ? 0.f : m;
            const float off0 = -mref * LOG2E, scT = LOG2E * invT, offT = off0 * invT;
            float a0 = 0.f, a1 = 0.f, aT = 0.f;
#pragma unroll
            for (int i = 0; i < 16; i += 2) {
              a0 += ex2_approx(fmaf(acc[i], LOG2E, off0));
              a1 += ex2_approx(fmaf(acc[i + 1], LOG2E, off0));
              if (two) aT += ex2_approx(fmaf(acc[i], scT, offT)) + ex2_approx(fmaf(acc[i + 1], scT, offT));
            }
            a0 += a1;
            s0 += a0;
            sT += two ? aT : a0;
          }
          // ---- candidates ---------------------------------------------------------------------------
          uint32_t mkK = 0, mkL = 0;
          if (cm >= thrL) {
#pragma unroll
            for (int i = 0; i < 16; ++i) mkL |= (uint32_t)(acc[i] >= thrL && acc[i] > -INFINITY) << i;
          }
          if (keys) {
            const float thr = thrK;
            // the whole chunk first: its best logit plus the noise bound of the largest leading bits among its
            // sixteen tokens bounds every key in it; then four tokens at a time, then singly
            const uint32_t m8 = __vmaxu2(__vmaxu2(__vmaxu2(cw0.x, cw0.y), __vmaxu2(cw0.z, cw0.w)),
                                         __vmaxu2(__vmaxu2(cw1.x, cw1.y), __vmaxu2(cw1.z, cw1.w)));
            const uint32_t c16all = max(m8 & 0xFFFFu, m8 >> 16);
            if (cm * invT + ghi[noise_bound_index(c16all)] >= thr && cm > -INFINITY) {
#pragma unroll
              for (int sg = 0; sg < 4; ++sg) {
                const uint4& cw = sg < 2 ? cw0 : cw1;
                const uint32_t wa = (sg & 1) ? cw.z : cw.x, wb = (sg & 1) ? cw.w : cw.y;
                const uint32_t m2 = __vmaxu2(wa, wb);
                const uint32_t c16m = max(m2 & 0xFFFFu, m2 >> 16);
                if (gmax[sg] * invT + ghi[noise_bound_index(c16m)] >= thr && gmax[sg] > -INFINITY) {
#pragma unroll
                  for (int i = 4 * sg; i < 4 * sg + 4; ++i) {
                    const uint32_t word = word_of(i < 8 ? cw0 : cw1, (i & 7) >> 1);
                    const uint32_t c16 = (word >> (16 * (i & 1))) & 0xFFFFu;
                    mkK |= (uint32_t)(acc[i] * invT + ghi[noise_bound_index(c16)] >= thr && acc[i] > -INFINITY) << i;
                  }
                }
              }
            }
          }
          uint32_t mk = mkK | mkL;
#pragma unroll 1
          while (mk) {   // rare: hand the token to the selector warp of this row
            const int i = __ffs(mk) - 1;
            mk &= mk - 1;
            const uint32_t kind = ((mkL >> i) & 1u) * KIND_TOP | ((mkK >> i) & 1u) * KIND_KEY;
            const uint32_t c16 = (pick8(cw0, cw1, i >> 1) >> (16 * (i & 1))) & 0xFFFFu;
            const unsigned idx = atomicAdd(sh.q_tail + sel, 1u);
            uint32_t spin = 0;
            while ((int)(idx - sh.q_head[sel]) >= QCAP) {   // queue full: the selector is behind
              if (*s_abort) break;
              if (++spin > wait_limit) { *s_abort = 1; if (a.err) atomicExch(a.err, 1); break; }
              __nanosleep(64);
            }
            uint4* slot = sh.q + sel * QCAP + (idx & (QCAP - 1));
            slot->x = (uint32_t)(v0 + i); slot->y = __float_as_uint(pick16(acc, i));
            slot->z = ztag | (kind << 12) | (c16 << 16);
            __threadfence_block();
            *reinterpret_cast<volatile uint32_t*>(&slot->w) = idx + 1u;   // tag: the entry is complete
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(t_empty + tb);
      }
      // this piece's sums; the row's record is put together when the group is over
      s_part[(0 * EPI_S + s) * 128 + row] = m; s_part[(1 * EPI_S + s) * 128 + row] = s0; s_part[(2 * EPI_S + s) * 128 + row] = sT;
      __threadfence_block();
      __syncwarp();
      if (lane == 0) atomicAdd((int*)s_done, alive ? 1 : (1 << 20));   // one tick per warp per group (a large one releases the others after a failed wait)
    } else if (warp == W_REFRESH) {
      // ======================= bounds-refresh warp ====================================================
      // keeps the shared-memory copies of every row's launch-wide pruning bounds current, so that the
      // other warps never wait on those (contended) global words
      for (uint32_t spin = 0; spin < wait_limit; ++spin) {
        if (*s_done >= (gg + 1) * EPI_WARPS || *s_abort) break;
        // (1) This CTA condenses the slots of the parents it is responsible for (parent p belongs to tile
        // p mod ntiles) into two words per parent; (2) every CTA reads the condensed words of its rows.
        // Only one CTA per parent reads the slot lines, which the whole launch is hitting with
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
          if (in && a.thr0) {   // never below the seed bounds
            rL[k] = max(rL[k], __ldcg(a.thr0 + p));
            rK[k] = max(rK[k], __ldcg(a.thr0 + (size_t)a.cap + p));
          }
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
          if (rr < per && p < P) { s_thr[pbase + rr] = rL[k]; s_thr[pbase + 128 + rr] = rK[k]; }
        }
        if (spin >= 48u) __nanosleep(500);   // poll flat out while the launch warms up, then back off
      }
      __syncwarp();
    } else if (warp >= W_SEL) {
      // ======================= selector warps ==========================================================
      const int sel = warp - W_SEL;
      unsigned head = sh.q_head[sel];
      const int done_target = (gg + 1) * EPI_WARPS;
      for (uint32_t spin = 0; spin < wait_limit; ++spin) {
        if (*s_abort) break;
        const bool finished = *s_done >= done_target;   // read before the tail: pushes precede the tick
        const unsigned tail = *reinterpret_cast<volatile unsigned*>(sh.q_tail + sel);
        const int avail = (int)(tail - head);
        if (avail <= 0) {
          if (finished) break;
          __nanosleep(100);
          continue;
        }
        spin = 0;
        const int n = min(avail, 32);
        uint4 e = make_uint4(0u, 0u, 0u, 0u);
        bool have = false;
        if (lane < n) {
          uint4* slot = sh.q + sel * QCAP + ((head + lane) & (QCAP - 1));
          uint32_t w = 0;
          for (uint32_t t = 0; t < wait_limit; ++t) {   // the producer writes right after claiming: a few cycles
            w = *reinterpret_cast<volatile uint32_t*>(&slot->w);
            if (w == head + lane + 1u || *s_abort) break;
          }
          have = (w == head + lane + 1u);
          __threadfence_block();
          if (have) { e.x = slot->x; e.y = slot->y; e.z = slot->z; }
        }
        __threadfence_block();
        __syncwarp();
        head += (unsigned)n;
        if (lane == 0) sh.q_head[sel] = head;   // the slots may be reused
        // candidates of one row are inserted one after the other (lanes of a row take turns)
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, have ? (int)(e.z & 0xFFu) : -1 - lane);
        const int turn = __popc(peers & ((1u << lane) - 1u));
        const int turns = __reduce_max_sync(0xFFFFFFFFu, have ? turn + 1 : 0);
        for (int t = 0; t < turns; ++t) {
          if (have && turn == t) select_candidate(a, sh, e, ghi, invT, K, tile, R, g, s_thr, pbase, true, lp_req, lp_hash);
          __syncwarp();
        }
      }
    } else if (warp == W_MMA && lane == 0) {
      // ======================= MMA issuer ===========================================================
      const uint32_t ws_addr = smem_u32(Ws), as_addr = smem_u32(As);
      // (UMMA) Blocks go to the tensor cores in pairs (blocks 2x and 2x + 1 belong to neighbouring splits, whose accumulator
      // buffers are neighbours in tensor memory, so one N = 128 instruction per K step fills both: issuing is what
      // limits this warp).  A pair needs the base-logit slabs of its 128 tokens: two bulk-tensor loads into one of
      // NUP ring slots (pair x of the kernel's running count uses slot x % NUP; a slot is free again as soon as the
      // MMAs that read it are done, long before the blocks are scanned).  Within the window of NUP requested pairs,
      // whichever pair has its buffers drained and its slabs landed is issued.  The first slabs are requested
      // before the A tile is complete: they do not depend on it.
      constexpr int NUP = NUB / 2;
      constexpr uint32_t SLAB = (uint32_t)UMMA_REQ * 128u;
      const int npair = (nblk + 1) / 2;
      int base = 0, unext = 0;        // first pair not yet issued; first pair whose slabs are not yet requested
      uint32_t done = 0;              // bit w: pair base + w is issued
      auto request_slabs = [&]() {
        while (unext < npair && unext < base + NUP) {
          const uint32_t gx = ul + (uint32_t)unext, slot = gx % NUP, use = gx / NUP;
          if (use >= 1 && !mbar_test_wait(u_free + slot, (use - 1) & 1)) break;
          const bool two = 2 * unext + 1 < nblk;
          mbar_expect_tx(u_full + slot, two ? 2u * SLAB : SLAB);
          tma_load_box3(Us + (size_t)slot * 2 * SLAB, &tmU, t0 + 2 * unext * BLK_N, u_depth, 0, u_full + slot);
          if (two) tma_load_box3(Us + (size_t)slot * 2 * SLAB + SLAB, &tmU, t0 + (2 * unext + 1) * BLK_N, u_depth, 0, u_full + slot);
          ++unext;
        }
      };
      if (UMMA) request_slabs();
      if (mbar_wait(a_full, gg & 1, s_abort, a.err, wait_limit)) {
        tc_fence_after();
        if (UMMA) {
          const uint32_t us_addr = smem_u32(Us);
          const int KU = UMMA_REQ / 16;   // extra K steps: the one-hot columns against the slabs' rows
          uint32_t spin = 0;
          while (base < npair) {
            request_slabs();
            bool progressed = false;
#pragma unroll
            for (int w = 0; w < NUP; ++w) {
              const int pr = base + w;
              if (pr >= unext || ((done >> w) & 1u)) continue;
              const int nb = 2 * pr;
              const bool two = nb + 1 < nblk;
              const int sp = nb % EPI_S;                      // even: the pair's splits are sp and sp + 1
              const int j = nb / EPI_S, h = j & 1, tb = sp + EPI_S * h;
              const int nuse0 = (nblk - sp + EPI_S - 1) / EPI_S, nuse1 = (nblk - sp - 1 + EPI_S - 1) / EPI_S;
              const int u0 = gg * ((nuse0 + 1 - h) >> 1) + (j >> 1), u1 = gg * ((nuse1 + 1 - h) >> 1) + (j >> 1);
              if (u0 >= 1 && !mbar_test_wait(t_empty + tb, (u0 - 1) & 1)) continue;
              if (two && u1 >= 1 && !mbar_test_wait(t_empty + tb + 1, (u1 - 1) & 1)) continue;
              if (use_tma && gg == gg_tile && !mbar_test_wait(w_full + nb * BLK_N / WBLK, tile_it & 1)) continue;
              const uint32_t gx = ul + (uint32_t)pr, slot = gx % NUP;
              if (!mbar_test_wait(u_full + slot, (gx / NUP) & 1)) continue;
              tc_fence_after();
              const uint32_t idesc = instr_desc(two ? 2 * BLK_N : BLK_N);
              const uint32_t d_tmem = tmem_base + (uint32_t)(tb * BLK_N);
              const uint32_t wb = ws_addr + (uint32_t)nb * slab_bytes, ub = us_addr + slot * 2u * SLAB;
              for (int ks = 0; ks < rp / 16; ++ks)
                mma_bf16(d_tmem, smem_desc(as_addr + (uint32_t)(ks >> 2) * a_slab_bytes + (uint32_t)(ks & 3) * 32u, 16u, 1024u),
                         smem_desc(wb + (uint32_t)ks * 2048u, slab_bytes, 1024u), idesc, ks > 0 ? 1u : 0u);
              for (int ks = 0; ks < KU; ++ks)
                mma_bf16(d_tmem, smem_desc(as_addr + (uint32_t)(rp / 64) * a_slab_bytes + (uint32_t)ks * 32u, 16u, 1024u),
                         smem_desc(ub + (uint32_t)ks * 2048u, SLAB, 1024u), idesc, 1u);
              mma_commit(t_full + tb);
              if (two) mma_commit(t_full + tb + 1);
              mma_commit(u_free + slot);
              done |= 1u << w;
              progressed = true;
            }
            while (done & 1u) { done >>= 1; ++base; }
            if (progressed) { spin = 0; continue; }
            if (*s_abort) break;
            if (++spin > wait_limit) { *s_abort = 1; if (a.err) atomicExch(a.err, 1); break; }
            if (spin > 8) __nanosleep(32);
          }
          ul += (uint32_t)npair;
        } else if (wring) {
          // Streaming form: the tile's 64-token slabs of W pass through a ring of `wring` slots, block nb of the
          // kernel's running count in slot nb % wring; a slot is free again when the MMAs that read it are done.
          // Blocks are issued in order, each as soon as its slab has landed and its accumulator buffer is drained;
          // slabs are requested as far ahead as the ring allows.
          int nb = 0, req = 0;
          uint32_t spin = 0;
          while (nb < nblk) {
            while (req < nblk && req < nb + wring) {
              const uint32_t gx = wl + (uint32_t)req, slot = gx % (uint32_t)wring, use = gx / (uint32_t)wring;
              if (use >= 1 && !mbar_test_wait(w_free + slot, (use - 1) & 1)) break;
              mbar_expect_tx(w_full + slot, slab_bytes);
              tma_load_box(Ws + (size_t)slot * slab_bytes, &tmW, t0 + req * BLK_N, 0, w_full + slot);
              ++req;
            }
            const int sp = nb % EPI_S, nuse = (nblk - sp + EPI_S - 1) / EPI_S;
            const int j = nb / EPI_S, h = j & 1, tb = sp + EPI_S * h;
            const int u = gg * ((nuse + 1 - h) >> 1) + (j >> 1);
            const uint32_t gx = wl + (uint32_t)nb, slot = gx % (uint32_t)wring;
            if (nb < req && (u < 1 || mbar_test_wait(t_empty + tb, (u - 1) & 1)) && mbar_test_wait(w_full + slot, (gx / (uint32_t)wring) & 1)) {
              tc_fence_after();
              const uint32_t idesc = instr_desc(BLK_N);
              const uint32_t d_tmem = tmem_base + (uint32_t)(tb * BLK_N);
              for (int ks = 0; ks < rp / 16; ++ks) {
                const uint64_t adesc = smem_desc(as_addr + (uint32_t)(ks >> 2) * a_slab_bytes + (uint32_t)(ks & 3) * 32u, 16u, 1024u);
                const uint64_t bdesc = smem_desc(ws_addr + slot * slab_bytes + (uint32_t)ks * 2048u, slab_bytes, 1024u);
                mma_bf16(d_tmem, adesc, bdesc, idesc, ks > 0 ? 1u : 0u);
              }
              mma_commit(t_full + tb);
              mma_commit(w_free + slot);
              ++nb;
              spin = 0;
              continue;
            }
            if (*s_abort) break;
            if (++spin > wait_limit) { *s_abort = 1; if (a.err) atomicExch(a.err, 1); break; }
            if (spin > 8) __nanosleep(32);
          }
          // gave up with slabs on their way: they write this CTA's shared memory, so wait for them (bounded)
          for (int x = nb; x < req; ++x) {
            const uint32_t gx = wl + (uint32_t)x, slot = gx % (uint32_t)wring;
            bool landed = false;
            for (uint32_t t = 0; t < WAIT_LIMIT && !landed; ++t) { landed = mbar_test_wait(w_full + slot, (gx / (uint32_t)wring) & 1); if (!landed) __nanosleep(100); }
          }
          wl += (uint32_t)nblk;
        } else {
        // each split's pipeline advances on its own: whichever buffer is drained (and whose W block has landed) is refilled
        int nxt[EPI_S];
#pragma unroll
        for (int i = 0; i < EPI_S; ++i) nxt[i] = i;
        int remaining = nblk;
        uint32_t spin = 0;
        while (remaining > 0) {
          bool progressed = false;
#pragma unroll
          for (int sp = 0; sp < EPI_S; ++sp) {
            const int nb = nxt[sp];
            if (nb >= nblk) continue;
            const int nuse = (nblk - sp + EPI_S - 1) / EPI_S;
            const int j = nb / EPI_S, h = j & 1, tb = sp + EPI_S * h;
            const int u = gg * ((nuse + 1 - h) >> 1) + (j >> 1);
            if (u >= 1 && !mbar_test_wait(t_empty + tb, (u - 1) & 1)) continue;
            if (use_tma && gg == gg_tile && !mbar_test_wait(w_full + nb * BLK_N / WBLK, tile_it & 1)) continue;
            tc_fence_after();
            const uint32_t idesc = instr_desc(BLK_N);
            const uint32_t d_tmem = tmem_base + (uint32_t)(tb * BLK_N);
            for (int ks = 0; ks < rp / 16; ++ks) {
              const uint64_t adesc = smem_desc(as_addr + (uint32_t)(ks >> 2) * a_slab_bytes + (uint32_t)(ks & 3) * 32u, 16u, 1024u);
              const uint64_t bdesc = smem_desc(ws_addr + (uint32_t)nb * slab_bytes + (uint32_t)ks * 2048u, slab_bytes, 1024u);
              mma_bf16(d_tmem, adesc, bdesc, idesc, ks > 0 ? 1u : 0u);
            }
            mma_commit(t_full + tb);
            nxt[sp] = nb + EPI_S;
            --remaining;
            progressed = true;
          }
          if (progressed) { spin = 0; continue; }
          if (*s_abort) break;
          if (++spin > wait_limit) { *s_abort = 1; if (a.err) atomicExch(a.err, 1); break; }
          if (spin > 8) __nanosleep(32);
        }
        }
      }
      if (UMMA && base < npair) {
        // gave up with slabs on their way: do not go on (to the tear-down) while a bulk load may still be writing
        // this CTA's shared memory
        for (int w = 0; w < NUP; ++w) {
          const int pr = base + w;
          if (pr >= unext || ((done >> w) & 1u)) continue;
          const uint32_t gx = ul + (uint32_t)pr, slot = gx % NUP;
          bool landed = false;
          for (uint32_t t = 0; t < WAIT_LIMIT && !landed; ++t) { landed = mbar_test_wait(u_full + slot, (gx / NUP) & 1); if (!landed) __nanosleep(100); }
        }
      }
    }
    // ---- the group is over: one record per row -----------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (*s_abort) { dead = true; break; }
    if (tid < 128) {
      const int row = tid;
      const int p = R > 1 ? row % per : g * 128 + row;
      if (p < P) {
        // the splits' (max, sums) in split order: the same bits on every run
        float m = -INFINITY, s0 = 0.f, sT = 0.f;
#pragma unroll
        for (int s = 0; s < EPI_S; ++s) {
          const float3 h = make_float3(s_part[(0 * EPI_S + s) * 128 + row], s_part[(1 * EPI_S + s) * 128 + row], s_part[(2 * EPI_S + s) * 128 + row]);
          if (h.x == -INFINITY) continue;
          if (h.x > m) { const float d = m - h.x; s0 *= __expf(d); sT *= __expf(d * invT); m = h.x; }
          const float d = h.x - m;
          s0 += h.y * __expf(d); sT += h.z * __expf(d * invT);
        }
        const int prow = pbase + (R > 1 ? row % per : row);
        const float gL = dec_f(s_thr[prow]), gK = dec_f(s_thr[128 + prow]);
        const float* L = sh.lists + (size_t)row * 5 * K;
        const int* Li = reinterpret_cast<const int*>(L);
        const int gslot = R > 1 ? row : g * 128 + row;
        float* rec = a.rec + ((size_t)tile * a.cap + gslot) * rw;
        int* reci = reinterpret_cast<int*>(rec) + 4;   // the lists go out as the bits they are (two of the five hold tokens)
        int nt = 0, nk = 0;
        for (int j = 0; j < 5 * K; ++j) reci[j] = Li[j];
        for (int j = 0; j < K; ++j) { nt += (Li[K + j] >= 0 && L[j] >= gL); nk += (Li[3 * K + j] >= 0 && L[2 * K + j] >= gK); }
        *reinterpret_cast<float4*>(rec) = make_float4(m, s0, sT, __int_as_float(nt | (nk << 8)));
      }
    }
    __syncthreads();
    ++gg;
  }
  if (!persist || dead) break;
  // ---- persistent form: merge, level step, next level -------------------------------------------------------
  {
    // queues, lists and partial sums are idle between scans; in the streaming form so is the (larger) ring of W slabs:
    // every slab of the level was consumed before its last group ended, and none is requested ahead of a level
    unsigned char* ov = wring ? Ws : reinterpret_cast<unsigned char*>(sh.q);
    const unsigned nexpect = gridDim.x + (pa.lost_arrival ? 1u : 0u);
    __threadfence();   // this CTA's records
    if (!grid_barrier(pa.barrier, nexpect, gen, wait_limit)) { dead = true; break; }
    if (tid < MERGE_THREADS) {
      MergeArgs mg = pa.mg;
      mg.P = P; mg.P_dev = nullptr;
      for (int p = blockIdx.x; p < P; p += gridDim.x) {
        if (BIGK) merge_parent<KMAX>(mg, p, P, *reinterpret_cast<MergeSmem*>(ov), tid, NamedSync<1, MERGE_THREADS>());
        else merge_parent<8>(mg, p, P, *reinterpret_cast<MergeSmem*>(ov), tid, NamedSync<1, MERGE_THREADS>());
      }
    }
    __threadfence();   // merged results
    if (!grid_barrier(pa.barrier, nexpect, gen, wait_limit)) { dead = true; break; }
    if (tid < LEVEL_THREADS) {
      for (int b = blockIdx.x; b < pa.ex.B; b += gridDim.x)
        level_step(pa.ex, lvl, (scout && lvl + 1 < pa.nlevels) ? 1 : 0, b, *reinterpret_cast<LevelSmem*>(ov),
                   ov + ((sizeof(LevelSmem) + 15) & ~(size_t)15), tid, NamedSync<2, LEVEL_THREADS>());
    }
    __syncthreads();
    for (int i = tid; i < NSEL * QCAP; i += MMA_THREADS) sh.q[i] = make_uint4(0u, 0u, 0u, 0u);   // the queues' tags start clean again
    __threadfence();   // next level's parent list and seed bounds
    if (!grid_barrier(pa.barrier, nexpect, gen, wait_limit)) { dead = true; break; }
    if (lvl + 1 >= pa.nlevels || __ldcg(pa.ex.lvl_count + lvl + 1) <= 0) break;
  }
  }
  // ---- the next tile of this CTA (never in the persistent form, whose grid covers the tiles) ---------------
  if (persist || dead || *s_abort || gg == gg_tile || tile + (int)gridDim.x >= a.ntiles) break;
  // Every block of the finished tile was drained, so the MMAs that read its W are done, and the barrier that ended
  // the last group has every thread past its scan: the W tile may be overwritten.
  tile += (int)gridDim.x; ++tile_it;
  t0 = tile * TV; tlen = min(TV, V - t0); nblk_w = (tlen + WBLK - 1) / WBLK;
  if (use_tma) { if (tid == 0) issue_w(); }
  else { fill_w_plain(); fence_async_smem(); __syncthreads(); }
  }
  if (dead && persist && tid == 0) { atomicExch(pa.barrier + 1, 1u); if (a.err) atomicExch(a.err, 1); }
  // ---- tear-down -----------------------------------------------------------------------------------
  if (use_tma && tid == 0 && w_issued && (*s_abort || dead || gg == gg_tile)) {
    // gave up somewhere, or nothing to score: do not leave while a bulk load may still be writing this
    // CTA's shared memory
    for (int nb = 0; nb < nblk_w; ++nb) {
      bool done = false;
      for (uint32_t i = 0; i < WAIT_LIMIT && !done; ++i) { done = mbar_test_wait(w_full + nb, tile_it & 1); if (!done) __nanosleep(100); }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == W_MMA) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// shared memory beside the W tile: A tile, noise tables, queues, lists, bounds, partial sums, barriers
static size_t mma_fixed_smem(const ts_config& c, bool umma) {
  const size_t rp = (size_t)(c.r + 63) / 64 * 64;
  const size_t K = (size_t)c.K;
  return (rp / 64 + (umma ? 1 : 0)) * 128 * 128 + (umma ? (size_t)NUB * UMMA_REQ * 128 : 0) + 512 * 4 + (size_t)NSEL * QCAP * 16 + 128 * 5 * K * 4 + 2 * 128 * 4 +
         2 * EPI_S * 128 * 4 + 3 * EPI_S * 128 * 4 + 512 * 4 + (1 + 2 * NBUF + 2 * MAX_BLK + 2 * NUB) * 8 + 64 + 1024;
}

// tile size for the tensor-core path: W tile + the rest within the shared-memory limit,
// a whole number of waves over the SMs
static bool choose_tile_mma_for(const ts_config& c, int num_sms, int max_smem, bool umma, TileCfg* out) {
  const size_t rp = (size_t)(c.r + 63) / 64 * 64;
  const size_t fixed = mma_fixed_smem(c, umma);
  out->umma = umma ? 1 : 0;
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
  out->smem = (size_t)(tv / 64) * rp * 128 + fixed;
  out->w_ring = 0;
  return out->ntiles <= 4096;
}

// Streaming form for ranks at which a resident W tile would take more than one wave of CTAs: one tile per SM, W
// in 64-token slabs through a ring that takes what shared memory is left (the scanning threads add the base logits).
static bool choose_stream_mma(const ts_config& c, int num_sms, int max_smem, TileCfg* out) {
  const size_t rp = (size_t)(c.r + 63) / 64 * 64;
  const size_t fixed = mma_fixed_smem(c, false);
  if ((size_t)max_smem < fixed + 3 * rp * 128) return false;
  int ring = (int)(((size_t)max_smem - fixed) / (rp * 128));
  if (ring > MAX_BLK) ring = MAX_BLK;
  const int tv = ((c.V + num_sms - 1) / num_sms + 63) / 64 * 64;
  if (tv > 4096) return false;
  out->TV = tv; out->ntiles = (c.V + tv - 1) / tv; out->umma = 0; out->w_ring = ring;
  out->smem = (size_t)ring * rp * 128 + fixed;
  return true;
}

// With room for the one-hot slab and the base-logit slabs (base logits through the MMA) unless that costs waves: at
// large ranks the W tile is what shared memory is short of, and every wave pays the kernel's set-up again.
bool choose_tile_mma(const ts_config& c, int num_sms, int max_smem, bool allow_stream, TileCfg* out) {
  TileCfg with{}, without{};
  const bool ok_with = choose_tile_mma_for(c, num_sms, max_smem, true, &with);
  const bool ok_without = choose_tile_mma_for(c, num_sms, max_smem, false, &without);
  auto waves = [&](const TileCfg& t) { return (t.ntiles + num_sms - 1) / num_sms; };
  TileCfg stream{};
  const bool ok_stream = allow_stream && choose_stream_mma(c, num_sms, max_smem, &stream);
  if (!ok_with && !ok_without && !ok_stream) return false;
  if (ok_with || ok_without) *out = (ok_with && (!ok_without || waves(with) <= waves(without))) ? with : without;
  if (ok_stream && ((!ok_with && !ok_without) || waves(*out) > 1)) *out = stream;
  return true;
}

cudaError_t score_mma_setup(ts_ctx* ctx) {
  cudaError_t e = cudaFuncSetAttribute(score_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->tile.smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(score_mma_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->tile.smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(score_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->tile.smem);
}

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

// Tensor map of the base logits U = [B][D][V] bf16 for boxes of 64 tokens x 1 depth x UMMA_REQ requests (requests past
// B arrive as zeros), in the 128-byte swizzle of a B-operand slab whose K rows are the requests.
static bool u_tensor_map(ts_ctx* ctx, const void* U, int B) {
  if (ctx->tma_state != 1 || !g_encode || ((uintptr_t)U & 15u) != 0 || B < 1 || B > UMMA_REQ) return false;
  if (ctx->tmapU_ptr == U && ctx->tmapU_B == B) return true;
  const ts_config& c = ctx->cfg;
  const cuuint64_t gdim[3] = {(cuuint64_t)c.V, (cuuint64_t)c.D, (cuuint64_t)B};
  const cuuint64_t gstride[2] = {(cuuint64_t)c.V * 2, (cuuint64_t)c.V * 2 * (cuuint64_t)c.D};
  const cuuint32_t box[3] = {64u, 1u, (cuuint32_t)UMMA_REQ};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  CUtensorMap tm;
  const CUresult rc = g_encode(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(U), gdim, gstride, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (rc != CUDA_SUCCESS) return false;
  memcpy(ctx->tmapU, &tm, sizeof(tm));
  ctx->tmapU_ptr = U; ctx->tmapU_B = B;
  return true;
}

// base logits through the tensor cores: every parent at one known depth, few enough requests, bulk-tensor loads available
static bool use_umma(ts_ctx* c, const ScoreArgs& a, bool persist, int use_tma) {
  return c->tile.umma && use_tma && (persist || a.u_depth >= 0) && a.u_B >= 1 && a.u_B <= UMMA_REQ && !(c->test_mode & TS_TEST_NO_UMMA) &&
         u_tensor_map(c, a.U, a.u_B);
}

cudaError_t launch_score_mma(const ts_ctx* ctx, const ScoreArgs& a, cudaStream_t st) {
  ts_ctx* c = const_cast<ts_ctx*>(ctx);
  const int use_tma = w_tensor_map(c, a.W) ? 1 : 0;
  CUtensorMap tm;
  memcpy(&tm, c->tmapW, sizeof(tm));
  PersistArgs pa{};   // pa.on = 0: one scan
  CUtensorMap tu;
  memset(&tu, 0, sizeof(tu));
  const bool umma = use_umma(c, a, false, use_tma);
  if (umma) memcpy(&tu, c->tmapU, sizeof(tu));
  const int grid = a.ntiles < ctx->num_sms ? a.ntiles : ctx->num_sms;   // one CTA per SM at most: a CTA takes its tiles in turn
  if (a.w_ring > 0 && !use_tma) return cudaErrorNotSupported;           // the streaming form moves W by bulk-tensor loads only
  const cudaError_t e = umma ? launch_kernel(score_mma_kernel<true>, grid, MMA_THREADS, ctx->tile.smem, st, a.pdl != 0, a, tm, use_tma, pa, tu)
                             : launch_kernel(score_mma_kernel<false>, grid, MMA_THREADS, ctx->tile.smem, st, a.pdl != 0, a, tm, use_tma, pa, tu);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// Shared memory that is idle between two scans (queues, lists, local thresholds, published bests, partial sums):
// the merge and the level step of the persistent form work in it.
static size_t persist_overlay_bytes(const ts_config& c) {
  return (size_t)NSEL * QCAP * 16 + (size_t)128 * 5 * c.K * 4 + 2 * 128 * 4 + 2 * EPI_S * 128 * 4 + 3 * EPI_S * 128 * 4;
}

bool persistent_supported(const ts_ctx* ctx, int B, int first_level) {
  const ts_config& c = ctx->cfg;
  if (!ctx->use_mma || (c.K > 8 && !ctx->tile.w_ring)) return false;   // (only the streaming form's instantiation carries the merge with 16-entry lists)
  if (ctx->few_ok) {
    // Levels that can hold only a few parents run on the few-parents kernel, which neither scouts nor takes seed bounds:
    // the cooperative launch must start at a level that the tensor-core kernel serves, and (unless it starts at the
    // root, where a seed launch precedes it) so must the level before, whose scouts feed its first seed bounds.
    long long bound = B;
    for (int l = 0; l < (first_level > 0 ? first_level - 1 : 0); ++l) bound = bound * c.K < (long long)B * c.Nmax ? bound * c.K : (long long)B * c.Nmax;
    if (bound <= FEW_MAX) return false;
  }
  if (ctx->tile.ntiles > ctx->num_sms) return false;          // every CTA must be resident: the phases are separated by grid barriers
  const size_t ov = ctx->tile.w_ring ? (size_t)ctx->tile.w_ring * ((size_t)(c.r + 63) / 64 * 64) * 128 : persist_overlay_bytes(c);
  return sizeof(MergeSmem) <= ov && ((sizeof(LevelSmem) + 15) & ~(size_t)15) + level_smem_bytes(c) <= ov;
}

cudaError_t launch_expand_persistent(const ts_ctx* ctx, const ScoreArgs& a, const PersistArgs& pa, cudaStream_t st) {
  ts_ctx* c = const_cast<ts_ctx*>(ctx);
  int use_tma = w_tensor_map(c, a.W) ? 1 : 0;
  CUtensorMap tm;
  memcpy(&tm, c->tmapW, sizeof(tm));
  CUtensorMap tu;
  memset(&tu, 0, sizeof(tu));
  const bool umma = use_umma(c, a, true, use_tma);
  if (umma) memcpy(&tu, c->tmapU, sizeof(tu));
  const void* fn = umma ? (const void*)score_mma_kernel<true>
                        : (ctx->cfg.K > 8 ? (const void*)score_mma_kernel<false, true> : (const void*)score_mma_kernel<false>);
  void* kargs[] = {(void*)&a, (void*)&tm, (void*)&use_tma, (void*)&pa, (void*)&tu};
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.ntiles); cfg.blockDim = dim3(MMA_THREADS); cfg.dynamicSmemBytes = ctx->tile.smem; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative; attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization; attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = c->persist_pdl >= 0 ? 2 : 1;
  cudaError_t e = cudaLaunchKernelExC(&cfg, fn, kargs);
  if (e != cudaSuccess && cfg.numAttrs == 2) {   // not accepted together: remember, and launch cooperative only
    (void)cudaGetLastError();
    c->persist_pdl = -1;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelExC(&cfg, fn, kargs);
  }
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ts
