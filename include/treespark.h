/*
 * treespark.h -- C ABI of the B200 (sm_100a) hot path of one TreeSpark decoding round.
 *
 * Three calls follow the round as the paper states it (Section 3.2, Algorithm 1, Section 3.3):
 *   ts_score_parents  parent-conditioned scoring with sibling candidates   (Eq. 1, Eq. 2)
 *   ts_expand_tree    calibrated best-first expansion with the theta stop  (Algorithm 1, Eq. 3, Section 3.5)
 *   ts_verify_tree    lossless verification, accepted path + bonus token   (Section 3.2 item 3, Section 3.3)
 *
 * Conventions
 *   - Every function returns a status (TS_OK = 0, negative = error).  No exception crosses the ABI.
 *   - Pointers marked DEVICE are CUDA device addresses owned by the caller and must be 16-byte
 *     aligned; pointers marked HOST are host addresses read during the call only.
 *   - The three hot calls allocate nothing, never synchronise with the host and enqueue all work on
 *     the caller's stream (a cudaStream_t passed as void*).  Scratch memory is the caller's
 *     workspace of at least ts_workspace_bytes() bytes; its contents are undefined between calls.
 *   - Problems found on the device (NaN logits, zero residual mass, a barrier that timed out) are
 *     reported per request in the caller's status[] array, readable after the stream has drained.
 *   - Indices: draft depth d of a PARENT is 0-based (the root has depth 0); its children live at
 *     depth d+1 in 1..D and are scored with base-logit row U[request][d].
 *   - Random numbers: Philox4x32-10, key = seed, counter = (index, path hash of the node (64 bit),
 *     request | stream << 24).  Stream 1/2 give the high / low 16 bits of the sampling uniform of
 *     token v (index = v / 8: one call serves eight consecutive tokens, one half-word each),
 *     stream 3 the accept uniform of sibling j,
 *     stream 4 the bonus uniform.  hash(root) = 0, hash(child) = splitmix64(hash(parent) XOR
 *     (token+1) * 0x9E3779B97F4A7C15).  A draw therefore depends on the node's token path only,
 *     never on the order in which nodes were materialised.
 */
#ifndef TREESPARK_H
#define TREESPARK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TS_OK 0
#define TS_ERR_INVALID (-1)      /* bad argument (NULL or misaligned pointer, size out of range) */
#define TS_ERR_UNSUPPORTED (-2)  /* configuration outside what the kernels are built for */
#define TS_ERR_WORKSPACE (-3)    /* workspace smaller than ts_workspace_bytes() */
#define TS_ERR_CUDA (-4)         /* a CUDA runtime call failed; see ts_last_error_string() */
#define TS_ERR_TIMEOUT (-5)      /* device status: a bounded device-side wait ran out */
#define TS_ERR_OVERFLOW (-6)     /* device status: an internal list overflowed */
#define TS_ERR_NUMERIC (-7)      /* device status: NaN logits or a residual without mass */

#define TS_DTYPE_F32 0
#define TS_DTYPE_BF16 1

#define TS_KMAX 16       /* largest sibling cap K */
#define TS_DMAX 16       /* largest block depth D */
#define TS_CALIB_KNOTS 16

/* per-request flag word written by ts_verify_tree: bits 0..7 flags, bits 8..23 the number of
 * vocabulary-wide residual reductions the walk of that request needed (T > 0; a statistic) */
#define TS_FLAG_ZERO_MASS 64u  /* a residual target lost all mass; the previous residual was kept */
#define TS_FLAGS_MASK 0xFFu

typedef struct ts_ctx ts_ctx;

typedef struct {
  int32_t V, D, r, K, Nmax;  /* vocabulary, block depth, Markov rank, sibling cap, node cap (root excluded) */
  int32_t max_batch;         /* largest B any call will pass */
  int32_t dt_U, dt_A, dt_W, dt_Z; /* TS_DTYPE_*; this build needs all four equal */
  int32_t calib_mode;        /* 0 = Platt scalars (Eq. 3), 1 = per-depth table of TS_CALIB_KNOTS knots */
  float platt_a, platt_b;    /* Eq. 3; the paper's fit is 0.67, -0.46 */
  float calib_lo, calib_hi;  /* knot range in logit(q0), knots uniform, linear interpolation, clamped */
  const float* calib_table;  /* HOST [D][16], non-decreasing in (0,1]; copied at create; NULL for mode 0 */
} ts_config;

/* Create / destroy a context on the current device.  Create copies the calibration table to the
 * device (the only allocation the library ever makes).  Errors: TS_ERR_INVALID, TS_ERR_UNSUPPORTED
 * (K > 16, D > 16, Nmax > 256, r > 256, mixed dtypes), TS_ERR_CUDA. */
int32_t ts_create(const ts_config* cfg, ts_ctx** out);
int32_t ts_destroy(ts_ctx* ctx);

/* Ablation switches for study (Section 5.5); 0, the default, is the method.  Takes effect for calls
 * issued afterwards.  TS_ABLATE_CALIB_QT: at T > 0 the calibrator of ts_expand_tree is fed the tempered
 * conditional q_T instead of the untempered q0 (the paper finds that this inflates the trees and loses
 * the advantage of the price rule).  The marginal-tree ablation needs no switch (pass zero head rows A),
 * nor does the raw priority (Platt mode with a = 1, b = 0). */
#define TS_ABLATE_CALIB_QT 1u
int32_t ts_set_ablation(ts_ctx* ctx, uint32_t flags);

/* Switches for the library's own tests (the paper has no counterpart; 0, the default, is the product).
 * They select kernel paths that the configuration or the device would otherwise select, and shorten
 * or break the bounded device-side waits so that their give-up path can be exercised without hanging
 * anything.  Call it right after ts_create, before ts_workspace_bytes and before any other call on the
 * context: the workspace size depends on the path.  Errors: TS_ERR_INVALID (unknown switch),
 * TS_ERR_UNSUPPORTED (the forced path has no tiling for this configuration), TS_ERR_CUDA.
 *   TS_TEST_FORCE_FMA     bf16 inputs run on the fp32 fused-multiply-add kernels (no tensor cores)
 *   TS_TEST_NO_TMA        the tensor-core kernels stage W with plain loads (no tensor map)
 *   TS_TEST_NO_FEW        levels with few parents run on the tile kernel too
 *   TS_TEST_NO_SEED       the tensor-core scoring kernel runs without seed bounds (no seed kernel ahead of it)
 *   TS_TEST_PERSIST       ts_expand_tree runs every level inside one cooperative launch (scan, merge and level
 *                         step separated by grid barriers; nothing is launched for empty levels) instead of one
 *                         launch per step of every level, where the configuration fits that kernel
 *   TS_TEST_NO_TAIL       ts_expand_tree launches every level's kernels one by one up to the last level, instead of
 *                         handing the levels from the fifth on (mostly empty) to one cooperative launch
 *   TS_TEST_NO_UMMA       the scanning threads of the tensor-core scoring kernel load the base logits themselves
 *                         instead of receiving them through the MMA (the path of batches above 32 requests)
 *   TS_TEST_SHORT_WAITS   bounded waits give up after 4096 polls instead of 2^22
 *   TS_TEST_LOST_ARRIVAL  the walk's grid barriers and the scoring kernel's operand barrier expect one
 *                         arrival more than will come: the waits run out, the kernels return, and the
 *                         requests are reported with TS_ERR_TIMEOUT in status[] */
#define TS_TEST_FORCE_FMA 1u
#define TS_TEST_NO_TMA 2u
#define TS_TEST_NO_FEW 4u
#define TS_TEST_NO_SEED 8u
#define TS_TEST_SHORT_WAITS 16u
#define TS_TEST_LOST_ARRIVAL 32u
#define TS_TEST_PERSIST 64u
#define TS_TEST_NO_UMMA 128u
#define TS_TEST_NO_TAIL 256u
int32_t ts_set_test_mode(ts_ctx* ctx, uint32_t flags);

/* Bytes of workspace the hot calls need for a batch of `batch` requests (<= max_batch). */
size_t ts_workspace_bytes(const ts_ctx* ctx, int32_t batch);

/* Human-readable description of the last error returned on this thread. */
const char* ts_last_error_string(void);

/*
 * Score P parents (Eq. 1; Section 3.2 item 1; Section 5.6 cost per scored node).
 * For parent i = (request parent_req[i], depth parent_depth[i] in [0,D), token parent_token[i]):
 *   l = U[req][depth][:] + A[token][:] . W          (never written to memory)
 *   lse0[i] = log sum exp(l),  lseT[i] = log sum exp(l / T)   (lseT = lse0 when T == 0)
 *   top_*  [i][K]: the K largest logits, value descending, ties to the lowest token
 *   draw_* [i][K]: T > 0: the K without-replacement draws from softmax(l/T) in draw order (Eq. 2),
 *                  realised as the K largest keys l_v/T - log(-log u_v); T == 0: a copy of top_*.
 * Layout: U DEVICE [B][D][V], A DEVICE [V][r], W DEVICE [r][V], all row-major in the context's
 * dtype.  parent_* DEVICE [P]; parent_hash = path hash of the parent node.  Outputs DEVICE.
 * P <= max_batch * Nmax.  Entries beyond the vocabulary size (K > V) hold token -1.
 */
int32_t ts_score_parents(ts_ctx* ctx, const void* U, const void* A, const void* W,
                         int32_t P, const int32_t* parent_req, const int32_t* parent_depth,
                         const int32_t* parent_token, const uint64_t* parent_hash,
                         float T, uint64_t seed,
                         float* lse0, float* lseT,
                         int32_t* top_tok, float* top_logit,
                         int32_t* draw_tok, float* draw_logit,
                         void* ws, size_t ws_bytes, void* stream);

/*
 * ts_score_parents_static -- ts_score_parents without a caller workspace.  (The paper has no
 * counterpart; this exists for deployment reasons only.)
 *
 * Who needs it: code that must score parents but is in no position to get device memory for the
 * library -- for example a plugin inside a serving process whose start-up phase has already handed
 * every free byte of HBM to the KV-cache pool, or a component whose rules forbid cudaMalloc on the
 * request path because it can stall the whole device.  Such a caller still owns its inputs and
 * outputs, but has nowhere to put the scratch that ts_score_parents keeps in `ws`.
 *
 * What it does instead: the per-tile records the scoring pass writes and the merge pass reads live in
 * one array of TS_STATIC_SCRATCH_BYTES (8 MiB) that is part of the library's device image.  Every GPU
 * that loads the library carries that array until the process ends.  The call makes no cudaMalloc,
 * cudaFree or other allocating call, and the results are the same as ts_score_parents'.
 *
 * Limits and rules:
 *   - The array bounds P: every parent slot needs one record of (4 + 5K) words (rounded up to 16 bytes)
 *     per vocabulary tile, plus its pruning-bound words (2K lines of 128 bytes), the array also holds 1 MiB
 *     of scratch for the seed-bound kernel, and slots come in blocks of 128 on the tensor-core path: 256
 *     parents for a 152k vocabulary with K = 8 in bf16 (140 tiles), a few hundred on the fp32 path.  A
 *     larger P is refused with TS_ERR_WORKSPACE and a message that names the limit; nothing is launched.
 *   - The context's device must be the current device.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress) and
 *     remembers it; make that first call before starting any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the last call left in it.
 *     Nothing in it needs clearing (each call overwrites all records it later reads), but two calls
 *     whose kernels overlap on the GPU (different streams, no ordering between them) race on it:
 *     keep calls on one stream, or order them with events.
 * Arguments are those of ts_score_parents minus ws / ws_bytes.
 */
#define TS_STATIC_SCRATCH_BYTES (8u << 20)
int32_t ts_score_parents_static(ts_ctx* ctx, const void* U, const void* A, const void* W,
                                int32_t P, const int32_t* parent_req, const int32_t* parent_depth,
                                const int32_t* parent_token, const uint64_t* parent_hash,
                                float T, uint64_t seed,
                                float* lse0, float* lseT,
                                int32_t* top_tok, float* top_logit,
                                int32_t* draw_tok, float* draw_logit,
                                void* stream);

/*
 * Build the draft trees of B requests (Algorithm 1 with the stop rule of Section 3.5).
 * Slots are admitted in non-increasing order of the candidate survival S(v) * p_hat(best unused
 * token | v) while fewer than Nmax nodes exist and that survival is >= theta[b]; the child token is
 * the best unused token (T == 0) or the next without-replacement draw (T > 0); S(child) = S(v) *
 * p_hat(child | v) with p_hat the calibrated estimate of Eq. 3 fed with the untempered q0.
 * theta[b] >= 1 selects the chain member of the price ladder (Section 4): one child per node,
 * exactly D nodes.  theta[b] == 0 is the fixed budget Nmax.
 *
 * Outputs (all DEVICE), nodes in canonical order: depth ascending, then parent's index, then
 * sibling rank.  Arrays are [B][Nmax] unless noted; entries >= n_nodes[b] are undefined.
 *   n_nodes [B]; tok; parent (-1 = root); depth (1..D); sib_rank (0-based draw order);
 *   logS = log survival; q0 = q0(token | parent); logqT = log q_T(token | parent) (log q0 at T == 0);
 *   logkey = log of the slot key the node was admitted under; pop_rank = best-first admission order;
 *   node_hash [B][Nmax+1] (slot 0 = root); node_lseT [B][Nmax+1] = log-normaliser of q_T(.|node)
 *   (slot 0 = root).  It is defined for the nodes whose conditional was computed: the root and every
 *   node that has children, plus scored nodes all of whose candidates were refused.  A node that was
 *   never a parent (depth D, survival below theta, or admitted when the tree was already full) holds
 *   NaN; ts_verify_tree needs the value only where a node has children;
 *   mask [B][Nmax][ceil(Nmax/64)]: ancestor bitmask, bit i of row i set, root implicit (the tree
 *   attention mask of Section 3.2 item 3; position id = depth);
 *   n_scored [B] = parent conditionals actually computed for the request (Eq. 1 evaluations): one per
 *   node on a level's parent list.  That is at least 1 + the number of nodes with children; it also
 *   counts nodes that were scored and later evicted by the cut to Nmax, and it does not count admitted
 *   nodes that never became parents.  status [B].
 * logkey, pop_rank, node_lseT, n_scored may be NULL.
 */
int32_t ts_expand_tree(ts_ctx* ctx, const void* U, const void* A, const void* W,
                       int32_t B, const int32_t* anchor_tok, const float* theta,
                       float T, uint64_t seed,
                       int32_t* n_nodes, int32_t* tok, int32_t* parent, int32_t* depth,
                       int32_t* sib_rank, float* logS, float* q0, float* logqT,
                       float* logkey, int32_t* pop_rank,
                       uint64_t* node_hash, float* node_lseT, uint64_t* mask,
                       int32_t* n_scored, int32_t* status,
                       void* ws, size_t ws_bytes, void* stream);

/*
 * Verify the trees against target logits (Section 3.2 item 3; Section 3.3).
 * Z DEVICE [rows][V] in dt_Z: request b owns rows z_row_off[b] .. z_row_off[b] + n_nodes[b];
 * its first row is the root, row 1+i is node i.  z_row_off DEVICE int64 [B+1].
 * T == 0: walk from the root to the child whose token equals argmax of the current row (ties to
 *   the lowest token) until none matches; the bonus token is that argmax.
 * T > 0: at a visited node the siblings are tested in draw order; sibling j is accepted with
 *   probability min(1, p_j(x) / q_j(x)), p_1 = softmax(Z[row]/T), q_j = q_T with earlier siblings
 *   removed and renormalised; after a rejection p_{j+1} = norm(max(p_j - q_j, 0)).  When no sibling
 *   is accepted the bonus token is drawn from the current residual by inverse CDF in token order.
 *   The proposal is recomputed from U, A, W; no per-node vocabulary vector is stored.
 *   logqT and node_lseT (from ts_expand_tree) are required when T > 0.
 * Outputs DEVICE: acc_len [B] in [0,D]; acc_node, acc_tok [B][D]; bonus_tok [B];
 *   edge_stat [B][Nmax] or NULL: T == 0 -> 1/0 "token equals the parent's target argmax" for every
 *   edge, T > 0 -> min(1, p(x)/q_T(x)) for every edge; flags [B]; status [B].
 * A request one of whose target rows holds a NaN or no finite mass (T > 0: also an infinite logit), or
 * whose tree carries a NaN proposal probability, is not walked: status TS_ERR_NUMERIC, acc_len 0,
 * bonus_tok -1, edge_stat 0; the other requests of the call are unaffected.
 */
int32_t ts_verify_tree(ts_ctx* ctx, const void* U, const void* A, const void* W,
                       const void* Z, const int64_t* z_row_off, int32_t B,
                       const int32_t* anchor_tok, const int32_t* n_nodes, const int32_t* tok,
                       const int32_t* parent, const int32_t* depth, const int32_t* sib_rank,
                       const uint64_t* node_hash, const float* logqT, const float* node_lseT,
                       float T, uint64_t seed,
                       int32_t* acc_len, int32_t* acc_node, int32_t* acc_tok, int32_t* bonus_tok,
                       float* edge_stat, uint32_t* flags, int32_t* status,
                       void* ws, size_t ws_bytes, void* stream);

/*
 * Cut the trees of a batch back to one node budget (Section 4, "per-request budget allocation").
 * The scheduler chooses the tree sizes N_b that maximise the expected number of accepted tokens under
 * a total of `budget` verified nodes; with concave per-request gain curves greedy water-filling does
 * it: the budget is handed out one node at a time to the request whose next candidate -- in its own
 * best-first admission order, pop_rank -- was admitted under the largest key (logkey; equal keys go
 * to the lowest request, then to the earlier admission).  The gain credited to a candidate is its
 * admission key, never a value drawn for it, so the resulting shapes stay within Proposition 1.
 * With budget = the number of candidates whose key is >= theta this is the theta stop rule.
 *
 * Input: the outputs of ts_expand_tree for the same B (DEVICE, same shapes), logkey and pop_rank
 * required.  The call keeps, per request, the keep[b] nodes admitted first, renumbers them in
 * canonical order (their relative order does not change), rewrites parent and mask to the new
 * numbering and moves every per-node array in place, node_hash and node_lseT (slot 0 = root) included;
 * n_nodes[b] becomes keep[b].  Array arguments other than n_nodes, logkey and pop_rank may be NULL and
 * are then skipped.  log_price DEVICE float[1] or NULL: logkey of the last node handed out, -inf when
 * none was.  budget >= the number of nodes leaves every tree as it is.  Trees of requests on the chain
 * member of the price ladder take part like any other.
 * One CTA selects the price, so the cost grows with B * Nmax (32,768 candidates at most in the
 * workloads this library is sized for).  Errors as for the other calls; nothing is launched on error.
 */
int32_t ts_allocate_budget(ts_ctx* ctx, int32_t B, int32_t budget,
                           int32_t* n_nodes, int32_t* tok, int32_t* parent, int32_t* depth,
                           int32_t* sib_rank, float* logS, float* q0, float* logqT,
                           float* logkey, int32_t* pop_rank,
                           uint64_t* node_hash, float* node_lseT, uint64_t* mask,
                           float* log_price, void* ws, size_t ws_bytes, void* stream);

/*
 * Inputs of the target forward over the flattened trees (Section 3.2 item 3: row i attends to its root
 * path only; a node's position is its depth below the anchor), in a dense layout an attention kernel
 * can take as is.  Per request Nmax + 1 rows: row 0 = the anchor (root), row 1 + i = node i.
 *   flat_tok [B][Nmax+1]: anchor token, then node tokens; -1 in unused rows.
 *   pos_ids  [B][Nmax+1]: base_pos[b] + depth (base_pos DEVICE [B] or NULL = 0); 0 in unused rows.
 *   dense_mask [B][Nmax+1][Nmax+1] float: 0 where the row may attend the column, -inf elsewhere.  An
 *     unused row attends to itself only (a softmax over it stays defined); no used row attends to an
 *     unused column.
 * n_nodes, tok, depth, mask as written by ts_expand_tree.  Any of the three outputs may be NULL.
 * All DEVICE.  No counterpart of this layout is fixed by the paper.
 */
int32_t ts_emit_attention_inputs(ts_ctx* ctx, int32_t B, const int32_t* anchor_tok, const int32_t* base_pos,
                                 const int32_t* n_nodes, const int32_t* tok, const int32_t* depth,
                                 const uint64_t* mask, int32_t* flat_tok, int32_t* pos_ids,
                                 float* dense_mask, void* stream);

/*
 * Calibration statistics from verified trees and the refit of the edge-acceptance map (Section 3.4).
 * Verification labels every materialised edge; the map p_hat (Eq. 3, or the per-depth table) is fitted on
 * the edges whose ancestors were all accepted, the population a path-survival product conditions on.
 *
 * stats: DEVICE uint64 [2][D][TS_CALIB_KNOTS][3], zeroed by the caller before the first call and added
 * to by every call (integer sums: rounds can be accumulated in any order, on any number of streams that
 * do not overlap).  Population 0 = every edge, 1 = edges whose ancestors were all accepted (the parent
 * is the root or lies on the committed path).  Row = depth of the edge's parent (the row of the
 * per-depth table that priced it); cell = the knot nearest to logit(q0) (knots uniform on
 * [calib_lo, calib_hi], the logit clamped to [-30, 30]).  Words of a cell: number of edges; sum of
 * labels in units of 2^-24; sum of (logit + 32) in units of 2^-24.  The label of an edge is edge_stat
 * of ts_verify_tree: 1/0 at T == 0, the first-stage acceptance probability at T > 0.
 *
 * ts_calib_accumulate: adds the edges of B verified trees.  n_nodes, parent, depth, q0 as written by
 * ts_expand_tree (or cut by ts_allocate_budget); acc_len, acc_node, edge_stat as written by
 * ts_verify_tree for those trees.  All DEVICE.
 *
 * ts_calib_refit: from the cells of `population`,
 *   platt DEVICE double[4] (or NULL) = a, b of the maximum-likelihood logistic map over the cells (each
 *     cell = its count of edges at its mean logit with its mean label; depths pooled; Newton's method
 *     from (0, 0), 1e-12 on the Hessian's diagonal, the step halved until the likelihood does not get
 *     worse, at most 100 steps, stop when both move by < 1e-12), the steps taken, the edges used;
 *   table DEVICE float[D][TS_CALIB_KNOTS] (or NULL) = per knot (label sum + 1) / (count + 2) of its cell
 *     (the rule-of-succession estimate: a cell whose edges were all rejected stays away from 0) where
 *     the cell has >= min_count edges, made non-decreasing per depth by weighted pool-adjacent-violators,
 *     knots without data interpolated linearly between neighbours with data and held constant outside,
 *     clamped to [1e-6, 1]; a depth without data takes its row from fallback (DEVICE float[D][16]), or,
 *     when fallback is NULL, from the context's own map sampled at the knots.
 * ts_calib_load_table: copies a DEVICE table [D][16] (non-decreasing rows in (0, 1], as ts_calib_refit
 *   writes them; not checked) into a context created in table mode, in stream order: calls issued after it
 *   on the same stream price edges with the new table.  TS_ERR_INVALID in Platt mode.
 */
int32_t ts_calib_accumulate(ts_ctx* ctx, int32_t B, const int32_t* n_nodes, const int32_t* parent,
                            const int32_t* depth, const float* q0, const int32_t* acc_len,
                            const int32_t* acc_node, const float* edge_stat, uint64_t* stats, void* stream);
int32_t ts_calib_refit(ts_ctx* ctx, const uint64_t* stats, int32_t population, int32_t min_count,
                       const float* fallback, float* table, double* platt, void* stream);
int32_t ts_calib_load_table(ts_ctx* ctx, const float* table, void* stream);

/*
 * Instrumentation (no counterpart in the paper): per-kernel device times and launch counts.
 * ts_profile_enable(capacity > 0) creates `capacity` CUDA event pairs and from then on every kernel
 * the hot calls launch is bracketed by an event pair on the caller's stream until the pairs run out;
 * capacity == 0 switches it off and frees the events.  Launches are always counted.
 * ts_profile_read waits for the recorded events (a host synchronisation: never call it inside a
 * timed region), adds up the elapsed milliseconds and launch counts per kernel id into ms[0..n) and
 * launches[0..n) (HOST arrays; ids >= n are dropped) and, when reset != 0, clears both.
 * ts_kernel_name gives the name of a kernel id, NULL past the last one.
 */
int32_t ts_profile_enable(ts_ctx* ctx, int32_t capacity);
int32_t ts_profile_read(ts_ctx* ctx, int32_t n, double* ms, int64_t* launches, int32_t reset);
const char* ts_kernel_name(int32_t id);

#ifdef __cplusplus
}
#endif
#endif /* TREESPARK_H */
