/*
 * TreeSpark CPU oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, double-precision restatement of one TreeSpark round as the paper defines it:
 * parent-conditioned scoring (Eq. 1), without-replacement sibling draws (Eq. 2), calibrated edge
 * estimates (Eq. 3), best-first expansion with the theta stop (Algorithm 1, Section 3.5), tree
 * mask emission (Section 3.2 item 3) and lossless verification (Section 3.3).  Only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may call it.  It shares no code with the
 * CUDA library and never includes its headers.
 *
 * Pinned by tests against: Philox known-answer vectors, softmax normalisation, the Platt closed
 * form, survival = product of edge estimates, brute-force slot enumeration on tiny trees, the
 * iterated arg-max chain, brute-force greedy target paths, the vector-form vs scalar-form sibling
 * residuals, and chi-square losslessness / sampling-order tests.
 * Parity unpinned: the individual sampled outcomes at T>0 (accepted length and tokens of one
 * seeded round) have no external reference beyond those distributional tests.
 */
#ifndef TREESPARK_ORACLE_H
#define TREESPARK_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORC_KMAX 16
#define ORC_DMAX 16
#define ORC_CALIB_KNOTS 16
#define ORC_TOPK_MARGIN 4e-6  /* relative gap below which two candidates count as a near-tie */

/* flag bits (per request) */
#define ORC_FLAG_NEAR_TOPK   1u   /* near-tie among candidates that decided a materialised child or its rank */
#define ORC_FLAG_NEAR_THETA  2u   /* a slot key within 1e-4 (log) of the stop price */
#define ORC_FLAG_NEAR_CAP    4u   /* last admitted and first excluded key within 1e-4 (log) at the node cap */
#define ORC_FLAG_NEAR_ACCEPT 8u   /* an accept test with |u - rho| below the accept margin */
#define ORC_FLAG_NEAR_CDF    16u  /* bonus draw within 1e-6 (relative mass) of a CDF step */
#define ORC_FLAG_SATURATED   32u  /* some q0 above 0.999: fp32 loses digits in 1-q0 */
#define ORC_FLAG_ZERO_MASS   64u  /* a residual lost all its mass; previous residual kept */

typedef struct {
  int32_t V, D, r, K, Nmax;
  int32_t calib_mode;            /* 0 = Platt scalars, 1 = per-depth table */
  double platt_a, platt_b;
  double calib_lo, calib_hi;     /* knot range in logit(q0) */
  const double* calib_table;     /* [D][16] when calib_mode == 1 */
  int32_t calib_input;           /* 0 = the calibrator is fed the untempered q0 (the method); 1 = it is fed
                                    q_T when T > 0 (the ablation of Section 5.5) */
} orc_config;

/* Philox4x32-10 (Salmon et al., SC'11). */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
/* path hash of a child given its parent's hash and its token; hash(root) = 0 */
uint64_t orc_path_hash(uint64_t parent_hash, int32_t token);
/* uniforms in (0,1) of the three library streams */
double orc_u_gumbel(uint64_t seed, int32_t req, uint64_t hash, int32_t v);
double orc_u_accept(uint64_t seed, int32_t req, uint64_t hash, int32_t j);
double orc_u_bonus(uint64_t seed, int32_t req, uint64_t hash);

/* calibrated edge estimate p-hat for a child of a parent at depth d, from t = logit q0 */
double orc_calib(const orc_config* cfg, int32_t d, double t);

/* logits of one parent: l[v] = U_row[v] + sum_k a_row[k] * W[k*V+v] */
void orc_logits(const orc_config* cfg, const float* U_row, const float* a_row, const float* W, double* l);

/* logit of q0(x) = l_x - log sum_{w != x} exp(l_w), given m = max l and s0 = sum exp(l - m) */
double orc_logit_q0(const double* l, int32_t V, int32_t x, double m, double s0);

/* Score one parent.  top_*: K best logits (value desc, ties lowest token).  draw_*: at T>0 the K
 * without-replacement draws in draw order (largest perturbed keys), at T==0 a copy of top_*.
 * margins (optional, may be NULL), 2K doubles: [j] = gap between the j-th and (j+1)-th largest logit
 * relative to max(1,|l|) (the (K+1)-th included), [K+j] = the same for the sampling keys. */
void orc_score_parent(const orc_config* cfg, const float* U_row, const float* a_row, const float* W,
                      double T, uint64_t seed, int32_t req, uint64_t hash,
                      double* lse0, double* lseT, int32_t* top_tok, double* top_logit,
                      int32_t* draw_tok, double* draw_logit, double* draw_key, double* margins);

/* Algorithm 1 for one request.  U_req = [D][V].  Outputs in canonical (BFS) order, arrays of Nmax
 * (node_hash: Nmax+1, slot 0 = root; mask: Nmax * ceil(Nmax/64) words).  Returns the node count. */
int32_t orc_expand_tree(const orc_config* cfg, const float* U_req, const float* A, const float* W,
                        int32_t anchor_tok, double theta, double T, uint64_t seed, int32_t req,
                        int32_t* tok, int32_t* parent, int32_t* depth, int32_t* sib_rank,
                        double* logS, double* q0, double* logqT, double* logkey, int32_t* pop_rank,
                        uint64_t* node_hash, uint64_t* mask, int32_t* n_scored, uint32_t* flags);

/* Verification of one request's tree.  Z = [(n+1)][V], row 0 = root, row 1+i = node i.
 * closed_form = 0: literal vector residual updates; 1: the scalar-sequence form of the same walk.
 * edge_stat may be NULL.  accept_margin: |u-rho| below it sets ORC_FLAG_NEAR_ACCEPT. */
void orc_verify_tree(const orc_config* cfg, const float* U_req, const float* A, const float* W,
                     const float* Z, int32_t anchor_tok, int32_t n, const int32_t* tok,
                     const int32_t* parent, const int32_t* depth, const int32_t* sib_rank,
                     const uint64_t* node_hash, double T, uint64_t seed, int32_t req,
                     int32_t closed_form, double accept_margin,
                     int32_t* acc_len, int32_t* acc_node, int32_t* acc_tok, int32_t* bonus_tok,
                     double* edge_stat, uint32_t* flags);

/* ---- test support: many seeded one-request rounds on a tiny vocabulary -------------------------
 * Z_path holds target logits for every token path of length 0..D: rows indexed by
 * path_index(path) = sum over prefix lengths of V^len offsets (root = 0; a path (x1..xk) has index
 * off_k + ((x1*V + x2)*V + ...), off_k = (V^k - 1)/(V - 1)).  For trial t the seed is seed0 + t.
 * mode 0: the method (sampled expansion + recursive rejection).
 * mode 1: biased control: deterministic top-k children with the same rejection walk.
 * hist1[V] counts the first committed token, hist2[V*V] the first two committed tokens. */
void orc_lossless_trials(const orc_config* cfg, const float* U_req, const float* A, const float* W,
                         const float* Z_path, int32_t anchor_tok, double theta, double T,
                         uint64_t seed0, int64_t trials, int32_t mode, int32_t closed_form,
                         int64_t* hist1, int64_t* hist2, double* mean_nodes, double* mean_acc);

/* ordered K-tuples drawn by the perturbed-key rule for one parent, counted into hist[V^K]
 * (index = ((x1*V)+x2)*V+...), trial t uses seed0 + t. */
void orc_draw_order_trials(const orc_config* cfg, const float* U_row, const float* a_row, const float* W,
                           double T, uint64_t seed0, int64_t trials, int64_t* hist);

#ifdef __cplusplus
}
#endif
#endif
