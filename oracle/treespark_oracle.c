/*
 * TreeSpark CPU oracle -- TEST INFRASTRUCTURE (see treespark_oracle.h).  Plain C, double precision,
 * literal heap, literal sequential walks, no blocking or fusion.
 */
#include "treespark_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------ */
/* Counter-based random numbers                                                                */
/* ------------------------------------------------------------------------------------------ */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static uint64_t splitmix64(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

uint64_t orc_path_hash(uint64_t parent_hash, int32_t token) {
  return splitmix64(parent_hash ^ (((uint64_t)(uint32_t)token + 1ull) * 0x9E3779B97F4A7C15ull));
}

enum { STREAM_GUMBEL_COARSE = 1, STREAM_GUMBEL_FINE = 2, STREAM_ACCEPT = 3, STREAM_BONUS = 4 };

static void stream_words(uint64_t seed, int32_t req, uint64_t hash, uint32_t stream, uint32_t index,
                         uint32_t out[4]) {
  uint32_t ctr[4], key[2];
  ctr[0] = index;
  ctr[1] = (uint32_t)hash;
  ctr[2] = (uint32_t)(hash >> 32);
  ctr[3] = ((uint32_t)req & 0xFFFFFFu) | (stream << 24);
  key[0] = (uint32_t)seed;
  key[1] = (uint32_t)(seed >> 32);
  orc_philox4x32_10(ctr, key, out);
}

/* The sampling uniform of token v is a 32-bit fraction: its high half comes from generator stream 1,
 * its low half from stream 2; each call of either stream serves eight consecutive tokens (one 16-bit
 * half-word per token). */
double orc_u_gumbel(uint64_t seed, int32_t req, uint64_t hash, int32_t v) {
  uint32_t w[4];
  const uint32_t vv = (uint32_t)v;
  stream_words(seed, req, hash, STREAM_GUMBEL_COARSE, vv >> 3, w);
  uint32_t coarse = (w[(vv & 7u) >> 1] >> (16u * (vv & 1u))) & 0xFFFFu;
  stream_words(seed, req, hash, STREAM_GUMBEL_FINE, vv >> 3, w);
  uint32_t fine = (w[(vv & 7u) >> 1] >> (16u * (vv & 1u))) & 0xFFFFu;
  uint32_t x = (coarse << 16) | fine;
  return ((double)x + 0.5) * (1.0 / 4294967296.0);
}

double orc_u_accept(uint64_t seed, int32_t req, uint64_t hash, int32_t j) {
  uint32_t w[4];
  stream_words(seed, req, hash, STREAM_ACCEPT, (uint32_t)j, w);
  return ((double)w[0] + 0.5) * (1.0 / 4294967296.0);
}

double orc_u_bonus(uint64_t seed, int32_t req, uint64_t hash) {
  uint32_t w[4];
  stream_words(seed, req, hash, STREAM_BONUS, 0u, w);
  return ((double)w[0] + 0.5) * (1.0 / 4294967296.0);
}

/* ------------------------------------------------------------------------------------------ */
/* Calibration (Eq. 3; the per-depth table is the benchmark's variant of it)                   */
/* ------------------------------------------------------------------------------------------ */

double orc_calib(const orc_config* cfg, int32_t d, double t) {
  if (t > 30.0) t = 30.0;
  if (t < -30.0) t = -30.0;
  if (cfg->calib_mode == 0) {
    return 1.0 / (1.0 + exp(-(cfg->platt_a * t + cfg->platt_b)));
  }
  const double* y = cfg->calib_table + (size_t)d * ORC_CALIB_KNOTS;
  double pos = (t - cfg->calib_lo) / (cfg->calib_hi - cfg->calib_lo) * (ORC_CALIB_KNOTS - 1);
  if (pos <= 0.0) return y[0];
  if (pos >= ORC_CALIB_KNOTS - 1) return y[ORC_CALIB_KNOTS - 1];
  int i = (int)floor(pos);
  double f = pos - i;
  return y[i] + f * (y[i + 1] - y[i]);
}

/* ------------------------------------------------------------------------------------------ */
/* Scoring (Eq. 1) and sibling draws (Eq. 2 via perturbed keys)                                */
/* ------------------------------------------------------------------------------------------ */

void orc_logits(const orc_config* cfg, const float* U_row, const float* a_row, const float* W, double* l) {
  const int V = cfg->V, r = cfg->r;
  for (int v = 0; v < V; ++v) {
    double acc = (double)U_row[v];
    for (int k = 0; k < r; ++k) acc += (double)a_row[k] * (double)W[(size_t)k * V + v];
    l[v] = acc;
  }
}

double orc_logit_q0(const double* l, int32_t V, int32_t x, double m, double s0) {
  double ex = exp(l[x] - m);
  double rest;
  if (ex <= 0.5 * s0) {
    rest = s0 - ex; /* loses at most one bit */
  } else {
    rest = 0.0;     /* dominant token: sum the others directly, no cancellation */
    for (int w = 0; w < V; ++w)
      if (w != x) rest += exp(l[w] - m);
  }
  if (rest <= 0.0) return 1e300;
  return (l[x] - m) - log(rest);
}

/* K passes of arg-max over not-yet-taken entries: value descending, ties to the lowest index.
 * Also returns in *next the best value left after the K picks (or -inf). */
static void select_top(const double* val, int V, int K, int32_t* out_idx, double* next) {
  char* taken = (char*)calloc((size_t)V, 1);
  for (int j = 0; j <= K; ++j) {
    int best = -1;
    for (int v = 0; v < V; ++v) {
      if (taken[v]) continue;
      if (best < 0 || val[v] > val[best]) best = v;
    }
    if (j < K) {
      out_idx[j] = best;
      if (best >= 0) taken[best] = 1;
    } else if (next) {
      *next = best >= 0 ? val[best] : -INFINITY;
    }
  }
  free(taken);
}

/* gap[j] = (value of pick j - value of pick j+1) / max(1, |value of pick j|); pick K is `next` */
static void rel_gaps(const double* val, const int32_t* idx, int K, double next, double* gap) {
  for (int j = 0; j < K; ++j) {
    gap[j] = INFINITY;
    if (idx[j] < 0) continue;
    double a = val[idx[j]];
    double b = (j + 1 < K) ? (idx[j + 1] >= 0 ? val[idx[j + 1]] : -INFINITY) : next;
    if (!(b > -INFINITY)) continue;
    double scale = fabs(a) > 1.0 ? fabs(a) : 1.0;
    gap[j] = (a - b) / scale;
  }
}

void orc_score_parent(const orc_config* cfg, const float* U_row, const float* a_row, const float* W,
                      double T, uint64_t seed, int32_t req, uint64_t hash,
                      double* lse0, double* lseT, int32_t* top_tok, double* top_logit,
                      int32_t* draw_tok, double* draw_logit, double* draw_key, double* margins) {
  const int V = cfg->V;
  int K = cfg->K < V ? cfg->K : V;
  double* l = (double*)malloc(sizeof(double) * (size_t)V);
  orc_logits(cfg, U_row, a_row, W, l);
  double m = l[0];
  for (int v = 1; v < V; ++v) if (l[v] > m) m = l[v];
  double s0 = 0.0;
  for (int v = 0; v < V; ++v) s0 += exp(l[v] - m);
  *lse0 = m + log(s0);
  if (T > 0.0) {
    double sT = 0.0;
    for (int v = 0; v < V; ++v) sT += exp((l[v] - m) / T);
    *lseT = m / T + log(sT);
  } else {
    *lseT = *lse0;
  }
  for (int j = 0; j < cfg->K; ++j) { top_tok[j] = -1; top_logit[j] = 0.0; draw_tok[j] = -1; draw_logit[j] = 0.0; if (draw_key) draw_key[j] = 0.0; }
  double next = -INFINITY;
  select_top(l, V, K, top_tok, &next);
  for (int j = 0; j < K; ++j) top_logit[j] = l[top_tok[j]];
  if (margins) {
    for (int j = 0; j < 2 * cfg->K; ++j) margins[j] = INFINITY;
    rel_gaps(l, top_tok, K, next, margins);
  }
  if (T > 0.0) {
    /* j-th without-replacement draw = j-th largest of l/T + Gumbel noise (equal in law to Eq. 2) */
    double* key = (double*)malloc(sizeof(double) * (size_t)V);
    for (int v = 0; v < V; ++v) {
      double u = orc_u_gumbel(seed, req, hash, v);
      key[v] = l[v] / T - log(-log(u));
    }
    select_top(key, V, K, draw_tok, &next);
    for (int j = 0; j < K; ++j) { draw_logit[j] = l[draw_tok[j]]; if (draw_key) draw_key[j] = key[draw_tok[j]]; }
    if (margins) rel_gaps(key, draw_tok, K, next, margins + cfg->K);
    free(key);
  } else {
    for (int j = 0; j < K; ++j) { draw_tok[j] = top_tok[j]; draw_logit[j] = top_logit[j]; if (draw_key) draw_key[j] = top_logit[j]; }
  }
  free(l);
}

/* ------------------------------------------------------------------------------------------ */
/* Algorithm 1                                                                                 */
/* ------------------------------------------------------------------------------------------ */

typedef struct {
  int parent;            /* internal index; root = 0, root's parent = -1 */
  int depth, sib, tok;
  uint64_t hash;
  double logS, q0, logqT, logkey;
  unsigned char path[ORC_DMAX];
  int scored, nchild;
  double lse0, lseT;
  int32_t top_tok[ORC_KMAX], draw_tok[ORC_KMAX];
  double top_logit[ORC_KMAX], draw_logit[ORC_KMAX];
  double gap_top[ORC_KMAX], gap_key[ORC_KMAX];
} node_t;

typedef struct {
  double logkey;
  int parent, j;
} slot_t;

/* strict "a is popped before b": key descending, then shallower first, then the sequence of
 * sibling ranks from the root in lexicographic order */
static int slot_before(const node_t* nodes, const slot_t* a, const slot_t* b) {
  if (a->logkey != b->logkey) return a->logkey > b->logkey;
  int da = nodes[a->parent].depth + 1, db = nodes[b->parent].depth + 1;
  if (da != db) return da < db;
  for (int i = 0; i < da - 1; ++i) {
    unsigned char pa = nodes[a->parent].path[i], pb = nodes[b->parent].path[i];
    if (pa != pb) return pa < pb;
  }
  return a->j < b->j;
}

static void heap_push(const node_t* nodes, slot_t* heap, int* n, slot_t s) {
  int i = (*n)++;
  heap[i] = s;
  while (i > 0) {
    int p = (i - 1) / 2;
    if (!slot_before(nodes, &heap[i], &heap[p])) break;
    slot_t t = heap[i]; heap[i] = heap[p]; heap[p] = t;
    i = p;
  }
}

static slot_t heap_pop(const node_t* nodes, slot_t* heap, int* n) {
  slot_t top = heap[0];
  heap[0] = heap[--(*n)];
  int i = 0;
  for (;;) {
    int a = 2 * i + 1, b = a + 1, best = i;
    if (a < *n && slot_before(nodes, &heap[a], &heap[best])) best = a;
    if (b < *n && slot_before(nodes, &heap[b], &heap[best])) best = b;
    if (best == i) break;
    slot_t t = heap[i]; heap[i] = heap[best]; heap[best] = t;
    i = best;
  }
  return top;
}

typedef struct {
  const orc_config* cfg;
  const float *U_req, *A, *W;
  double T, theta_log;
  uint64_t seed;
  int32_t req;
  int K_eff, N_eff, force_topk;
  uint32_t flags;
  int n_scored;
} expand_ctx;

static void score_node(expand_ctx* c, node_t* nd) {
  const orc_config* cfg = c->cfg;
  double margins[2 * ORC_KMAX];
  double top_logit[ORC_KMAX], draw_logit[ORC_KMAX];
  orc_score_parent(cfg, c->U_req + (size_t)nd->depth * cfg->V, c->A + (size_t)nd->tok * cfg->r, c->W,
                   c->force_topk ? 0.0 : c->T, c->seed, c->req, nd->hash,
                   &nd->lse0, &nd->lseT, nd->top_tok, top_logit, nd->draw_tok, draw_logit, NULL, margins);
  for (int j = 0; j < cfg->K; ++j) {
    nd->top_logit[j] = top_logit[j]; nd->draw_logit[j] = draw_logit[j];
    nd->gap_top[j] = margins[j]; nd->gap_key[j] = margins[cfg->K + j];
  }
  if (c->force_topk && c->T > 0.0) {
    /* biased control: children are the modes, but the proposal is still q_T */
    double* l = (double*)malloc(sizeof(double) * (size_t)cfg->V);
    orc_logits(cfg, c->U_req + (size_t)nd->depth * cfg->V, c->A + (size_t)nd->tok * cfg->r, c->W, l);
    double m = l[0];
    for (int v = 1; v < cfg->V; ++v) if (l[v] > m) m = l[v];
    double sT = 0.0;
    for (int v = 0; v < cfg->V; ++v) sT += exp((l[v] - m) / c->T);
    nd->lseT = m / c->T + log(sT);
    free(l);
  }
  nd->scored = 1;
  c->n_scored++;
}

/* logit q0 of token x (logit lx) under a scored parent.  With q = exp(lx - lse0) at most one half,
 * logit q = log q - log(1 - q) is free of cancellation; for a dominant token the "all other tokens"
 * sum is taken directly from the parent's recomputed logit vector. */
static double edge_logit_q0(expand_ctx* c, const node_t* nd, int x, double lx) {
  const orc_config* cfg = c->cfg;
  /* ablation: the calibrator sees the tempered conditional q_T instead of q0 */
  const int tempered = cfg->calib_input == 1 && c->T > 0.0;
  const double scale = tempered ? 1.0 / c->T : 1.0;
  double lq = tempered ? lx / c->T - nd->lseT : lx - nd->lse0;
  double qv = exp(lq);
  if (qv <= 0.5) return lq - log1p(-qv);
  double* l = (double*)malloc(sizeof(double) * (size_t)cfg->V);
  orc_logits(cfg, c->U_req + (size_t)nd->depth * cfg->V, c->A + (size_t)nd->tok * cfg->r, c->W, l);
  if (tempered) for (int v = 0; v < cfg->V; ++v) l[v] *= scale;
  double m = l[0];
  for (int v = 1; v < cfg->V; ++v) if (l[v] > m) m = l[v];
  double s0 = 0.0;
  for (int v = 0; v < cfg->V; ++v) s0 += exp(l[v] - m);
  double t = orc_logit_q0(l, cfg->V, x, m, s0);
  free(l);
  return t;
}

/* index in the top list of the best token of q0(.|v) not yet among v's first j children */
static int best_unused(const expand_ctx* c, const node_t* nd, int j) {
  if (c->T == 0.0 || c->force_topk) return j;
  for (int i = 0; i < c->K_eff; ++i) {
    int t = nd->top_tok[i], used = 0;
    for (int u = 0; u < j; ++u) if (nd->draw_tok[u] == t) used = 1;
    if (!used) return i;
  }
  return -1;
}

static double slot_key(expand_ctx* c, const node_t* nd, int j) {
  int i = best_unused(c, nd, j);
  double t = edge_logit_q0(c, nd, nd->top_tok[i], nd->top_logit[i]);
  double key = nd->logS + log(orc_calib(c->cfg, nd->depth, t));
  if (c->theta_log > -INFINITY && fabs(key - c->theta_log) < 1e-4) c->flags |= ORC_FLAG_NEAR_THETA;
  return key;
}

static int32_t expand_impl(const orc_config* cfg, const float* U_req, const float* A, const float* W,
                           int32_t anchor_tok, double theta, double T, uint64_t seed, int32_t req,
                           int force_topk,
                           int32_t* tok, int32_t* parent, int32_t* depth, int32_t* sib_rank,
                           double* logS, double* q0, double* logqT, double* logkey, int32_t* pop_rank,
                           uint64_t* node_hash, uint64_t* mask, int32_t* n_scored, uint32_t* flags) {
  expand_ctx c;
  memset(&c, 0, sizeof(c));
  c.cfg = cfg; c.U_req = U_req; c.A = A; c.W = W; c.T = T; c.seed = seed; c.req = req;
  c.force_topk = force_topk;
  c.K_eff = cfg->K < cfg->V ? cfg->K : cfg->V;
  c.N_eff = cfg->Nmax;
  if (theta >= 1.0) { /* chain member of the price ladder: one child per node, D nodes, no stop */
    c.K_eff = 1;
    c.N_eff = cfg->D < cfg->Nmax ? cfg->D : cfg->Nmax;
    theta = 0.0;
  }
  c.theta_log = theta > 0.0 ? log(theta) : -INFINITY;

  node_t* nodes = (node_t*)calloc((size_t)c.N_eff + 1, sizeof(node_t));
  slot_t* heap = (slot_t*)malloc(sizeof(slot_t) * (size_t)(2 * c.N_eff + 4));
  int heap_n = 0, n = 0; /* n = materialised nodes, internal indices 1..n */

  nodes[0].parent = -1; nodes[0].depth = 0; nodes[0].tok = anchor_tok; nodes[0].hash = 0; nodes[0].logS = 0.0;
  if (cfg->D > 0 && c.N_eff > 0) {
    score_node(&c, &nodes[0]);
    slot_t s = { slot_key(&c, &nodes[0], 0), 0, 0 };
    heap_push(nodes, heap, &heap_n, s);
  }
  double last_admitted = INFINITY;
  while (n < c.N_eff && heap_n > 0) {
    slot_t s = heap_pop(nodes, heap, &heap_n);
    if (s.logkey < c.theta_log) { heap_n = 0; break; } /* best remaining candidate is below its price */
    node_t* v = &nodes[s.parent];
    int xc = (T == 0.0 || force_topk) ? v->top_tok[s.j] : v->draw_tok[s.j];
    double lx = (T == 0.0 || force_topk) ? v->top_logit[s.j] : v->draw_logit[s.j];
    node_t* cn = &nodes[++n];
    cn->parent = s.parent; cn->depth = v->depth + 1; cn->sib = s.j; cn->tok = xc;
    cn->hash = orc_path_hash(v->hash, xc);
    memcpy(cn->path, v->path, sizeof(cn->path));
    cn->path[v->depth] = (unsigned char)s.j;
    double t = edge_logit_q0(&c, v, xc, lx);
    double ph = orc_calib(cfg, v->depth, t);
    cn->logS = v->logS + log(ph);
    cn->q0 = exp(lx - v->lse0);
    if (cn->q0 > 0.999) c.flags |= ORC_FLAG_SATURATED;
    cn->logqT = (T > 0.0) ? lx / T - v->lseT : lx - v->lse0;
    cn->logkey = s.logkey;
    last_admitted = s.logkey;
    v->nchild = s.j + 1;
    if (cn->depth < cfg->D) {
      score_node(&c, cn);
      slot_t sc = { slot_key(&c, cn, 0), n, 0 };
      heap_push(nodes, heap, &heap_n, sc);
    }
    if (v->nchild < c.K_eff) {
      slot_t sv = { slot_key(&c, v, v->nchild), s.parent, v->nchild };
      heap_push(nodes, heap, &heap_n, sv);
    }
  }
  /* a near-tie among a parent's candidates matters only where it decides which token becomes, or
   * in what order tokens become, one of its materialised children */
  for (int i = 0; i <= n; ++i) {
    const node_t* nd = &nodes[i];
    if (!nd->scored) continue;
    const double* gap = (T == 0.0 || force_topk) ? nd->gap_top : nd->gap_key;
    for (int j = 0; j < nd->nchild && j < cfg->K; ++j)
      if (gap[j] < ORC_TOPK_MARGIN) c.flags |= ORC_FLAG_NEAR_TOPK;
  }
  if (n == c.N_eff && heap_n > 0) {
    double rest = heap[0].logkey;
    double scale = fabs(rest) > 1.0 ? fabs(rest) : 1.0;
    /* bitwise-equal keys come from one parent's unchanged "best unused token" bound (sibling slots
     * at T>0); the (depth, rank path) order settles those identically in any arithmetic */
    if (rest >= c.theta_log && last_admitted != rest && (last_admitted - rest) < 1e-4 * scale)
      c.flags |= ORC_FLAG_NEAR_CAP;
  }

  /* canonical order: depth ascending, then the parent's canonical index, then sibling rank */
  int* canon_of = (int*)malloc(sizeof(int) * (size_t)(n + 1)); /* internal -> canonical (root = -1) */
  int* order = (int*)malloc(sizeof(int) * (size_t)(n + 1));    /* canonical -> internal */
  canon_of[0] = -1;
  int placed = 0;
  for (int d = 1; d <= cfg->D && placed < n; ++d) {
    /* parents at depth d-1 in canonical order: the root, or canonical indices of depth d-1 */
    int first_parent = (d == 1) ? -1 : 0;
    int last_parent = (d == 1) ? 0 : placed; /* exclusive bound on canonical index */
    for (int pc = first_parent; pc < last_parent; ++pc) {
      int pint = (pc < 0) ? 0 : order[pc];
      if (nodes[pint].depth != d - 1) continue;
      for (int j = 0; j < cfg->K; ++j)
        for (int i = 1; i <= n; ++i)
          if (nodes[i].parent == pint && nodes[i].sib == j) { canon_of[i] = placed; order[placed++] = i; }
    }
  }
  const int words = (cfg->Nmax + 63) / 64;
  node_hash[0] = 0;
  for (int ci = 0; ci < n; ++ci) {
    const node_t* nd = &nodes[order[ci]];
    tok[ci] = nd->tok;
    parent[ci] = canon_of[nd->parent];
    depth[ci] = nd->depth;
    sib_rank[ci] = nd->sib;
    logS[ci] = nd->logS;
    q0[ci] = nd->q0;
    logqT[ci] = nd->logqT;
    logkey[ci] = nd->logkey;
    pop_rank[ci] = order[ci] - 1;
    node_hash[ci + 1] = nd->hash;
    /* tree attention mask: a node sees its root path and itself */
    for (int w = 0; w < words; ++w)
      mask[(size_t)ci * words + w] = parent[ci] >= 0 ? mask[(size_t)parent[ci] * words + w] : 0ull;
    mask[(size_t)ci * words + ci / 64] |= 1ull << (ci % 64);
  }
  *n_scored = c.n_scored;
  *flags = c.flags;
  free(order); free(canon_of); free(heap); free(nodes);
  return n;
}

int32_t orc_expand_tree(const orc_config* cfg, const float* U_req, const float* A, const float* W,
                        int32_t anchor_tok, double theta, double T, uint64_t seed, int32_t req,
                        int32_t* tok, int32_t* parent, int32_t* depth, int32_t* sib_rank,
                        double* logS, double* q0, double* logqT, double* logkey, int32_t* pop_rank,
                        uint64_t* node_hash, uint64_t* mask, int32_t* n_scored, uint32_t* flags) {
  return expand_impl(cfg, U_req, A, W, anchor_tok, theta, T, seed, req, 0, tok, parent, depth, sib_rank,
                     logS, q0, logqT, logkey, pop_rank, node_hash, mask, n_scored, flags);
}

/* ------------------------------------------------------------------------------------------ */
/* Verification (Section 3.2 item 3, Section 3.3)                                              */
/* ------------------------------------------------------------------------------------------ */

static int argmax_f(const float* z, int V) {
  int best = 0;
  for (int w = 1; w < V; ++w) if (z[w] > z[best]) best = w;
  return best;
}

static void softmax_T(const float* z, int V, double T, double* p) {
  double m = z[0];
  for (int w = 1; w < V; ++w) if ((double)z[w] > m) m = z[w];
  double s = 0.0;
  for (int w = 0; w < V; ++w) { p[w] = exp(((double)z[w] - m) / T); s += p[w]; }
  for (int w = 0; w < V; ++w) p[w] /= s;
}

static void softmax_d(const double* l, int V, double T, double* q) {
  double m = l[0];
  for (int w = 1; w < V; ++w) if (l[w] > m) m = l[w];
  double s = 0.0;
  for (int w = 0; w < V; ++w) { q[w] = exp((l[w] - m) / T); s += q[w]; }
  for (int w = 0; w < V; ++w) q[w] /= s;
}

/* inverse CDF in token order: smallest w with cumulative mass > u * total */
static int inverse_cdf(const double* mass, int V, double u, uint32_t* flags) {
  double total = 0.0;
  for (int w = 0; w < V; ++w) total += mass[w];
  double target = u * total, cum = 0.0;
  int pick = -1, last_pos = 0;
  for (int w = 0; w < V; ++w) {
    double before = cum;
    cum += mass[w];
    if (mass[w] > 0.0) last_pos = w;
    if (pick < 0 && cum > target) {
      pick = w;
      if (fabs(before - target) < 1e-6 * total || fabs(cum - target) < 1e-6 * total) *flags |= ORC_FLAG_NEAR_CDF;
    }
  }
  if (pick < 0) { pick = last_pos; *flags |= ORC_FLAG_NEAR_CDF; }
  return pick;
}

void orc_verify_tree(const orc_config* cfg, const float* U_req, const float* A, const float* W,
                     const float* Z, int32_t anchor_tok, int32_t n, const int32_t* tok,
                     const int32_t* parent, const int32_t* depth, const int32_t* sib_rank,
                     const uint64_t* node_hash, double T, uint64_t seed, int32_t req,
                     int32_t closed_form, double accept_margin,
                     int32_t* acc_len, int32_t* acc_node, int32_t* acc_tok, int32_t* bonus_tok,
                     double* edge_stat, uint32_t* flags) {
  const int V = cfg->V;
  uint32_t fl = 0;
  double* p = (double*)malloc(sizeof(double) * (size_t)V);
  double* q = (double*)malloc(sizeof(double) * (size_t)V);
  double* l = (double*)malloc(sizeof(double) * (size_t)V);
  double* keep = (double*)malloc(sizeof(double) * (size_t)V);
  char* used = (char*)malloc((size_t)V);

  /* per-edge statistics for every materialised edge (labels for calibration, Section 3.4) */
  if (edge_stat) {
    for (int v = -1; v < n; ++v) {
      int has_child = 0;
      for (int i = 0; i < n; ++i) if (parent[i] == v) has_child = 1;
      if (!has_child) continue;
      const float* zrow = Z + (size_t)(v + 1) * V;
      if (T == 0.0) {
        int g = argmax_f(zrow, V);
        for (int i = 0; i < n; ++i) if (parent[i] == v) edge_stat[i] = (tok[i] == g) ? 1.0 : 0.0;
      } else {
        int dv = v < 0 ? 0 : depth[v];
        int xv = v < 0 ? anchor_tok : tok[v];
        softmax_T(zrow, V, T, p);
        orc_logits(cfg, U_req + (size_t)dv * V, A + (size_t)xv * cfg->r, W, l);
        softmax_d(l, V, T, q);
        for (int i = 0; i < n; ++i)
          if (parent[i] == v) { double ratio = p[tok[i]] / q[tok[i]]; edge_stat[i] = ratio < 1.0 ? ratio : 1.0; }
      }
    }
  }

  int cur = -1, acc = 0;
  for (;;) {
    /* children of cur in draw order */
    int child[ORC_KMAX], m = 0;
    for (int j = 0; j < cfg->K; ++j)
      for (int i = 0; i < n; ++i)
        if (parent[i] == cur && sib_rank[i] == j) child[m++] = i;
    const float* zrow = Z + (size_t)(cur + 1) * V;
    uint64_t hcur = node_hash[cur + 1];
    if (T == 0.0) {
      int g = argmax_f(zrow, V), hit = -1;
      for (int j = 0; j < m; ++j) if (tok[child[j]] == g) hit = child[j];
      if (hit < 0) { *bonus_tok = g; break; }
      acc_node[acc] = hit; acc_tok[acc] = g; ++acc; cur = hit;
      continue;
    }
    softmax_T(zrow, V, T, p);
    int accepted = -1;
    if (m > 0) {
      int dv = cur < 0 ? 0 : depth[cur];
      int xv = cur < 0 ? anchor_tok : tok[cur];
      orc_logits(cfg, U_req + (size_t)dv * V, A + (size_t)xv * cfg->r, W, l);
      softmax_d(l, V, T, q);
    }
    if (!closed_form) {
      /* literal: p is the normalised residual target, q^(j) the renormalised residual proposal */
      memset(used, 0, (size_t)V);
      double Qused = 0.0;
      for (int j = 0; j < m && accepted < 0; ++j) {
        int x = tok[child[j]];
        double qj = q[x] / (1.0 - Qused);
        double ratio = p[x] / qj;
        double rho = ratio < 1.0 ? ratio : 1.0;
        double u = orc_u_accept(seed, req, hcur, j);
        if (fabs(u - rho) < accept_margin && rho < 1.0) fl |= ORC_FLAG_NEAR_ACCEPT;
        if (u < rho) { accepted = child[j]; break; }
        memcpy(keep, p, sizeof(double) * (size_t)V);
        double sum = 0.0;
        for (int w = 0; w < V; ++w) {
          double qw = used[w] ? 0.0 : q[w] / (1.0 - Qused);
          double d = p[w] - qw;
          p[w] = d > 0.0 ? d : 0.0;
          sum += p[w];
        }
        if (sum <= 1e-30) { memcpy(p, keep, sizeof(double) * (size_t)V); fl |= ORC_FLAG_ZERO_MASS; }
        else for (int w = 0; w < V; ++w) p[w] /= sum;
        used[x] = 1;
        Qused += q[x];
      }
      if (accepted < 0) { *bonus_tok = inverse_cdf(p, V, orc_u_bonus(seed, req, hcur), &fl); break; }
    } else {
      /* scalar form: unnormalised residual R(w) = max(p(w) - C q(w), 0) for untested tokens and
       * frozen at max(p(x_i) - C_i q(x_i), 0) for tested siblings; Zj = sum R; c_j = Zj/(1 - Qused) */
      double C = 0.0, Zj = 1.0, Qused = 0.0;
      int fx[ORC_KMAX]; double fC[ORC_KMAX]; int nf = 0;
      for (int j = 0; j < m && accepted < 0; ++j) {
        int x = tok[child[j]];
        double cj = Zj / (1.0 - Qused);
        double num = p[x] / q[x] - C;
        if (num < 0.0) num = 0.0;
        double ratio = num / cj;
        double rho = ratio < 1.0 ? ratio : 1.0;
        double u = orc_u_accept(seed, req, hcur, j);
        if (fabs(u - rho) < accept_margin && rho < 1.0) fl |= ORC_FLAG_NEAR_ACCEPT;
        if (u < rho) { accepted = child[j]; break; }
        double Cn = C + cj;
        double Zn = 0.0;
        for (int w = 0; w < V; ++w) {
          int frozen = (w == x);
          for (int i = 0; i < nf; ++i) if (fx[i] == w) frozen = 1;
          if (frozen) continue;
          double d = p[w] - Cn * q[w];
          if (d > 0.0) Zn += d;
        }
        double fsum = 0.0;
        for (int i = 0; i < nf; ++i) { double d = p[fx[i]] - fC[i] * q[fx[i]]; if (d > 0.0) fsum += d; }
        double dx = p[x] - Cn * q[x];
        if (dx < 0.0) dx = 0.0;
        if (Zn + fsum + dx <= 1e-30 * Zj) { /* residual lost its mass: keep the previous one */
          fl |= ORC_FLAG_ZERO_MASS;
          fx[nf] = x; fC[nf] = C; ++nf;
        } else {
          fx[nf] = x; fC[nf] = Cn; ++nf;
          C = Cn; Zj = Zn + fsum + dx;
        }
        Qused += q[x];
      }
      if (accepted < 0) {
        for (int w = 0; w < V; ++w) {
          double Cw = C;
          for (int i = 0; i < nf; ++i) if (fx[i] == w) Cw = fC[i];
          double d = (m > 0) ? p[w] - Cw * q[w] : p[w];
          keep[w] = d > 0.0 ? d : 0.0;
        }
        *bonus_tok = inverse_cdf(keep, V, orc_u_bonus(seed, req, hcur), &fl);
        break;
      }
    }
    acc_node[acc] = accepted; acc_tok[acc] = tok[accepted]; ++acc; cur = accepted;
  }
  *acc_len = acc;
  *flags = fl;
  free(used); free(keep); free(l); free(q); free(p);
}

/* ------------------------------------------------------------------------------------------ */
/* Test support                                                                                */
/* ------------------------------------------------------------------------------------------ */

static int64_t path_index(const int32_t* tok, const int32_t* parent, int node, int V) {
  /* node = -1 is the root */
  int32_t seq[ORC_DMAX]; int len = 0;
  for (int i = node; i >= 0; i = parent[i]) seq[len++] = tok[i];
  int64_t off = 0, pw = 1;
  for (int k = 0; k < len; ++k) { off += pw; pw *= V; }
  int64_t idx = 0;
  for (int k = len - 1; k >= 0; --k) idx = idx * V + seq[k];
  return off + idx;
}

void orc_lossless_trials(const orc_config* cfg, const float* U_req, const float* A, const float* W,
                         const float* Z_path, int32_t anchor_tok, double theta, double T,
                         uint64_t seed0, int64_t trials, int32_t mode, int32_t closed_form,
                         int64_t* hist1, int64_t* hist2, double* mean_nodes, double* mean_acc) {
  const int V = cfg->V, N = cfg->Nmax, words = (N + 63) / 64;
  int32_t *tok = malloc(sizeof(int32_t) * N), *par = malloc(sizeof(int32_t) * N), *dep = malloc(sizeof(int32_t) * N),
          *sib = malloc(sizeof(int32_t) * N), *pop = malloc(sizeof(int32_t) * N);
  double *logS = malloc(sizeof(double) * N), *q0 = malloc(sizeof(double) * N), *lq = malloc(sizeof(double) * N),
         *lk = malloc(sizeof(double) * N);
  uint64_t *hash = malloc(sizeof(uint64_t) * (N + 1)), *mask = malloc(sizeof(uint64_t) * (size_t)N * words);
  float* Z = malloc(sizeof(float) * (size_t)(N + 1) * V);
  int32_t acc_node[ORC_DMAX], acc_tok[ORC_DMAX];
  double sum_nodes = 0.0, sum_acc = 0.0;
  memset(hist1, 0, sizeof(int64_t) * V);
  memset(hist2, 0, sizeof(int64_t) * V * V);
  for (int64_t t = 0; t < trials; ++t) {
    uint64_t seed = seed0 + (uint64_t)t;
    int32_t n_scored; uint32_t fl;
    int n = expand_impl(cfg, U_req, A, W, anchor_tok, theta, T, seed, 0, mode == 1,
                        tok, par, dep, sib, logS, q0, lq, lk, pop, hash, mask, &n_scored, &fl);
    for (int i = -1; i < n; ++i)
      memcpy(Z + (size_t)(i + 1) * V, Z_path + (size_t)path_index(tok, par, i, V) * V, sizeof(float) * V);
    int32_t acc_len, bonus;
    orc_verify_tree(cfg, U_req, A, W, Z, anchor_tok, n, tok, par, dep, sib, hash, T, seed, 0,
                    closed_form, 0.0, &acc_len, acc_node, acc_tok, &bonus, NULL, &fl);
    int first = acc_len >= 1 ? acc_tok[0] : bonus;
    hist1[first]++;
    if (acc_len >= 1) {
      int second = acc_len >= 2 ? acc_tok[1] : bonus;
      hist2[(size_t)first * V + second]++;
    }
    sum_nodes += n; sum_acc += acc_len;
  }
  *mean_nodes = sum_nodes / (double)trials;
  *mean_acc = sum_acc / (double)trials;
  free(Z); free(mask); free(hash); free(lk); free(lq); free(q0); free(logS);
  free(pop); free(sib); free(dep); free(par); free(tok);
}

void orc_draw_order_trials(const orc_config* cfg, const float* U_row, const float* a_row, const float* W,
                           double T, uint64_t seed0, int64_t trials, int64_t* hist) {
  const int V = cfg->V, K = cfg->K;
  int64_t size = 1;
  for (int j = 0; j < K; ++j) size *= V;
  memset(hist, 0, sizeof(int64_t) * (size_t)size);
  int32_t top_tok[ORC_KMAX], draw_tok[ORC_KMAX];
  double top_logit[ORC_KMAX], draw_logit[ORC_KMAX], lse0, lseT;
  for (int64_t t = 0; t < trials; ++t) {
    orc_score_parent(cfg, U_row, a_row, W, T, seed0 + (uint64_t)t, 0, 0ull, &lse0, &lseT,
                     top_tok, top_logit, draw_tok, draw_logit, NULL, NULL);
    int64_t idx = 0;
    for (int j = 0; j < K; ++j) idx = idx * V + draw_tok[j];
    hist[idx]++;
  }
}
