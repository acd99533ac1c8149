/*
 * CPU oracle for the MaxScore router (arXiv 2508.12801).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, deliberately
 * unoptimised restatement of what the router computes, written from the
 * paper's definitions.  It shares no code with the CUDA library and must
 * never be called from the product path; only tests, the smoke check and
 * the CPU-baseline leg of the benchmark use it.
 *
 * Arithmetic: double precision for floating point, int64 keys (with
 * __int128 totals) for the assignment problem.
 *
 * Stages (paper passage each follows):
 *   mso_capacity            Sec. 2.3, c = cf * k * n / e ; Algorithm 1 step 1
 *   mso_gate                Eq. 2, x . W_g  (plus the optional expert bias)
 *   mso_softtopk_fwd/bwd    Eq. 6 (reading "ITERMASK", see below) and its derivative
 *   mso_keys_from_scores    fixed-point keys of the affinities A (Eq. 8 objective)
 *   mso_keys_from_scores_hashed   the same plus the 12-bit position hash the library documents
 *   mso_keys_from_logits    int16-quantised logits with a hashed tie-break
 *   mso_flow_ssp            Eq. 7-8 on the network of Table 1, solved by
 *                           successive shortest augmenting paths (SPFA), Sec. 3.2
 *   mso_flow_condensed      the same method with the path search done on the
 *                           expert-level residual graph (for the large configs)
 *   mso_flow_bruteforce     Eq. 7-8 by enumeration (tiny inputs)
 *   mso_flow_certificate    optimality / uniqueness check of a given P
 *   mso_index_build, mso_dispatch, mso_combine      Eq. 1 through E x C buffers
 *   mso_combine_bwd, mso_gate_bwd                   derivatives of Eq. 1 and Eq. 2
 *   mso_aux_loss            Eq. 9
 *
 * Reading of Eq. 6 ("ITERMASK"): SoftTopk^(0) = 0; level j (1-based) adds a
 * softmax with temperature t over the entries that are NOT among the j-1
 * largest; ties go to the lowest expert index.
 *
 * Every function here is pinned by tests/test_oracle_*.py against closed
 * forms, library routines, brute force or invariants.  "Parity unpinned"
 * against the paper: mso_softtopk_rankscale_fwd/bwd, the literal readings of
 * Eq. 6 (pinned by the formula's own special cases only: the paper prints no
 * value that tells the readings of Eq. 6 apart), and the second stage of
 * mso_alg1_top1_sinkhorn (the paper names Sinkhorn but gives neither its
 * regulariser, nor its iteration count, nor how the plan is rounded; pinned by
 * what the mathematics fixes: marginals, the LP optimum on tiny cases, plain
 * top-2 under loose capacity).
 *   mso_softtopk_rankscale_fwd/bwd   Eq. 6 read literally (rank-scaled softmax)
 *   mso_itertopk_fwd/bwd             IterTopk of Table 2 and its derivative
 *   mso_alg1_top1_sinkhorn           Algorithm 1: top-1, then Sinkhorn on the residual problem (k = 2);
 *                                    Sinkhorn's regulariser, iteration count and rounding are this build's
 *                                    reading: parity unpinned against the paper
 *   mso_iterative_reroute            top-k with capacity, then greedy rerouting of the dropped pairs
 *                                    (Sec. 2.3; the serving orders are this build's reading)
 *   mso_aux_loss_grad                derivative of Eq. 9 with respect to A
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef __int128 i128;

#define MSO_OK 0
#define MSO_ERR_ARG 1
#define MSO_ERR_INFEASIBLE 2
#define MSO_ERR_ALLOC 3

/* ------------------------------------------------------------------ */
/* Capacity: C = ceil(cf * T * k / E)  (Sec. 2.3; Algorithm 1 step 1). */
/* cf is given as a rational cf_num / cf_den so the ceiling is exact.   */
int64_t mso_capacity(int64_t T, int64_t k, int64_t E, int64_t cf_num, int64_t cf_den) {
  i128 num = (i128)cf_num * T * k;
  i128 den = (i128)cf_den * E;
  return (int64_t)((num + den - 1) / den);
}

/* Feasible iff every token can get k distinct experts under capacity C. */
int mso_feasible(int64_t T, int64_t k, int64_t E, int64_t C) {
  if (k > E) return 0;
  int64_t cap = C < T ? C : T;
  return (i128)E * cap >= (i128)T * k;
}

/* ------------------------------------------------------------------ */
/* Gate, Eq. 2:  L[i][j] = sum_m H[i][m] * W[m][j] (+ bias[j]).         */
/* H is [T,d], W is [d,E] as the paper writes x . W_g, both row-major.  */
void mso_gate(int64_t T, int64_t d, int64_t E, const double *H, const double *W,
              const double *bias, double *L) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < T; ++i) {
    for (int64_t j = 0; j < E; ++j) {
      double acc = 0.0;
      for (int64_t m = 0; m < d; ++m) acc += H[i * d + m] * W[m * E + j];
      if (bias) acc += bias[j];
      L[i * E + j] = acc;
    }
  }
}

/* ------------------------------------------------------------------ */
/* SoftTopk forward, Eq. 6, one token at a time.                        */
static void softtopk_row(int64_t E, int64_t k, double t, const double *a, double *y,
                         char *sel) {
  for (int64_t i = 0; i < E; ++i) { y[i] = 0.0; sel[i] = 0; }
  for (int64_t level = 0; level < k; ++level) {
    /* largest unmasked entry, lowest index on ties */
    int64_t arg = -1;
    for (int64_t i = 0; i < E; ++i)
      if (!sel[i] && (arg < 0 || a[i] > a[arg])) arg = i;
    if (arg < 0) return;
    double m = a[arg];
    double Z = 0.0;
    for (int64_t i = 0; i < E; ++i)
      if (!sel[i]) Z += exp((a[i] - m) / t);
    for (int64_t i = 0; i < E; ++i)
      if (!sel[i]) y[i] += exp((a[i] - m) / t) / Z;
    sel[arg] = 1; /* masked from the next level on */
  }
}

int mso_softtopk_fwd(int64_t T, int64_t E, int64_t k, double t, const double *L, double *A) {
  if (k < 1 || k > E || !(t > 0.0)) return MSO_ERR_ARG;
#pragma omp parallel
  {
    char *sel = (char *)malloc((size_t)E);
#pragma omp for schedule(static)
    for (int64_t i = 0; i < T; ++i) softtopk_row(E, k, t, L + i * E, A + i * E, sel);
    free(sel);
  }
  return MSO_OK;
}

/* SoftTopk backward: the masks are held constant; level j is a softmax  */
/* q over its unmasked set U_j, so                                       */
/*   da_l = (1/t) * sum_{j : l in U_j} q_l * (g_l - sum_{i in U_j} g_i q_i). */
int mso_softtopk_bwd(int64_t T, int64_t E, int64_t k, double t, const double *L,
                     const double *G, double *dL) {
  if (k < 1 || k > E || !(t > 0.0)) return MSO_ERR_ARG;
#pragma omp parallel
  {
    char *sel = (char *)malloc((size_t)E);
    double *q = (double *)malloc(sizeof(double) * (size_t)E);
#pragma omp for schedule(static)
    for (int64_t r = 0; r < T; ++r) {
      const double *a = L + r * E, *g = G + r * E;
      double *da = dL + r * E;
      for (int64_t i = 0; i < E; ++i) { da[i] = 0.0; sel[i] = 0; }
      for (int64_t level = 0; level < k; ++level) {
        int64_t arg = -1;
        for (int64_t i = 0; i < E; ++i)
          if (!sel[i] && (arg < 0 || a[i] > a[arg])) arg = i;
        if (arg < 0) break;
        double m = a[arg], Z = 0.0;
        for (int64_t i = 0; i < E; ++i)
          if (!sel[i]) Z += exp((a[i] - m) / t);
        double gq = 0.0;
        for (int64_t i = 0; i < E; ++i)
          if (!sel[i]) { q[i] = exp((a[i] - m) / t) / Z; gq += g[i] * q[i]; }
        for (int64_t i = 0; i < E; ++i)
          if (!sel[i]) da[i] += q[i] * (g[i] - gq) / t;
        sel[arg] = 1;
      }
    }
    free(sel); free(q);
  }
  return MSO_OK;
}

/* ------------------------------------------------------------------ */
/* Keys for the assignment problem.                                     */

/* Float mode: fixed-point image of the affinities, w = rne(A * 2^40).  */
void mso_keys_from_scores(int64_t n, const double *A, int64_t *w) {
  for (int64_t i = 0; i < n; ++i) w[i] = llrint(ldexp(A[i], 40));
}

/* Float mode as the library solves it: the same fixed-point image plus a 12-bit  */
/* multiplicative hash of the entry's position (i*E + j) * 2654435761 mod 2^32,   */
/* top 12 bits.  The hash only separates exact ties between equal scores; it adds */
/* less than 2^12 units of 2^-40 (under 4e-9) to any key.                          */
void mso_keys_from_scores_hashed(int64_t T, int64_t E, const double *A, int64_t *w) {
  for (int64_t i = 0; i < T; ++i)
    for (int64_t j = 0; j < E; ++j) {
      uint32_t pos = (uint32_t)(i * E + j);
      w[i * E + j] = llrint(ldexp(A[i * E + j], 40)) + (int64_t)((pos * 2654435761u) >> 20);
    }
}

/* 32-bit finaliser of MurmurHash3 (Appleby, public domain). */
static uint32_t fmix32(uint32_t h) {
  h ^= h >> 16; h *= 0x85ebca6bu; h ^= h >> 13; h *= 0xc2b2ae35u; h ^= h >> 16;
  return h;
}

/* Integer mode: q = clamp(rne(L * 2^shift)) as int16; tie-break          */
/* r = top 20 bits of fmix32(i*E + j + seed * 0x9E3779B9);                */
/* w = q * 2^S + r with S = 20 + ceil(log2(T*k)), so that the summed      */
/* perturbation of any assignment stays below one step of q.              */
int mso_tiebreak_shift(int64_t T, int64_t k) {
  int64_t n = T * k; int s = 0;
  while (((int64_t)1 << s) < n) ++s;
  return 20 + s;
}

void mso_keys_from_logits(int64_t T, int64_t E, int64_t k, const float *L, int shift,
                          uint32_t seed, int64_t *w, int16_t *q_out) {
  int S = mso_tiebreak_shift(T, k);
  for (int64_t i = 0; i < T; ++i)
    for (int64_t j = 0; j < E; ++j) {
      /* the product by a power of two is exact in float; rintf is round-to-nearest-even */
      float scaled = rintf(ldexpf(L[i * E + j], shift));
      if (scaled > 32767.0f) scaled = 32767.0f;
      if (scaled < -32768.0f) scaled = -32768.0f;
      int64_t q = (int64_t)scaled;
      uint32_t r = fmix32((uint32_t)(i * E + j) + seed * 0x9E3779B9u) >> 12;
      w[i * E + j] = q * ((int64_t)1 << S) + (int64_t)r;
      if (q_out) q_out[i * E + j] = (int16_t)q;
    }
}

/* ------------------------------------------------------------------ */
/* Textbook min-cost max-flow on the network of Table 1:                 */
/*   source -> token_i   cap k  cost 0                                   */
/*   token_i -> expert_j cap 1  cost -w_ij                               */
/*   expert_j -> sink    cap C  cost 0                                   */
/* Successive shortest augmenting paths, each found by SPFA (queue-based */
/* Bellman-Ford), until the sink is unreachable.                         */
typedef struct { int32_t to, cap; int64_t cost; } arc_t;

int mso_flow_ssp(int64_t T, int64_t E, int64_t k, int64_t C, const int64_t *w,
                 int32_t *expert_idx, int32_t *load, int64_t *flow_value) {
  if (!mso_feasible(T, k, E, C)) return MSO_ERR_INFEASIBLE;
  int64_t N = T + E + 2, S = 0, SINK = T + E + 1;
  int64_t M = 2 * (T + T * E + E);
  arc_t *arc = (arc_t *)malloc(sizeof(arc_t) * (size_t)M);
  int64_t *first = (int64_t *)malloc(sizeof(int64_t) * (size_t)(N + 1));
  i128 *dist = (i128 *)malloc(sizeof(i128) * (size_t)N);
  int64_t *prev_arc = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
  int64_t *queue = (int64_t *)malloc(sizeof(int64_t) * (size_t)(N + 1));
  char *inq = (char *)malloc((size_t)N);
  if (!arc || !first || !dist || !prev_arc || !queue || !inq) return MSO_ERR_ALLOC;
  /* adjacency in CSR form; arc a and its reverse sit at a and rev(a) = partner[] */
  int64_t *partner = (int64_t *)malloc(sizeof(int64_t) * (size_t)M);
  int64_t *deg = (int64_t *)calloc((size_t)(N + 1), sizeof(int64_t));
  /* degrees */
  deg[S] = T;
  for (int64_t i = 0; i < T; ++i) deg[1 + i] = 1 + E;
  for (int64_t j = 0; j < E; ++j) deg[1 + T + j] = T + 1;
  deg[SINK] = E;
  first[0] = 0;
  for (int64_t v = 0; v < N; ++v) first[v + 1] = first[v] + deg[v];
  int64_t *fill = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
  for (int64_t v = 0; v < N; ++v) fill[v] = first[v];
#define ADD_ARC(u, v, c, cst)                                                   \
  do {                                                                          \
    int64_t a_ = fill[u]++, b_ = fill[v]++;                                     \
    arc[a_].to = (int32_t)(v); arc[a_].cap = (int32_t)(c); arc[a_].cost = (cst); \
    arc[b_].to = (int32_t)(u); arc[b_].cap = 0; arc[b_].cost = -(cst);          \
    partner[a_] = b_; partner[b_] = a_;                                         \
  } while (0)
  for (int64_t i = 0; i < T; ++i) ADD_ARC(S, 1 + i, k, 0);
  for (int64_t i = 0; i < T; ++i)
    for (int64_t j = 0; j < E; ++j) ADD_ARC(1 + i, 1 + T + j, 1, -w[i * E + j]);
  for (int64_t j = 0; j < E; ++j) ADD_ARC(1 + T + j, SINK, C, 0);
#undef ADD_ARC
  const i128 INF = ((i128)1) << 120;
  int64_t flow = 0;
  for (;;) {
    for (int64_t v = 0; v < N; ++v) { dist[v] = INF; inq[v] = 0; prev_arc[v] = -1; }
    int64_t qh = 0, qt = 0, qn = 0;
    dist[S] = 0; queue[qt] = S; qt = (qt + 1) % (N + 1); qn = 1; inq[S] = 1;
    while (qn > 0) {
      int64_t u = queue[qh]; qh = (qh + 1) % (N + 1); --qn; inq[u] = 0;
      for (int64_t a = first[u]; a < first[u + 1]; ++a) {
        if (arc[a].cap <= 0) continue;
        int64_t v = arc[a].to;
        i128 nd = dist[u] + arc[a].cost;
        if (nd < dist[v]) {
          dist[v] = nd; prev_arc[v] = a;
          if (!inq[v]) { queue[qt] = v; qt = (qt + 1) % (N + 1); ++qn; inq[v] = 1; }
        }
      }
    }
    if (prev_arc[SINK] < 0) break; /* no augmenting path remains */
    /* bottleneck is 1 because every path crosses a unit token->expert arc */
    for (int64_t v = SINK; v != S;) {
      int64_t a = prev_arc[v];
      arc[a].cap -= 1; arc[partner[a]].cap += 1;
      v = arc[partner[a]].to;
    }
    ++flow;
  }
  /* read the assignment off the saturated token->expert arcs */
  for (int64_t j = 0; j < E; ++j) load[j] = 0;
  int rc = MSO_OK;
  for (int64_t i = 0; i < T; ++i) {
    int64_t c = 0;
    for (int64_t a = first[1 + i]; a < first[2 + i]; ++a) {
      int64_t v = arc[a].to;
      if (v >= 1 + T && v < 1 + T + E && arc[a].cap == 0) {
        if (c < k) expert_idx[i * k + c] = (int32_t)(v - 1 - T);
        ++c; load[v - 1 - T] += 1;
      }
    }
    if (c != k) rc = MSO_ERR_INFEASIBLE;
    /* ascending expert index within the token */
    for (int64_t x = 1; x < (c < k ? c : k); ++x)
      for (int64_t y = x; y > 0 && expert_idx[i * k + y] < expert_idx[i * k + y - 1]; --y) {
        int32_t tmp = expert_idx[i * k + y]; expert_idx[i * k + y] = expert_idx[i * k + y - 1];
        expert_idx[i * k + y - 1] = tmp;
      }
  }
  if (flow_value) *flow_value = flow;
  free(arc); free(first); free(dist); free(prev_arc); free(queue); free(inq);
  free(partner); free(deg); free(fill);
  return rc;
}

/* ------------------------------------------------------------------ */
/* Brute force for Eq. 7-8: enumerate every choice of k experts per     */
/* token, keep those with all loads <= C, maximise sum of keys.         */
/* Returns the optimum, how many assignments attain it, and the first   */
/* optimal assignment in enumeration order.  For T <= 8, E <= 4 only.   */
int mso_flow_bruteforce(int64_t T, int64_t E, int64_t k, int64_t C, const int64_t *w,
                        int64_t *best_total, int64_t *n_optimal, int32_t *expert_idx) {
  if (T > 10 || E > 6 || k > E) return MSO_ERR_ARG;
  int masks[64]; int nm = 0;
  for (int m = 0; m < (1 << E); ++m) if (__builtin_popcount(m) == k) masks[nm++] = m;
  int choice[16]; int best_choice[16];
  for (int i = 0; i < T; ++i) choice[i] = 0;
  int found = 0; i128 best = 0; int64_t count = 0;
  for (;;) {
    int ld[8] = {0}; i128 tot = 0; int ok = 1;
    for (int i = 0; i < T && ok; ++i)
      for (int j = 0; j < E; ++j)
        if (masks[choice[i]] >> j & 1) {
          tot += w[i * E + j];
          if (++ld[j] > C) { ok = 0; break; }
        }
    if (ok) {
      if (!found || tot > best) { best = tot; count = 1; found = 1; memcpy(best_choice, choice, sizeof(choice)); }
      else if (tot == best) ++count;
    }
    int p = (int)T - 1;
    while (p >= 0 && ++choice[p] == nm) { choice[p] = 0; --p; }
    if (p < 0) break;
  }
  if (!found) return MSO_ERR_INFEASIBLE;
  *best_total = (int64_t)best; *n_optimal = count;
  for (int i = 0; i < T; ++i) {
    int c = 0;
    for (int j = 0; j < E; ++j) if (masks[best_choice[i]] >> j & 1) expert_idx[i * k + c++] = j;
  }
  return MSO_OK;
}

/* ------------------------------------------------------------------ */
/* Expert-level residual graph of an assignment P (nodes 0..E-1 are the */
/* experts, node E is the sink side "Z"):                               */
/*   D[e][f] = min over tokens i with P_ie = 1, P_if = 0 of w_ie - w_if */
/*             (the loss of moving one token from e to f)               */
/*   D[f][Z] = 0 if load_f < C ;  D[Z][e] = 0 if load_e > 0.            */
/* P is optimal iff this graph has no negative cycle; it is the only    */
/* optimum iff every cycle is strictly positive.                        */
#define BIG ((i128)1 << 100)

static void build_D(int64_t T, int64_t E, int64_t k, int64_t C, const int64_t *w,
                    const int32_t *expert_idx, const int32_t *load, i128 *D, int32_t *who) {
  int64_t n = E + 1;
  for (int64_t a = 0; a < n * n; ++a) { D[a] = BIG; if (who) who[a] = -1; }
  char *in = (char *)malloc((size_t)E);
  for (int64_t i = 0; i < T; ++i) {
    memset(in, 0, (size_t)E);
    for (int64_t c = 0; c < k; ++c) in[expert_idx[i * k + c]] = 1;
    for (int64_t c = 0; c < k; ++c) {
      int64_t e = expert_idx[i * k + c];
      for (int64_t f = 0; f < E; ++f) {
        if (in[f]) continue;
        i128 loss = (i128)w[i * E + e] - (i128)w[i * E + f];
        if (loss < D[e * n + f]) { D[e * n + f] = loss; if (who) who[e * n + f] = (int32_t)i; }
      }
    }
  }
  for (int64_t e = 0; e < E; ++e) {
    if (load[e] < C) D[e * n + E] = 0;
    if (load[e] > 0) D[E * n + e] = 0;
  }
  free(in);
}

/* result: 0 = not optimal (negative cycle), 1 = optimal but a zero     */
/* cycle exists (other optima), 2 = uniquely optimal.                   */
/* prices[E] receives dual prices p_e >= 0 when optimal.                */
/* Also checks the invariants: k distinct experts per token, ascending, */
/* loads match and stay <= C; returns -1 if any fails.                  */
int mso_flow_certificate(int64_t T, int64_t E, int64_t k, int64_t C, const int64_t *w,
                         const int32_t *expert_idx, int64_t *prices) {
  int64_t n = E + 1;
  int32_t *load = (int32_t *)calloc((size_t)E, sizeof(int32_t));
  for (int64_t i = 0; i < T; ++i)
    for (int64_t c = 0; c < k; ++c) {
      int32_t e = expert_idx[i * k + c];
      if (e < 0 || e >= E) { free(load); return -1; }
      if (c > 0 && expert_idx[i * k + c - 1] >= e) { free(load); return -1; }
      load[e] += 1;
    }
  for (int64_t e = 0; e < E; ++e) if (load[e] > C) { free(load); return -1; }
  i128 *D = (i128 *)malloc(sizeof(i128) * (size_t)(n * n));
  build_D(T, E, k, C, w, expert_idx, load, D, NULL);
  /* G = the expert-only part of D, kept apart for the uniqueness test: in  */
  /* the full graph Z -> e -> Z is always a zero cycle (take a unit off the  */
  /* arc expert_e -> sink and put it back), which is no second optimum.      */
  i128 *G = (i128 *)malloc(sizeof(i128) * (size_t)(E * E));
  for (int64_t a = 0; a < E; ++a)
    for (int64_t b = 0; b < E; ++b) G[a * E + b] = D[a * n + b];
  /* all-pairs shortest walks (Floyd-Warshall); diagonals start at +inf so  */
  /* that [v][v] ends as the cheapest cycle through v                       */
  for (int64_t m = 0; m < n; ++m)
    for (int64_t a = 0; a < n; ++a) {
      if (D[a * n + m] >= BIG) continue;
      for (int64_t b = 0; b < n; ++b) {
        if (D[m * n + b] >= BIG) continue;
        i128 via = D[a * n + m] + D[m * n + b];
        if (via < D[a * n + b]) D[a * n + b] = via;
      }
    }
  for (int64_t m = 0; m < E; ++m)
    for (int64_t a = 0; a < E; ++a) {
      if (G[a * E + m] >= BIG) continue;
      for (int64_t b = 0; b < E; ++b) {
        if (G[m * E + b] >= BIG) continue;
        i128 via = G[a * E + m] + G[m * E + b];
        if (via < G[a * E + b]) G[a * E + b] = via;
      }
    }
  int result = 2;
  for (int64_t v = 0; v < n; ++v)
    if (D[v * n + v] < 0) { result = 0; break; }
  if (result) {
    /* a zero cycle among the experts, or a zero walk from an expert to a    */
    /* different expert with room (a cycle through Z), is a second optimum   */
    for (int64_t a = 0; a < E && result == 2; ++a)
      for (int64_t b = 0; b < E; ++b) {
        if (a == b) { if (G[a * E + a] == 0) { result = 1; break; } }
        else if (load[b] < C && G[a * E + b] == 0) { result = 1; break; }
      }
  }
  free(G);
  if (result > 0 && prices) {
    /* potentials: pi_v = min(0, cheapest walk into v from any node), so    */
    /* pi_f <= pi_e + D[e][f] on every arc.  The price of expert e is        */
    /* p_e = pi_Z - pi_e: the arcs e -> f then say w_ie - p_e >= w_if - p_f  */
    /* for every token in e and not in f, the arcs Z -> e give p_e >= 0      */
    /* where load_e > 0 and the arcs f -> Z give p_f <= 0 where load_f < C.  */
    /* An empty expert may come out negative; raising it to 0 keeps every    */
    /* token's preference and no token sits there.                           */
    i128 piZ = 0;
    for (int64_t a = 0; a < n; ++a) if (D[a * n + E] < piZ) piZ = D[a * n + E];
    for (int64_t e = 0; e < E; ++e) {
      i128 pie = 0;
      for (int64_t a = 0; a < n; ++a) if (D[a * n + e] < pie) pie = D[a * n + e];
      i128 p = piZ - pie;
      prices[e] = (int64_t)(p < 0 ? 0 : p);
    }
  }
  free(D); free(load);
  return result;
}

/* Dual objective of Eq. 8 at prices p:                                 */
/*   sum_i (sum of the k largest of w_ie - p_e) + C * sum_e p_e.        */
/* Equals the primal optimum exactly when p is optimal (strong duality   */
/* of the totally unimodular flow LP).  Written as two int64 halves.     */
void mso_dual_value(int64_t T, int64_t E, int64_t k, int64_t C, const int64_t *w,
                    const int64_t *p, int64_t *hi, uint64_t *lo) {
  i128 tot = 0;
  i128 *v = (i128 *)malloc(sizeof(i128) * (size_t)E);
  for (int64_t i = 0; i < T; ++i) {
    for (int64_t e = 0; e < E; ++e) v[e] = (i128)w[i * E + e] - (i128)p[e];
    for (int64_t c = 0; c < k; ++c) { /* selection of the k largest */
      int64_t arg = c;
      for (int64_t e = c + 1; e < E; ++e) if (v[e] > v[arg]) arg = e;
      i128 tmp = v[c]; v[c] = v[arg]; v[arg] = tmp;
      tot += v[c];
    }
  }
  for (int64_t e = 0; e < E; ++e) tot += (i128)C * p[e];
  free(v);
  *hi = (int64_t)(tot >> 64); *lo = (uint64_t)tot;
}

void mso_primal_value(int64_t T, int64_t E, int64_t k, const int64_t *w,
                      const int32_t *expert_idx, int64_t *hi, uint64_t *lo) {
  i128 tot = 0;
  for (int64_t i = 0; i < T; ++i)
    for (int64_t c = 0; c < k; ++c) tot += w[i * E + expert_idx[i * k + c]];
  *hi = (int64_t)(tot >> 64); *lo = (uint64_t)tot;
}

/* ------------------------------------------------------------------ */
/* Successive shortest paths with the path search on the expert-level   */
/* graph.  Start: every token takes its k largest keys (the min-cost    */
/* flow when the expert->sink capacities are ignored).  Then, while an  */
/* expert holds more than C tokens, find the cheapest walk from the set  */
/* of overloaded experts to an expert with room (Bellman-Ford on E+1     */
/* nodes; all cycles are non-negative, so it terminates) and move one    */
/* token along each of its arcs.  The rows of D touched by the walk are  */
/* rebuilt from the token lists.  Same optimum as mso_flow_ssp; checked  */
/* against it in the tests.                                              */
int mso_flow_condensed(int64_t T, int64_t E, int64_t k, int64_t C, const int64_t *w,
                       int32_t *expert_idx, int32_t *load, int64_t *n_augment) {
  if (!mso_feasible(T, k, E, C)) return MSO_ERR_INFEASIBLE;
  int64_t n = E; /* expert nodes only; room is a node property here */
  /* member[i*E+e] = 1 iff P_ie = 1 */
  char *member = (char *)calloc((size_t)(T * E), 1);
  for (int64_t e = 0; e < E; ++e) load[e] = 0;
  for (int64_t i = 0; i < T; ++i) {
    for (int64_t c = 0; c < k; ++c) {
      int64_t arg = -1;
      for (int64_t e = 0; e < E; ++e)
        if (!member[i * E + e] && (arg < 0 || w[i * E + e] > w[i * E + arg])) arg = e;
      member[i * E + arg] = 1; load[arg] += 1;
    }
  }
  i128 *D = (i128 *)malloc(sizeof(i128) * (size_t)(n * n));
  int32_t *who = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n * n));
  i128 *dist = (i128 *)malloc(sizeof(i128) * (size_t)n);
  int64_t *pred = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
  char *dirty = (char *)malloc((size_t)n);
  for (int64_t e = 0; e < n; ++e) dirty[e] = 1;
  int64_t aug = 0;
  for (;;) {
    /* rebuild the rows marked dirty: D[e][f] over tokens in e and not in f */
    for (int64_t e = 0; e < n; ++e) {
      if (!dirty[e]) continue;
      for (int64_t f = 0; f < n; ++f) { D[e * n + f] = BIG; who[e * n + f] = -1; }
    }
    for (int64_t i = 0; i < T; ++i)
      for (int64_t e = 0; e < n; ++e) {
        if (!dirty[e] || !member[i * E + e]) continue;
        for (int64_t f = 0; f < n; ++f) {
          if (member[i * E + f]) continue;
          i128 loss = (i128)w[i * E + e] - (i128)w[i * E + f];
          if (loss < D[e * n + f]) { D[e * n + f] = loss; who[e * n + f] = (int32_t)i; }
        }
      }
    /* a token that joined expert f may have been the cheapest mover of some
       arc into f from another of its experts; those arcs' rows were marked too */
    for (int64_t e = 0; e < n; ++e) dirty[e] = 0;
    int any_over = 0;
    for (int64_t e = 0; e < n; ++e) {
      if (load[e] > C) { dist[e] = 0; any_over = 1; } else dist[e] = BIG;
      pred[e] = -1;
    }
    if (!any_over) break;
    for (int64_t round = 0; round < n; ++round) {
      int changed = 0;
      for (int64_t e = 0; e < n; ++e) {
        if (dist[e] >= BIG) continue;
        for (int64_t f = 0; f < n; ++f) {
          if (D[e * n + f] >= BIG) continue;
          i128 nd = dist[e] + D[e * n + f];
          if (nd < dist[f]) { dist[f] = nd; pred[f] = e; changed = 1; }
        }
      }
      if (!changed) break;
    }
    int64_t target = -1;
    for (int64_t f = 0; f < n; ++f)
      if (load[f] < C && dist[f] < BIG && (target < 0 || dist[f] < dist[target])) target = f;
    if (target < 0) { free(member); free(D); free(who); free(dist); free(pred); free(dirty); return MSO_ERR_INFEASIBLE; }
    /* move one token along each arc of the walk, from the far end back */
    int64_t f = target;
    load[target] += 1;
    while (pred[f] >= 0) {
      int64_t e = pred[f];
      int64_t i = who[e * n + f];
      member[i * E + e] = 0; member[i * E + f] = 1;
      /* rows to rebuild: e (lost i), f (gained i), and every other expert of i
         (its arc into f may have been using i, and its arc into e may now use i) */
      for (int64_t g = 0; g < n; ++g) if (member[i * E + g]) dirty[g] = 1;
      dirty[e] = 1;
      f = e;
    }
    load[f] -= 1; /* f is now the overloaded start of the walk */
    ++aug;
  }
  for (int64_t i = 0; i < T; ++i) {
    int64_t c = 0;
    for (int64_t e = 0; e < E; ++e) if (member[i * E + e]) expert_idx[i * k + c++] = (int32_t)e;
  }
  if (n_augment) *n_augment = aug;
  free(member); free(D); free(who); free(dist); free(pred); free(dirty);
  return MSO_OK;
}

/* ------------------------------------------------------------------ */
/* Index build: the slot of token i in expert e is the rank of i among  */
/* the tokens assigned to e, in ascending token index.  Unused slots of */
/* slot_token hold -1 (padding of the capacity-shaped buffers, Sec. 2.3).*/
int mso_index_build(int64_t T, int64_t E, int64_t k, int64_t C, const int32_t *expert_idx,
                    int32_t *slot_idx, int32_t *slot_token, int32_t *load) {
  for (int64_t e = 0; e < E; ++e) load[e] = 0;
  for (int64_t a = 0; a < E * C; ++a) slot_token[a] = -1;
  for (int64_t i = 0; i < T; ++i)
    for (int64_t c = 0; c < k; ++c) {
      int32_t e = expert_idx[i * k + c];
      if (e < 0 || e >= E || load[e] >= C) return MSO_ERR_ARG;
      slot_idx[i * k + c] = load[e];
      slot_token[(int64_t)e * C + load[e]] = (int32_t)i;
      load[e] += 1;
    }
  return MSO_OK;
}

/* Dispatch: xdisp[e][s][:] = src[slot_token[e][s]][:], zero rows for   */
/* padding.  Pure data movement on rows of row_bytes bytes.             */
void mso_dispatch(int64_t E, int64_t C, int64_t row_bytes, const void *src,
                  const int32_t *slot_token, void *dst) {
  for (int64_t a = 0; a < E * C; ++a) {
    char *out = (char *)dst + a * row_bytes;
    if (slot_token[a] < 0) memset(out, 0, (size_t)row_bytes);
    else memcpy(out, (const char *)src + (int64_t)slot_token[a] * row_bytes, (size_t)row_bytes);
  }
}

/* Combine, Eq. 1: Y[i][:] = sum over the token's experts, in ascending  */
/* expert index, of gate_w[i][c] * yexp[e][slot][:].  gate_w NULL means  */
/* unit weights (the adjoint of dispatch).                               */
void mso_combine(int64_t T, int64_t d, int64_t k, int64_t C, const double *yexp,
                 const int32_t *expert_idx, const int32_t *slot_idx, const double *gate_w,
                 double *Y) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < T; ++i) {
    for (int64_t m = 0; m < d; ++m) Y[i * d + m] = 0.0;
    for (int64_t c = 0; c < k; ++c) {
      int64_t row = (int64_t)expert_idx[i * k + c] * C + slot_idx[i * k + c];
      double g = gate_w ? gate_w[i * k + c] : 1.0;
      for (int64_t m = 0; m < d; ++m) Y[i * d + m] += g * yexp[row * d + m];
    }
  }
}

/* Derivative of Eq. 1 with P held fixed:                               */
/*   dyexp[e][s][:] = gate_w[i][c] * dY[i][:]   (zero rows for padding)  */
/*   dgate_w[i][c]  = <dY[i][:], yexp[e][s][:]>                          */
void mso_combine_bwd(int64_t T, int64_t d, int64_t E, int64_t k, int64_t C, const double *dY,
                     const double *yexp, const int32_t *expert_idx, const int32_t *slot_idx,
                     const double *gate_w, double *dyexp, double *dgate_w) {
  for (int64_t a = 0; a < E * C * d; ++a) dyexp[a] = 0.0;
  for (int64_t i = 0; i < T; ++i)
    for (int64_t c = 0; c < k; ++c) {
      int64_t row = (int64_t)expert_idx[i * k + c] * C + slot_idx[i * k + c];
      double dot = 0.0;
      for (int64_t m = 0; m < d; ++m) {
        dyexp[row * d + m] = gate_w[i * k + c] * dY[i * d + m];
        dot += dY[i * d + m] * yexp[row * d + m];
      }
      dgate_w[i * k + c] = dot;
    }
}

/* Derivative of Eq. 2:  dW = H^T dL  ([d,E]),  dH = dL W^T  ([T,d]).    */
void mso_gate_bwd(int64_t T, int64_t d, int64_t E, const double *H, const double *W,
                  const double *dL, double *dW, double *dH) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < d; ++m)
    for (int64_t j = 0; j < E; ++j) {
      double acc = 0.0;
      for (int64_t i = 0; i < T; ++i) acc += H[i * d + m] * dL[i * E + j];
      dW[m * E + j] = acc;
    }
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < T; ++i)
    for (int64_t m = 0; m < d; ++m) {
      double acc = 0.0;
      for (int64_t j = 0; j < E; ++j) acc += dL[i * E + j] * W[m * E + j];
      dH[i * d + m] = acc;
    }
}

/* Auxiliary load-balance loss, Eq. 9:                                  */
/*   L_aux = lambda / e * sum_j mean_i(A_ij) * mean_i(P_ij).            */
double mso_aux_loss(int64_t T, int64_t E, int64_t k, double lambda, const double *A,
                    const int32_t *expert_idx) {
  double tot = 0.0;
  for (int64_t j = 0; j < E; ++j) {
    double sa = 0.0, sp = 0.0;
    for (int64_t i = 0; i < T; ++i) {
      sa += A[i * E + j];
      for (int64_t c = 0; c < k; ++c) if (expert_idx[i * k + c] == j) sp += 1.0;
    }
    tot += (sa / (double)T) * (sp / (double)T);
  }
  return lambda * tot / (double)E;
}

/* Gradient of Eq. 9 with respect to the affinities, P held constant (it is  */
/* binary): dL_aux/dA_ij = lambda / (e n^2) * sum_i' P_i'j, the same for     */
/* every token i, so one value per expert is returned.                       */
void mso_aux_loss_grad(int64_t T, int64_t E, int64_t k, double lambda, const int32_t *expert_idx,
                       double *dA_col) {
  for (int64_t j = 0; j < E; ++j) {
    double sp = 0.0;
    for (int64_t i = 0; i < T; ++i)
      for (int64_t c = 0; c < k; ++c) if (expert_idx[i * k + c] == j) sp += 1.0;
    dA_col[j] = lambda * sp / ((double)E * (double)T * (double)T);
  }
}

/* ------------------------------------------------------------------ */
/* The literal readings of Eq. 6 ("RANKSCALE").  Read as printed, the   */
/* recursion adds t * Softmax(a)_i (softmax over ALL experts, t a       */
/* factor) at every level at which entry i is not masked, so an entry   */
/* of rank r (1 = largest, ties: lowest index first) ends up with       */
/*     y_i = p_i * (beta + t * min(r_i - delta, k)),  p = Softmax(a).    */
/* (beta, delta) = (0, 0): base 0, level j masks the j-1 largest;       */
/* (beta, delta) = (1, 1): base Softmax(a), level j masks the j largest. */
/* The paper prints no value that tells these readings (or ITERMASK)    */
/* apart: parity unpinned against the paper; the pins are the formula's */
/* own special cases (tests/test_oracle_softtopk.py).                   */
static void rank_of_row(int64_t E, const double *a, int64_t *rank) {
  for (int64_t i = 0; i < E; ++i) {
    int64_t r = 1;
    for (int64_t j = 0; j < E; ++j)
      if (a[j] > a[i] || (a[j] == a[i] && j < i)) ++r;
    rank[i] = r;
  }
}

int mso_softtopk_rankscale_fwd(int64_t T, int64_t E, int64_t k, double t, double beta, int64_t delta,
                               const double *L, double *A) {
  if (k < 1 || k > E) return MSO_ERR_ARG;
  int64_t *rank = (int64_t *)malloc(sizeof(int64_t) * (size_t)E);
  if (!rank) return MSO_ERR_ALLOC;
  for (int64_t r = 0; r < T; ++r) {
    const double *a = L + r * E;
    double m = a[0], Z = 0.0;
    for (int64_t i = 1; i < E; ++i) if (a[i] > m) m = a[i];
    for (int64_t i = 0; i < E; ++i) Z += exp(a[i] - m);
    rank_of_row(E, a, rank);
    for (int64_t i = 0; i < E; ++i) {
      int64_t c = rank[i] - delta; if (c > k) c = k;
      A[r * E + i] = exp(a[i] - m) / Z * (beta + t * (double)c);
    }
  }
  free(rank);
  return MSO_OK;
}

/* Backward with the ranks held constant: y = s (.) p with s fixed, so   */
/* da_l = p_l * (g_l s_l - sum_i g_i s_i p_i), the softmax Jacobian      */
/* applied to g (.) s.                                                   */
int mso_softtopk_rankscale_bwd(int64_t T, int64_t E, int64_t k, double t, double beta, int64_t delta,
                               const double *L, const double *G, double *dL) {
  if (k < 1 || k > E) return MSO_ERR_ARG;
  int64_t *rank = (int64_t *)malloc(sizeof(int64_t) * (size_t)E);
  double *p = (double *)malloc(sizeof(double) * (size_t)E);
  if (!rank || !p) { free(rank); free(p); return MSO_ERR_ALLOC; }
  for (int64_t r = 0; r < T; ++r) {
    const double *a = L + r * E, *g = G + r * E;
    double m = a[0], Z = 0.0;
    for (int64_t i = 1; i < E; ++i) if (a[i] > m) m = a[i];
    for (int64_t i = 0; i < E; ++i) Z += exp(a[i] - m);
    rank_of_row(E, a, rank);
    double dot = 0.0;
    for (int64_t i = 0; i < E; ++i) {
      int64_t c = rank[i] - delta; if (c > k) c = k;
      p[i] = exp(a[i] - m) / Z;
      dot += g[i] * (beta + t * (double)c) * p[i];
    }
    for (int64_t i = 0; i < E; ++i) {
      int64_t c = rank[i] - delta; if (c > k) c = k;
      dL[r * E + i] = p[i] * (g[i] * (beta + t * (double)c) - dot);
    }
  }
  free(rank); free(p);
  return MSO_OK;
}

/* ------------------------------------------------------------------ */
/* IterTopk of Table 2: y^(0) = 0 and, for level l = 1..k,               */
/*     y^(l) = y^(l-1) + g(x; 1 - y^(l-1)),   g(x; w)_j = w_j e^{x_j} / sum_i w_i e^{x_i}.  */
/* Every level adds a distribution, so the result sums to k.  Table 2    */
/* carries no temperature: the logits enter as they are.                 */
int mso_itertopk_fwd(int64_t T, int64_t E, int64_t k, const double *L, double *A) {
  if (k < 1 || k > E) return MSO_ERR_ARG;
  for (int64_t r = 0; r < T; ++r) {
    const double *x = L + r * E; double *y = A + r * E;
    double m = x[0];
    for (int64_t j = 1; j < E; ++j) if (x[j] > m) m = x[j];
    for (int64_t j = 0; j < E; ++j) y[j] = 0.0;
    for (int64_t l = 0; l < k; ++l) {
      double s = 0.0;
      for (int64_t j = 0; j < E; ++j) s += (1.0 - y[j]) * exp(x[j] - m);
      /* all increments of a level come from the y of the level before */
      for (int64_t j = 0; j < E; ++j) y[j] = y[j] + (1.0 - y[j]) * exp(x[j] - m) / s;
    }
  }
  return MSO_OK;
}

/* Derivative of IterTopk: dL = J^T G, by reverse accumulation through   */
/* the k levels.  With z_j = e^{x_j - m}, u_j = w_j z_j, s = sum u,      */
/* r = u / s: given the gradient rb of r,                                */
/*   ub_j = (rb_j - sum_i rb_i r_i) / s,  wb_j = ub_j z_j,  zb_j += ub_j w_j, */
/* and since w = 1 - y^(l-1), the gradient of y^(l-1) is that of y^(l)   */
/* minus wb.  Finally dx_j = zb_j z_j (the shift m drops out: IterTopk   */
/* does not change when a constant is added to every logit).             */
int mso_itertopk_bwd(int64_t T, int64_t E, int64_t k, const double *L, const double *G, double *dL) {
  if (k < 1 || k > E) return MSO_ERR_ARG;
  double *w = (double *)malloc(sizeof(double) * (size_t)(k * E));   /* w of every level */
  double *z = (double *)malloc(sizeof(double) * (size_t)E);
  double *yb = (double *)malloc(sizeof(double) * (size_t)E);
  double *zb = (double *)malloc(sizeof(double) * (size_t)E);
  double *ss = (double *)malloc(sizeof(double) * (size_t)k);
  if (!w || !z || !yb || !zb || !ss) { free(w); free(z); free(yb); free(zb); free(ss); return MSO_ERR_ALLOC; }
  for (int64_t r = 0; r < T; ++r) {
    const double *x = L + r * E, *g = G + r * E;
    double m = x[0];
    for (int64_t j = 1; j < E; ++j) if (x[j] > m) m = x[j];
    for (int64_t j = 0; j < E; ++j) { z[j] = exp(x[j] - m); yb[j] = g[j]; zb[j] = 0.0; }
    /* forward, keeping each level's weights and normaliser */
    for (int64_t j = 0; j < E; ++j) w[j] = 1.0;
    for (int64_t l = 0; l < k; ++l) {
      double s = 0.0;
      for (int64_t j = 0; j < E; ++j) s += w[l * E + j] * z[j];
      ss[l] = s;
      if (l + 1 < k)
        for (int64_t j = 0; j < E; ++j) w[(l + 1) * E + j] = w[l * E + j] - w[l * E + j] * z[j] / s;
    }
    for (int64_t l = k - 1; l >= 0; --l) {
      const double s = ss[l];
      double dot = 0.0;
      for (int64_t j = 0; j < E; ++j) dot += yb[j] * (w[l * E + j] * z[j] / s);
      for (int64_t j = 0; j < E; ++j) {
        const double ub = (yb[j] - dot) / s;
        zb[j] += ub * w[l * E + j];
        yb[j] -= ub * z[j];              /* gradient of y^(l-1): through the sum and through w = 1 - y^(l-1) */
      }
    }
    for (int64_t j = 0; j < E; ++j) dL[r * E + j] = zb[j] * z[j];
  }
  free(w); free(z); free(yb); free(zb); free(ss);
  return MSO_OK;
}

/* ------------------------------------------------------------------ */
/* Iterative rerouting (Sec. 2.3, the Switch Transformers paragraph;     */
/* the assignment step of "MaxScore-I", Sec. 4.1 Baselines).             */
/* Stage 1: every token's k choices by descending affinity (ties: lowest */
/* expert index); choice level 1 of all tokens is served first, then     */
/* level 2, ..., within a level in ascending token index; a pair is      */
/* accepted while its expert holds fewer than C tokens, else dropped.    */
/* Stage 2: the dropped pairs, in ascending token index and within a     */
/* token in level order, are each given to the expert of highest         */
/* affinity among those that still have room and that the token does not */
/* hold (ties: lowest index); if there is none the slot stays empty.     */
/* The paper fixes neither order: both are this build's reading.         */
/* Outputs: expert_idx [T,k] ascending with -1 (empty) last, load [E],   */
/* counts[0] = pairs dropped in stage 1, counts[1] = slots left empty.   */
int mso_iterative_reroute(int64_t T, int64_t E, int64_t k, int64_t C, const double *A,
                          int32_t *expert_idx, int32_t *load, int64_t *counts) {
  if (k < 1 || k > E || C < 0) return MSO_ERR_ARG;
  int32_t *choice = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T * k));   /* [T][k], level order */
  unsigned char *held = (unsigned char *)calloc((size_t)(T * E), 1);
  unsigned char *dropped = (unsigned char *)calloc((size_t)(T * k), 1);
  if (!choice || !held || !dropped) { free(choice); free(held); free(dropped); return MSO_ERR_ALLOC; }
  for (int64_t i = 0; i < T; ++i) {
    const double *a = A + i * E;
    for (int64_t r = 0; r < k; ++r) {
      int64_t best = -1;
      for (int64_t j = 0; j < E; ++j) {
        int taken = 0;
        for (int64_t q = 0; q < r; ++q) if (choice[i * k + q] == j) taken = 1;
        if (taken) continue;
        if (best < 0 || a[j] > a[best]) best = j;
      }
      choice[i * k + r] = (int32_t)best;
    }
  }
  for (int64_t j = 0; j < E; ++j) load[j] = 0;
  int64_t ndrop = 0, nempty = 0;
  for (int64_t r = 0; r < k; ++r)
    for (int64_t i = 0; i < T; ++i) {
      const int32_t e = choice[i * k + r];
      if (load[e] < C) { load[e] += 1; held[i * E + e] = 1; }
      else { dropped[i * k + r] = 1; ++ndrop; }
    }
  for (int64_t i = 0; i < T; ++i)
    for (int64_t r = 0; r < k; ++r) {
      if (!dropped[i * k + r]) continue;
      const double *a = A + i * E;
      int64_t best = -1;
      for (int64_t j = 0; j < E; ++j) {
        if (load[j] >= C || held[i * E + j]) continue;
        if (best < 0 || a[j] > a[best]) best = j;
      }
      if (best < 0) { ++nempty; continue; }
      load[best] += 1; held[i * E + best] = 1;
    }
  for (int64_t i = 0; i < T; ++i) {
    int64_t n = 0;
    for (int64_t j = 0; j < E; ++j) if (held[i * E + j]) expert_idx[i * k + n++] = (int32_t)j;
    while (n < k) expert_idx[i * k + n++] = -1;
  }
  counts[0] = ndrop; counts[1] = nempty;
  free(choice); free(held); free(dropped);
  return MSO_OK;
}

/* ------------------------------------------------------------------ */
/* Algorithm 1: maximum score routing for top-2 (Sec. 3.2): top-1, then  */
/* Sinkhorn on what is left.  Steps as the algorithm numbers them:       */
/*   1  c_j = C                       (the caller's capacity, 2n/e in the paper)   */
/*   2  a = the affinities A          (given)                            */
/*   4  mask = one-hot of argmax_j a_ij (ties: lowest expert index)      */
/*   5  the masked pair is removed from the second stage                 */
/*   6  c_j = max(0, c_j - sum_i mask_ij)                                */
/*   7  k_i = 1                                                          */
/*   8-9  Sinkhorn for max sum P_ij a_ij over rows summing to 1 and      */
/*        columns within c.                                              */
/* What the paper leaves open, and the reading taken (all "parity        */
/* unpinned against the paper"):                                         */
/*   - Sinkhorn: entropic regularisation eps, kernel K_ij = exp((a_ij -  */
/*     m_i) / eps) over the unmasked pairs (m_i the row maximum, which   */
/*     the row scaling absorbs), `iters` rounds of                       */
/*         u_i = 1 / sum_j K_ij v_j,  t_j = sum_i u_i K_ij,  v_j = min(1, c_j / t_j)  */
/*     (columns are capped, not forced to equal c: the residual          */
/*     capacities sum to at least n), then a last row scaling.  Its      */
/*     fixed point has rows summing to 1 and every column either         */
/*     uncapped (v = 1) or exactly full: the optimality conditions of    */
/*     the entropic problem with capacity upper bounds.                  */
/*   - rounding: token i takes argmax_j of its plan row (ties: lowest    */
/*     index); per expert the first c_j such tokens in ascending token   */
/*     index are kept, the rest lose their second expert (-1).           */
/*   - top-1 pairs are never dropped here, even beyond C (step 6 clips   */
/*     the residual at 0); the E x C buffers drop them downstream.       */
/* Outputs: first/second [T] (second = -1: dropped), plan [T,E] (may be  */
/* NULL), resid [E] residual capacities, counts[0] = top-1 pairs beyond  */
/* C, counts[1] = second choices dropped.                                */
int mso_alg1_top1_sinkhorn(int64_t T, int64_t E, int64_t C, const double *A, double eps, int64_t iters,
                           int32_t *first, int32_t *second, double *plan, int64_t *resid, int64_t *counts) {
  if (E < 2 || C < 0 || !(eps > 0.0) || iters < 0) return MSO_ERR_ARG;
  double *K = (double *)malloc(sizeof(double) * (size_t)(T * E));
  double *u = (double *)malloc(sizeof(double) * (size_t)T);
  double *v = (double *)malloc(sizeof(double) * (size_t)E);
  double *t = (double *)malloc(sizeof(double) * (size_t)E);
  int64_t *cnt = (int64_t *)calloc((size_t)E, sizeof(int64_t));
  if (!K || !u || !v || !t || !cnt) { free(K); free(u); free(v); free(t); free(cnt); return MSO_ERR_ALLOC; }
  /* steps 4-6 */
  for (int64_t i = 0; i < T; ++i) {
    const double *a = A + i * E;
    int64_t best = 0;
    for (int64_t j = 1; j < E; ++j) if (a[j] > a[best]) best = j;
    first[i] = (int32_t)best; cnt[best] += 1;
  }
  int64_t over = 0;
  for (int64_t j = 0; j < E; ++j) {
    resid[j] = C - cnt[j] > 0 ? C - cnt[j] : 0;
    if (cnt[j] > C) over += cnt[j] - C;
  }
  /* steps 7-9 */
  for (int64_t i = 0; i < T; ++i) {
    const double *a = A + i * E;
    double m = -INFINITY;
    for (int64_t j = 0; j < E; ++j) if (j != first[i] && a[j] > m) m = a[j];
    for (int64_t j = 0; j < E; ++j) K[i * E + j] = (j == first[i]) ? 0.0 : exp((a[j] - m) / eps);
  }
  for (int64_t j = 0; j < E; ++j) v[j] = resid[j] > 0 ? 1.0 : 0.0;
  for (int64_t it = 0; it <= iters; ++it) {
    for (int64_t i = 0; i < T; ++i) {
      double s = 0.0;
      for (int64_t j = 0; j < E; ++j) s += K[i * E + j] * v[j];
      u[i] = s > 0.0 ? 1.0 / s : 0.0;
    }
    if (it == iters) break;                 /* the last row scaling */
    for (int64_t j = 0; j < E; ++j) t[j] = 0.0;
    for (int64_t i = 0; i < T; ++i)
      for (int64_t j = 0; j < E; ++j) t[j] += u[i] * K[i * E + j];
    for (int64_t j = 0; j < E; ++j) {
      if (resid[j] <= 0) v[j] = 0.0;
      else v[j] = (t[j] > (double)resid[j]) ? (double)resid[j] / t[j] : 1.0;
    }
  }
  int64_t *taken = (int64_t *)calloc((size_t)E, sizeof(int64_t));
  if (!taken) { free(K); free(u); free(v); free(t); free(cnt); return MSO_ERR_ALLOC; }
  int64_t dropped = 0;
  for (int64_t i = 0; i < T; ++i) {
    int64_t best = -1; double pb = 0.0;
    for (int64_t j = 0; j < E; ++j) {
      const double p = u[i] * K[i * E + j] * v[j];
      if (plan) plan[i * E + j] = p;
      if (p > pb) { pb = p; best = j; }     /* strictly larger: ties keep the lowest index; zero mass is no choice */
    }
    if (best >= 0 && taken[best] < resid[best]) { taken[best] += 1; second[i] = (int32_t)best; }
    else { second[i] = -1; ++dropped; }
  }
  counts[0] = over; counts[1] = dropped;
  free(K); free(u); free(v); free(t); free(cnt); free(taken);
  return MSO_OK;
}
