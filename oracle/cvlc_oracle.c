/*
 * CPU oracle for the Fed-CVLC per-round compression path (test infrastructure
 * only; see cvlc_oracle.h).  One thread, plain loops, the paper's steps in the
 * paper's order.  Build: gcc -O2 -ffp-contract=off -shared -fPIC.
 *
 * Notation follows the paper: d coordinates, k transmitted, R packets, P_r
 * records in packet r, y_r bits per value, s bits per position ID, b packet
 * bits, H header bits, B the scale-down constant, beta = 2*alpha + 1.
 */
#include "cvlc_oracle.h"

#include <float.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ======================================================================== */
/* Spec math: log2 / exp2 built from IEEE + - * / only, so that any machine   */
/* that evaluates the same operations in the same order gets the same bits.  */
/* ======================================================================== */

static double bits_to_double(uint64_t u) {
  double v;
  memcpy(&v, &u, 8);
  return v;
}
static uint64_t double_to_bits(double v) {
  uint64_t u;
  memcpy(&u, &v, 8);
  return u;
}

/* log2 of a positive, finite, normal double.
 * v = m * 2^e with m in [1,2); fold m into (sqrt(1/2), sqrt(2)];
 * ln m = 2 atanh(t), t = (m-1)/(m+1), as the odd series up to t^25. */
double cvlc_log2_oracle(double v) {
  uint64_t bits = double_to_bits(v);
  int e = (int)((bits >> 52) & 0x7FF) - 1023;
  double m = bits_to_double((bits & 0x000FFFFFFFFFFFFFull) | 0x3FF0000000000000ull);
  if (m > 1.4142135623730951) {
    m = m / 2.0;
    e = e + 1;
  }
  double t = (m - 1.0) / (m + 1.0);
  double q = t * t;
  double p = 1.0 / 25.0;
  for (int j = 11; j >= 0; --j) p = p * q + 1.0 / (double)(2 * j + 1);
  double ln_m = (2.0 * t) * p;
  return (double)e + ln_m * 1.4426950408889634;
}

/* 2^v for |v| <= 1000: v = n + r, |r| <= 1/2, e^(r ln 2) as a degree-20 Taylor
 * polynomial in Horner form, then n added to the exponent field. */
double cvlc_exp2_oracle(double v) {
  double n = floor(v + 0.5);
  double r = v - n;
  double u = r * 0.6931471805599453;
  double p = 1.0;
  for (int j = 20; j >= 1; --j) p = 1.0 + (u / (double)j) * p;
  int64_t ni = (int64_t)n;
  uint64_t pb = double_to_bits(p);
  pb = (uint64_t)((int64_t)pb + ni * ((int64_t)1 << 52));
  return bits_to_double(pb);
}

/* a^beta for a >= 1 */
double cvlc_powr_oracle(double a, double beta) { return cvlc_exp2_oracle(beta * cvlc_log2_oracle(a)); }

/* ======================================================================== */
/* Philox4x32-10, written from the published definition (Salmon, Moraes,     */
/* Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11).        */
/* ======================================================================== */

void cvlc_philox4x32_10_oracle(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The random word of coordinate `coord`: counter (coord lo, coord hi, client, round),
 * key (seed lo, seed hi), output word 0. */
uint32_t cvlc_philox_coord_oracle(uint64_t seed, uint32_t client_id, uint32_t round, uint64_t coord) {
  uint32_t ctr[4] = {(uint32_t)coord, (uint32_t)(coord >> 32), client_id, round};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  cvlc_philox4x32_10_oracle(ctr, key, out);
  return out[0];
}

/* ======================================================================== */
/* Keys, histogram, power-law exponent (Definition 1; Algorithm 1, step 1)   */
/* ======================================================================== */

static uint32_t key_of(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  return u & 0x7FFFFFFFu;
}

/* h[j] = number of coordinates whose magnitude key has top bits j
 * (8 exponent bits and the 4 leading mantissa bits). */
int cvlc_histogram_oracle(const float* x, uint64_t d, uint64_t h[ORC_HIST_BINS]) {
  memset(h, 0, sizeof(uint64_t) * ORC_HIST_BINS);
  int nonfinite = 0;
  for (uint64_t i = 0; i < d; ++i) {
    uint32_t key = key_of(x[i]);
    if (key >= 0x7F800000u) nonfinite = 1;
    h[key >> 19] += 1;
  }
  return nonfinite ? ORC_ERR_NONFINITE_INPUT : ORC_OK;
}

/* Least squares of log2|U{l}| on log2 l (Definition 1: |U{l}| <= phi * l^alpha)
 * over the histogram's survival counts: the point of bin j is
 * (log2 N_j, log2 of the bin's lower edge), N_j = #{key >> 19 >= j}, for the
 * non-empty normal bins in the upper half of the ranks. */
void cvlc_alpha_fit_oracle(const uint64_t h[ORC_HIST_BINS], uint64_t d, double* alpha, double* alpha_q) {
  static uint64_t N[ORC_HIST_BINS + 1];
  N[ORC_HIST_BINS] = 0;
  for (int j = ORC_HIST_BINS - 1; j >= 0; --j) N[j] = N[j + 1] + h[j];
  double n = 0.0, Sx = 0.0, Sy = 0.0, Sxx = 0.0, Sxy = 0.0;
  for (int j = 16; j <= 4079; ++j) {
    if (h[j] == 0) continue;
    if (N[j] < 1 || N[j] > d / 2) continue;
    double X = cvlc_log2_oracle((double)N[j]);
    double Y = (double)((j >> 4) - 127) + cvlc_log2_oracle(1.0 + (double)(j & 15) / 16.0);
    n = n + 1.0;
    Sx = Sx + X;
    Sy = Sy + Y;
    Sxx = Sxx + X * X;
    Sxy = Sxy + X * Y;
  }
  double den = n * Sxx - Sx * Sx;
  double a;
  if (n < 2.0 || !(den > 0.0))
    a = -1.0;
  else
    a = (n * Sxy - Sx * Sy) / den;
  double aq = floor(a * 256.0 + 0.5) / 256.0;
  if (aq < -4.0) aq = -4.0;
  if (aq > -1.0 / 256.0) aq = -1.0 / 256.0;
  if (aq == -0.5) aq = -0.5 - 1.0 / 256.0; /* beta = 0 would make d^beta - 1 vanish */
  *alpha = a;
  *alpha_q = aq;
}

/* ======================================================================== */
/* Packet constraint (Eq. (3)) and per-length coefficients (Eq. (5))         */
/* ======================================================================== */

static int params_ok(const orc_params* p) {
  if (!p) return 0;
  if (p->d < 2 || p->d > ((uint64_t)1 << 31)) return 0;
  if (p->packet_bits == 0 || (p->packet_bits % 32) != 0) return 0;
  if (p->header_bits < 80 || p->header_bits >= p->packet_bits) return 0;
  if (p->quantizer != ORC_QUANT_PQ && p->quantizer != ORC_QUANT_QSGD) return 0;
  if (p->max_code_bits < 1 || p->max_code_bits > ORC_MAX_Y) return 0;
  if (!(p->scale_B >= 1.0) || !(p->scale_B < 1e300)) return 0;
  return 1;
}

/* s = ceil(log2 d) (Section IV-C); R = floor(budget / b); cap(y) = the most
 * records P that satisfy P*(s+y) + H <= b. */
int cvlc_derive_oracle(const orc_params* p, uint32_t* s_out, uint32_t* R_out, uint32_t cap[ORC_MAX_Y + 1]) {
  if (!params_ok(p)) return ORC_ERR_INVALID_ARG;
  uint32_t s = 1;
  while (((uint64_t)1 << s) < p->d) ++s;
  uint64_t R = p->budget_bits / p->packet_bits;
  if (R == 0) return ORC_ERR_BUDGET_TOO_SMALL;
  if (R > 0xFFFFFFFFull) return ORC_ERR_BUDGET_TOO_LARGE;
  for (uint32_t y = 0; y <= ORC_MAX_Y; ++y) cap[y] = 0;
  for (uint32_t y = 1; y <= p->max_code_bits; ++y) cap[y] = (p->packet_bits - p->header_bits) / (s + y);
  if (cap[p->max_code_bits] < 1) return ORC_ERR_PACKET_TOO_SMALL;
  *s_out = s;
  *R_out = (uint32_t)R;
  return ORC_OK;
}

size_t cvlc_stream_bytes_oracle(const orc_params* p) {
  uint64_t R = p->budget_bits / p->packet_bits;
  return (size_t)(64 + R * (p->packet_bits / 8));
}

/* Magnitude levels of a y-bit QSGD code.  The paper gives every record y bits and lets
 * QSGD quantize absolute values; it does not say where the sign goes.  Here the top bit of
 * the code is the sign and the other y - 1 bits hold a level 0..s_q, s_q = 2^(y-1) - 1, so a
 * record stays s + y bits wide and Eq. (3) holds unchanged.  One bit cannot hold a level. */
static uint32_t qsgd_levels(uint32_t y) { return (y >= 2) ? (uint32_t)((((uint64_t)1) << (y - 1)) - 1) : 0u; }

/* Quantization error factor with P = cap(y) values at y bits (Appendix, case study).
 * PQ:   Q = P / (2^y - 1)^2, 2^y - 1 being the intervals between its 2^y centroids.
 * QSGD: Q = min(P / s_q^2, sqrt(P) / s_q), the paper's min(Q_1, Q_2) with its level count
 *       (printed as 2^y) replaced by the s_q levels the record format really has. */
static double Q_of(uint32_t quantizer, uint32_t cap_y, uint32_t y) {
  if (quantizer == ORC_QUANT_QSGD) {
    if (y < 2) return INFINITY;
    double sq = (double)qsgd_levels(y);
    double Q1 = (double)cap_y / (sq * sq);
    double Q2 = sqrt((double)cap_y) / sq;
    return (Q1 < Q2) ? Q1 : Q2;
  }
  double L = (double)(((uint64_t)1 << y) - 1);
  return (double)cap_y / (L * L);
}

double cvlc_quant_error_Q_oracle(const orc_params* p, uint32_t y) {
  uint32_t s, R, cap[ORC_MAX_Y + 1];
  if (cvlc_derive_oracle(p, &s, &R, cap) != ORC_OK || y < 1 || y > p->max_code_bits) return NAN;
  return Q_of(p->quantizer, cap[y], y);
}

/* The bracket of Eq. (5) is c = Q/B^2 + 1/B_c^2 with 1/B_c = 1 - 1/B; g = 1 - c is
 * what a packet gains over sparsifying its coordinates. */
static double g_of(double Q, double B) {
  double c = Q / (B * B) + (1.0 - 1.0 / B) * (1.0 - 1.0 / B);
  return 1.0 - c;
}

double cvlc_coeff_g_oracle(const orc_params* p, uint32_t y) {
  double Q = cvlc_quant_error_Q_oracle(p, y);
  return g_of(Q, p->scale_B);
}

/* Scale of a first round: 1 + Q of an 8-bit packet (the paper takes B from the previous
 * round's max Q + 1; there is no previous round yet). */
double cvlc_default_scale_oracle(const orc_params* p) {
  orc_params q = *p;
  q.scale_B = 1.0;
  q.max_code_bits = ORC_MAX_Y;
  if (!params_ok(&q)) return NAN;
  uint32_t s = 1;
  while (((uint64_t)1 << s) < p->d) ++s;
  uint32_t cap8 = (p->packet_bits - p->header_bits) / (s + 8);
  return 1.0 + Q_of(p->quantizer, cap8, 8);
}

/* Planner context: candidate lengths and their coefficients */
typedef struct {
  uint64_t d;
  uint32_t R;
  int nY;
  uint32_t Y[ORC_MAX_Y + 1];   /* ascending */
  double g[ORC_MAX_Y + 1];     /* by length */
  double Q[ORC_MAX_Y + 1];     /* by length */
  uint32_t cap[ORC_MAX_Y + 1]; /* by length */
  uint32_t y_min;
  double beta, D;
  uint64_t n_evals;
} plan_ctx;

static int ctx_init(plan_ctx* c, const orc_params* p, uint32_t* s_out) {
  uint32_t s, R;
  int rc = cvlc_derive_oracle(p, &s, &R, c->cap);
  if (rc != ORC_OK) return rc;
  *s_out = s;
  c->d = p->d;
  c->R = R;
  c->n_evals = 0;
  c->y_min = 0;
  c->nY = 0;
  for (uint32_t y = 1; y <= p->max_code_bits; ++y) {
    c->Q[y] = Q_of(p->quantizer, c->cap[y], y);
    c->g[y] = g_of(c->Q[y], p->scale_B);
    if (c->y_min == 0 && c->g[y] > 0.0) c->y_min = y;
  }
  if (c->y_min == 0) return ORC_ERR_SCALE_TOO_SMALL;
  c->nY = 0;
  for (uint32_t y = c->y_min; y <= p->max_code_bits; ++y) {
    /* a length that fits no more records than the next longer one is dominated */
    if (y == p->max_code_bits || c->cap[y] > c->cap[y + 1]) c->Y[c->nY++] = y;
  }
  return ORC_OK;
}

int cvlc_candidates_oracle(const orc_params* p, uint32_t Y[ORC_MAX_Y + 1]) {
  plan_ctx c;
  uint32_t s;
  if (ctx_init(&c, p, &s) != ORC_OK) return 0;
  for (int i = 0; i < c.nY; ++i) Y[i] = c.Y[i];
  return c.nY;
}

static void ctx_set_beta(plan_ctx* c, double beta) {
  c->beta = beta;
  c->D = cvlc_powr_oracle((double)c->d, beta) - 1.0;
}

/* Share of ||U||^2 carried by the top Z ranks under Definition 1:
 * sum_{l<=Z} l^(2 alpha) ~ ((Z+1)^beta - 1) / (d^beta - 1), the boundary the first
 * term of Eq. (5) uses (d^beta - (k+1)^beta), applied to every packet boundary. */
static double energy_E(const plan_ctx* c, uint64_t Z) {
  return (cvlc_powr_oracle((double)(Z + 1), c->beta) - 1.0) / c->D;
}

/* F(n) = 1 - gamma, gamma of Eq. (5) with the packets grouped by code length as in
 * Eq. (1): packets are laid out longest code first, so the group of length y covers
 * ranks (W_prev, W]. */
static double objective_F(plan_ctx* c, const uint32_t n[ORC_MAX_Y + 1]) {
  uint64_t W = 0;
  double Eprev = 0.0, F = 0.0;
  c->n_evals += 1;
  for (int i = c->nY - 1; i >= 0; --i) {
    uint32_t y = c->Y[i];
    if (n[y] == 0) continue;
    W += (uint64_t)n[y] * (uint64_t)c->cap[y];
    double Ecur = energy_E(c, W);
    F = F + c->g[y] * (Ecur - Eprev);
    Eprev = Ecur;
  }
  if (W > c->d) return -INFINITY;
  return F;
}

double cvlc_objective_oracle(const orc_params* p, double beta, const uint32_t n_y[ORC_MAX_Y + 1]) {
  plan_ctx c;
  uint32_t s;
  if (ctx_init(&c, p, &s) != ORC_OK) return NAN;
  ctx_set_beta(&c, beta);
  uint32_t n[ORC_MAX_Y + 1];
  memset(n, 0, sizeof n);
  for (int i = 0; i < c.nY; ++i) n[c.Y[i]] = n_y[c.Y[i]];
  return objective_F(&c, n);
}

/* Atomic operation (Section IV-C): two lengths a > c share X = n_a + n_c packets;
 * choose the split that maximises F (minimises gamma).  F is discretely concave in
 * the split (Lemma 2), so the first t with F(t+1) <= F(t) is found by bisection. */
static int atomic_op(plan_ctx* c, uint32_t n[ORC_MAX_Y + 1], uint32_t a, uint32_t cc) {
  uint32_t X = n[a] + n[cc];
  if (X == 0) return 0;
  uint32_t na0 = n[a], nc0 = n[cc];
  uint32_t lo = 0, hi = X;
  while (lo < hi) {
    uint32_t mid = lo + (hi - lo) / 2;
    n[a] = mid + 1; n[cc] = X - (mid + 1);
    double F1 = objective_F(c, n);
    n[a] = mid; n[cc] = X - mid;
    double F0 = objective_F(c, n);
    if (F1 > F0) lo = mid + 1; else hi = mid;
  }
  int moved = 0;
  if (lo != na0) {
    n[a] = lo; n[cc] = X - lo;
    double Fnew = objective_F(c, n);
    n[a] = na0; n[cc] = nc0;
    double Fold = objective_F(c, n);
    if (Fnew > Fold) { n[a] = lo; n[cc] = X - lo; moved = 1; }
  } else {
    n[a] = na0; n[cc] = nc0;
  }
  return moved;
}

static void plan_fill(orc_plan* plan, plan_ctx* c, uint32_t s, const uint32_t n[ORC_MAX_Y + 1],
                      double alpha, double alpha_q) {
  memset(plan, 0, sizeof *plan);
  plan->s = s;
  plan->R = c->R;
  plan->y_min = c->y_min;
  plan->n_lengths = (uint32_t)c->nY;
  plan->alpha = alpha;
  plan->alpha_q = alpha_q;
  plan->beta = c->beta;
  uint64_t k = 0;
  double Qmax = 0.0;
  for (uint32_t y = 1; y <= ORC_MAX_Y; ++y) {
    plan->cap[y] = c->cap[y];
    plan->n_y[y] = n[y];
    k += (uint64_t)n[y] * c->cap[y];
    if (n[y] > 0 && c->Q[y] > Qmax) Qmax = c->Q[y];
  }
  plan->k = k;
  double F = objective_F(c, n);
  plan->gamma = 1.0 - F;
  plan->B_next = 1.0 + Qmax;
  plan->n_evals = c->n_evals;
}

/* Algorithm 1, steps 2-14, on integer code lengths: start from equal packets, then
 * repeat atomic operations on pairs of lengths until no pair can be improved. */
int cvlc_plan_from_alpha_oracle(const orc_params* p, double alpha_q, orc_plan* plan) {
  plan_ctx c;
  uint32_t s;
  int rc = ctx_init(&c, p, &s);
  if (rc != ORC_OK) return rc;
  ctx_set_beta(&c, 2.0 * alpha_q + 1.0);

  uint32_t n[ORC_MAX_Y + 1];
  /* equal packets: the best admissible single-length plan, ties to the longer code */
  int best = -1;
  double bestF = -INFINITY;
  for (int i = 0; i < c.nY; ++i) {
    memset(n, 0, sizeof n);
    n[c.Y[i]] = c.R;
    double F = objective_F(&c, n);
    if (F == -INFINITY) continue;
    if (best < 0 || F >= bestF) { best = i; bestF = F; }
  }
  if (best < 0) return ORC_ERR_BUDGET_TOO_LARGE;
  memset(n, 0, sizeof n);
  n[c.Y[best]] = c.R;

  for (int round = 0; round < 64; ++round) {
    /* phase A: neighbouring lengths, until a sweep moves nothing */
    for (int sweep = 0; sweep < 256; ++sweep) {
      int moved = 0;
      for (int i = c.nY - 1; i >= 1; --i) moved |= atomic_op(&c, n, c.Y[i], c.Y[i - 1]);
      if (!moved) break;
    }
    /* phase B: every pair once */
    int movedB = 0;
    for (int i = c.nY - 1; i >= 1; --i)
      for (int j = i - 1; j >= 0; --j) movedB |= atomic_op(&c, n, c.Y[i], c.Y[j]);
    if (!movedB) break;
  }
  plan_fill(plan, &c, s, n, alpha_q, alpha_q);
  return ORC_OK;
}

/* Section IV-C, last paragraph: a client may send the distribution of its update to the
 * parameter server, which solves the problem and returns k and the P_r.  The distribution
 * is the 4096-bin histogram of |x|: Algorithm 1 uses the update only through alpha. */
int cvlc_plan_from_histogram_oracle(const uint64_t h[ORC_HIST_BINS], const orc_params* p, orc_plan* plan) {
  if (!params_ok(p)) return ORC_ERR_INVALID_ARG;
  uint64_t total = 0;
  for (int j = 0; j < ORC_HIST_BINS; ++j) total += h[j];
  if (total != p->d) return ORC_ERR_INVALID_ARG;
  /* bins of exponent 255: Inf and NaN */
  for (int j = (int)(0x7F800000u >> 19); j < ORC_HIST_BINS; ++j)
    if (h[j] != 0) return ORC_ERR_NONFINITE_INPUT;
  double alpha, alpha_q;
  cvlc_alpha_fit_oracle(h, p->d, &alpha, &alpha_q);
  int rc = cvlc_plan_from_alpha_oracle(p, alpha_q, plan);
  if (rc == ORC_OK) plan->alpha = alpha;
  return rc;
}

int cvlc_plan_oracle(const float* x, const orc_params* p, orc_plan* plan) {
  if (!params_ok(p)) return ORC_ERR_INVALID_ARG;
  static uint64_t h[ORC_HIST_BINS];
  int rc = cvlc_histogram_oracle(x, p->d, h);
  if (rc != ORC_OK) return rc;
  return cvlc_plan_from_histogram_oracle(h, p, plan);
}

/* Degenerate plan: every packet at one length y ("Top_k plus y-bit quantization",
 * the baselines of Section V). */
int cvlc_plan_fixed_oracle(const orc_params* p, uint32_t y, orc_plan* plan) {
  if (!params_ok(p)) return ORC_ERR_INVALID_ARG;
  if (y < 1 || y > p->max_code_bits) return ORC_ERR_INVALID_ARG;
  if (p->quantizer == ORC_QUANT_QSGD && y < 2) return ORC_ERR_INVALID_ARG;
  plan_ctx c;
  uint32_t s;
  int rc = ctx_init(&c, p, &s);
  if (rc != ORC_OK && rc != ORC_ERR_SCALE_TOO_SMALL) return rc;
  if ((uint64_t)c.R * c.cap[y] > p->d) return ORC_ERR_BUDGET_TOO_LARGE;
  /* evaluate gamma with the single length y as the only candidate */
  c.nY = 1;
  c.Y[0] = y;
  c.Q[y] = Q_of(p->quantizer, c.cap[y], y);
  c.g[y] = g_of(c.Q[y], p->scale_B);
  c.y_min = y;
  ctx_set_beta(&c, 2.0 * (-1.0) + 1.0);
  uint32_t n[ORC_MAX_Y + 1];
  memset(n, 0, sizeof n);
  n[y] = c.R;
  plan_fill(plan, &c, s, n, -1.0, -1.0);
  return ORC_OK;
}

/* ======================================================================== */
/* Problem P2 with real-valued packet sizes (Section IV-C): enumerate k, and   */
/* for every k tune P_1 .. P_R two consecutive packets at a time               */
/* ======================================================================== */

/* What a real-valued packet of P records contributes per unit of energy: the bracket of
 * Eq. (5) with the code length the packet constraint leaves, y = (b - H) / P - s. */
static double packet_cost(double P, double bH, double s, uint32_t quantizer, double B) {
  double y = bH / P - s;
  double Q;
  if (quantizer == ORC_QUANT_QSGD) {
    double sq = cvlc_exp2_oracle(y - 1.0) - 1.0;
    double Q1 = P / (sq * sq);
    double Q2 = sqrt(P) / sq;
    Q = (Q1 < Q2) ? Q1 : Q2;
  } else {
    double L = cvlc_exp2_oracle(y) - 1.0;
    Q = P / (L * L);
  }
  return Q / (B * B) + (1.0 - 1.0 / B) * (1.0 - 1.0 / B);
}

/* share of the energy in the top Z ranks for real Z (same boundary as energy_E) */
static double energy_real(double Z, double beta, double D) { return (cvlc_powr_oracle(Z + 1.0, beta) - 1.0) / D; }

/* Eq. (7): the part of gamma that the split of X = P_{r-1} + P_r records between the packets r-1 and r
 * decides, as a function of p = P_r; Z0 = Z_{r-2}, Z2 = Z_r. */
static double pair_f(double p, double X, double Z0, double Z2, double bH, double s, uint32_t quantizer, double B,
                     double beta, double D) {
  double Em = energy_real(Z0 + (X - p), beta, D);
  double hi_part = packet_cost(p, bH, s, quantizer, B) * (energy_real(Z2, beta, D) - Em);
  double lo_part = packet_cost(X - p, bH, s, quantizer, B) * (Em - energy_real(Z0, beta, D));
  return hi_part + lo_part;
}

int cvlc_plan_literal_oracle(const orc_params* p, double alpha_q, uint32_t n_k, uint32_t max_sweeps, uint64_t* k_grid,
                             double* gamma_of_k, uint32_t* sweeps_of_k, uint64_t* k_star, double* gamma_star, double* P_star) {
  if (!params_ok(p) || n_k < 1 || n_k > 4096 || max_sweeps < 1 || !(alpha_q < 0.0) || alpha_q == -0.5) return ORC_ERR_INVALID_ARG;
  uint32_t si, R, cap[ORC_MAX_Y + 1];
  int rc = cvlc_derive_oracle(p, &si, &R, cap);
  if (rc != ORC_OK) return rc;
  const uint32_t y_lo = (p->quantizer == ORC_QUANT_QSGD) ? 2u : 1u; /* a one-bit QSGD code holds no level */
  if (p->max_code_bits < y_lo) return ORC_ERR_INVALID_ARG;
  const double s = (double)si, bH = (double)(p->packet_bits - p->header_bits), B = p->scale_B;
  const double P_min = bH / (s + (double)p->max_code_bits), P_max = bH / (s + (double)y_lo);
  /* the range of k: at least one record per packet and no code longer than max_code_bits, no code shorter than
   * y_lo, no more than d coordinates */
  double klo = ceil((double)R * P_min), khi = floor((double)R * P_max);
  if (klo < (double)R) klo = (double)R;
  if (khi > (double)p->d) khi = (double)p->d;
  if (!(klo <= khi)) return ORC_ERR_BUDGET_TOO_LARGE;
  const uint64_t k_lo = (uint64_t)klo, k_hi = (uint64_t)khi;
  const double beta = 2.0 * alpha_q + 1.0;
  const double D = cvlc_powr_oracle((double)p->d, beta) - 1.0;
  const double tol = P_max * (1.0 / 1073741824.0);

  double* P = (double*)malloc(sizeof(double) * (size_t)R);
  double* Z = (double*)malloc(sizeof(double) * ((size_t)R + 1));
  if (!P || !Z) { free(P); free(Z); return ORC_ERR_INVALID_ARG; }
  int have = 0;
  for (uint32_t ik = 0; ik < n_k; ++ik) {
    /* equidistant values of k (Section IV-D) */
    uint64_t k = (n_k == 1) ? k_lo : k_lo + (uint64_t)(((unsigned __int128)ik * (k_hi - k_lo)) / (n_k - 1));
    for (uint32_t r = 0; r < R; ++r) P[r] = (double)k / (double)R; /* equal packets */
    uint32_t sweep = 0;
    for (; sweep < max_sweeps; ++sweep) {
      Z[0] = 0.0;
      for (uint32_t r = 0; r < R; ++r) Z[r + 1] = Z[r] + P[r];
      double moved = 0.0;
      for (uint32_t r = 1; r < R; ++r) { /* packets r-1 and r (0-based), the later one the larger (Eq. (4)) */
        double X = P[r - 1] + P[r], Z0 = Z[r - 1], Z2 = Z[r + 1];
        double lo = X / 2.0, hi = X - P_min;
        if (lo < P_min) lo = P_min;
        if (lo < X - P_max) lo = X - P_max;
        if (hi > P_max) hi = P_max;
        if (!(lo < hi)) continue;
        /* the atomic operation: f is strongly convex in p (Lemma 2); eight times, 32 equidistant points of the
         * bracket are tried and the bracket shrinks to the neighbours of the best one */
        double best_x = lo;
        for (int round = 0; round < 8; ++round) {
          double step = (hi - lo) / 31.0;
          int best_j = 0;
          double best_f = 0.0;
          for (int j = 0; j < 32; ++j) {
            double xj = (j == 31) ? hi : lo + (double)j * step;
            double fj = pair_f(xj, X, Z0, Z2, bH, s, p->quantizer, B, beta, D);
            if (j == 0 || fj < best_f) { best_f = fj; best_j = j; }
          }
          double nlo = (best_j == 0) ? lo : lo + (double)(best_j - 1) * step;
          double nhi = (best_j >= 30) ? hi : lo + (double)(best_j + 1) * step;
          best_x = (best_j == 31) ? hi : lo + (double)best_j * step;
          lo = nlo;
          hi = nhi;
        }
        double f_new = pair_f(best_x, X, Z0, Z2, bH, s, p->quantizer, B, beta, D);
        double f_old = pair_f(P[r], X, Z0, Z2, bH, s, p->quantizer, B, beta, D);
        if (f_new < f_old) {
          double delta = fabs(best_x - P[r]);
          if (delta > moved) moved = delta;
          P[r - 1] = X - best_x;
          P[r] = best_x;
          Z[r] = Z0 + P[r - 1];
        }
      }
      if (!(moved > tol)) { ++sweep; break; }
    }
    /* Eq. (5) at these packet sizes */
    Z[0] = 0.0;
    for (uint32_t r = 0; r < R; ++r) Z[r + 1] = Z[r] + P[r];
    double gamma = 1.0 - energy_real(Z[R], beta, D);
    double Eprev = 0.0;
    for (uint32_t r = 0; r < R; ++r) {
      double Ecur = energy_real(Z[r + 1], beta, D);
      gamma = gamma + packet_cost(P[r], bH, s, p->quantizer, B) * (Ecur - Eprev);
      Eprev = Ecur;
    }
    if (k_grid) k_grid[ik] = k;
    if (gamma_of_k) gamma_of_k[ik] = gamma;
    if (sweeps_of_k) sweeps_of_k[ik] = sweep;
    if (!have || gamma < *gamma_star) {
      have = 1;
      *gamma_star = gamma;
      *k_star = k;
      if (P_star) memcpy(P_star, P, sizeof(double) * (size_t)R);
    }
  }
  free(P);
  free(Z);
  return ORC_OK;
}

/* ======================================================================== */
/* Ranking ("ranked in a descending order of their absolute values")          */
/* ======================================================================== */

static int cmp_desc_u64(const void* a, const void* b) {
  uint64_t x = *(const uint64_t*)a, y = *(const uint64_t*)b;
  return (x < y) - (x > y);
}

/* Order: magnitude key descending, ties by ascending index.  The pair is packed
 * as key * 2^32 + (2^32 - 1 - index) so one descending sort gives that order. */
int cvlc_rank_oracle(const float* x, uint64_t d, uint64_t k, uint32_t* idx_out) {
  if (k > d) return ORC_ERR_INVALID_ARG;
  uint64_t* comp = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)d);
  if (!comp) return ORC_ERR_INVALID_ARG;
  for (uint64_t i = 0; i < d; ++i) comp[i] = ((uint64_t)key_of(x[i]) << 32) | (uint64_t)(0xFFFFFFFFu - (uint32_t)i);
  qsort(comp, (size_t)d, sizeof(uint64_t), cmp_desc_u64);
  for (uint64_t r = 0; r < k; ++r) idx_out[r] = 0xFFFFFFFFu - (uint32_t)(comp[r] & 0xFFFFFFFFu);
  free(comp);
  return ORC_OK;
}

/* ======================================================================== */
/* PQ stochastic quantization (uniform centroids on [min,max], each value     */
/* mapped to its upper or lower centroid, unbiased)                           */
/* ======================================================================== */

uint32_t cvlc_pq_quantize_oracle(float x, float lo, float hi, uint32_t y, uint32_t rnd) {
  if (hi == lo) return 0;
  double L = (double)(((uint64_t)1 << y) - 1);
  double num = (double)x - (double)lo;
  double den = (double)hi - (double)lo;
  double t = (num / den) * L;
  double j0 = floor(t);
  if (j0 > L) j0 = L;
  double frac = t - j0;
  double u = (double)rnd * (1.0 / 4294967296.0);
  uint32_t code = (uint32_t)j0;
  if (u < frac) code += 1;
  return code;
}

float cvlc_pq_dequantize_oracle(uint32_t code, float lo, float hi, uint32_t y) {
  if (hi == lo) return lo;
  double L = (double)(((uint64_t)1 << y) - 1);
  double den = (double)hi - (double)lo;
  return (float)((double)lo + (double)code * (den / L));
}

/* ======================================================================== */
/* QSGD stochastic quantization (Alistarh et al.): |x| / ||segment||_2 is      */
/* rounded up or down onto the grid {0, 1/s_q, ..., 1}, unbiased; the sign is  */
/* kept.  Section IV-C: the header carries the l2-norm as the centroid         */
/* distribution (32 bits).                                                     */
/* ======================================================================== */

/* l2-norm of a packet's values: squares (exact in double) added in rank order in double,
 * square root, rounded to fp32; a result beyond the fp32 range is stored as FLT_MAX. */
float cvlc_qsgd_norm_oracle(const float* v, uint32_t n) {
  double sum = 0.0;
  for (uint32_t j = 0; j < n; ++j) sum = sum + (double)v[j] * (double)v[j];
  double r = sqrt(sum);
  if (r > (double)FLT_MAX) return FLT_MAX;
  return (float)r;
}

/* code = sign bit (bit y-1) | level (bits 0..y-2) */
uint32_t cvlc_qsgd_quantize_oracle(float x, float norm, uint32_t y, uint32_t rnd) {
  uint32_t sq = qsgd_levels(y);
  uint32_t sign = (x < 0.0f) ? 1u : 0u;
  uint32_t level = 0;
  if (norm > 0.0f) {
    double a = fabs((double)x);
    double t = (a / (double)norm) * (double)sq;
    double j0 = floor(t);
    if (j0 > (double)sq) j0 = (double)sq;
    double frac = t - j0;
    double u = (double)rnd * (1.0 / 4294967296.0);
    level = (uint32_t)j0;
    if (u < frac) level += 1;
    if (level > sq) level = sq; /* only when |x| > norm, i.e. the norm was cut to FLT_MAX */
  }
  return (sign << (y - 1)) | level;
}

float cvlc_qsgd_dequantize_oracle(uint32_t code, float norm, uint32_t y) {
  uint32_t sq = qsgd_levels(y);
  uint32_t level = code & sq; /* s_q = 2^(y-1) - 1 is also the mask of the level bits */
  double mag = (double)level * ((double)norm / (double)sq);
  float v = (float)mag;
  return ((code >> (y - 1)) & 1u) ? -v : v;
}

/* ======================================================================== */
/* Bit stream (packet layout of Fig. 2: header with s, y_r and the centroid   */
/* distribution, then (PID, CID) pairs)                                       */
/* ======================================================================== */

/* bit i of a packet is bit (i mod 32) of its (i / 32)-th little-endian 32-bit word */
static void put_bits(uint8_t* pkt, uint64_t bitpos, uint64_t value, uint32_t width) {
  for (uint32_t i = 0; i < width; ++i) {
    uint64_t bp = bitpos + i;
    if ((value >> i) & 1) pkt[bp >> 3] |= (uint8_t)(1u << (bp & 7));
  }
}
static uint64_t get_bits(const uint8_t* pkt, uint64_t bitpos, uint32_t width) {
  uint64_t v = 0;
  for (uint32_t i = 0; i < width; ++i) {
    uint64_t bp = bitpos + i;
    if ((pkt[bp >> 3] >> (bp & 7)) & 1) v |= ((uint64_t)1 << i);
  }
  return v;
}

static void put_le(uint8_t* p, uint64_t v, int nbytes) {
  for (int i = 0; i < nbytes; ++i) p[i] = (uint8_t)(v >> (8 * i));
}
static uint64_t get_le(const uint8_t* p, int nbytes) {
  uint64_t v = 0;
  for (int i = 0; i < nbytes; ++i) v |= (uint64_t)p[i] << (8 * i);
  return v;
}

static float canon(float x) { return (key_of(x) == 0) ? 0.0f : x; }
static uint32_t float_bits(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  return u;
}
static float bits_float(uint32_t u) {
  float x;
  memcpy(&x, &u, 4);
  return x;
}

/* Algorithm 1, steps 15-17: packet r takes the next P_r ranked coordinates and
 * quantizes them with y_r bits; everything not sent is zero at the receiver. */
int cvlc_encode_oracle(const float* x, const orc_params* p, const orc_plan* plan, uint8_t* stream,
                       size_t capacity, uint32_t* ranked_idx_out) {
  if (!params_ok(p) || !plan) return ORC_ERR_INVALID_ARG;
  uint32_t s, R, cap[ORC_MAX_Y + 1];
  int rc = cvlc_derive_oracle(p, &s, &R, cap);
  if (rc != ORC_OK) return rc;
  if (plan->R != R || plan->s != s) return ORC_ERR_INVALID_ARG;
  size_t total = cvlc_stream_bytes_oracle(p);
  if (capacity < total) return ORC_ERR_OUTPUT_TOO_SMALL;
  uint64_t k = 0, nsum = 0;
  for (uint32_t y = 1; y <= ORC_MAX_Y; ++y) {
    if (plan->n_y[y] && cap[y] == 0) return ORC_ERR_INVALID_ARG;
    k += (uint64_t)plan->n_y[y] * cap[y];
    nsum += plan->n_y[y];
  }
  if (nsum != R || k != plan->k || k > p->d) return ORC_ERR_INVALID_ARG;
  for (uint64_t i = 0; i < p->d; ++i)
    if (key_of(x[i]) >= 0x7F800000u) return ORC_ERR_NONFINITE_INPUT;

  uint32_t* rank = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)(k ? k : 1));
  if (!rank) return ORC_ERR_INVALID_ARG;
  rc = cvlc_rank_oracle(x, p->d, k, rank);
  if (rc != ORC_OK) { free(rank); return rc; }
  if (ranked_idx_out) memcpy(ranked_idx_out, rank, sizeof(uint32_t) * (size_t)k);

  memset(stream, 0, total);
  /* global header, 64 bytes, little-endian */
  put_le(stream + 0, 0x434C5643u, 4);
  put_le(stream + 4, 1, 2);
  put_le(stream + 6, p->quantizer, 1);
  put_le(stream + 7, s, 1);
  put_le(stream + 8, p->d, 8);
  put_le(stream + 16, R, 4);
  put_le(stream + 20, p->packet_bits, 4);
  put_le(stream + 24, p->header_bits, 4);
  put_le(stream + 28, p->client_id, 4);
  put_le(stream + 32, p->seed, 8);
  put_le(stream + 40, p->round, 4);
  put_le(stream + 44, 0, 4);
  put_le(stream + 48, double_to_bits(p->scale_B), 8);
  put_le(stream + 56, k, 8);

  const uint32_t pkt_bytes = p->packet_bits / 8;
  uint64_t Z = 0; /* ranks already packed */
  uint32_t r = 0;
  for (int y = ORC_MAX_Y; y >= 1; --y) {      /* longest codes first: P_1 <= ... <= P_R */
    for (uint32_t q = 0; q < plan->n_y[y]; ++q, ++r) {
      uint8_t* pkt = stream + 64 + (size_t)r * pkt_bytes;
      uint32_t P = cap[y];
      float lo = 0.0f, hi = 0.0f, norm = 0.0f;
      put_bits(pkt, 0, s, 8);
      put_bits(pkt, 8, (uint64_t)y, 8);
      if (p->quantizer == ORC_QUANT_QSGD) {
        /* centroid distribution of QSGD: the l2-norm of the packet's values (32 bits) */
        if (y < 2) { free(rank); return ORC_ERR_INVALID_ARG; }
        float* seg = (float*)malloc(sizeof(float) * (size_t)P);
        if (!seg) { free(rank); return ORC_ERR_INVALID_ARG; }
        for (uint32_t j = 0; j < P; ++j) seg[j] = canon(x[rank[Z + j]]);
        norm = cvlc_qsgd_norm_oracle(seg, P);
        free(seg);
        put_bits(pkt, 16, float_bits(norm), 32);
      } else {
        /* centroid distribution of PQ: minimum and maximum of the packet's values (64 bits) */
        lo = canon(x[rank[Z]]);
        hi = lo;
        for (uint32_t j = 1; j < P; ++j) {
          float v = canon(x[rank[Z + j]]);
          if (v < lo) lo = v;
          if (v > hi) hi = v;
        }
        put_bits(pkt, 16, float_bits(lo), 32);
        put_bits(pkt, 48, float_bits(hi), 32);
      }
      for (uint32_t j = 0; j < P; ++j) {
        uint32_t pid = rank[Z + j];
        uint32_t rnd = cvlc_philox_coord_oracle(p->seed, p->client_id, p->round, pid);
        uint32_t code = (p->quantizer == ORC_QUANT_QSGD)
                            ? cvlc_qsgd_quantize_oracle(canon(x[pid]), norm, (uint32_t)y, rnd)
                            : cvlc_pq_quantize_oracle(canon(x[pid]), lo, hi, (uint32_t)y, rnd);
        uint64_t bitpos = (uint64_t)p->header_bits + (uint64_t)j * (s + (uint32_t)y);
        put_bits(pkt, bitpos, pid, s);
        put_bits(pkt, bitpos + s, code, (uint32_t)y);
      }
      Z += P;
    }
  }
  free(rank);
  return ORC_OK;
}

/* ======================================================================== */
/* Unframed stream (version 2): the same records without the packet frame.    */
/* Section IV-C fixes one length per packet and a fixed packet size only       */
/* because of the header a real network needs; Proposition 1 itself groups the */
/* top-k by code length.  Here the groups are kept (the records of packet r,   */
/* longest codes first, with the packet's own centroid distribution, so the    */
/* plan and its error bound are unchanged), but a block is as long as its      */
/* records need: no s / y_r fields (a table of n_y and cap(y) in the stream    */
/* header says which block has which length), no padding, and the position IDs */
/* of a block are sorted and sent as differences in a Golomb-Rice code.        */
/* ======================================================================== */

/* Rice parameter of a block of P records out of d coordinates: the gaps between sorted positions are about
 * d / P, so the low m = floor(log2(d / P)) bits go out verbatim and the rest in unary. */
static uint32_t rice_param(uint64_t d, uint32_t P) {
  uint64_t g = d / (uint64_t)P;
  uint32_t m = 0;
  while (g >= 2) { g >>= 1; ++m; }
  return m;
}

static int cmp_u64_asc(const void* a, const void* b) {
  uint64_t x = *(const uint64_t*)a, y = *(const uint64_t*)b;
  return (x > y) - (x < y);
}

size_t cvlc_unframed_header_bytes_oracle(uint32_t R) { return 64 + 33 * 4 * 2 + 8 + (size_t)R * 8; }

/* upper bound of the stream size: per block 64 header bits and per record 1 + m + y bits, plus fewer than 2P unary
 * one-bits per block (the differences of a block add up to less than d, and 2^m > d / (2P)) */
size_t cvlc_unframed_capacity_oracle(const orc_params* p) {
  uint32_t s, R, cap[ORC_MAX_Y + 1];
  if (cvlc_derive_oracle(p, &s, &R, cap) != ORC_OK) return 0;
  uint64_t worst = 0;
  for (uint32_t y = 1; y <= p->max_code_bits; ++y) {
    uint64_t bits = 64 + (uint64_t)cap[y] * (1 + rice_param(p->d, cap[y]) + y) + 2 * (uint64_t)cap[y];
    if (bits > worst) worst = bits;
  }
  return cvlc_unframed_header_bytes_oracle(R) + (size_t)((worst * R + 63) / 64) * 8;
}

int cvlc_encode_unframed_oracle(const float* x, const orc_params* p, const orc_plan* plan, uint8_t* stream,
                                size_t capacity, size_t* bytes_out) {
  if (!params_ok(p) || !plan) return ORC_ERR_INVALID_ARG;
  uint32_t s, R, cap[ORC_MAX_Y + 1];
  int rc = cvlc_derive_oracle(p, &s, &R, cap);
  if (rc != ORC_OK) return rc;
  if (plan->R != R || plan->s != s) return ORC_ERR_INVALID_ARG;
  uint64_t k = 0, nsum = 0;
  for (uint32_t y = 1; y <= ORC_MAX_Y; ++y) {
    if (plan->n_y[y] && cap[y] == 0) return ORC_ERR_INVALID_ARG;
    k += (uint64_t)plan->n_y[y] * cap[y];
    nsum += plan->n_y[y];
  }
  if (nsum != R || k != plan->k || k > p->d) return ORC_ERR_INVALID_ARG;
  if (capacity < cvlc_unframed_capacity_oracle(p)) return ORC_ERR_OUTPUT_TOO_SMALL;
  for (uint64_t i = 0; i < p->d; ++i)
    if (key_of(x[i]) >= 0x7F800000u) return ORC_ERR_NONFINITE_INPUT;

  uint32_t* rank = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)(k ? k : 1));
  if (!rank) return ORC_ERR_INVALID_ARG;
  rc = cvlc_rank_oracle(x, p->d, k, rank);
  if (rc != ORC_OK) { free(rank); return rc; }

  const size_t head = cvlc_unframed_header_bytes_oracle(R);
  memset(stream, 0, capacity);
  put_le(stream + 0, 0x434C5643u, 4);
  put_le(stream + 4, 2, 2); /* version 2: unframed */
  put_le(stream + 6, p->quantizer, 1);
  put_le(stream + 7, s, 1);
  put_le(stream + 8, p->d, 8);
  put_le(stream + 16, R, 4);
  put_le(stream + 20, p->packet_bits, 4);
  put_le(stream + 24, p->header_bits, 4);
  put_le(stream + 28, p->client_id, 4);
  put_le(stream + 32, p->seed, 8);
  put_le(stream + 40, p->round, 4);
  put_le(stream + 44, 0, 4);
  put_le(stream + 48, double_to_bits(p->scale_B), 8);
  put_le(stream + 56, k, 8);
  for (uint32_t y = 0; y <= ORC_MAX_Y; ++y) {
    put_le(stream + 64 + 4 * y, plan->n_y[y], 4);
    put_le(stream + 64 + 132 + 4 * y, cap[y], 4);
  }
  uint8_t* dir = stream + 64 + 264 + 8; /* bit offset of every block inside the body */
  uint8_t* body = stream + head;
  uint64_t bit = 0, Z = 0;
  uint32_t r = 0;
  uint64_t* recs = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(cap[1] ? cap[1] : 1));
  float* seg = (float*)malloc(sizeof(float) * (size_t)(cap[1] ? cap[1] : 1));
  if (!recs || !seg) { free(rank); free(recs); free(seg); return ORC_ERR_INVALID_ARG; }
  for (int y = ORC_MAX_Y; y >= 1; --y) {
    for (uint32_t q = 0; q < plan->n_y[y]; ++q, ++r) {
      uint32_t P = cap[y];
      uint32_t m = rice_param(p->d, P);
      put_le(dir + 8 * (size_t)r, bit, 8);
      /* the block's centroid distribution is that of the packet it replaces: over its records in rank order */
      float lo = 0.0f, hi = 0.0f, norm = 0.0f;
      if (p->quantizer == ORC_QUANT_QSGD) {
        if (y < 2) { free(rank); free(recs); free(seg); return ORC_ERR_INVALID_ARG; }
        for (uint32_t j = 0; j < P; ++j) seg[j] = canon(x[rank[Z + j]]);
        norm = cvlc_qsgd_norm_oracle(seg, P);
        lo = norm;
      } else {
        lo = canon(x[rank[Z]]);
        hi = lo;
        for (uint32_t j = 1; j < P; ++j) {
          float v = canon(x[rank[Z + j]]);
          if (v < lo) lo = v;
          if (v > hi) hi = v;
        }
      }
      put_bits(body, bit, float_bits(lo), 32);
      put_bits(body, bit + 32, float_bits(hi), 32);
      bit += 64;
      /* records in ascending position */
      for (uint32_t j = 0; j < P; ++j) recs[j] = rank[Z + j];
      qsort(recs, P, sizeof(uint64_t), cmp_u64_asc);
      uint64_t prev = 0; /* one past the previous position */
      for (uint32_t j = 0; j < P; ++j) {
        uint32_t pid = (uint32_t)recs[j];
        uint32_t rnd = cvlc_philox_coord_oracle(p->seed, p->client_id, p->round, pid);
        uint32_t code = (p->quantizer == ORC_QUANT_QSGD)
                            ? cvlc_qsgd_quantize_oracle(canon(x[pid]), norm, (uint32_t)y, rnd)
                            : cvlc_pq_quantize_oracle(canon(x[pid]), lo, hi, (uint32_t)y, rnd);
        uint64_t delta = (uint64_t)pid - prev; /* positions skipped since the previous record */
        uint64_t quo = delta >> m;
        for (uint64_t u = 0; u < quo; ++u) put_bits(body, bit + u, 1, 1);
        bit += quo + 1; /* quo ones, then a zero */
        put_bits(body, bit, delta & (((uint64_t)1 << m) - 1), m);
        bit += m;
        put_bits(body, bit, code, (uint32_t)y);
        bit += (uint32_t)y;
        prev = (uint64_t)pid + 1;
      }
      Z += P;
    }
  }
  put_le(stream + 64 + 264, bit, 8);
  *bytes_out = head + (size_t)((bit + 63) / 64) * 8;
  free(rank);
  free(recs);
  free(seg);
  return ORC_OK;
}

/* ======================================================================== */
/* Parameter-server side: w_{t+1} = w_t - (1/|S_t|) sum_i U_i (Section III,   */
/* step 3), with U_i rebuilt from the packets and divided by B_i               */
/* ======================================================================== */

typedef struct {
  uint32_t s, R, packet_bits, header_bits, quantizer;
  uint64_t d;
  double B;
} stream_head;

static int parse_head_any(const uint8_t* st, uint64_t nbytes, uint64_t d, stream_head* h, uint32_t version);

static int parse_head(const uint8_t* st, uint64_t nbytes, uint64_t d, stream_head* h) { return parse_head_any(st, nbytes, d, h, 1); }

static int parse_head_any(const uint8_t* st, uint64_t nbytes, uint64_t d, stream_head* h, uint32_t version) {
  if (nbytes < 64) return ORC_ERR_BAD_STREAM;
  if (get_le(st, 4) != 0x434C5643u) return ORC_ERR_BAD_STREAM;
  if (get_le(st + 4, 2) != version) return ORC_ERR_BAD_STREAM;
  h->quantizer = (uint32_t)get_le(st + 6, 1);
  if (h->quantizer != ORC_QUANT_PQ && h->quantizer != ORC_QUANT_QSGD) return ORC_ERR_BAD_STREAM;
  h->s = (uint32_t)get_le(st + 7, 1);
  h->d = get_le(st + 8, 8);
  h->R = (uint32_t)get_le(st + 16, 4);
  h->packet_bits = (uint32_t)get_le(st + 20, 4);
  h->header_bits = (uint32_t)get_le(st + 24, 4);
  h->B = bits_to_double(get_le(st + 48, 8));
  if (h->d != d) return ORC_ERR_BAD_STREAM;
  uint32_t s = 1;
  while (((uint64_t)1 << s) < d) ++s;
  if (h->s != s) return ORC_ERR_BAD_STREAM;
  if (h->packet_bits == 0 || h->packet_bits % 32) return ORC_ERR_BAD_STREAM;
  if (h->header_bits < 80 || h->header_bits >= h->packet_bits) return ORC_ERR_BAD_STREAM;
  if (version == 1 && 64 + (uint64_t)h->R * (h->packet_bits / 8) != nbytes) return ORC_ERR_BAD_STREAM;
  if (!(h->B >= 1.0) || !(h->B < 1e300)) return ORC_ERR_BAD_STREAM;
  return ORC_OK;
}

/* Decode + aggregate of unframed (version 2) streams: the same arithmetic as for packets */
int cvlc_decode_aggregate_unframed_oracle(const uint8_t* const* streams, const uint64_t* stream_bytes,
                                          const float* weights, uint32_t n_clients, double weight_total,
                                          uint64_t d, float* out, int accumulate) {
  if (d < 2 || d > ((uint64_t)1 << 31) || n_clients == 0) return ORC_ERR_INVALID_ARG;
  double W = weight_total;
  if (W == 0.0) {
    for (uint32_t i = 0; i < n_clients; ++i) W = W + (double)weights[i];
  }
  if (!(W > 0.0)) return ORC_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n_clients; ++i)
    if (!(weights[i] > 0.0f) || !isfinite(weights[i])) return ORC_ERR_INVALID_ARG;
  double* acc = (double*)calloc((size_t)d, sizeof(double));
  if (!acc) return ORC_ERR_INVALID_ARG;
  int rc = ORC_OK;
  for (uint32_t i = 0; i < n_clients && rc == ORC_OK; ++i) {
    stream_head h;
    const uint8_t* st = streams[i];
    rc = parse_head_any(st, stream_bytes[i], d, &h, 2);
    if (rc != ORC_OK) break;
    const size_t head = cvlc_unframed_header_bytes_oracle(h.R);
    if (stream_bytes[i] < head) { rc = ORC_ERR_BAD_STREAM; break; }
    uint32_t n_y[ORC_MAX_Y + 1], cap[ORC_MAX_Y + 1];
    uint64_t blocks = 0;
    for (uint32_t y = 0; y <= ORC_MAX_Y; ++y) {
      n_y[y] = (uint32_t)get_le(st + 64 + 4 * y, 4);
      cap[y] = (uint32_t)get_le(st + 64 + 132 + 4 * y, 4);
      blocks += n_y[y];
      if (n_y[y] && (y == 0 || cap[y] == 0)) rc = ORC_ERR_BAD_STREAM;
    }
    uint64_t total_bits = get_le(st + 64 + 264, 8);
    if (rc != ORC_OK || blocks != h.R || head + ((total_bits + 63) / 64) * 8 != stream_bytes[i]) { rc = ORC_ERR_BAD_STREAM; break; }
    const uint8_t* dir = st + 64 + 264 + 8;
    const uint8_t* body = st + head;
    float coef = (float)((double)weights[i] / (W * h.B));
    uint32_t r = 0;
    for (int y = ORC_MAX_Y; y >= 1 && rc == ORC_OK; --y) {
      for (uint32_t q = 0; q < n_y[y] && rc == ORC_OK; ++q, ++r) {
        uint32_t P = cap[y];
        uint32_t m = rice_param(d, P);
        uint64_t bit = get_le(dir + 8 * (size_t)r, 8);
        if (bit + 64 > total_bits) { rc = ORC_ERR_BAD_STREAM; break; }
        float lo = bits_float((uint32_t)get_bits(body, bit, 32));
        float hi = bits_float((uint32_t)get_bits(body, bit + 32, 32));
        bit += 64;
        if (h.quantizer == ORC_QUANT_QSGD) {
          uint32_t nb = float_bits(lo);
          if (y < 2 || nb >= 0x7F800000u) { rc = ORC_ERR_BAD_STREAM; break; }
        } else if (!isfinite(lo) || !isfinite(hi) || lo > hi) { rc = ORC_ERR_BAD_STREAM; break; }
        uint64_t prev = 0;
        for (uint32_t j = 0; j < P; ++j) {
          uint64_t quo = 0;
          while (bit < total_bits && get_bits(body, bit, 1)) { ++quo; ++bit; }
          if (bit + 1 + m + (uint32_t)y > total_bits) { rc = ORC_ERR_BAD_STREAM; break; }
          bit += 1;
          uint64_t delta = (quo << m) | get_bits(body, bit, m);
          bit += m;
          uint32_t code = (uint32_t)get_bits(body, bit, (uint32_t)y);
          bit += (uint32_t)y;
          uint64_t pid = prev + delta;
          if (pid >= d) { rc = ORC_ERR_BAD_STREAM; break; }
          prev = pid + 1;
          float v = (h.quantizer == ORC_QUANT_QSGD) ? cvlc_qsgd_dequantize_oracle(code, lo, (uint32_t)y)
                                                    : cvlc_pq_dequantize_oracle(code, lo, hi, (uint32_t)y);
          acc[pid] = acc[pid] + (double)coef * (double)v;
        }
        /* blocks follow one another without gaps: a block ends where the directory says the next one starts */
        uint64_t next = (r + 1 < h.R) ? get_le(dir + 8 * ((size_t)r + 1), 8) : total_bits;
        if (rc == ORC_OK && bit != next) rc = ORC_ERR_BAD_STREAM;
      }
    }
  }
  if (rc == ORC_OK) {
    for (uint64_t i = 0; i < d; ++i) {
      if (accumulate)
        out[i] = (float)((double)out[i] + acc[i]);
      else
        out[i] = (float)acc[i];
    }
  }
  free(acc);
  return rc;
}

int cvlc_decode_aggregate_oracle(const uint8_t* const* streams, const uint64_t* stream_bytes,
                                 const float* weights, uint32_t n_clients, double weight_total,
                                 uint64_t d, float* out, int accumulate) {
  if (d < 2 || d > ((uint64_t)1 << 31) || n_clients == 0) return ORC_ERR_INVALID_ARG;
  double W = weight_total;
  if (W == 0.0) {
    for (uint32_t i = 0; i < n_clients; ++i) W = W + (double)weights[i];
  }
  if (!(W > 0.0)) return ORC_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n_clients; ++i)
    if (!(weights[i] > 0.0f) || !isfinite(weights[i])) return ORC_ERR_INVALID_ARG; /* weights are finite and positive */
  double* acc = (double*)calloc((size_t)d, sizeof(double));
  if (!acc) return ORC_ERR_INVALID_ARG;
  int rc = ORC_OK;
  for (uint32_t i = 0; i < n_clients && rc == ORC_OK; ++i) {
    stream_head h;
    rc = parse_head(streams[i], stream_bytes[i], d, &h);
    if (rc != ORC_OK) break;
    float coef = (float)((double)weights[i] / (W * h.B));
    uint32_t y_prev = ORC_MAX_Y;
    for (uint32_t r = 0; r < h.R; ++r) {
      const uint8_t* pkt = streams[i] + 64 + (size_t)r * (h.packet_bits / 8);
      uint32_t s = (uint32_t)get_bits(pkt, 0, 8);
      uint32_t y = (uint32_t)get_bits(pkt, 8, 8);
      if (s != h.s || y < 1 || y > ORC_MAX_Y || y > y_prev) { rc = ORC_ERR_BAD_STREAM; break; }
      y_prev = y;
      float lo = bits_float((uint32_t)get_bits(pkt, 16, 32));
      float hi = bits_float((uint32_t)get_bits(pkt, 48, 32));
      if (h.quantizer == ORC_QUANT_QSGD) {
        /* lo is the norm field: a finite, non-negative fp32; the code needs a sign and a level bit */
        uint32_t nb = (uint32_t)get_bits(pkt, 16, 32);
        if (y < 2 || nb >= 0x7F800000u) { rc = ORC_ERR_BAD_STREAM; break; }
      } else {
        /* PQ: the two centroid fields are the packet's minimum and maximum, finite and in that order */
        if (!isfinite(lo) || !isfinite(hi) || lo > hi) { rc = ORC_ERR_BAD_STREAM; break; }
      }
      uint32_t P = (h.packet_bits - h.header_bits) / (s + y);
      for (uint32_t j = 0; j < P; ++j) {
        uint64_t bitpos = (uint64_t)h.header_bits + (uint64_t)j * (s + y);
        uint64_t pid = get_bits(pkt, bitpos, s);
        uint32_t code = (uint32_t)get_bits(pkt, bitpos + s, y);
        if (pid >= d) { rc = ORC_ERR_BAD_STREAM; break; }
        float v = (h.quantizer == ORC_QUANT_QSGD) ? cvlc_qsgd_dequantize_oracle(code, lo, y)
                                                  : cvlc_pq_dequantize_oracle(code, lo, hi, y);
        acc[pid] = acc[pid] + (double)coef * (double)v;
      }
      if (rc != ORC_OK) break;
    }
  }
  if (rc == ORC_OK) {
    for (uint64_t i = 0; i < d; ++i) {
      if (accumulate)
        out[i] = (float)((double)out[i] + acc[i]);
      else
        out[i] = (float)acc[i];
    }
  }
  free(acc);
  return rc;
}

/* Error compensation (Section II: Top_k "with an error compensation mechanism", Stich et al.): the client keeps
 * what compression lost and adds it to its next update.  compensated = memory + update is what gets compressed
 * this round; the new memory is compensated - U_hat, U_hat being the update the parameter server rebuilds from the
 * stream: the dequantized value divided by B on the transmitted coordinates, zero elsewhere. */
void cvlc_ec_accumulate_oracle(float* memory, const float* update, uint64_t d) {
  for (uint64_t i = 0; i < d; ++i) memory[i] = memory[i] + update[i];
}

int cvlc_ec_residual_oracle(const float* compensated, const uint8_t* stream, uint64_t stream_bytes, uint64_t d,
                            float* memory_out) {
  stream_head h;
  int rc = parse_head(stream, stream_bytes, d, &h);
  if (rc != ORC_OK) return rc;
  for (uint64_t i = 0; i < d; ++i) memory_out[i] = compensated[i];
  for (uint32_t r = 0; r < h.R; ++r) {
    const uint8_t* pkt = stream + 64 + (size_t)r * (h.packet_bits / 8);
    uint32_t y = (uint32_t)get_bits(pkt, 8, 8);
    if (y < 1 || y > ORC_MAX_Y) return ORC_ERR_BAD_STREAM;
    float lo = bits_float((uint32_t)get_bits(pkt, 16, 32));
    float hi = bits_float((uint32_t)get_bits(pkt, 48, 32));
    uint32_t P = (h.packet_bits - h.header_bits) / (h.s + y);
    for (uint32_t j = 0; j < P; ++j) {
      uint64_t bitpos = (uint64_t)h.header_bits + (uint64_t)j * (h.s + y);
      uint64_t pid = get_bits(pkt, bitpos, h.s);
      uint32_t code = (uint32_t)get_bits(pkt, bitpos + h.s, y);
      if (pid >= d) return ORC_ERR_BAD_STREAM;
      float v = (h.quantizer == ORC_QUANT_QSGD) ? cvlc_qsgd_dequantize_oracle(code, lo, y)
                                                : cvlc_pq_dequantize_oracle(code, lo, hi, y);
      float u_hat = (float)((double)v / h.B);
      memory_out[pid] = canon(compensated[pid]) - u_hat;
    }
  }
  return ORC_OK;
}

/* Section III, step 3: w_{t+1} = w_t - (weighted mean of the decoded updates), in fp32 */
int cvlc_decode_apply_oracle(const uint8_t* const* streams, const uint64_t* stream_bytes,
                             const float* weights, uint32_t n_clients, double weight_total,
                             uint64_t d, float* model) {
  float* agg = (float*)malloc(sizeof(float) * (size_t)d);
  if (!agg) return ORC_ERR_INVALID_ARG;
  int rc = cvlc_decode_aggregate_oracle(streams, stream_bytes, weights, n_clients, weight_total, d, agg, 0);
  if (rc == ORC_OK)
    for (uint64_t i = 0; i < d; ++i) model[i] = model[i] - agg[i];
  free(agg);
  return rc;
}
