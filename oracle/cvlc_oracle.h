/*
 * CPU oracle for the Fed-CVLC per-round compression path.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, single-threaded, deliberately
 * slow restatement of the method, written from the paper, that the CUDA
 * library is compared against.  It shares no code with the CUDA library and
 * must never be linked or called from the product path; only the tests, the
 * smoke check and the benchmark's CPU-baseline leg use it.
 *
 * All pointers are HOST pointers.  Every function is deterministic.
 * Floating point: IEEE-754 binary64, round to nearest even, no fused
 * multiply-add (build with -ffp-contract=off), operations in written order.
 *
 * Parity pins (see tests, "-m 'not gpu'"): every exported function is checked
 * against something other than itself; none is "parity unpinned".
 */
#ifndef CVLC_ORACLE_H
#define CVLC_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  ORC_OK = 0,
  ORC_ERR_INVALID_ARG = 1,
  ORC_ERR_BUDGET_TOO_SMALL = 2,
  ORC_ERR_BUDGET_TOO_LARGE = 3,
  ORC_ERR_PACKET_TOO_SMALL = 4,
  ORC_ERR_NONFINITE_INPUT = 5,
  ORC_ERR_OUTPUT_TOO_SMALL = 7,
  ORC_ERR_BAD_STREAM = 8,
  ORC_ERR_SCALE_TOO_SMALL = 12
};

#define ORC_HIST_BINS 4096
#define ORC_MAX_Y 32
#define ORC_QUANT_PQ 0u   /* uniform centroids on [min, max] of the packet (Suresh et al.) */
#define ORC_QUANT_QSGD 1u /* sign and level of |x| / l2-norm of the packet (Alistarh et al.) */

typedef struct {
  uint64_t d;             /* number of coordinates */
  uint64_t budget_bits;   /* uplink budget of this client this round, bits */
  uint32_t packet_bits;   /* b  (Section IV-C: 1500 bytes) */
  uint32_t header_bits;   /* H  (Eq. (2)) */
  uint32_t quantizer;     /* ORC_QUANT_PQ or ORC_QUANT_QSGD */
  uint32_t max_code_bits; /* largest candidate code length, <= 32 */
  double scale_B;         /* B of the scaling operation (Section IV-B) */
  uint64_t seed;          /* Philox key */
  uint32_t client_id;     /* Philox counter word 2 */
  uint32_t round;         /* Philox counter word 3 */
} orc_params;

typedef struct {
  uint32_t s;             /* bits per position ID */
  uint32_t R;             /* packets */
  uint32_t y_min;         /* shortest length with a useful coefficient */
  uint32_t n_lengths;     /* |Y*| */
  uint64_t k;             /* transmitted coordinates */
  double alpha;           /* fitted decay exponent before rounding */
  double alpha_q;         /* rounded to 1/256 and clamped */
  double beta;            /* 2*alpha_q + 1 */
  double gamma;           /* error-bound value of the chosen plan, Eq. (5) */
  double B_next;          /* 1 + max Q over used lengths */
  uint32_t n_y[ORC_MAX_Y + 1]; /* packets per code length */
  uint32_t cap[ORC_MAX_Y + 1]; /* records per packet per code length */
  uint64_t n_evals;       /* objective evaluations spent (diagnostic) */
} orc_plan;

/* --- spec math ---------------------------------------------------------- */
double cvlc_log2_oracle(double v);
double cvlc_exp2_oracle(double v);
double cvlc_powr_oracle(double a, double beta);

/* --- Philox4x32-10 (Salmon et al., SC'11) ------------------------------- */
void cvlc_philox4x32_10_oracle(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
uint32_t cvlc_philox_coord_oracle(uint64_t seed, uint32_t client_id, uint32_t round, uint64_t coord);

/* --- planning ------------------------------------------------------------ */
int cvlc_histogram_oracle(const float* x, uint64_t d, uint64_t h[ORC_HIST_BINS]);
void cvlc_alpha_fit_oracle(const uint64_t h[ORC_HIST_BINS], uint64_t d, double* alpha, double* alpha_q);
int cvlc_derive_oracle(const orc_params* p, uint32_t* s, uint32_t* R, uint32_t cap[ORC_MAX_Y + 1]);
double cvlc_default_scale_oracle(const orc_params* p);
size_t cvlc_stream_bytes_oracle(const orc_params* p);
/* coefficient g(y) = 1 - (Q(y)/B^2 + (1-1/B)^2) of Eq. (5); Q of the chosen quantizer (Appendix, case study) */
double cvlc_coeff_g_oracle(const orc_params* p, uint32_t y);
double cvlc_quant_error_Q_oracle(const orc_params* p, uint32_t y);
/* F(n) = 1 - gamma for packet counts n_y (index = code length) at exponent beta; -inf if inadmissible */
double cvlc_objective_oracle(const orc_params* p, double beta, const uint32_t n_y[ORC_MAX_Y + 1]);
/* Y*: candidate lengths, ascending; returns their number */
int cvlc_candidates_oracle(const orc_params* p, uint32_t Y[ORC_MAX_Y + 1]);
int cvlc_plan_from_alpha_oracle(const orc_params* p, double alpha, orc_plan* plan);
int cvlc_plan_oracle(const float* x, const orc_params* p, orc_plan* plan);
/* planning at the parameter server from a client's histogram (Section IV-C, last paragraph) */
int cvlc_plan_from_histogram_oracle(const uint64_t h[ORC_HIST_BINS], const orc_params* p, orc_plan* plan);
int cvlc_plan_fixed_oracle(const orc_params* p, uint32_t y, orc_plan* plan);

/* Problem P2 with real-valued packet sizes, as Section IV-C solves it: k runs over n_k equidistant values of
 * its range; for each, P_1 .. P_R start equal and consecutive packets are re-split (atomic operation on Eq. (7),
 * a fixed 8 x 32-point bracketing search) in sweeps r = 2 .. R until a sweep moves no packet by more than
 * 2^-30 of the largest packet, or max_sweeps; gamma of Eq. (5) with y_r = (b - H) / P_r - s picks k*.  A plan
 * only (real-valued code lengths cannot be packed).  Outputs: k_grid, gamma_of_k, sweeps_of_k (n_k entries each,
 * may be NULL), k_star, gamma_star, P_star (R doubles, may be NULL). */
int cvlc_plan_literal_oracle(const orc_params* p, double alpha_q, uint32_t n_k, uint32_t max_sweeps, uint64_t* k_grid,
                             double* gamma_of_k, uint32_t* sweeps_of_k, uint64_t* k_star, double* gamma_star,
                             double* P_star);

/* --- encoding ------------------------------------------------------------ */
/* first k ranks of the order (|x| descending, index ascending) */
int cvlc_rank_oracle(const float* x, uint64_t d, uint64_t k, uint32_t* idx_out);
uint32_t cvlc_pq_quantize_oracle(float x, float lo, float hi, uint32_t y, uint32_t rnd);
float cvlc_pq_dequantize_oracle(uint32_t code, float lo, float hi, uint32_t y);
/* QSGD: y >= 2; code = sign << (y-1) | level, level in 0..2^(y-1)-1 */
float cvlc_qsgd_norm_oracle(const float* v, uint32_t n);
uint32_t cvlc_qsgd_quantize_oracle(float x, float norm, uint32_t y, uint32_t rnd);
float cvlc_qsgd_dequantize_oracle(uint32_t code, float norm, uint32_t y);
int cvlc_encode_oracle(const float* x, const orc_params* p, const orc_plan* plan, uint8_t* stream,
                       size_t capacity, uint32_t* ranked_idx_out /* k entries or NULL */);

/* --- unframed stream (version 2): the packets' records without the frame; blocks in the packets' order, each with
 * its centroid distribution (64 bits) and its records sorted by position, positions as Golomb-Rice coded
 * differences, lengths and capacities in a table of the stream header, a directory of block offsets ------------- */
size_t cvlc_unframed_header_bytes_oracle(uint32_t R);
size_t cvlc_unframed_capacity_oracle(const orc_params* p);
int cvlc_encode_unframed_oracle(const float* x, const orc_params* p, const orc_plan* plan, uint8_t* stream,
                                size_t capacity, size_t* bytes_out);
int cvlc_decode_aggregate_unframed_oracle(const uint8_t* const* streams, const uint64_t* stream_bytes,
                                          const float* weights, uint32_t n_clients, double weight_total,
                                          uint64_t d, float* out, int accumulate);

/* --- decoding ------------------------------------------------------------ */
int cvlc_decode_aggregate_oracle(const uint8_t* const* streams, const uint64_t* stream_bytes,
                                 const float* weights, uint32_t n_clients, double weight_total,
                                 uint64_t d, float* out, int accumulate);
/* error compensation: memory <- memory + update before compression; memory_out = compensated - (what the server
 * rebuilds from the stream) after it */
void cvlc_ec_accumulate_oracle(float* memory, const float* update, uint64_t d);
int cvlc_ec_residual_oracle(const float* compensated, const uint8_t* stream, uint64_t stream_bytes, uint64_t d,
                            float* memory_out);
/* model <- model - aggregate (Section III, step 3) */
int cvlc_decode_apply_oracle(const uint8_t* const* streams, const uint64_t* stream_bytes,
                             const float* weights, uint32_t n_clients, double weight_total,
                             uint64_t d, float* model);

#ifdef __cplusplus
}
#endif
#endif
