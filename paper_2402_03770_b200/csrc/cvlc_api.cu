// C ABI of libcvlc: argument validation, derived constants, workspace carving and
// stream-ordered kernel launches.  No device allocation, no CPU fallback.  Process-wide state is
// limited to what include/cvlc.h lists (per-device set-up flags, two events per device for
// cvlc_compress_batch, launch counters, the profiling events, the scratch of the allocation-free
// decode); host calls are not thread-safe.
#include <math.h>
#include <string.h>

#include "cvlc_common.cuh"

using namespace cvlc;

namespace {

struct Derived {
  uint32_t s, R;
  uint32_t cap[CVLC_MAX_CODE_BITS + 1];
};

bool params_ok(const cvlc_params* p) {
  if (!p) return false;
  if (p->d < 2 || p->d > (1ull << 31)) return false;
  if (p->packet_bits == 0 || (p->packet_bits % 32) != 0) return false;
  if (p->header_bits < 80 || p->header_bits >= p->packet_bits) return false;
  if (p->quantizer != CVLC_QUANT_PQ && p->quantizer != CVLC_QUANT_QSGD) return false;
  if (p->max_code_bits < 1 || p->max_code_bits > CVLC_MAX_CODE_BITS) return false;
  if (!(p->scale_B >= 1.0) || !(p->scale_B < 1e300)) return false;
  return true;
}

uint32_t position_bits(uint64_t d) {  // s = ceil(log2 d)  (Section IV-C)
  uint32_t s = 1;
  while ((1ull << s) < d) ++s;
  return s;
}

// Packet constraint Eq. (3) packed maximally: cap(y) = floor((b - H) / (s + y)); R = floor(budget / b).
int derive(const cvlc_params* p, Derived* D) {
  if (!params_ok(p)) return CVLC_ERR_INVALID_ARG;
  D->s = position_bits(p->d);
  const uint64_t R = p->budget_bits / p->packet_bits;
  if (R == 0) return CVLC_ERR_BUDGET_TOO_SMALL;
  if (R > 0xFFFFFFFFull) return CVLC_ERR_BUDGET_TOO_LARGE;
  D->R = (uint32_t)R;
  for (uint32_t y = 0; y <= CVLC_MAX_CODE_BITS; ++y) D->cap[y] = 0;
  for (uint32_t y = 1; y <= p->max_code_bits; ++y) D->cap[y] = (p->packet_bits - p->header_bits) / (D->s + y);
  if (D->cap[p->max_code_bits] < 1) return CVLC_ERR_PACKET_TOO_SMALL;
  return CVLC_OK;
}

// Error factor Q of P = cap(y) values at y bits (Appendix, case study) and the coefficient of Eq. (5):
// g = 1 - (Q / B^2 + (1 - 1/B)^2).  PQ: Q = P / (2^y - 1)^2.  QSGD: Q = min(P / s_q^2, sqrt(P) / s_q) with
// the s_q = 2^(y-1) - 1 levels its y-bit code holds beside the sign; one bit holds none.  Plain IEEE
// operations in this order; the host compiler is told not to contract them (-ffp-contract=off).
double quant_Q(uint32_t quantizer, uint32_t cap_y, uint32_t y) {
  if (quantizer == CVLC_QUANT_QSGD) {
    if (y < 2) return INFINITY;
    const double sq = (double)((1ull << (y - 1)) - 1ull);
    const double Q1 = (double)cap_y / (sq * sq);
    const double Q2 = sqrt((double)cap_y) / sq;
    return (Q1 < Q2) ? Q1 : Q2;
  }
  const double L = (double)((1ull << y) - 1ull);
  return (double)cap_y / (L * L);
}
double coeff_g(double Q, double B) {
  const double c = Q / (B * B) + (1.0 - 1.0 / B) * (1.0 - 1.0 / B);
  return 1.0 - c;
}

// Checks one client's parameters and fills the shape shared by a batch.  The per-length
// coefficients are rebuilt on the device from scale_B with the same IEEE operations; the host
// evaluates them here only to reject parameters for which no length is usable.
int build_shape(const cvlc_params* p, uint32_t fixed_y, Shape* S) {
  Derived D;
  const int rc = derive(p, &D);
  if (rc != CVLC_OK) return rc;
  memset(S, 0, sizeof *S);
  S->d = p->d;
  S->s = D.s;
  S->R = D.R;
  S->packet_bits = p->packet_bits;
  S->header_bits = p->header_bits;
  S->quantizer = p->quantizer;
  S->max_code_bits = p->max_code_bits;
  S->fixed_y = fixed_y;
  for (uint32_t y = 0; y <= CVLC_MAX_CODE_BITS; ++y) S->cap[y] = D.cap[y];
  if (fixed_y) {
    if (fixed_y > p->max_code_bits) return CVLC_ERR_INVALID_ARG;
    if (p->quantizer == CVLC_QUANT_QSGD && fixed_y < 2) return CVLC_ERR_INVALID_ARG;
    if ((uint64_t)D.R * D.cap[fixed_y] > p->d) return CVLC_ERR_BUDGET_TOO_LARGE;
    return CVLC_OK;
  }
  bool usable = false;
  for (uint32_t y = 1; y <= p->max_code_bits; ++y)
    if (coeff_g(quant_Q(p->quantizer, D.cap[y], y), p->scale_B) > 0.0) usable = true;
  if (!usable) return CVLC_ERR_SCALE_TOO_SMALL;
  // an admissible single-length plan must exist: the longest code sends the fewest coordinates
  if ((uint64_t)D.R * D.cap[p->max_code_bits] > p->d) return CVLC_ERR_BUDGET_TOO_LARGE;
  return CVLC_OK;
}

bool same_shape(const cvlc_params& a, const cvlc_params& b) {
  return a.d == b.d && a.budget_bits / a.packet_bits == b.budget_bits / b.packet_bits && a.packet_bits == b.packet_bits &&
         a.header_bits == b.header_bits && a.quantizer == b.quantizer && a.max_code_bits == b.max_code_bits;
}

bool aligned(const void* p, size_t a) { return p && (reinterpret_cast<uintptr_t>(p) % a) == 0; }

size_t plan_ws_bytes_of(uint64_t d, uint32_t n) { return plan_ws_bytes(make_partition(d, n), n); }

// the packing kernel assembles one packet per warp, four warps per block, in shared memory (QSGD: each next to the
// squares of the packet's values): four of them must fit
bool pack_fits(const Shape& S) {
  return 4 * ((size_t)S.packet_bits / 8 + 16 + (S.quantizer == CVLC_QUANT_QSGD ? (size_t)S.cap[1] * 8 : 0)) <= 200 * 1024;
}

}  // namespace

extern "C" {

int cvlc_version(void) { return 100; }

const char* cvlc_status_string(int status) {
  switch (status) {
    case CVLC_OK: return "ok";
    case CVLC_ERR_INVALID_ARG: return "invalid argument";
    case CVLC_ERR_BUDGET_TOO_SMALL: return "budget below one packet";
    case CVLC_ERR_BUDGET_TOO_LARGE: return "budget sends more than d coordinates";
    case CVLC_ERR_PACKET_TOO_SMALL: return "packet cannot hold one record";
    case CVLC_ERR_NONFINITE_INPUT: return "non-finite value in the update";
    case CVLC_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case CVLC_ERR_OUTPUT_TOO_SMALL: return "output buffer too small";
    case CVLC_ERR_BAD_STREAM: return "malformed stream";
    case CVLC_ERR_DEVICE_TIMEOUT: return "device-side wait ran out";
    case CVLC_ERR_CUDA: return "CUDA error";
    case CVLC_ERR_NOT_IMPLEMENTED: return "not implemented";
    case CVLC_ERR_SCALE_TOO_SMALL: return "scale_B too small for every code length";
    case CVLC_ERR_PLAN_MISMATCH: return "plan does not match parameters or update";
    default: return "unknown status";
  }
}

int cvlc_set_device(int device) { return cudaSetDevice(device) == cudaSuccess ? CVLC_OK : CVLC_ERR_CUDA; }

size_t cvlc_stream_bytes(const cvlc_params* p) {
  if (!params_ok(p)) return 0;
  const uint64_t R = p->budget_bits / p->packet_bits;
  return (size_t)(CVLC_STREAM_HEADER_BYTES + R * (p->packet_bits / 8));
}

double cvlc_default_scale(const cvlc_params* p) {
  if (!p) return NAN;
  cvlc_params q = *p;
  q.scale_B = 1.0;
  q.max_code_bits = CVLC_MAX_CODE_BITS;
  if (!params_ok(&q)) return NAN;
  const uint32_t s = position_bits(q.d);
  const uint32_t cap8 = (q.packet_bits - q.header_bits) / (s + 8);
  return 1.0 + quant_Q(p->quantizer, cap8, 8);
}

size_t cvlc_plan_workspace_bytes(const cvlc_params* p) { return cvlc_plan_batch_workspace_bytes(p, 1); }

size_t cvlc_plan_batch_workspace_bytes(const cvlc_params* p, uint32_t n) {
  if (!params_ok(p) || n == 0 || n > CVLC_MAX_BATCH) return 0;
  return plan_ws_bytes_of(p->d, n);
}

size_t cvlc_encode_workspace_bytes(const cvlc_params* p) { return cvlc_encode_batch_workspace_bytes(p, 1, 0); }

size_t cvlc_encode_batch_workspace_bytes(const cvlc_params* p, uint32_t n, uint64_t max_candidates) {
  if (!params_ok(p) || n == 0 || n > CVLC_MAX_BATCH) return 0;
  const uint64_t cap = (max_candidates == 0 || max_candidates > p->d) ? p->d : max_candidates;
  return enc_layout(p->d, n, cap).total;
}

size_t cvlc_decode_workspace_bytes(uint32_t n_clients) {
  if (n_clients == 0 || n_clients > CVLC_MAX_CLIENTS_PER_CALL) return 0;
  return dec_ws_bytes(n_clients);
}

int cvlc_plan_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, uint32_t fixed_y,
                    cvlc_plan_t* plans_dev, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  if (!x_dev || !params || n == 0 || n > CVLC_MAX_BATCH || fixed_y > CVLC_MAX_CODE_BITS) return CVLC_ERR_INVALID_ARG;
  Shape S;
  ClientDesc desc[CVLC_MAX_BATCH];
  for (uint32_t i = 0; i < n; ++i) {
    Shape Si;
    const int rc = build_shape(&params[i], fixed_y, i == 0 ? &S : &Si);
    if (rc != CVLC_OK) return rc;
    if (i && !same_shape(params[0], params[i])) return CVLC_ERR_INVALID_ARG;
    if (!aligned(x_dev[i], 16)) return CVLC_ERR_INVALID_ARG;
    desc[i].x = x_dev[i];
    desc[i].plan = plans_dev + i;
    desc[i].stream = nullptr;
    desc[i].seed = params[i].seed;
    desc[i].scale_B = params[i].scale_B;
    desc[i].client_id = params[i].client_id;
    desc[i].round = params[i].round;
  }
  if (!aligned(plans_dev, 8) || !aligned(ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (ws_bytes < plan_ws_bytes_of(S.d, n)) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  return launch_plan(desc, n, S, ws_dev, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CVLC_OK : CVLC_ERR_CUDA;
}

int cvlc_histogram_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, uint64_t* hist_dev,
                         void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  if (!x_dev || !params || n == 0 || n > CVLC_MAX_BATCH) return CVLC_ERR_INVALID_ARG;
  Shape S;
  ClientDesc desc[CVLC_MAX_BATCH];
  for (uint32_t i = 0; i < n; ++i) {
    Derived D;
    const int rc = derive(&params[i], &D);
    if (rc != CVLC_OK) return rc;
    if (params[i].d != params[0].d) return CVLC_ERR_INVALID_ARG;
    if (!aligned(x_dev[i], 16)) return CVLC_ERR_INVALID_ARG;
    memset(&desc[i], 0, sizeof desc[i]);
    desc[i].x = x_dev[i];
  }
  memset(&S, 0, sizeof S);
  S.d = params[0].d;
  if (!aligned(hist_dev, 8) || !aligned(ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (ws_bytes < plan_ws_bytes_of(S.d, n)) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  return launch_histogram(desc, n, S, ws_dev, reinterpret_cast<unsigned long long*>(hist_dev),
                          static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CVLC_OK : CVLC_ERR_CUDA;
}

int cvlc_plan_from_histogram_batch(const uint64_t* hist_dev, const cvlc_params* params, uint32_t n,
                                   cvlc_plan_t* plans_dev, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  if (!hist_dev || !params || n == 0 || n > CVLC_MAX_BATCH) return CVLC_ERR_INVALID_ARG;
  Shape S;
  ClientDesc desc[CVLC_MAX_BATCH];
  for (uint32_t i = 0; i < n; ++i) {
    Shape Si;
    const int rc = build_shape(&params[i], 0, i == 0 ? &S : &Si);
    if (rc != CVLC_OK) return rc;
    if (i && !same_shape(params[0], params[i])) return CVLC_ERR_INVALID_ARG;
    memset(&desc[i], 0, sizeof desc[i]);
    desc[i].plan = plans_dev + i;
    desc[i].seed = params[i].seed;
    desc[i].scale_B = params[i].scale_B;
    desc[i].client_id = params[i].client_id;
    desc[i].round = params[i].round;
  }
  if (!aligned(hist_dev, 8) || !aligned(plans_dev, 8) || !aligned(ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (ws_bytes < plan_ws_bytes_of(S.d, n)) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  return launch_plan_from_hist(desc, n, S, reinterpret_cast<const unsigned long long*>(hist_dev), ws_dev,
                               static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CVLC_OK : CVLC_ERR_CUDA;
}

size_t cvlc_plan_literal_workspace_bytes(const cvlc_params* p, uint32_t n_k) {
  Derived D;
  if (derive(p, &D) != CVLC_OK || n_k == 0 || n_k > kLiteralMaxK || D.R > kLiteralMaxR) return 0;
  return literal_ws_bytes(n_k, D.R);
}

int cvlc_plan_literal(const cvlc_params* p, double alpha_q, uint32_t n_k, uint32_t max_sweeps, cvlc_literal_plan_t* out_dev,
                      double* P_star_dev, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  Derived D;
  const int rc = derive(p, &D);
  if (rc != CVLC_OK) return rc;
  if (n_k == 0 || n_k > kLiteralMaxK || max_sweeps == 0 || !(alpha_q < 0.0) || alpha_q == -0.5 || D.R > kLiteralMaxR)
    return CVLC_ERR_INVALID_ARG;
  const uint32_t y_lo = (p->quantizer == CVLC_QUANT_QSGD) ? 2u : 1u;  // a one-bit QSGD code holds no level
  if (p->max_code_bits < y_lo) return CVLC_ERR_INVALID_ARG;
  if (!aligned(out_dev, 8) || !aligned(ws_dev, 256) || (P_star_dev && !aligned(P_star_dev, 8))) return CVLC_ERR_INVALID_ARG;
  if (ws_bytes < literal_ws_bytes(n_k, D.R)) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  // the range of k: no code longer than max_code_bits or shorter than y_lo, at least one record per packet, at
  // most d coordinates (plain IEEE operations, compiled without contraction)
  const double s = (double)D.s, bH = (double)(p->packet_bits - p->header_bits);
  const double P_min = bH / (s + (double)p->max_code_bits), P_max = bH / (s + (double)y_lo);
  double klo = ceil((double)D.R * P_min), khi = floor((double)D.R * P_max);
  if (klo < (double)D.R) klo = (double)D.R;
  if (khi > (double)p->d) khi = (double)p->d;
  if (!(klo <= khi)) return CVLC_ERR_BUDGET_TOO_LARGE;
  const double tol = P_max * (1.0 / 1073741824.0);
  return launch_plan_literal(*p, alpha_q, D.s, D.R, n_k, max_sweeps, (unsigned long long)klo, (unsigned long long)khi, P_min,
                             P_max, tol, out_dev, P_star_dev, ws_dev, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

int cvlc_plan(const float* x_dev, const cvlc_params* p, cvlc_plan_t* plan_dev, void* ws_dev, size_t ws_bytes,
              void* cuda_stream) {
  return cvlc_plan_batch(&x_dev, p, 1, 0, plan_dev, ws_dev, ws_bytes, cuda_stream);
}

int cvlc_plan_fixed(const float* x_dev, const cvlc_params* p, uint32_t y, cvlc_plan_t* plan_dev, void* ws_dev,
                    size_t ws_bytes, void* cuda_stream) {
  if (y < 1 || y > CVLC_MAX_CODE_BITS) return CVLC_ERR_INVALID_ARG;
  return cvlc_plan_batch(&x_dev, p, 1, y, plan_dev, ws_dev, ws_bytes, cuda_stream);
}

static int encode_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, const cvlc_plan_t* plans_dev,
                        const void* plan_ws_dev, uint8_t* const* streams_dev, size_t stream_capacity,
                        uint64_t max_candidates, void* ws_dev, size_t ws_bytes, void* cuda_stream, int write_residual) {
  if (!x_dev || !params || !streams_dev || n == 0 || n > CVLC_MAX_BATCH) return CVLC_ERR_INVALID_ARG;
  Shape S;
  ClientDesc desc[CVLC_MAX_BATCH];
  for (uint32_t i = 0; i < n; ++i) {
    Derived D;
    const int rc = derive(&params[i], &D);
    if (rc != CVLC_OK) return rc;
    if (i && !same_shape(params[0], params[i])) return CVLC_ERR_INVALID_ARG;
    if (!aligned(x_dev[i], 16) || !aligned(streams_dev[i], 16)) return CVLC_ERR_INVALID_ARG;
    if (i == 0) {
      memset(&S, 0, sizeof S);
      S.d = params[0].d;
      S.s = D.s;
      S.R = D.R;
      S.packet_bits = params[0].packet_bits;
      S.header_bits = params[0].header_bits;
      S.quantizer = params[0].quantizer;
      S.max_code_bits = params[0].max_code_bits;
      for (uint32_t y = 0; y <= CVLC_MAX_CODE_BITS; ++y) S.cap[y] = D.cap[y];
    }
    desc[i].x = x_dev[i];
    desc[i].plan = const_cast<cvlc_plan_t*>(plans_dev) + i;
    desc[i].stream = streams_dev[i];
    desc[i].seed = params[i].seed;
    desc[i].scale_B = params[i].scale_B;
    desc[i].client_id = params[i].client_id;
    desc[i].round = params[i].round;
  }
  if (!aligned(plans_dev, 8) || !aligned(ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (plan_ws_dev && !aligned(plan_ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (stream_capacity < cvlc_stream_bytes(&params[0])) return CVLC_ERR_OUTPUT_TOO_SMALL;
  const uint64_t cap = (max_candidates == 0 || max_candidates > S.d) ? S.d : max_candidates;
  if (ws_bytes < enc_layout(S.d, n, cap).total) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  if (!pack_fits(S)) return CVLC_ERR_INVALID_ARG;
  if (S.R > 0x7FFFFFFFu || n > 65535) return CVLC_ERR_INVALID_ARG;
  return launch_encode(desc, n, S, cap, plan_ws_dev, ws_dev, static_cast<cudaStream_t>(cuda_stream), nullptr, write_residual) ==
                 cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

int cvlc_encode_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, const cvlc_plan_t* plans_dev,
                      const void* plan_ws_dev, uint8_t* const* streams_dev, size_t stream_capacity,
                      uint64_t max_candidates, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  return encode_batch(x_dev, params, n, plans_dev, plan_ws_dev, streams_dev, stream_capacity, max_candidates, ws_dev,
                      ws_bytes, cuda_stream, 0);
}

int cvlc_encode_batch_ec(float* const* memory_dev, const cvlc_params* params, uint32_t n, const cvlc_plan_t* plans_dev,
                         const void* plan_ws_dev, uint8_t* const* streams_dev, size_t stream_capacity,
                         uint64_t max_candidates, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  return encode_batch(const_cast<const float* const*>(memory_dev), params, n, plans_dev, plan_ws_dev, streams_dev,
                      stream_capacity, max_candidates, ws_dev, ws_bytes, cuda_stream, 1);
}

// ---- unframed stream (version 2) ------------------------------------------------------

static bool unframed_fits(const Derived& D, const cvlc_params* p, size_t* capacity_out) {
  const uint32_t y_lo = (p->quantizer == CVLC_QUANT_QSGD) ? 2u : 1u;
  if (p->max_code_bits < y_lo || D.cap[y_lo] > kUfMaxRecords) return false;
  uint64_t worst = 0;
  for (uint32_t y = 1; y <= p->max_code_bits; ++y) {
    const uint64_t bits = 64 + (uint64_t)D.cap[y] * (1 + uf_rice_param(p->d, D.cap[y]) + y) + 2 * (uint64_t)D.cap[y];
    if (bits > worst) worst = bits;
  }
  if (capacity_out) *capacity_out = (uf_head_bytes(D.R) + (size_t)((worst * D.R + 63) / 64) * 8 + 15) & ~(size_t)15;
  return true;
}

size_t cvlc_unframed_stream_capacity(const cvlc_params* p) {
  Derived D;
  size_t cap = 0;
  if (derive(p, &D) != CVLC_OK || !unframed_fits(D, p, &cap)) return 0;
  return cap;
}

size_t cvlc_unframed_workspace_bytes(const cvlc_params* p, uint32_t n) {
  Derived D;
  if (derive(p, &D) != CVLC_OK || n == 0 || n > CVLC_MAX_BATCH) return 0;
  return uf_ws_bytes(n, D.R);
}

int cvlc_encode_unframed_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, const cvlc_plan_t* plans_dev,
                               const void* plan_ws_dev, uint8_t* const* streams_dev, size_t stream_capacity,
                               uint64_t* stream_bytes_dev, uint64_t max_candidates, void* enc_ws_dev, size_t enc_ws_bytes,
                               void* uf_ws_dev, size_t uf_ws_bytes_given, void* cuda_stream) {
  if (!x_dev || !params || !streams_dev || n == 0 || n > CVLC_MAX_BATCH) return CVLC_ERR_INVALID_ARG;
  Shape S;
  ClientDesc desc[CVLC_MAX_BATCH];
  size_t need_capacity = 0;
  for (uint32_t i = 0; i < n; ++i) {
    Derived D;
    const int rc = derive(&params[i], &D);
    if (rc != CVLC_OK) return rc;
    if (i && !same_shape(params[0], params[i])) return CVLC_ERR_INVALID_ARG;
    if (!aligned(x_dev[i], 16) || !aligned(streams_dev[i], 16)) return CVLC_ERR_INVALID_ARG;
    if (i == 0) {
      if (!unframed_fits(D, &params[0], &need_capacity)) return CVLC_ERR_INVALID_ARG;  // blocks of more than 2048 records
      memset(&S, 0, sizeof S);
      S.d = params[0].d;
      S.s = D.s;
      S.R = D.R;
      S.packet_bits = params[0].packet_bits;
      S.header_bits = params[0].header_bits;
      S.quantizer = params[0].quantizer;
      S.max_code_bits = params[0].max_code_bits;
      for (uint32_t y = 0; y <= CVLC_MAX_CODE_BITS; ++y) S.cap[y] = D.cap[y];
    }
    desc[i].x = x_dev[i];
    desc[i].plan = const_cast<cvlc_plan_t*>(plans_dev) + i;
    desc[i].stream = streams_dev[i];
    desc[i].seed = params[i].seed;
    desc[i].scale_B = params[i].scale_B;
    desc[i].client_id = params[i].client_id;
    desc[i].round = params[i].round;
  }
  if (!aligned(plans_dev, 8) || !aligned(enc_ws_dev, 256) || !aligned(uf_ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (plan_ws_dev && !aligned(plan_ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (stream_bytes_dev && !aligned(stream_bytes_dev, 8)) return CVLC_ERR_INVALID_ARG;
  if (stream_capacity < need_capacity) return CVLC_ERR_OUTPUT_TOO_SMALL;
  const uint64_t cap = (max_candidates == 0 || max_candidates > S.d) ? S.d : max_candidates;
  if (enc_ws_bytes < enc_layout(S.d, n, cap).total || uf_ws_bytes_given < uf_ws_bytes(n, S.R)) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  if (S.R > 0x7FFFFFFFu || n > 65535) return CVLC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (launch_encode(desc, n, S, cap, plan_ws_dev, enc_ws_dev, st, nullptr, kPackNone) != cudaSuccess) return CVLC_ERR_CUDA;
  return launch_pack_unframed(desc, n, S, cap, stream_capacity, enc_ws_dev, uf_ws_dev,
                              reinterpret_cast<unsigned long long*>(stream_bytes_dev), st) == cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

int cvlc_decode_aggregate_unframed(const uint8_t* const* streams_dev, const uint64_t* stream_bytes_dev, const float* weights_dev,
                                   uint32_t n_clients, double weight_total, uint64_t d, float* out_dev, int accumulate,
                                   void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  if (n_clients == 0 || n_clients > CVLC_MAX_CLIENTS_PER_CALL) return CVLC_ERR_INVALID_ARG;
  if (d < 2 || d > (1ull << 31)) return CVLC_ERR_INVALID_ARG;
  if (!(weight_total >= 0.0) || !(weight_total < 1e300)) return CVLC_ERR_INVALID_ARG;
  if (!aligned(streams_dev, 8) || !aligned(stream_bytes_dev, 8) || !aligned(weights_dev, 4) || !aligned(out_dev, 16) ||
      !aligned(ws_dev, 256))
    return CVLC_ERR_INVALID_ARG;
  if (ws_bytes < dec_ws_bytes(n_clients)) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  return launch_decode_unframed(streams_dev, stream_bytes_dev, weights_dev, n_clients, weight_total, d, position_bits(d), out_dev,
                                accumulate ? 1 : 0, ws_dev, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

int cvlc_ec_accumulate_batch(float* const* memory_dev, const float* const* update_dev, uint32_t n, uint64_t d,
                             void* cuda_stream) {
  if (!memory_dev || !update_dev || n == 0 || n > CVLC_MAX_BATCH || d < 2 || d > (1ull << 31)) return CVLC_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n; ++i)
    if (!aligned(memory_dev[i], 16) || !aligned(update_dev[i], 16) || memory_dev[i] == update_dev[i]) return CVLC_ERR_INVALID_ARG;
  return launch_ec_accumulate(memory_dev, update_dev, n, d, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CVLC_OK
                                                                                                                  : CVLC_ERR_CUDA;
}

// Two events per device order the two streams of cvlc_compress_batch (created on first use, kept until exit).
static cudaError_t compress_events(cudaEvent_t* fork, cudaEvent_t* join) {
  static cudaEvent_t ev[64][2];
  static bool made[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!made[dev]) {
    for (int i = 0; i < 2; ++i) {
      e = cudaEventCreateWithFlags(&ev[dev][i], cudaEventDisableTiming);
      if (e != cudaSuccess) return e;
    }
    made[dev] = true;
  }
  *fork = ev[dev][0];
  *join = ev[dev][1];
  return cudaSuccess;
}

int cvlc_compress_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, uint32_t fixed_y,
                        cvlc_plan_t* plans_dev, uint8_t* const* streams_dev, size_t stream_capacity,
                        uint64_t max_candidates, void* plan_ws_dev, size_t plan_ws_bytes, void* enc_ws_dev,
                        size_t enc_ws_bytes, void* cuda_stream, void* side_stream) {
  if (!x_dev || !params || !streams_dev || n == 0 || n > CVLC_MAX_BATCH || fixed_y > CVLC_MAX_CODE_BITS) return CVLC_ERR_INVALID_ARG;
  Shape S;
  ClientDesc desc[CVLC_MAX_BATCH];
  for (uint32_t i = 0; i < n; ++i) {
    Shape Si;
    const int rc = build_shape(&params[i], fixed_y, i == 0 ? &S : &Si);
    if (rc != CVLC_OK) return rc;
    if (i && !same_shape(params[0], params[i])) return CVLC_ERR_INVALID_ARG;
    if (!aligned(x_dev[i], 16) || !aligned(streams_dev[i], 16)) return CVLC_ERR_INVALID_ARG;
    desc[i].x = x_dev[i];
    desc[i].plan = plans_dev + i;
    desc[i].stream = streams_dev[i];
    desc[i].seed = params[i].seed;
    desc[i].scale_B = params[i].scale_B;
    desc[i].client_id = params[i].client_id;
    desc[i].round = params[i].round;
  }
  if (!aligned(plans_dev, 8) || !aligned(plan_ws_dev, 256) || !aligned(enc_ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (plan_ws_bytes < plan_ws_bytes_of(S.d, n)) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  if (stream_capacity < cvlc_stream_bytes(&params[0])) return CVLC_ERR_OUTPUT_TOO_SMALL;
  const uint64_t cap = (max_candidates == 0 || max_candidates > S.d) ? S.d : max_candidates;
  if (enc_ws_bytes < enc_layout(S.d, n, cap).total) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  if (!pack_fits(S)) return CVLC_ERR_INVALID_ARG;
  if (S.R > 0x7FFFFFFFu || n > 65535) return CVLC_ERR_INVALID_ARG;
  cudaStream_t main_st = static_cast<cudaStream_t>(cuda_stream), side_st = static_cast<cudaStream_t>(side_stream);
  const bool two = side_stream != nullptr && side_st != main_st;
  Shape Senc = S;
  Senc.fixed_y = 0;
  if (launch_plan_front(desc, n, S, plan_ws_dev, main_st) != cudaSuccess) return CVLC_ERR_CUDA;
  if (!two) {
    if (launch_plan_back(desc, n, S, plan_ws_dev, main_st) != cudaSuccess) return CVLC_ERR_CUDA;
    return launch_encode(desc, n, Senc, cap, plan_ws_dev, enc_ws_dev, main_st, nullptr, kPackFramed) == cudaSuccess ? CVLC_OK : CVLC_ERR_CUDA;
  }
  // the length tuning reads the histograms' fit only; selection and ranking do not need its result
  cudaEvent_t fork, join;
  if (compress_events(&fork, &join) != cudaSuccess) return CVLC_ERR_CUDA;
  if (cudaEventRecord(fork, main_st) != cudaSuccess || cudaStreamWaitEvent(side_st, fork, 0) != cudaSuccess) return CVLC_ERR_CUDA;
  if (launch_plan_back(desc, n, S, plan_ws_dev, side_st) != cudaSuccess) return CVLC_ERR_CUDA;
  if (cudaEventRecord(join, side_st) != cudaSuccess) return CVLC_ERR_CUDA;
  return launch_encode(desc, n, Senc, cap, plan_ws_dev, enc_ws_dev, main_st, join, kPackFramed) == cudaSuccess ? CVLC_OK : CVLC_ERR_CUDA;
}

int cvlc_encode(const float* x_dev, const cvlc_params* p, const cvlc_plan_t* plan_dev, const void* plan_ws_dev,
                uint8_t* stream_dev, size_t stream_capacity, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  return cvlc_encode_batch(&x_dev, p, 1, plan_dev, plan_ws_dev, &stream_dev, stream_capacity, 0, ws_dev, ws_bytes,
                           cuda_stream);
}

int cvlc_decode_aggregate(const uint8_t* const* streams_dev, const uint64_t* stream_bytes_dev, const float* weights_dev,
                          uint32_t n_clients, double weight_total, uint64_t d, float* out_dev, int accumulate,
                          void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  if (n_clients == 0 || n_clients > CVLC_MAX_CLIENTS_PER_CALL) return CVLC_ERR_INVALID_ARG;
  if (d < 2 || d > (1ull << 31)) return CVLC_ERR_INVALID_ARG;
  if (!(weight_total >= 0.0) || !(weight_total < 1e300)) return CVLC_ERR_INVALID_ARG;
  if (!aligned(streams_dev, 8) || !aligned(stream_bytes_dev, 8) || !aligned(weights_dev, 4) || !aligned(out_dev, 16) ||
      !aligned(ws_dev, 256))
    return CVLC_ERR_INVALID_ARG;
  if (ws_bytes < dec_ws_bytes(n_clients)) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  return launch_decode(streams_dev, stream_bytes_dev, weights_dev, n_clients, weight_total, d, position_bits(d), out_dev,
                       accumulate ? 1 : 0, ws_dev, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

int cvlc_decode_apply(const uint8_t* const* streams_dev, const uint64_t* stream_bytes_dev, const float* weights_dev,
                      uint32_t n_clients, double weight_total, uint64_t d, float* model_dev, float* aggregate_dev,
                      void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  if (!aligned(model_dev, 16) || model_dev == aggregate_dev) return CVLC_ERR_INVALID_ARG;
  const int rc = cvlc_decode_aggregate(streams_dev, stream_bytes_dev, weights_dev, n_clients, weight_total, d,
                                       aggregate_dev, 0, ws_dev, ws_bytes, cuda_stream);
  if (rc != CVLC_OK) return rc;
  return launch_apply(model_dev, aggregate_dev, d, ws_dev, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

int cvlc_read_status(const void* plan_or_ws_dev, void* cuda_stream) {
  if (!plan_or_ws_dev) return CVLC_ERR_INVALID_ARG;
  int32_t v = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&v, plan_or_ws_dev, sizeof v, cudaMemcpyDeviceToHost, st) != cudaSuccess) return CVLC_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return CVLC_ERR_CUDA;
  return (int)v;
}

int cvlc_selftest_wait(uint64_t* word_dev, int32_t* status_dev, uint32_t max_polls, void* cuda_stream) {
  if (!aligned(word_dev, 8) || !aligned(status_dev, 4) || max_polls == 0 || max_polls > (1u << 20)) return CVLC_ERR_INVALID_ARG;
  return launch_selftest_wait(reinterpret_cast<unsigned long long*>(word_dev), status_dev, max_polls,
                              static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

int cvlc_selftest_philox(uint64_t seed, uint32_t client_id, uint32_t round, uint64_t first, uint64_t n, uint32_t* out_dev,
                         void* cuda_stream) {
  if (!aligned(out_dev, 4)) return CVLC_ERR_INVALID_ARG;
  return launch_selftest_philox(seed, client_id, round, first, n, out_dev, static_cast<cudaStream_t>(cuda_stream)) ==
                 cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

int cvlc_selftest_math(const double* in_dev, uint64_t n, double* log2_out_dev, double* exp2_out_dev, double* div_out_dev,
                       double* div_ref_dev, void* cuda_stream) {
  if (!aligned(in_dev, 8)) return CVLC_ERR_INVALID_ARG;
  return launch_selftest_math(in_dev, n, log2_out_dev, exp2_out_dev, div_out_dev, div_ref_dev,
                              static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
}

}  // extern "C"
