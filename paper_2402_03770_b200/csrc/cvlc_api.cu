// C ABI of libcvlc: argument validation, derived constants, workspace carving and
// stream-ordered kernel launches.  No allocation, no global state, no CPU fallback.
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
  if (p->quantizer != 0) return false;
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

// PQ error factor Q = P / (2^y - 1)^2 (Appendix, case study) and the coefficient of Eq. (5):
// g = 1 - (Q / B^2 + (1 - 1/B)^2).  Plain IEEE operations in this order; the host compiler is
// told not to contract them (-ffp-contract=off).
double quant_Q(uint32_t cap_y, uint32_t y) {
  const double L = (double)((1ull << y) - 1ull);
  return (double)cap_y / (L * L);
}
double coeff_g(double Q, double B) {
  const double c = Q / (B * B) + (1.0 - 1.0 / B) * (1.0 - 1.0 / B);
  return 1.0 - c;
}

int build_tables(const cvlc_params* p, uint32_t fixed_y, PlanTables* T) {
  Derived D;
  const int rc = derive(p, &D);
  if (rc != CVLC_OK) return rc;
  memset(T, 0, sizeof *T);
  T->d = p->d;
  T->s = D.s;
  T->R = D.R;
  T->fixed_y = fixed_y;
  for (uint32_t y = 0; y <= CVLC_MAX_CODE_BITS; ++y) T->cap[y] = D.cap[y];
  if (fixed_y) {
    if (fixed_y > p->max_code_bits) return CVLC_ERR_INVALID_ARG;
    if ((uint64_t)D.R * D.cap[fixed_y] > p->d) return CVLC_ERR_BUDGET_TOO_LARGE;
    T->nY = 1;
    T->y_min = fixed_y;
    T->Y[0] = fixed_y;
    T->capY[0] = D.cap[fixed_y];
    T->QY[0] = quant_Q(D.cap[fixed_y], fixed_y);
    T->gY[0] = coeff_g(T->QY[0], p->scale_B);
    return CVLC_OK;
  }
  double Q[CVLC_MAX_CODE_BITS + 1], g[CVLC_MAX_CODE_BITS + 1];
  uint32_t y_min = 0;
  for (uint32_t y = 1; y <= p->max_code_bits; ++y) {
    Q[y] = quant_Q(D.cap[y], y);
    g[y] = coeff_g(Q[y], p->scale_B);
    if (y_min == 0 && g[y] > 0.0) y_min = y;
  }
  if (y_min == 0) return CVLC_ERR_SCALE_TOO_SMALL;
  T->y_min = y_min;
  uint32_t nY = 0;
  for (uint32_t y = y_min; y <= p->max_code_bits; ++y) {
    // a length that fits no more records than the next longer one is dominated
    if (y == p->max_code_bits || D.cap[y] > D.cap[y + 1]) {
      T->Y[nY] = y;
      T->capY[nY] = D.cap[y];
      T->QY[nY] = Q[y];
      T->gY[nY] = g[y];
      ++nY;
    }
  }
  T->nY = nY;
  // an admissible single-length plan must exist: the longest code sends the fewest coordinates
  if ((uint64_t)D.R * D.cap[p->max_code_bits] > p->d) return CVLC_ERR_BUDGET_TOO_LARGE;
  return CVLC_OK;
}

bool aligned(const void* p, size_t a) { return p && (reinterpret_cast<uintptr_t>(p) % a) == 0; }

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
  return 1.0 + quant_Q(cap8, 8);
}

size_t cvlc_plan_workspace_bytes(const cvlc_params* p) { return params_ok(p) ? kPlanWsBytes : 0; }

size_t cvlc_encode_workspace_bytes(const cvlc_params* p) { return params_ok(p) ? enc_layout(p->d).total : 0; }

size_t cvlc_decode_workspace_bytes(uint32_t n_clients) {
  if (n_clients == 0 || n_clients > CVLC_MAX_CLIENTS_PER_CALL) return 0;
  return dec_ws_bytes(n_clients);
}

static int plan_common(const float* x_dev, const cvlc_params* p, uint32_t fixed_y, cvlc_plan_t* plan_dev, void* ws_dev,
                       size_t ws_bytes, void* cuda_stream) {
  PlanTables T;
  const int rc = build_tables(p, fixed_y, &T);
  if (rc != CVLC_OK) return rc;
  if (!aligned(x_dev, 16) || !aligned(plan_dev, 8) || !aligned(ws_dev, 256)) return CVLC_ERR_INVALID_ARG;
  if (ws_bytes < kPlanWsBytes) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  return launch_plan(x_dev, T, plan_dev, ws_dev, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CVLC_OK
                                                                                                        : CVLC_ERR_CUDA;
}

int cvlc_plan(const float* x_dev, const cvlc_params* p, cvlc_plan_t* plan_dev, void* ws_dev, size_t ws_bytes,
              void* cuda_stream) {
  return plan_common(x_dev, p, 0, plan_dev, ws_dev, ws_bytes, cuda_stream);
}

int cvlc_plan_fixed(const float* x_dev, const cvlc_params* p, uint32_t y, cvlc_plan_t* plan_dev, void* ws_dev,
                    size_t ws_bytes, void* cuda_stream) {
  if (y < 1 || y > CVLC_MAX_CODE_BITS) return CVLC_ERR_INVALID_ARG;
  return plan_common(x_dev, p, y, plan_dev, ws_dev, ws_bytes, cuda_stream);
}

int cvlc_encode(const float* x_dev, const cvlc_params* p, const cvlc_plan_t* plan_dev, uint8_t* stream_dev,
                size_t stream_capacity, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  Derived D;
  const int rc = derive(p, &D);
  if (rc != CVLC_OK) return rc;
  if (!aligned(x_dev, 16) || !aligned(plan_dev, 8) || !aligned(stream_dev, 16) || !aligned(ws_dev, 256))
    return CVLC_ERR_INVALID_ARG;
  if (stream_capacity < cvlc_stream_bytes(p)) return CVLC_ERR_OUTPUT_TOO_SMALL;
  if (ws_bytes < enc_layout(p->d).total) return CVLC_ERR_WORKSPACE_TOO_SMALL;
  const uint32_t max_cap = D.cap[1];
  if ((size_t)max_cap * 8 > 200 * 1024) return CVLC_ERR_INVALID_ARG;  // a packet's records are staged in shared memory
  return launch_encode(x_dev, *p, D.s, D.R, max_cap, plan_dev, stream_dev, ws_dev,
                       static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? CVLC_OK
             : CVLC_ERR_CUDA;
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

int cvlc_read_status(const void* plan_or_ws_dev, void* cuda_stream) {
  if (!plan_or_ws_dev) return CVLC_ERR_INVALID_ARG;
  int32_t v = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&v, plan_or_ws_dev, sizeof v, cudaMemcpyDeviceToHost, st) != cudaSuccess) return CVLC_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return CVLC_ERR_CUDA;
  return (int)v;
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
