// Internal declarations shared by the libcvlc translation units (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "../../include/cvlc.h"

namespace cvlc {

constexpr int kNumSM = 148;  // B200: grids are sized in multiples of this

// ---- workspace layouts (byte offsets; every region 256-byte aligned) ----------

// plan workspace
constexpr size_t kPlanWsStatus = 0;      // int32 status, uint32 nonfinite flag at +4
constexpr size_t kPlanWsHist = 256;      // uint64[4096]
constexpr size_t kPlanWsBytes = kPlanWsHist + CVLC_HIST_BINS * 8;

// encode workspace header (first 256 bytes), all zeroed at the start of a call
struct EncHeader {
  int32_t status;            // byte 0
  uint32_t pad0;
  uint32_t select_ticket;    // tile tickets of the selection kernel
  uint32_t sort_ticket[4];   // tile tickets of the four digit passes
  uint32_t pad1;
  unsigned long long n_selected;  // candidates written by the selection kernel
};
constexpr size_t kEncWsSortHist = 256;                 // uint64[4][256] digit histograms
constexpr size_t kEncWsSelectState = 256 + 4 * 256 * 8;  // uint64[n_select_tiles]

constexpr int kSelectThreads = 256;
constexpr int kSelectVecPerThread = 4;                       // float4 loads per thread per tile
constexpr int kSelectTile = kSelectThreads * kSelectVecPerThread * 4;  // 4096 coordinates

constexpr int kSortThreads = 256;
constexpr int kSortItemsPerThread = 8;
constexpr int kSortTile = kSortThreads * kSortItemsPerThread;  // 2048 pairs
constexpr int kSortPasses = 4;                                 // digits of 8,8,8,7 bits

struct EncLayout {
  uint64_t n_select_tiles;
  uint64_t max_sort_tiles;
  size_t off_select_state;
  size_t off_sort_state;   // uint64[4][max_sort_tiles][256]
  size_t off_buf_a;        // uint64[d]
  size_t off_buf_b;        // uint64[d]
  size_t total;
};

#ifdef __CUDACC__
#define CVLC_HD __host__ __device__
#else
#define CVLC_HD
#endif

CVLC_HD constexpr size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

static inline EncLayout enc_layout(uint64_t d) {
  EncLayout L;
  L.n_select_tiles = (d + kSelectTile - 1) / kSelectTile;
  L.max_sort_tiles = (d + kSortTile - 1) / kSortTile;
  L.off_select_state = kEncWsSelectState;
  L.off_sort_state = align256(L.off_select_state + L.n_select_tiles * 8);
  L.off_buf_a = align256(L.off_sort_state + (size_t)kSortPasses * L.max_sort_tiles * 256 * 8);
  L.off_buf_b = align256(L.off_buf_a + d * 8);
  L.total = align256(L.off_buf_b + d * 8);
  return L;
}

// decode workspace
constexpr size_t kDecWsStatus = 0;     // int32 status
constexpr size_t kDecWsTotalPkts = 8;  // uint32 total packets
constexpr size_t kDecWsCoef = 256;     // float[n]
CVLC_HD constexpr size_t dec_off_prefix(uint32_t n) { return align256(kDecWsCoef + (size_t)n * 4); }  // uint32[n+1]
CVLC_HD constexpr size_t dec_off_meta(uint32_t n) { return align256(dec_off_prefix(n) + ((size_t)n + 1) * 4); }
// per client: packet_bits, header_bits (uint32 each)
CVLC_HD constexpr size_t dec_ws_bytes(uint32_t n) { return align256(dec_off_meta(n) + (size_t)n * 8); }

// ---- host-side tables handed to the planning kernel -----------------------------

struct PlanTables {
  uint64_t d;
  uint32_t s, R;
  uint32_t nY;                               // candidate lengths
  uint32_t y_min;
  uint32_t fixed_y;                          // 0 = tune; otherwise every packet at this length
  uint32_t pad;
  uint32_t Y[CVLC_MAX_CODE_BITS];            // candidate lengths, ascending
  uint32_t capY[CVLC_MAX_CODE_BITS];         // cap(Y[i])
  double gY[CVLC_MAX_CODE_BITS];             // coefficient g(Y[i]) of Eq. (5)
  double QY[CVLC_MAX_CODE_BITS];             // PQ error factor Q(Y[i])
  uint32_t cap[CVLC_MAX_CODE_BITS + 1];      // cap(y) for every y
};

// ---- launch accounting and optional per-kernel timing ------------------------------

enum KernelId {
  kKZeroWords = 0, kKHist, kKPlan, kKEncodeInit, kKSelect, kKSortHist, kKSortPass, kKPack, kKDecodePrepare,
  kKFillZero, kKDecode, kKSelftest, kNumKernelIds
};

// Called around every kernel launch.  Counts launches; when a kernel has been selected with
// cvlc_profile_select, records a CUDA event pair on the launching stream around it.
void launch_begin(int kernel_id, cudaStream_t st);
void launch_end(int kernel_id, cudaStream_t st);

struct LaunchScope {
  int id;
  cudaStream_t st;
  LaunchScope(int id_, cudaStream_t st_) : id(id_), st(st_) { launch_begin(id, st); }
  ~LaunchScope() { launch_end(id, st); }
};

// ---- launchers (one per translation unit) ---------------------------------------

cudaError_t launch_plan(const float* x, const PlanTables& T, cvlc_plan_t* plan, void* ws, cudaStream_t st);
cudaError_t launch_encode(const float* x, const cvlc_params& p, uint32_t s, uint32_t R, uint32_t max_cap,
                          const cvlc_plan_t* plan, uint8_t* stream, void* ws, cudaStream_t st);
cudaError_t launch_decode(const uint8_t* const* streams, const uint64_t* stream_bytes, const float* weights,
                          uint32_t n, double weight_total, uint64_t d, uint32_t s, float* out, int accumulate,
                          void* ws, cudaStream_t st);
cudaError_t launch_selftest_philox(uint64_t seed, uint32_t client_id, uint32_t round, uint64_t first, uint64_t n,
                                   uint32_t* out, cudaStream_t st);
cudaError_t launch_selftest_math(const double* in, uint64_t n, double* l2, double* e2, double* dv, double* dr,
                                 cudaStream_t st);

// ---- device helpers ---------------------------------------------------------------

#ifdef __CUDACC__

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds of two 32x32->64
// multiplies with the constants 0xD2511F53 / 0xCD9E8D57, key bumped by the Weyl
// constants 0x9E3779B9 / 0xBB67AE85 after every round.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// random word of one coordinate: counter (coord lo, coord hi, client, round), key = seed
__device__ __forceinline__ uint32_t philox_coord(uint64_t seed, uint32_t client_id, uint32_t round, uint64_t coord) {
  const uint4 r = philox4x32_10(make_uint4((uint32_t)coord, (uint32_t)(coord >> 32), client_id, round),
                                make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
  return r.x;
}

__device__ __forceinline__ void set_status(int32_t* status, int32_t code) {
  // first error wins
  atomicCAS(status, 0, code);
}

#endif  // __CUDACC__

}  // namespace cvlc
