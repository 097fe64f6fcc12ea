// Internal declarations shared by the libcvlc translation units (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "../../include/cvlc.h"

namespace cvlc {

constexpr int kNumSM = 148;  // B200: grids are sized in multiples of this

#ifdef __CUDACC__
#define CVLC_HD __host__ __device__
#else
#define CVLC_HD
#endif

CVLC_HD constexpr size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// ---- a batch of clients -------------------------------------------------------------
// Every kernel of the plan / encode path works on a batch of clients that share the problem
// shape (d, budget, packet and header size, candidate lengths) and differ in their update,
// scale and Philox identifiers.  The per-client descriptors travel as a kernel parameter
// (no host-to-device copy, no device-side table to keep alive); kernels are instantiated
// for a small and a large descriptor capacity.

struct ClientDesc {
  const float* x;      // the update, d fp32
  cvlc_plan_t* plan;   // written by the plan kernels, read by the encode kernels
  uint8_t* stream;     // encode output (unused while planning)
  uint64_t seed;       // Philox key
  double scale_B;      // B of the scaling operation
  uint32_t client_id;  // Philox counter word 2
  uint32_t round;      // Philox counter word 3
};

constexpr int kSmallBatch = 4;
constexpr int kLargeBatch = CVLC_MAX_BATCH;

template <int CAP>
struct BatchDesc {
  uint32_t n;
  uint32_t pad;
  ClientDesc c[CAP];
};

struct Shape {
  uint64_t d;
  uint32_t s, R;
  uint32_t packet_bits, header_bits, quantizer, max_code_bits;
  uint32_t fixed_y;  // 0 = tune the lengths; otherwise every packet at this length
  uint32_t pad;
  uint32_t cap[CVLC_MAX_CODE_BITS + 1];  // records per packet per code length
};

// ---- workspace layouts (byte offsets; every region 256-byte aligned) ----------

// The histogram and the selection kernel stream the clients' updates as one concatenated
// array of units (a unit = one float4; every client ends with one ragged-tail unit) cut into
// equal contiguous chunks, several per thread block (the histogram takes them round-robin, the
// selection by ticket, because its cost per chunk depends on how many candidates it holds).
// A segment is the part of one client inside one chunk; with chunk q and client c both
// non-decreasing along the array, q + c numbers the segments uniquely.
constexpr int kStreamThreads = 512;
constexpr int kChunksPerBlock = 8;
struct Partition {
  uint64_t units;         // per client: d / 4 float4 units + 1 tail unit
  uint64_t total;         // units * n
  uint64_t chunk;         // units per chunk
  uint32_t n_chunks;
  uint32_t grid;          // blocks
  uint32_t max_segments;  // n_chunks + n
  uint32_t pad;
};
CVLC_HD inline Partition make_partition(uint64_t d, uint32_t n) {
  Partition P;
  P.units = (d >> 2) + 1;
  P.total = P.units * n;
  uint64_t grid = (P.total + 4 * kStreamThreads - 1) / (4 * kStreamThreads);
  if (grid > (uint64_t)(2 * kNumSM)) grid = 2 * kNumSM;
  if (grid == 0) grid = 1;
  P.grid = (uint32_t)grid;
  // chunks of at least 16 tiles of 2048 units, at most kChunksPerBlock per block
  uint64_t n_chunks = P.total / (16 * 4 * kStreamThreads);
  if (n_chunks > grid * kChunksPerBlock) n_chunks = grid * kChunksPerBlock;
  if (n_chunks < grid) n_chunks = grid;
  P.chunk = (P.total + n_chunks - 1) / n_chunks;
  P.n_chunks = (uint32_t)((P.total + P.chunk - 1) / P.chunk);
  P.max_segments = P.n_chunks + n;
  P.pad = 0;
  return P;
}

// Rows: the float4 units of a segment are also grouped into rows of 16 units (64 coordinates, half of a warp-wide
// load).  The histogram kernel leaves the largest magnitude key of every row; once the selection threshold is known
// the planner lists, per segment and in ascending order, the rows that hold a candidate (a key at or above the
// threshold).  The selection kernel works through that list 128 rows (one tile of its staging buffers) at a time:
// rows without candidates are neither read nor looked at.  Both tables are indexed by row; row r of the segment that
// starts at position p0 of the concatenated array sits at 128 * (p0 / 2048 + segment id) + r, so that the index
// ranges of different segments do not overlap.
constexpr int kRowUnits = 16;
constexpr int kTileUnits = 2048;                    // 2048 float4 = 8192 coordinates: a tile of the selection kernel
constexpr int kTileRows = kTileUnits / kRowUnits;   // 128
CVLC_HD inline uint64_t row_tiles_total(const Partition& P) { return P.total / kTileUnits + P.max_segments + 1; }
CVLC_HD inline uint64_t seg_first_tile(uint64_t p0, uint32_t seg) { return p0 / kTileUnits + seg; }

// plan workspace:
//   [0] PlanWsHeader | [256] uint64 hist[n][4096] | uint32 nonfinite[n] | uint64 tune_key[n][2] | uint32 leader[n]
//   | uint32 seg_count[S] | uint64 seg_prefix[S] | uint32 seg_rows[S] | uint32 row_max[64 * tiles]
//   | uint32 row_list[64 * tiles] | uint32 seg_hist[S][4096]          (S = max_segments, tiles = row_tiles_total)
// tune_key = (bits of alpha_q, bits of scale_B): clients of a batch with equal keys have the same code lengths;
// leader[c] = the first client of the batch with c's key (it runs the length tuning, the others copy its result).
struct PlanWsHeader {
  int32_t status;   // byte 0
  uint32_t n;       // clients of the batch the workspace was filled for
  uint64_t d;
  uint32_t n_chunks;
  uint32_t magic;   // set when the segment tables are valid
};
constexpr uint32_t kPlanWsMagic = 0x53454743u;
constexpr size_t kPlanWsHist = 256;
CVLC_HD constexpr size_t plan_off_flags(uint32_t n) { return kPlanWsHist + (size_t)n * CVLC_HIST_BINS * 8; }
CVLC_HD constexpr size_t plan_off_keys(uint32_t n) { return align256(plan_off_flags(n) + (size_t)n * 4); }
CVLC_HD constexpr size_t plan_off_leader(uint32_t n) { return align256(plan_off_keys(n) + (size_t)n * 16); }
CVLC_HD constexpr size_t plan_off_seg_count(uint32_t n) { return align256(plan_off_leader(n) + (size_t)n * 4); }
CVLC_HD constexpr size_t plan_off_seg_prefix(uint32_t n, uint32_t S) { return align256(plan_off_seg_count(n) + (size_t)S * 4); }
CVLC_HD constexpr size_t plan_off_seg_rows(uint32_t n, uint32_t S) { return align256(plan_off_seg_prefix(n, S) + (size_t)S * 8); }
CVLC_HD constexpr size_t plan_off_row_max(uint32_t n, uint32_t S) { return align256(plan_off_seg_rows(n, S) + (size_t)S * 4); }
CVLC_HD constexpr size_t plan_off_row_list(uint32_t n, uint32_t S, uint64_t tiles) {
  return align256(plan_off_row_max(n, S) + (size_t)tiles * kTileRows * 4);
}
CVLC_HD constexpr size_t plan_off_seg_hist(uint32_t n, uint32_t S, uint64_t tiles) {
  return align256(plan_off_row_list(n, S, tiles) + (size_t)tiles * kTileRows * 4);
}
CVLC_HD constexpr size_t plan_ws_bytes(uint32_t n, uint32_t S, uint64_t tiles) {
  return align256(plan_off_seg_hist(n, S, tiles) + (size_t)S * CVLC_HIST_BINS * 4);
}
CVLC_HD inline size_t plan_ws_bytes(const Partition& P, uint32_t n) { return plan_ws_bytes(n, P.max_segments, row_tiles_total(P)); }

// encode workspace header (first 256 bytes), zeroed at the start of a call
struct EncHeader {
  int32_t status;           // byte 0
  uint32_t select_ticket;   // tile tickets of the selection kernel
  uint32_t sort_ticket[4];  // tile tickets of the four digit passes
  uint32_t total_sort_tiles;
  uint32_t max_sort_tiles;  // largest per-client tile count of this batch
};

constexpr int kSelectThreads = 512;
constexpr int kSelectVecPerThread = 4;                                 // float4 loads per thread per tile
constexpr int kSelectTile = kSelectThreads * kSelectVecPerThread * 4;  // 8192 coordinates

constexpr int kSortThreads = 256;
constexpr int kSortItemsPerThread = 20;  // 128 registers per thread hold a tile without spilling: two blocks per SM
constexpr int kSortMinBlocks = 2;
constexpr int kSortTile = kSortThreads * kSortItemsPerThread;  // 5120 pairs
constexpr int kSortPasses = 4;                                 // digits of 9,9,9,4 bits
constexpr int kDigitBits = 9;
constexpr int kDigits = 1 << kDigitBits;                       // 512 digit values

struct EncLayout {
  uint32_t n;
  uint64_t capacity;             // candidate slots per client
  uint64_t select_tiles;         // per client
  uint64_t sort_tiles_max;       // per client
  size_t off_n_selected;         // uint64[n]
  size_t off_sort_prefix;        // uint32[n + 1]: first sort tile of every client
  size_t off_pass_mask;          // uint32[n]: digit passes that are constant for the client
  size_t off_ghist;              // uint64[n][4][512] digit histograms
  size_t off_gbase;              // uint64[n][4][512] their exclusive scans
  size_t off_select_state;       // uint64[n][select_tiles]
  size_t off_sort_state;         // uint64[4][n * sort_tiles_max][512]
  size_t off_buf_a, off_buf_b;   // uint64[n][capacity]
  size_t total;
};

static inline EncLayout enc_layout(uint64_t d, uint32_t n, uint64_t capacity) {
  EncLayout L;
  L.n = n;
  L.capacity = capacity;
  L.select_tiles = (d + kSelectTile - 1) / kSelectTile;
  L.sort_tiles_max = (capacity + kSortTile - 1) / kSortTile;
  L.off_n_selected = 256;
  L.off_sort_prefix = align256(L.off_n_selected + (size_t)n * 8);
  L.off_pass_mask = align256(L.off_sort_prefix + ((size_t)n + 1) * 4);
  L.off_ghist = align256(L.off_pass_mask + (size_t)n * 4);
  L.off_gbase = align256(L.off_ghist + (size_t)n * kSortPasses * kDigits * 8);
  L.off_select_state = align256(L.off_gbase + (size_t)n * kSortPasses * kDigits * 8);
  L.off_sort_state = align256(L.off_select_state + (size_t)n * L.select_tiles * 8);
  L.off_buf_a = align256(L.off_sort_state + (size_t)kSortPasses * n * L.sort_tiles_max * kDigits * 8);
  L.off_buf_b = align256(L.off_buf_a + (size_t)n * capacity * 8);
  L.total = align256(L.off_buf_b + (size_t)n * capacity * 8);
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

// ---- launch accounting and optional per-kernel timing ------------------------------

enum KernelId {
  kKZeroWords = 0, kKHist, kKPlanFit, kKPlanTune, kKPlanFinish, kKEncodeInit, kKSelect, kKSelectLookback, kKSortHist, kKSortScan,
  kKSortPass, kKPack, kKDecodePrepare, kKFillZero, kKPrefetchL2, kKDecode, kKNoallocStatus, kKSelftest, kKHistCheck, kKApply,
  kKPlanLiteral, kKEcAccumulate, kKPackUnframed, kKDecodeUnframed, kNumKernelIds
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

// Planning is launched in two parts.  The front (histogram, exponent fit, selection threshold, per-segment candidate
// counts) is all the selection and ranking kernels need; the back (length tuning, copied to the clients that share a
// tuning key) is only needed by the packing kernel, so it may run on another stream next to selection and ranking.
cudaError_t launch_plan_front(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws, cudaStream_t st);
cudaError_t launch_plan_back(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws, cudaStream_t st);
cudaError_t launch_plan(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws, cudaStream_t st);
cudaError_t launch_histogram(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws,
                             unsigned long long* hist_out, cudaStream_t st);
cudaError_t launch_plan_from_hist(const ClientDesc* clients, uint32_t n, const Shape& shape,
                                  const unsigned long long* hist, void* ws, cudaStream_t st);
// workspace of cvlc_plan_literal: per value of k its value, its error bound, its sweeps and its packet sizes
CVLC_HD constexpr size_t literal_off_k(uint32_t) { return 256; }
CVLC_HD constexpr size_t literal_off_gamma(uint32_t n_k) { return align256(literal_off_k(n_k) + (size_t)n_k * 8); }
CVLC_HD constexpr size_t literal_off_sweeps(uint32_t n_k) { return align256(literal_off_gamma(n_k) + (size_t)n_k * 8); }
CVLC_HD constexpr size_t literal_off_P(uint32_t n_k) { return align256(literal_off_sweeps(n_k) + (size_t)n_k * 4); }
CVLC_HD constexpr size_t literal_ws_bytes(uint32_t n_k, uint32_t R) { return align256(literal_off_P(n_k) + (size_t)n_k * R * 8); }
constexpr uint32_t kLiteralMaxR = 2048;   // packet sizes and their running sums of one k live in shared memory
constexpr uint32_t kLiteralMaxK = 4096;
cudaError_t launch_plan_literal(const cvlc_params& p, double alpha_q, uint32_t s, uint32_t R, uint32_t n_k, uint32_t max_sweeps,
                                unsigned long long k_lo, unsigned long long k_hi, double P_min, double P_max, double tol,
                                cvlc_literal_plan_t* out, double* P_star, void* ws, cudaStream_t st);
cudaError_t launch_apply(float* model, const float* agg, uint64_t d, const void* dec_ws, cudaStream_t st);
// wait_before_pack: an event the stream waits for right before the packing kernel (the length tuning on
// another stream), or nullptr
// write_residual: kPackFramed = packets only; kPackResidual = the packing kernel also turns the encoder's input into
// the error-compensation memory (the input buffers are written: every sent coordinate loses what the parameter
// server rebuilds for it); kPackNone = selection and ranking only (the unframed writer follows)
constexpr int kPackFramed = 0, kPackResidual = 1, kPackNone = 2;
cudaError_t launch_encode(const ClientDesc* clients, uint32_t n, const Shape& shape, uint64_t capacity,
                          const void* plan_ws, void* ws, cudaStream_t st, cudaEvent_t wait_before_pack, int write_residual);
cudaError_t launch_ec_accumulate(float* const* memory, const float* const* update, uint32_t n, uint64_t d, cudaStream_t st);
// unframed stream (version 2)
constexpr uint32_t kUfMaxRecords = 2048;  // records of a block (it is sorted and assembled in one warp's shared memory)
constexpr size_t kUfTables = 64, kUfTotalBits = 64 + 264, kUfDirectory = 64 + 264 + 8;
CVLC_HD constexpr size_t uf_head_bytes(uint32_t R) { return kUfDirectory + (size_t)R * 8; }
CVLC_HD constexpr size_t uf_off_ticket() { return 256; }
CVLC_HD constexpr size_t uf_off_state(uint32_t n) { return align256(uf_off_ticket() + (size_t)n * 4); }
CVLC_HD constexpr size_t uf_ws_bytes(uint32_t n, uint32_t R) { return align256(uf_off_state(n) + (size_t)n * R * 8); }
CVLC_HD inline uint32_t uf_rice_param(uint64_t d, uint32_t P) {  // floor(log2(d / P)), 0 when d < 2 P
  uint64_t g = d / (uint64_t)P;
  uint32_t m = 0;
  while (g >= 2) {
    g >>= 1;
    ++m;
  }
  return m;
}
cudaError_t launch_pack_unframed(const ClientDesc* clients, uint32_t n, const Shape& shape, uint64_t capacity,
                                 size_t stream_capacity, void* enc_ws, void* uf_ws, unsigned long long* sizes_out, cudaStream_t st);
cudaError_t launch_decode_unframed(const uint8_t* const* streams, const uint64_t* stream_bytes, const float* weights,
                                   uint32_t n, double weight_total, uint64_t d, uint32_t s, float* out, int accumulate,
                                   void* ws, cudaStream_t st);
cudaError_t launch_fill_zero(float* out, uint64_t d, cudaStream_t st);
cudaError_t launch_selftest_wait(unsigned long long* word, int32_t* status, uint32_t max_polls, cudaStream_t st);
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
    const unsigned long long p0 = (unsigned long long)0xD2511F53u * c.x, p1 = (unsigned long long)0xCD9E8D57u * c.z;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0, hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
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

// The same word with the ten round keys worked out once per client instead of once per coordinate.
struct PhiloxRoundKeys {
  uint32_t x[10], y[10];
};
__device__ __forceinline__ PhiloxRoundKeys philox_round_keys(uint64_t seed) {
  PhiloxRoundKeys rk;
  uint32_t kx = (uint32_t)seed, ky = (uint32_t)(seed >> 32);
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    rk.x[i] = kx;
    rk.y[i] = ky;
    kx += 0x9E3779B9u;
    ky += 0xBB67AE85u;
  }
  return rk;
}
__device__ __forceinline__ uint32_t philox_coord(const PhiloxRoundKeys& rk, uint32_t client_id, uint32_t round, uint32_t coord) {
  uint4 c = make_uint4(coord, 0u, client_id, round);  // coordinates are below 2^32: counter word 1 is zero
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const unsigned long long p0 = (unsigned long long)0xD2511F53u * c.x, p1 = (unsigned long long)0xCD9E8D57u * c.z;
    c = make_uint4((uint32_t)(p1 >> 32) ^ c.y ^ rk.x[i], (uint32_t)p1, (uint32_t)(p0 >> 32) ^ c.w ^ rk.y[i], (uint32_t)p0);
  }
  return c.x;
}

__device__ __forceinline__ void set_status(int32_t* status, int32_t code) {
  // first error wins
  atomicCAS(status, 0, code);
}

#endif  // __CUDACC__

}  // namespace cvlc
