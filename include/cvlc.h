/*
 * libcvlc: Fed-CVLC per-round compression on one NVIDIA B200 (sm_100a).
 *
 * A client compresses its fp32 model update U (d coordinates) into R fixed-size
 * packets: the k largest |U| are ranked, split into packets, packet r carries P_r
 * (position ID, centroid ID) pairs at y_r bits per value, and the code lengths y_r
 * are tuned to minimise the error bound gamma under the packet and budget
 * constraints (paper: Section IV-B "three operations", Eq. (3), Proposition 2 /
 * Eq. (5), Algorithm 1, packet format of Fig. 2).  The parameter server decodes
 * the packets of many clients and forms their weighted average (Section III,
 * step 3).
 *
 * Conventions
 *  - Every function returns a status (0 = CVLC_OK); nothing throws, prints or aborts.
 *  - Pointers named *_dev are DEVICE pointers owned by the caller; cvlc_params is
 *    read from HOST memory at call time.  The library allocates no device memory
 *    and only enqueues kernels on `cuda_stream` (a cudaStream_t passed as void*;
 *    NULL = the legacy default stream).
 *  - State the library keeps in the process, all of it outside the data path: per-device
 *    flags saying that kernel attributes have been set; two CUDA events per device used by
 *    cvlc_compress_batch to order its two streams; the launch counters and, while
 *    cvlc_profile_select is active, the profiling events; the built-in scratch of
 *    cvlc_decode_aggregate_noalloc and its cached device address.  cvlc_set_device changes
 *    the calling thread's current device.  None of this is synchronised: call the library
 *    from one host thread at a time.
 *  - Host-detectable errors are returned at once.  Errors only the device can see
 *    (non-finite input, malformed stream, a wait that ran out) are written to the
 *    status word at byte 0 of the plan / workspace and read with cvlc_read_status;
 *    after such an error the outputs are unspecified, but no access is out of
 *    bounds and no kernel waits without limit.
 *  - Workspaces: 256-byte aligned, sized by the *_workspace_bytes calls, private to
 *    one call in flight (two calls that overlap on the GPU need two workspaces).
 *  - There is no CPU fallback: without a CUDA device every launch call returns
 *    CVLC_ERR_CUDA.
 */
#ifndef CVLC_H
#define CVLC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  CVLC_OK = 0,
  CVLC_ERR_INVALID_ARG = 1,
  CVLC_ERR_BUDGET_TOO_SMALL = 2,    /* budget below one packet */
  CVLC_ERR_BUDGET_TOO_LARGE = 3,    /* even the longest code would send more than d coordinates */
  CVLC_ERR_PACKET_TOO_SMALL = 4,    /* a packet cannot hold one record of the longest code */
  CVLC_ERR_NONFINITE_INPUT = 5,     /* Inf or NaN in the update (device-detected) */
  CVLC_ERR_WORKSPACE_TOO_SMALL = 6,
  CVLC_ERR_OUTPUT_TOO_SMALL = 7,
  CVLC_ERR_BAD_STREAM = 8,          /* malformed stream (device-detected) */
  CVLC_ERR_DEVICE_TIMEOUT = 9,      /* a bounded device-side wait ran out */
  CVLC_ERR_CUDA = 10,
  CVLC_ERR_NOT_IMPLEMENTED = 11,
  CVLC_ERR_SCALE_TOO_SMALL = 12,    /* scale_B violates B > (Q+1)/2 for every code length */
  CVLC_ERR_PLAN_MISMATCH = 13       /* plan does not belong to these params / this update */
};

#define CVLC_MAX_CODE_BITS 32
#define CVLC_HIST_BINS 4096
#define CVLC_STREAM_HEADER_BYTES 64
#define CVLC_STREAM_MAGIC 0x434C5643u
#define CVLC_MAX_CLIENTS_PER_CALL 4096
#define CVLC_MAX_BATCH 512

/* The two quantizers of the paper's experiments (Section V; Appendix, case study).  Both put uniform
 * centroids behind a y-bit centroid ID, so a record is s + y bits for either (Eq. (3)).
 *  PQ    centroids = 2^y points on [min, max] of the packet's values; the header's centroid
 *        distribution is {min, max} (64 bits); Q = P / (2^y - 1)^2.
 *  QSGD  quantizes |x| against the l2-norm of the packet's values, which is the header's centroid
 *        distribution (32 bits, then 32 zero bits).  The paper leaves the place of the sign open:
 *        here the top bit of the centroid ID is the sign and the other y - 1 bits hold a level
 *        0..s_q, s_q = 2^(y-1) - 1, value = sign * level * norm / s_q.  Lengths start at y = 2;
 *        Q = min(P / s_q^2, sqrt(P) / s_q), the paper's min(Q_1, Q_2) at this level count.
 *        The norm is sqrt(sum of squares added in rank order in double) rounded to fp32. */
#define CVLC_QUANT_PQ 0u
#define CVLC_QUANT_QSGD 1u

/* Problem statement of Section IV-C: the update has d coordinates, the client may
 * send budget_bits this round in packets of packet_bits (b) with header_bits (H)
 * of header each; lengths are chosen from 1..max_code_bits (Section IV-B, "Y kinds
 * of codes"), coordinates outside the top k get 0 bits. */
typedef struct cvlc_params {
  uint64_t d;             /* coordinates, 2 <= d <= 2^31 */
  uint64_t budget_bits;   /* uplink budget of this client this round; R = floor(budget_bits / packet_bits) */
  uint32_t packet_bits;   /* b; multiple of 32; the paper uses 12000 (1500 bytes).  cvlc_encode assembles one
                             packet per warp, four warps per thread block, in shared memory: 4 * (b / 8 + 16,
                             plus 8 * cap(1) bytes with QSGD) must stay within 200 KB, else INVALID_ARG */
  uint32_t header_bits;   /* H; 80 <= H < b; 80 = s (8) + y_r (8) + min,max (64), Fig. 2 */
  uint32_t quantizer;     /* CVLC_QUANT_PQ or CVLC_QUANT_QSGD */
  uint32_t max_code_bits; /* 1..32 */
  double scale_B;         /* B >= 1 of the scaling operation; cvlc_default_scale() in the first round */
  uint64_t seed;          /* Philox4x32-10 key */
  uint32_t client_id;     /* Philox counter word 2 */
  uint32_t round;         /* Philox counter word 3 */
} cvlc_params;

/* Device-resident plan, 512 bytes, written by cvlc_plan / cvlc_plan_fixed. */
typedef struct cvlc_plan_t {
  int32_t status;         /* byte 0: device status word */
  uint32_t s;             /* bits per position ID, ceil(log2 d) */
  uint32_t R;             /* packets */
  uint32_t y_min;         /* shortest length with a positive coefficient in Eq. (5) */
  uint32_t n_lengths;     /* number of candidate lengths */
  uint32_t thresh_bin;    /* selection threshold: the histogram bin that holds rank min(d, R * cap(shortest
                             candidate length)), an upper bound of k that is known before the lengths are tuned */
  uint64_t k;             /* transmitted coordinates, sum of n_y * cap */
  uint64_t n_candidates;  /* coordinates in bins >= thresh_bin (>= k): what the encoder selects and ranks */
  double alpha;           /* fitted decay exponent of Definition 1 */
  double alpha_q;         /* alpha rounded to 1/256 and clamped */
  double beta;            /* 2 * alpha_q + 1 */
  double gamma;           /* Eq. (5) at the chosen lengths */
  double B_next;          /* 1 + max Q over the used lengths: scale_B for the next round */
  uint32_t n_y[CVLC_MAX_CODE_BITS + 1]; /* packets per code length; packets are laid out longest code first */
  uint32_t cap[CVLC_MAX_CODE_BITS + 1]; /* records per packet per code length: floor((b - H) / (s + y)) */
  uint32_t top_bin;       /* highest non-empty histogram bin */
  uint32_t reserved0;
  uint8_t reserved[512 - 88 - 2 * 4 * (CVLC_MAX_CODE_BITS + 1)];
} cvlc_plan_t;

/* --- host-only helpers (no GPU work) --------------------------------------- */

int cvlc_version(void);
const char* cvlc_status_string(int status);
/* Selects the CUDA device the following calls launch on (one process drives one GPU). */
int cvlc_set_device(int device);

/* 64 + floor(budget_bits / b) * b / 8: global header plus R whole packets (the
 * budget bR of Section IV-C is met exactly in whole packets).  0 on invalid params. */
size_t cvlc_stream_bytes(const cvlc_params* p);
/* 1 + Q(cap(8), 8): the scale of a first round (Proposition 1, footnote: B is taken
 * from the previous round's max Q + 1).  NaN on invalid params. */
double cvlc_default_scale(const cvlc_params* p);
size_t cvlc_plan_workspace_bytes(const cvlc_params* p);
size_t cvlc_encode_workspace_bytes(const cvlc_params* p);
size_t cvlc_decode_workspace_bytes(uint32_t n_clients);

/* --- the hot path ----------------------------------------------------------- */

/*
 * Algorithm 1, steps 1-14.  Reads the update x_dev (d fp32, 16-byte aligned),
 * builds the 4096-bin magnitude histogram, fits the power-law exponent of
 * Definition 1 and tunes the per-packet code lengths by repeated atomic
 * operations (Section IV-C, Lemma 2, Theorem 1) on integer lengths, minimising
 * gamma of Eq. (5) under Eq. (3).  Writes *plan_dev.  After the call the 4096
 * uint64 histogram counts sit at byte 256 of the workspace.
 * Errors: INVALID_ARG, BUDGET_*, PACKET_TOO_SMALL, SCALE_TOO_SMALL,
 * WORKSPACE_TOO_SMALL (host); NONFINITE_INPUT (device, in plan_dev->status).
 */
int cvlc_plan(const float* x_dev, const cvlc_params* p, cvlc_plan_t* plan_dev, void* ws_dev,
              size_t ws_bytes, void* cuda_stream);

/*
 * Degenerate plan with every packet at code length y: Top_k sparsification plus
 * y-bit quantization, the baselines of Section V that the method contains as
 * special cases (Section I).  Same arguments and errors as cvlc_plan.
 */
int cvlc_plan_fixed(const float* x_dev, const cvlc_params* p, uint32_t y, cvlc_plan_t* plan_dev,
                    void* ws_dev, size_t ws_bytes, void* cuda_stream);

/*
 * Planning at the parameter server (Section IV-C, last paragraph: a client with limited capacity
 * sends the distribution of its update, the server solves the problem and returns k and the P_r).
 * The distribution is the 4096-bin histogram of |x| that cvlc_plan itself works from
 * (bin = (bits(x) & 0x7FFFFFFF) >> 19): Algorithm 1 uses the update only through alpha.
 *
 * cvlc_histogram_batch: hist_dev receives n * 4096 uint64 counts, client after client; x_dev and
 * params as in cvlc_plan_batch (only d is used; all clients share it).  The workspace is sized by
 * cvlc_plan_batch_workspace_bytes and is NOT a plan workspace afterwards.
 *
 * cvlc_plan_from_histogram_batch: hist_dev holds n * 4096 uint64 counts (device memory, 8-byte
 * aligned); plans_dev receives the same plans cvlc_plan_batch makes from the updates themselves.
 * Such a plan comes without the per-chunk candidate counts: the client encodes with
 * plan_ws_dev = NULL (passing this call's workspace there is refused with PLAN_MISMATCH).
 * Errors: as cvlc_plan_batch (host); device-detected, in the plan's status word and at byte 0 of
 * ws_dev: INVALID_ARG when a histogram's counts do not add up to d, NONFINITE_INPUT when a bin of
 * exponent 255 is not empty.
 */
int cvlc_histogram_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, uint64_t* hist_dev,
                         void* ws_dev, size_t ws_bytes, void* cuda_stream);
int cvlc_plan_from_histogram_batch(const uint64_t* hist_dev, const cvlc_params* params, uint32_t n,
                                   cvlc_plan_t* plans_dev, void* ws_dev, size_t ws_bytes, void* cuda_stream);

/*
 * Problem P2 of Section IV-C as the paper solves it, with real-valued packet sizes P_1 <= ... <= P_R and code
 * lengths y_r = (b - H) / P_r - s: k runs over n_k equidistant values of its range (Section IV-D, "equidistant
 * spanning search"); for every k the packets start equal and consecutive packets are re-split by the atomic
 * operation on Eq. (7) (Lemma 2: strongly convex in the split) in sweeps r = 2 .. R until a sweep moves no packet
 * by more than 2^-30 of the largest packet, or max_sweeps; Eq. (5) then picks k*.  The result is a plan only:
 * real-valued code lengths cannot be packed, so cvlc_encode does not take it; it serves to compare its error
 * bound with the integer-length rule of cvlc_plan (whose alpha_q is the input here).  The atomic operation is a
 * bracketing search (8 rounds of 32 equidistant splits, one per lane); the sweep inside one k is sequential, as
 * the algorithm states, and the values of k run side by side, one warp each.  The number of sweeps grows about
 * with R^2: meant for R up to a few dozen.
 *  out_dev          the result header (64 bytes); status at byte 0
 *  P_star_dev       R doubles: the packet sizes at k*, or NULL
 *  ws_dev           cvlc_plan_literal_workspace_bytes(p, n_k) bytes; afterwards it holds, per value of k, at byte 256
 *                   the values of k (uint64), then 256-byte aligned their error bounds (double), their sweeps
 *                   (uint32) and their packet sizes (R doubles each)
 * Errors: INVALID_ARG (alpha_q not below 0 or equal to -1/2, n_k outside 1 .. 4096, max_sweeps == 0, more than
 * 2048 packets), BUDGET_*, PACKET_TOO_SMALL, WORKSPACE_TOO_SMALL.
 */
typedef struct cvlc_literal_plan_t {
  int32_t status;
  uint32_t R;           /* packets */
  uint32_t n_k;         /* values of k tried */
  uint32_t sweeps;      /* sweeps spent at k* */
  uint64_t k_star;      /* the value of k with the smallest error bound (the first one on ties) */
  double gamma_star;    /* Eq. (5) there */
  double alpha_q, beta;
  uint8_t reserved[16];
} cvlc_literal_plan_t;
size_t cvlc_plan_literal_workspace_bytes(const cvlc_params* p, uint32_t n_k);
int cvlc_plan_literal(const cvlc_params* p, double alpha_q, uint32_t n_k, uint32_t max_sweeps,
                      cvlc_literal_plan_t* out_dev, double* P_star_dev, void* ws_dev, size_t ws_bytes,
                      void* cuda_stream);

/*
 * Algorithm 1, steps 15-17.  Ranks the coordinates of x_dev by |x| (ties by
 * ascending index), gives packet r the next cap(y_r) ranks, stores the packet's
 * centroid distribution (PQ: minimum and maximum; QSGD: l2-norm), quantizes each value
 * stochastically onto the uniform centroids of its y_r-bit code (unbiased; random word
 * = Philox4x32-10 of the coordinate index) and packs (position ID, centroid ID) pairs
 * behind the packet header (Fig. 2).
 * stream_dev (16-byte aligned) receives cvlc_stream_bytes(p) bytes.
 * plan_dev must come from cvlc_plan / cvlc_plan_fixed on the same x_dev and params.
 * plan_ws_dev: the workspace that call used, untouched since (it holds per-chunk candidate
 * counts that let the selection run without any exchange between thread blocks, and the list
 * of the 64-coordinate rows that hold a candidate, so that the rest of the update is not read
 * a second time), or NULL when it is gone or the plan came from elsewhere: the selection then
 * reads the whole update and computes its output offsets itself with a decoupled look-back
 * scan across blocks (slower).
 * Errors: INVALID_ARG, OUTPUT_TOO_SMALL, WORKSPACE_TOO_SMALL (host); PLAN_MISMATCH,
 * DEVICE_TIMEOUT (device, at byte 0 of ws_dev).
 */
int cvlc_encode(const float* x_dev, const cvlc_params* p, const cvlc_plan_t* plan_dev,
                const void* plan_ws_dev, uint8_t* stream_dev, size_t stream_capacity, void* ws_dev,
                size_t ws_bytes, void* cuda_stream);

/*
 * Batched forms: the same kernels over n clients (n <= CVLC_MAX_BATCH) in one set of
 * launches, for a process that compresses many clients' updates on one GPU.  All clients
 * of a batch share d, the packet count floor(budget_bits / b), b, H, the quantizer and
 * max_code_bits (else INVALID_ARG); scale_B, seed, client_id and round are per client.
 *  x_dev        HOST array of n device pointers (each update d fp32, 16-byte aligned)
 *  params       HOST array of n cvlc_params
 *  fixed_y      0 = tune the lengths (cvlc_plan); 1..32 = every packet at this length
 *  plans_dev    DEVICE array of n plans; plans_dev[i].status carries client i's status and
 *               byte 0 of the workspace the first error of the batch
 *  streams_dev  HOST array of n device pointers, each with stream_capacity bytes
 *  max_candidates  candidate slots per client in the encode workspace; 0 = d (always
 *               enough).  A plan whose n_candidates exceeds it makes the whole batch fail
 *               with WORKSPACE_TOO_SMALL (device-detected, byte 0 of the workspace).
 * A device-detected error in one client (non-finite input, plan mismatch) stops the
 * encoding of the whole batch.  After cvlc_plan_batch the histogram of client i sits at
 * byte 256 + 32768 * i of the workspace.  plan_ws_dev (see cvlc_encode) must be the workspace
 * of the cvlc_plan_batch call on the same n clients in the same order, or NULL.
 */
size_t cvlc_plan_batch_workspace_bytes(const cvlc_params* p, uint32_t n);
size_t cvlc_encode_batch_workspace_bytes(const cvlc_params* p, uint32_t n, uint64_t max_candidates);
int cvlc_plan_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, uint32_t fixed_y,
                    cvlc_plan_t* plans_dev, void* ws_dev, size_t ws_bytes, void* cuda_stream);
int cvlc_encode_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n,
                      const cvlc_plan_t* plans_dev, const void* plan_ws_dev, uint8_t* const* streams_dev,
                      size_t stream_capacity, uint64_t max_candidates, void* ws_dev, size_t ws_bytes,
                      void* cuda_stream);

/*
 * Error compensation (Section II: Top_k sparsification is used "with an error compensation mechanism"; the paper
 * gives no rule of its own, so this is the cited one): the client keeps a memory of what compression lost.
 * A round with it: cvlc_ec_accumulate_batch (memory <- memory + update, fp32), cvlc_plan_batch on the memory,
 * cvlc_encode_batch_ec on the memory.  cvlc_encode_batch_ec is cvlc_encode_batch, except that its input buffers
 * are also its output: when it returns, every transmitted coordinate of memory_dev[i] has given up what the
 * parameter server rebuilds for it, fp32(centroid value / B), in one fp32 subtraction, and every other coordinate
 * is unchanged: the memory for the next round.  (The selection reads the buffers before the packing kernel writes
 * them; cvlc_plan's workspace stays valid for this one encode call.)
 *  memory_dev / update_dev   HOST arrays of n device pointers (d fp32 each, 16-byte aligned, distinct)
 * Errors as cvlc_encode_batch; cvlc_ec_accumulate_batch: INVALID_ARG.
 */
int cvlc_ec_accumulate_batch(float* const* memory_dev, const float* const* update_dev, uint32_t n, uint64_t d,
                             void* cuda_stream);
int cvlc_encode_batch_ec(float* const* memory_dev, const cvlc_params* params, uint32_t n, const cvlc_plan_t* plans_dev,
                         const void* plan_ws_dev, uint8_t* const* streams_dev, size_t stream_capacity,
                         uint64_t max_candidates, void* ws_dev, size_t ws_bytes, void* cuda_stream);

/*
 * Unframed stream (version 2).  Section IV-C gives every packet one code length and a fixed size because a packet
 * on a real network needs a header; Proposition 1 / Eq. (1) itself only groups the top-k coordinates by code
 * length.  This format keeps the plan's groups (block r = the records of packet r, longest codes first, with that
 * packet's centroid distribution, so k, the lengths and the error bound are those of cvlc_plan) and drops the
 * frame: no s / y_r fields (a table of n_y and cap(y) in the stream header), no padding, and the position IDs of
 * a block are sorted and sent as Golomb-Rice coded differences (parameter floor(log2(d / P)) for a block of P
 * records).  Records then differ in length: their bit offsets are an exclusive prefix sum of the per-record code
 * lengths (warp scans inside a block, a decoupled look-back across the blocks of a client).  The layout is in the
 * header of csrc/cvlc_unframed.cu.  A stream decodes to exactly the aggregate of the framed stream of the same plan.
 *  stream_capacity      bytes of every output buffer, at least cvlc_unframed_stream_capacity(p) (0: the shape is not
 *                       supported: a block may hold at most 2048 records, i.e. (b - H) / (s + 1) <= 2048)
 *  stream_bytes_dev     DEVICE array of n uint64 that receives the streams' lengths (they depend on the data), or NULL;
 *                       the length is also 336 + 8 R + 8 * ceil(total bits / 64) with the total at byte 328 of the stream
 *  uf_ws_dev            cvlc_unframed_workspace_bytes(p, n) bytes
 * Other arguments and errors as cvlc_encode_batch / cvlc_decode_aggregate (which takes framed streams only; the two
 * decoders refuse each other's streams with BAD_STREAM).
 */
size_t cvlc_unframed_stream_capacity(const cvlc_params* p);
size_t cvlc_unframed_workspace_bytes(const cvlc_params* p, uint32_t n);
int cvlc_encode_unframed_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, const cvlc_plan_t* plans_dev,
                               const void* plan_ws_dev, uint8_t* const* streams_dev, size_t stream_capacity,
                               uint64_t* stream_bytes_dev, uint64_t max_candidates, void* enc_ws_dev, size_t enc_ws_bytes,
                               void* uf_ws_dev, size_t uf_ws_bytes, void* cuda_stream);
int cvlc_decode_aggregate_unframed(const uint8_t* const* streams_dev, const uint64_t* stream_bytes_dev,
                                   const float* weights_dev, uint32_t n_clients, double weight_total, uint64_t d,
                                   float* out_dev, int accumulate, void* ws_dev, size_t ws_bytes, void* cuda_stream);

/*
 * cvlc_plan_batch followed by cvlc_encode_batch (with the plan's workspace) in one call: Algorithm 1 from the
 * update to the packets.  Selection and ranking need the histogram but not the tuned lengths (they work on
 * the candidates down to an upper bound of k, see cvlc_plan_t::thresh_bin), so with a second stream the
 * length tuning (Algorithm 1 steps 2-14, a latency-bound computation that leaves the memory system idle)
 * runs on side_stream next to them and is joined right before the packets are assembled.
 *  plan_ws_dev / enc_ws_dev   workspaces sized by cvlc_plan_batch_workspace_bytes and
 *                             cvlc_encode_batch_workspace_bytes (with the same max_candidates)
 *  side_stream                a second stream of the same device, or NULL / the same stream: everything
 *                             runs on cuda_stream in order.  When the call returns, cuda_stream is
 *                             ordered after all work of the call; side_stream needs no further care.
 * Other arguments, results and errors as the two calls; device-detected errors are at byte 0 of either
 * workspace.  Uses two CUDA events per device that are created at the first two-stream call on that
 * device (make it outside of any stream capture).
 */
int cvlc_compress_batch(const float* const* x_dev, const cvlc_params* params, uint32_t n, uint32_t fixed_y,
                        cvlc_plan_t* plans_dev, uint8_t* const* streams_dev, size_t stream_capacity,
                        uint64_t max_candidates, void* plan_ws_dev, size_t plan_ws_bytes, void* enc_ws_dev,
                        size_t enc_ws_bytes, void* cuda_stream, void* side_stream);

/*
 * Parameter-server aggregation (Section III, step 3) fused with decoding: for every
 * record of every client, value = min + CID * (max - min) / (2^y - 1) (PQ; the QSGD value is
 * given with CVLC_QUANT_QSGD; every stream names its quantizer in its header), scaled by
 * 1/B_i (Section IV-B, scaling) and by weight_i / weight_total, added into
 * out_dev[PID].  Uniform weights give the paper's 1/|S_t| average.
 *  streams_dev       device array of n_clients device pointers (each 16-byte aligned)
 *  stream_bytes_dev  device array of n_clients stream lengths
 *  weights_dev       device array of n_clients fp32 weights (> 0)
 *  weight_total      0 = sum of this call's weights; otherwise the total over all
 *                    batches when the clients are fed in several calls
 *  out_dev           d fp32; overwritten when accumulate == 0, added to when 1
 * A vector of more than 24 Mi coordinates is filled window by window (one pass over the
 * streams per window) so that the additions stay in the L2 cache; the result does not
 * depend on it.
 * Errors: INVALID_ARG, WORKSPACE_TOO_SMALL (host); BAD_STREAM (device, at byte 0
 * of ws_dev).
 */
int cvlc_decode_aggregate(const uint8_t* const* streams_dev, const uint64_t* stream_bytes_dev,
                          const float* weights_dev, uint32_t n_clients, double weight_total,
                          uint64_t d, float* out_dev, int accumulate, void* ws_dev, size_t ws_bytes,
                          void* cuda_stream);

/*
 * The same aggregation as cvlc_decode_aggregate for callers that cannot allocate device
 * memory (the paper has no counterpart to this entry point; it exists for integration).
 * Such callers are, for example, code that runs inside another framework's memory pool
 * with no spare capacity, a plugin that is forbidden to call cudaMalloc after start-up,
 * or a real-time serving loop where an allocation could stall on the driver.  Instead of
 * a workspace argument the call uses a scratch array built into the library (a few KB per
 * GPU, held from library load to process exit), so it handles at most
 * CVLC_NOALLOC_MAX_CLIENTS clients per call; more returns CVLC_ERR_WORKSPACE_TOO_SMALL
 * and launches nothing.  It calls no cudaMalloc / cudaFree and no allocating routine.
 *  - All arguments as in cvlc_decode_aggregate, plus status_dev: one int32 of the
 *    caller's device memory that receives the device status (0 or CVLC_ERR_BAD_STREAM,
 *    ...) when the stream reaches that point; read it after synchronising.
 *  - The first call on each device looks the scratch's device address up (with that
 *    device current); make that first call outside of any stream capture.
 *  - Every call on a device shares the one scratch.  Each call resets what it needs, so
 *    calls that run one after another are independent, but two calls whose kernels may
 *    overlap on the GPU (different streams, no ordering between them) race on it: order
 *    them, or use cvlc_decode_aggregate with separate workspaces.
 */
#define CVLC_NOALLOC_MAX_CLIENTS 256
int cvlc_decode_aggregate_noalloc(const uint8_t* const* streams_dev, const uint64_t* stream_bytes_dev,
                                  const float* weights_dev, uint32_t n_clients, double weight_total,
                                  uint64_t d, float* out_dev, int accumulate, int32_t* status_dev,
                                  void* cuda_stream);

/*
 * The parameter server's model step (Section III, step 3): w_{t+1} = w_t - aggregate.
 * cvlc_decode_aggregate into aggregate_dev (d fp32, overwritten; kept for the caller), then
 * model_dev[i] -= aggregate_dev[i] in fp32.  Two kernels rather than atomics straight into the
 * model: adding a hundred small terms one by one to a large weight would round a hundred times.
 * After a device-detected decode error the model is left untouched.  Other arguments and errors
 * as cvlc_decode_aggregate; model_dev 16-byte aligned and distinct from aggregate_dev.
 */
int cvlc_decode_apply(const uint8_t* const* streams_dev, const uint64_t* stream_bytes_dev, const float* weights_dev,
                      uint32_t n_clients, double weight_total, uint64_t d, float* model_dev, float* aggregate_dev,
                      void* ws_dev, size_t ws_bytes, void* cuda_stream);

/* Waits for cuda_stream and returns the status word at byte 0 of a plan or workspace. */
int cvlc_read_status(const void* plan_or_ws_dev, void* cuda_stream);

/* --- diagnostic entry points (used by the parity tests) --------------------- */

/* out_dev[4*i .. 4*i+3] = Philox4x32-10(counter (i_lo, i_hi, client_id, round), key seed)
 * for i = first .. first + n - 1 (Salmon et al., SC'11). */
int cvlc_selftest_philox(uint64_t seed, uint32_t client_id, uint32_t round, uint64_t first,
                         uint64_t n, uint32_t* out_dev, void* cuda_stream);
/* The planner's series arithmetic: log2_out[i] = log2(in[i]) (in > 0), exp2_out[i] =
 * 2^in[i] (|in| <= 1000), div_out[i*20 + j-1] = in[i] / j for j = 1..20 (the constant
 * divisions of the exp2 series), div_ref the same by IEEE division. */
int cvlc_selftest_math(const double* in_dev, uint64_t n, double* log2_out_dev, double* exp2_out_dev,
                       double* div_out_dev, double* div_ref_dev, void* cuda_stream);

/* The bounded wait every look-back scan of the library uses (a block polls a state word of an earlier
 * tile at most 2^20 times, then gives up), run on word_dev (8 bytes; a value below 2^62 counts as "not
 * published yet") with a limit of max_polls (1 .. 2^20): when the wait runs out the kernel writes
 * CVLC_ERR_DEVICE_TIMEOUT to *status_dev (if that still holds 0) and returns.  Nothing hangs. */
int cvlc_selftest_wait(uint64_t* word_dev, int32_t* status_dev, uint32_t max_polls, void* cuda_stream);

/* Launch accounting: number of kernels this library has launched in this process
 * (all kernels when kernel_name is NULL or "", else the named one, e.g. "k_hist").  Kernel names: k_zero_words,
 * k_hist, k_plan_fit, k_plan_tune, k_plan_finish, k_encode_init, k_select, k_select_lookback, k_sort_hist,
 * k_sort_scan, k_sort_pass, k_pack, k_decode_prepare, k_fill_zero, k_prefetch_l2, k_decode,
 * k_noalloc_publish_status, k_selftest, k_hist_check, k_apply, k_plan_literal, k_ec_accumulate, k_pack_unframed, k_decode_unframed. */
unsigned long long cvlc_launch_count(const char* kernel_name);
/* Optional kernel timing: after cvlc_profile_select(name, n) the next n launches of that kernel
 * ("*" = of every kernel) are bracketed by a CUDA event pair on their own stream;
 * cvlc_profile_read synchronises the device and returns how many launches of `kernel_name`
 * (NULL, "" or "*" = all) were timed and their summed duration.  cvlc_profile_select(NULL, 0)
 * switches it off and frees the events.  Single-threaded use. */
int cvlc_profile_select(const char* kernel_name, uint32_t max_launches);
int cvlc_profile_reset(void);
int cvlc_profile_read(const char* kernel_name, uint32_t* launches, double* total_ms);

#ifdef __cplusplus
}
#endif
#endif
