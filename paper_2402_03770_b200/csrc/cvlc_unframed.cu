// Unframed stream (version 2): the records of every packet without the packet frame.
//
// Section IV-C gives every packet one code length and a fixed size because a real network needs a header per
// packet; Proposition 1 itself only groups the top-k coordinates by code length.  Here the groups of the plan are
// kept (block r holds the records of packet r, longest codes first, with that packet's centroid distribution, so
// the plan and its error bound are unchanged), but a block is exactly as long as its records need: no s / y_r
// fields (a table of n_y and cap(y) in the stream header tells which block has which length), no padding, and the
// position IDs of a block are sorted and sent as differences in a Golomb-Rice code.  Records therefore have
// different lengths: bit offsets come from an exclusive prefix sum of the per-record code lengths, inside a block
// by warp scans, across the blocks of a client by a decoupled look-back.
//
// Layout (little-endian, bit i of the body = bit i mod 32 of its 32-bit word i / 32):
//   bytes 0..63    the global header of version 1 with version = 2
//   64..195        n_y[0..32] (uint32): blocks per code length;   196..327  cap[0..32]: records per block
//   328..335       total bits of the body (uint64);   336..  directory: R x uint64 bit offsets of the blocks
//   body           blocks in descending code length: lo (32), hi (32) [PQ min, max; QSGD norm, 0], then the block's
//                  records in ascending position: Rice(position - previous position - 1; previous = -1 at the start
//                  of a block) then the centroid ID (y bits).  Rice parameter m = floor(log2(d / P)); a value v
//                  goes out as v >> m one-bits, a zero bit, the low m bits.
//   size           336 + 8 R + 8 * ceil(total bits / 64) bytes
#include "cvlc_common.cuh"
#include "cvlc_lookback.cuh"
#include "cvlc_quant.cuh"

namespace cvlc {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kUfThreads = 128;
constexpr int kUfWarps = kUfThreads / 32;

// every byte of the output buffers starts at zero: block boundaries share words (they are OR-ed in) and the
// stream ends with zero padding
template <int CAP>
__global__ void __launch_bounds__(256)
k_uf_clear(const __grid_constant__ BatchDesc<CAP> batch, size_t words16, unsigned char* uf_ws, size_t ws_words) {
  const size_t gtid = (size_t)blockIdx.x * 256 + threadIdx.x, gstride = (size_t)gridDim.x * 256;
  const size_t total = words16 * batch.n;
  for (size_t i = gtid; i < total; i += gstride) {
    const uint32_t c = (uint32_t)(i / words16);
    reinterpret_cast<uint4*>(batch.c[c].stream)[i - (size_t)c * words16] = make_uint4(0u, 0u, 0u, 0u);
  }
  for (size_t i = gtid; i < ws_words; i += gstride) reinterpret_cast<uint32_t*>(uf_ws)[i] = 0u;
}

__device__ __forceinline__ void or_bits(uint32_t* img, uint32_t pos, unsigned long long value) {  // up to 64 bits at bit pos
  const uint32_t w = pos >> 5, sh = pos & 31u;
  const unsigned long long lo64 = value << sh;
  const uint32_t p0 = (uint32_t)lo64, p1 = (uint32_t)(lo64 >> 32);
  const uint32_t p2 = sh ? (uint32_t)(value >> (64 - sh)) : 0u;
  if (p0) atomicOr(img + w, p0);
  if (p1) atomicOr(img + w + 1, p1);
  if (p2) atomicOr(img + w + 2, p2);
}

__device__ __forceinline__ void or_ones(uint32_t* img, uint32_t pos, uint32_t count) {  // `count` one-bits from bit pos
  while (count) {
    const uint32_t sh = pos & 31u;
    const uint32_t nb = (32u - sh < count) ? 32u - sh : count;
    const uint32_t mask = (nb == 32u) ? 0xFFFFFFFFu : (((1u << nb) - 1u) << sh);
    atomicOr(img + (pos >> 5), mask);
    pos += nb;
    count -= nb;
  }
}

// One warp writes one block.  Blocks are handed out by a per-client ticket, so every earlier block of the client is
// being written or done when a warp looks back for its bit offset.
template <int CAP, bool QSGD>
__global__ void __launch_bounds__(kUfThreads)
k_pack_unframed(const __grid_constant__ BatchDesc<CAP> batch, const __grid_constant__ Shape shape, unsigned char* enc_ws,
                const __grid_constant__ EncLayout L, unsigned char* uf_ws, uint32_t n_pad, uint32_t img_words,
                uint32_t warp_bytes, unsigned long long* __restrict__ sizes_out) {
  extern __shared__ __align__(16) unsigned char s_uf[];
  __shared__ int s_err;
  EncHeader* hdr = reinterpret_cast<EncHeader*>(enc_ws);
  if (threadIdx.x == 0) s_err = *reinterpret_cast<const volatile int32_t*>(&hdr->status);
  __syncthreads();
  if (s_err != 0) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t c = blockIdx.y;
  const ClientDesc& cd = batch.c[c];
  const cvlc_plan_t* __restrict__ plan = cd.plan;
  const uint32_t R = shape.R;
  unsigned char* s_mine = s_uf + (size_t)warp * warp_bytes;
  unsigned long long* rec = reinterpret_cast<unsigned long long*>(s_mine);                 // [n_pad] position << 32 | value bits
  uint32_t* img = reinterpret_cast<uint32_t*>(s_mine + (size_t)n_pad * 8);                 // [img_words + 2] the block's bits
  double* sqv = reinterpret_cast<double*>(s_mine + (size_t)n_pad * 8 + ((((size_t)img_words + 2) * 4 + 15) & ~(size_t)15));
  uint32_t* ticket = reinterpret_cast<uint32_t*>(uf_ws + uf_off_ticket());
  unsigned long long* state = reinterpret_cast<unsigned long long*>(uf_ws + uf_off_state(batch.n)) + (size_t)c * R;
  uint32_t* stream_words = reinterpret_cast<uint32_t*>(cd.stream);
  uint32_t* body = stream_words + uf_head_bytes(R) / 4;

  const uint32_t mask = reinterpret_cast<const uint32_t*>(enc_ws + L.off_pass_mask)[c];
  const int flips = __popc(~mask & ((1u << kSortPasses) - 1u));
  const unsigned long long* __restrict__ sorted =
      reinterpret_cast<const unsigned long long*>(enc_ws + ((flips & 1) ? L.off_buf_b : L.off_buf_a)) + (size_t)c * L.capacity;

  // block -> its code length and first rank: lane l holds length 32 - l with the inclusive sums of blocks and records
  const uint32_t yl = CVLC_MAX_CODE_BITS - lane;
  const uint32_t ny = plan->n_y[yl];
  const uint32_t capl = plan->cap[yl];
  const unsigned long long nz = (unsigned long long)ny * capl;
  uint32_t cum = ny;
  unsigned long long zc = nz;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t a = __shfl_up_sync(kFull, cum, off);
    const unsigned long long b = __shfl_up_sync(kFull, zc, off);
    if (lane >= off) {
      cum += a;
      zc += b;
    }
  }
  {
    const uint32_t tot_blocks = __shfl_sync(kFull, cum, 31);
    const unsigned long long tot_records = __shfl_sync(kFull, zc, 31);
    const bool qsgd_one_bit = QSGD && __shfl_sync(kFull, ny, 31) != 0;
    if (tot_blocks != R || tot_records != plan->k || tot_records == 0 || tot_records > plan->n_candidates || qsgd_one_bit) {
      if (blockIdx.x == 0 && threadIdx.x == 0) set_status(&hdr->status, CVLC_ERR_PLAN_MISMATCH);
      return;
    }
  }

  uint32_t r = 0;
  if (lane == 0) r = atomicAdd(ticket + c, 1u);
  r = __shfl_sync(kFull, r, 0);
  if (r >= R) return;
  const unsigned hit = __ballot_sync(kFull, r < cum);
  const int src_lane = __ffs(hit) - 1;
  const uint32_t y = CVLC_MAX_CODE_BITS - (uint32_t)src_lane;
  const unsigned long long Z = __shfl_sync(kFull, (zc - nz) + (unsigned long long)(r - (cum - ny)) * capl, src_lane);
  const uint32_t P = __shfl_sync(kFull, capl, src_lane);
  const uint32_t m = uf_rice_param(shape.d, P);
  const unsigned long long* __restrict__ seg = sorted + Z;
  const PhiloxRoundKeys rk = philox_round_keys(cd.seed);

  // ---- the block's records and its centroid distribution (over the records in rank order, as for a packet)
  float vmin = CUDART_INF_F, vmax = -CUDART_INF_F;
  for (uint32_t j = lane; j < n_pad; j += 32) {
    unsigned long long e = ~0ull;  // padding sorts to the end
    if (j < P) {
      const unsigned long long pair = seg[j];
      const uint32_t key = (uint32_t)(pair >> 32);
      const uint32_t b = key ? (key | ((uint32_t)pair & 0x80000000u)) : 0u;  // -0 is stored as +0
      e = ((unsigned long long)((uint32_t)pair & 0x7FFFFFFFu) << 32) | b;
      if constexpr (QSGD) {
        const double a = (double)__uint_as_float(key);
        sqv[j] = __dmul_rn(a, a);
      } else {
        const float v = __uint_as_float(b);
        vmin = fminf(vmin, v);
        vmax = fmaxf(vmax, v);
      }
    }
    rec[j] = e;
  }
  for (uint32_t w = lane; w < img_words + 2; w += 32) img[w] = 0u;
  __syncwarp();
  float lo, hi;
  if constexpr (QSGD) {
    float norm = 0.0f;
    if (lane == 0) norm = qsgd_norm_of_squares(sqv, P);
    lo = __shfl_sync(kFull, norm, 0);
    hi = 0.0f;
  } else {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      vmin = fminf(vmin, __shfl_xor_sync(kFull, vmin, off));
      vmax = fmaxf(vmax, __shfl_xor_sync(kFull, vmax, off));
    }
    lo = vmin;
    hi = vmax;
  }

  // ---- ascending position: bitonic network over the n_pad slots
  for (uint32_t k = 2; k <= n_pad; k <<= 1) {
    for (uint32_t jj = k >> 1; jj > 0; jj >>= 1) {
      for (uint32_t t = lane; t < n_pad / 2; t += 32) {
        const uint32_t i = ((t & ~(jj - 1)) << 1) | (t & (jj - 1));  // the lower index of the t-th pair at distance jj
        const uint32_t p = i | jj;
        const unsigned long long a = rec[i], b = rec[p];
        const bool up = (i & k) == 0;
        if ((a > b) == up) {
          rec[i] = b;
          rec[p] = a;
        }
      }
      __syncwarp();
    }
  }

  // ---- records, 32 at a time: code, length, offset by a warp scan, bits OR-ed into the block's image
  if (lane == 0) {
    img[0] = __float_as_uint(lo);
    img[1] = __float_as_uint(hi);
  }
  __syncwarp();
  const double Lc = (double)((1ull << y) - 1ull);
  const double dlo = (double)lo;
  const double den = __dsub_rn((double)hi, dlo);
  const double pq_scale = (hi != lo) ? __ddiv_rn(Lc, den) : 0.0;
  const uint32_t sq = QSGD ? (uint32_t)((1ull << (y - 1)) - 1ull) : 0u;
  const double sqd = (double)sq, dn = (double)lo;
  const double q_scale = (QSGD && lo > 0.0f) ? __ddiv_rn(sqd, dn) : 0.0;
  uint32_t carry = 64;
  for (uint32_t base = 0; base < P; base += 32) {
    const uint32_t j = base + lane;
    const bool valid = j < P;
    uint32_t len = 0, quo = 0;
    unsigned long long tail = 0;
    if (valid) {
      const unsigned long long e = rec[j];
      const uint32_t pid = (uint32_t)(e >> 32), b = (uint32_t)e;
      const uint32_t prev = j ? (uint32_t)(rec[j - 1] >> 32) + 1u : 0u;
      const uint32_t delta = pid - prev;
      quo = delta >> m;
      uint32_t code = 0;
      const double u = __dmul_rn((double)philox_coord(rk, cd.client_id, cd.round, pid), 1.0 / 4294967296.0);
      if constexpr (QSGD) {
        const uint32_t key = b & 0x7FFFFFFFu;
        uint32_t level = 0;
        if (lo > 0.0f) level = qsgd_quantize_level((double)__uint_as_float(key), dn, sqd, sq, q_scale, u);
        code = ((key ? (b >> 31) : 0u) << (y - 1)) | level;
      } else if (hi != lo) {
        code = pq_quantize(__dsub_rn((double)__uint_as_float(b), dlo), den, Lc, pq_scale, u);
      }
      // after the unary part: the zero bit, the low m bits of the difference, the centroid ID
      tail = ((unsigned long long)(delta & ((1u << m) - 1u)) << 1) | ((unsigned long long)code << (1 + m));
      len = quo + 1u + m + y;
    }
    uint32_t incl = len;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t o = __shfl_up_sync(kFull, incl, off);
      if (lane >= off) incl += o;
    }
    if (valid) {
      const uint32_t pos = carry + incl - len;
      or_ones(img, pos, quo);
      or_bits(img, pos + quo, tail);
    }
    carry += __shfl_sync(kFull, incl, 31);
  }
  __syncwarp();
  const uint32_t block_bits = carry;

  // ---- bit offset of the block: decoupled look-back over the client's earlier blocks, 32 at a time
  if (lane == 0) st_relaxed(state + r, (r == 0 ? kFlagPrefix : kFlagAgg) | block_bits);
  unsigned long long run = 0;
  if (r > 0) {
    long long top = (long long)r - 1;
    while (true) {
      const long long idx = top - lane;
      unsigned long long sv = kFlagPrefix;  // before the client's first block: nothing
      if (idx >= 0) {
        sv = wait_state(state + idx, &hdr->status);
        if (sv == 0) sv = kFlagPrefix;  // gave up (status set): close the chain, the results are void
      }
      const unsigned is_prefix = __ballot_sync(kFull, (sv & kFlagMask) == kFlagPrefix);
      unsigned long long val = sv & kValMask;
      if (is_prefix && lane > __ffs(is_prefix) - 1) val = 0;  // everything behind the nearest prefix is inside it
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) val += __shfl_xor_sync(kFull, val, off);
      run += val;
      if (is_prefix) break;
      top -= 32;
    }
    if (lane == 0) st_relaxed(state + r, kFlagPrefix | (run + block_bits));
  }

  // ---- the image goes out shifted to its bit offset; the first and the last word are shared with the neighbours
  {
    const uint32_t shift = (uint32_t)(run & 31ull);
    const size_t w0 = (size_t)(run >> 5);
    const uint32_t n_out = (shift + block_bits + 31) >> 5;
    for (uint32_t ow = lane; ow < n_out; ow += 32) {
      uint32_t v = img[ow] << shift;  // img has two zero words behind its last used one
      if (shift && ow) v |= img[ow - 1] >> (32 - shift);
      if (ow == 0 || ow == n_out - 1) {
        if (v) atomicOr(body + w0 + ow, v);
      } else {
        body[w0 + ow] = v;
      }
    }
    if (lane == 0) {
      unsigned long long* dir = reinterpret_cast<unsigned long long*>(cd.stream + kUfDirectory);
      dir[r] = run;
      if (r == R - 1) {
        const unsigned long long total = run + block_bits;
        *reinterpret_cast<unsigned long long*>(cd.stream + kUfTotalBits) = total;
        if (sizes_out) sizes_out[c] = uf_head_bytes(R) + ((total + 63) / 64) * 8;
      }
    }
  }

  // ---- stream header and the tables of lengths, by the warp that wrote block 0
  if (r == 0) {
    if (lane < 16) {
      uint32_t v = 0;
      const unsigned long long Bbits = (unsigned long long)__double_as_longlong(cd.scale_B);
      const unsigned long long k = plan->k;
      switch (lane) {
        case 0: v = CVLC_STREAM_MAGIC; break;
        case 1: v = 2u | (shape.quantizer << 16) | (shape.s << 24); break;
        case 2: v = (uint32_t)shape.d; break;
        case 3: v = (uint32_t)(shape.d >> 32); break;
        case 4: v = R; break;
        case 5: v = shape.packet_bits; break;
        case 6: v = shape.header_bits; break;
        case 7: v = cd.client_id; break;
        case 8: v = (uint32_t)cd.seed; break;
        case 9: v = (uint32_t)(cd.seed >> 32); break;
        case 10: v = cd.round; break;
        case 11: v = 0; break;
        case 12: v = (uint32_t)Bbits; break;
        case 13: v = (uint32_t)(Bbits >> 32); break;
        case 14: v = (uint32_t)k; break;
        default: v = (uint32_t)(k >> 32); break;
      }
      stream_words[lane] = v;
    }
    uint32_t* tab = stream_words + kUfTables / 4;
    tab[lane] = plan->n_y[lane];
    tab[33 + lane] = plan->cap[lane];
    if (lane == 0) {
      tab[32] = plan->n_y[32];
      tab[33 + 32] = plan->cap[32];
    }
  }
}

template <int CAP>
static cudaError_t launch_pack_unframed_t(const ClientDesc* clients, uint32_t n, const Shape& shape, uint64_t capacity,
                                          size_t stream_capacity, void* enc_ws, void* uf_ws, unsigned long long* sizes_out,
                                          cudaStream_t st) {
  static bool attr_done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && !attr_done[dev]) {
    e = cudaFuncSetAttribute(k_pack_unframed<CAP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_pack_unframed<CAP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  BatchDesc<CAP> batch;
  batch.n = n;
  batch.pad = 0;
  for (uint32_t i = 0; i < n; ++i) batch.c[i] = clients[i];
  const EncLayout L = enc_layout(shape.d, n, capacity);
  const bool qsgd = shape.quantizer == CVLC_QUANT_QSGD;
  // the largest block: cap of the shortest admissible length
  const uint32_t y_lo = qsgd ? 2u : 1u;
  const uint32_t P_max = shape.cap[y_lo];
  uint32_t n_pad = 2;
  while (n_pad < P_max) n_pad <<= 1;
  // bits of a block: 64 of header, per record 1 + m + y, fewer than 2 P one-bits of unary parts in all
  uint64_t bits = 0;
  for (uint32_t y = y_lo; y <= shape.max_code_bits; ++y) {
    const uint64_t b = 64 + (uint64_t)shape.cap[y] * (1 + uf_rice_param(shape.d, shape.cap[y]) + y) + 2 * (uint64_t)shape.cap[y];
    if (b > bits) bits = b;
  }
  const uint32_t img_words = (uint32_t)((bits + 31) / 32);
  const size_t warp_bytes = (size_t)n_pad * 8 + ((((size_t)img_words + 2) * 4 + 15) & ~(size_t)15) + (qsgd ? (size_t)P_max * 8 : 0);
  {
    LaunchScope ls(kKZeroWords, st);
    k_uf_clear<CAP><<<4 * kNumSM, 256, 0, st>>>(batch, stream_capacity / 16, static_cast<unsigned char*>(uf_ws),
                                                 uf_ws_bytes(n, shape.R) / 4);
  }
  {
    LaunchScope ls(kKPackUnframed, st);
    const unsigned grid = (shape.R + kUfWarps - 1) / kUfWarps;
    if (qsgd)
      k_pack_unframed<CAP, true><<<dim3(grid, n), kUfThreads, warp_bytes * kUfWarps, st>>>(
          batch, shape, static_cast<unsigned char*>(enc_ws), L, static_cast<unsigned char*>(uf_ws), n_pad, img_words,
          (uint32_t)warp_bytes, sizes_out);
    else
      k_pack_unframed<CAP, false><<<dim3(grid, n), kUfThreads, warp_bytes * kUfWarps, st>>>(
          batch, shape, static_cast<unsigned char*>(enc_ws), L, static_cast<unsigned char*>(uf_ws), n_pad, img_words,
          (uint32_t)warp_bytes, sizes_out);
  }
  return cudaGetLastError();
}

cudaError_t launch_pack_unframed(const ClientDesc* clients, uint32_t n, const Shape& shape, uint64_t capacity,
                                 size_t stream_capacity, void* enc_ws, void* uf_ws, unsigned long long* sizes_out, cudaStream_t st) {
  if (n <= (uint32_t)kSmallBatch)
    return launch_pack_unframed_t<kSmallBatch>(clients, n, shape, capacity, stream_capacity, enc_ws, uf_ws, sizes_out, st);
  return launch_pack_unframed_t<kLargeBatch>(clients, n, shape, capacity, stream_capacity, enc_ws, uf_ws, sizes_out, st);
}

// ===================================================================================
// parameter server: decode + dequantize + weighted scatter-accumulate of unframed streams
// ===================================================================================

constexpr int kUfPrepThreads = 1024;

// validates the headers and tables, derives the per-client coefficients and the prefix of block counts
__global__ void __launch_bounds__(kUfPrepThreads)
k_uf_decode_prepare(const uint8_t* const* __restrict__ streams, const uint64_t* __restrict__ stream_bytes,
                    const float* __restrict__ weights, uint32_t n, double weight_total, uint64_t d, uint32_t s, unsigned char* ws) {
  __shared__ double s_part[kUfPrepThreads / 32];
  __shared__ uint32_t s_cnt[kUfPrepThreads / 32];
  __shared__ double s_W;
  __shared__ uint32_t s_carry;
  int32_t* status = reinterpret_cast<int32_t*>(ws + kDecWsStatus);
  float* coef = reinterpret_cast<float*>(ws + kDecWsCoef);
  uint32_t* prefix = reinterpret_cast<uint32_t*>(ws + dec_off_prefix(n));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    *status = 0;
    s_carry = 0;
  }
  double wsum = 0.0;
  for (uint32_t i = tid; i < n; i += kUfPrepThreads) wsum += (double)weights[i];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) wsum += __shfl_xor_sync(kFull, wsum, off);
  if (lane == 0) s_part[warp] = wsum;
  __syncthreads();
  if (tid == 0) {
    double W = 0.0;
    for (int w = 0; w < kUfPrepThreads / 32; ++w) W += s_part[w];
    s_W = (weight_total != 0.0) ? weight_total : W;
  }
  __syncthreads();
  const double W = s_W;
  if (tid == 0 && !(W > 0.0)) set_status(status, CVLC_ERR_INVALID_ARG);
  for (uint32_t base = 0; base < n; base += kUfPrepThreads) {
    const uint32_t i = base + tid;
    uint32_t R = 0;
    if (i < n) {
      const uint8_t* st = streams[i];
      const uint64_t nbytes = stream_bytes[i];
      bool ok = (st != nullptr) && ((reinterpret_cast<uintptr_t>(st) & 15) == 0) && nbytes >= kUfDirectory;
      if (ok) {
        const uint32_t* hw = reinterpret_cast<const uint32_t*>(st);
        const uint32_t magic = hw[0], ver_q_s = hw[1];
        const uint64_t sd = (uint64_t)hw[2] | ((uint64_t)hw[3] << 32);
        const uint32_t sR = hw[4], pb = hw[5], hb = hw[6];
        const double B = __longlong_as_double((long long)((uint64_t)hw[12] | ((uint64_t)hw[13] << 32)));
        const uint32_t quantizer = (ver_q_s >> 16) & 0xFF;
        ok = (magic == CVLC_STREAM_MAGIC) && ((ver_q_s & 0xFFFF) == 2) && (quantizer <= CVLC_QUANT_QSGD) && ((ver_q_s >> 24) == s) &&
             (sd == d) && (pb != 0) && ((pb & 31) == 0) && (hb >= 80) && (hb < pb) && (B >= 1.0) && (B < 1e300) &&
             (nbytes >= uf_head_bytes(sR));
        if (ok) {
          const uint32_t* tab = hw + kUfTables / 4;
          unsigned long long blocks = 0;
          for (uint32_t y = 0; y <= CVLC_MAX_CODE_BITS; ++y) {
            const uint32_t ny = tab[y], cp = tab[33 + y];
            blocks += ny;
            if (ny && (y == 0 || cp == 0 || cp > kUfMaxRecords || (quantizer == CVLC_QUANT_QSGD && y < 2))) ok = false;
          }
          const unsigned long long total = *reinterpret_cast<const unsigned long long*>(st + kUfTotalBits);
          ok = ok && blocks == sR && uf_head_bytes(sR) + ((total + 63) / 64) * 8 == nbytes;
        }
        if (ok) {
          R = sR;
          const float wi = weights[i];
          if (!(wi > 0.0f) || __float_as_uint(wi) >= 0x7F800000u) set_status(status, CVLC_ERR_INVALID_ARG);
          coef[i] = (float)((double)wi / (W * B));
        }
      }
      if (!ok) {
        set_status(status, CVLC_ERR_BAD_STREAM);
        coef[i] = 0.0f;
      }
    }
    uint32_t incl = R;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t o = __shfl_up_sync(kFull, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) s_cnt[warp] = incl;
    __syncthreads();
    uint32_t below = s_carry;
    for (int w = 0; w < warp; ++w) below += s_cnt[w];
    if (i < n) prefix[i] = below + incl - R;
    __syncthreads();
    if (tid == kUfPrepThreads - 1) s_carry = below + incl;
    __syncthreads();
  }
  if (tid == 0) prefix[n] = s_carry;
}

// 64 bits of the body from bit pos on (zero beyond its last word)
__device__ __forceinline__ unsigned long long uf_peek(const uint32_t* __restrict__ body, unsigned long long n_words, unsigned long long pos) {
  const unsigned long long w = pos >> 5;
  const uint32_t sh = (uint32_t)(pos & 31ull);
  const unsigned long long a = (w < n_words) ? __ldg(body + w) : 0u, b = (w + 1 < n_words) ? __ldg(body + w + 1) : 0u;
  unsigned long long v = (a | (b << 32)) >> sh;
  if (sh) {
    const unsigned long long c2 = (w + 2 < n_words) ? __ldg(body + w + 2) : 0u;
    v |= c2 << (64 - sh);
  }
  return v;
}

constexpr int kUfDecThreads = 128;

// one warp per block: lane 0 walks the block's bits (the unary parts make that sequential) and leaves position and
// centroid ID of every record in shared memory; the warp then dequantizes and accumulates
__global__ void __launch_bounds__(kUfDecThreads)
k_decode_unframed(const uint8_t* const* __restrict__ streams, uint32_t n, uint64_t d, float* __restrict__ out, unsigned char* ws) {
  extern __shared__ uint32_t s_dec[];  // [n + 1] block prefix, then per warp kUfMaxRecords positions and codes
  __shared__ int s_err;
  int32_t* status = reinterpret_cast<int32_t*>(ws + kDecWsStatus);
  const float* coef = reinterpret_cast<const float*>(ws + kDecWsCoef);
  const uint32_t* prefix = reinterpret_cast<const uint32_t*>(ws + dec_off_prefix(n));
  if (threadIdx.x == 0) s_err = *reinterpret_cast<const volatile int32_t*>(status);
  for (uint32_t i = threadIdx.x; i <= n; i += kUfDecThreads) s_dec[i] = prefix[i];
  __syncthreads();
  if (s_err != 0) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* s_pid = s_dec + (n + 1) + (size_t)warp * 2 * kUfMaxRecords;
  uint32_t* s_cid = s_pid + kUfMaxRecords;
  const uint32_t total = s_dec[n];
  const uint32_t warps_total = gridDim.x * (kUfDecThreads / 32);
  for (uint32_t g = blockIdx.x * (kUfDecThreads / 32) + warp; g < total; g += warps_total) {
    uint32_t lo_c = 0, hi_c = n;
    while (hi_c - lo_c > 1) {
      const uint32_t mid = (lo_c + hi_c) >> 1;
      if (s_dec[mid] <= g) lo_c = mid; else hi_c = mid;
    }
    const uint32_t c = lo_c, r = g - s_dec[c];
    const uint8_t* st = streams[c];
    const uint32_t* hw = reinterpret_cast<const uint32_t*>(st);
    const uint32_t R = hw[4], quantizer = (hw[1] >> 16) & 0xFF;
    const uint32_t* tab = hw + kUfTables / 4;
    // the block's length: lane l holds length 32 - l and the inclusive count of blocks down to it
    const uint32_t ny = tab[CVLC_MAX_CODE_BITS - lane], cp = tab[33 + CVLC_MAX_CODE_BITS - lane];
    uint32_t cum = ny;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t a = __shfl_up_sync(kFull, cum, off);
      if (lane >= off) cum += a;
    }
    const unsigned hit = __ballot_sync(kFull, r < cum);
    const int src_lane = __ffs(hit) - 1;  // the tables add up to R: checked by the prepare kernel
    const uint32_t y = CVLC_MAX_CODE_BITS - (uint32_t)src_lane;
    const uint32_t P = __shfl_sync(kFull, cp, src_lane);
    const uint32_t m = uf_rice_param(d, P);
    const unsigned long long total_bits = *reinterpret_cast<const unsigned long long*>(st + kUfTotalBits);
    const unsigned long long n_words = ((total_bits + 63) / 64) * 2;
    const uint32_t* body = hw + uf_head_bytes(R) / 4;
    unsigned long long pos = reinterpret_cast<const unsigned long long*>(st + kUfDirectory)[r];
    __syncwarp();  // the previous block's records have been read
    int bad = 0;
    float lo = 0.f, hi = 0.f;
    if (pos + 64 > total_bits) {
      bad = 1;
    } else {
      const unsigned long long h = uf_peek(body, n_words, pos);
      lo = __uint_as_float((uint32_t)h);
      hi = __uint_as_float((uint32_t)(h >> 32));
      pos += 64;
      const bool qsgd = quantizer == CVLC_QUANT_QSGD;
      if (qsgd && __float_as_uint(lo) >= 0x7F800000u) bad = 1;
      if (!qsgd && ((__float_as_uint(lo) & 0x7FFFFFFFu) >= 0x7F800000u || (__float_as_uint(hi) & 0x7FFFFFFFu) >= 0x7F800000u || lo > hi)) bad = 1;
    }
    if (!bad && lane == 0) {
      unsigned long long prev = 0;
      const unsigned long long code_mask = (1ull << y) - 1ull, low_mask = (1ull << m) - 1ull;
      for (uint32_t j = 0; j < P; ++j) {
        unsigned long long quo = 0;
        while (true) {  // the unary part: at most total_bits one-bits, checked below
          const unsigned long long v = uf_peek(body, n_words, pos);
          const int ones = (~v == 0ull) ? 64 : __ffsll((long long)~v) - 1;
          quo += ones;
          pos += ones;
          if (ones < 64 || pos >= total_bits) break;
        }
        if (pos + 1 + m + y > total_bits) {
          bad = 1;
          break;
        }
        const unsigned long long v = uf_peek(body, n_words, pos + 1);
        const unsigned long long pid = prev + ((quo << m) | (v & low_mask));
        if (pid >= d) {
          bad = 1;
          break;
        }
        s_pid[j] = (uint32_t)pid;
        s_cid[j] = (uint32_t)((v >> m) & code_mask);
        pos += 1 + m + y;
        prev = pid + 1;
      }
      // blocks follow one another without gaps: this one ends where the directory says the next one starts
      const unsigned long long next = (r + 1 < R) ? reinterpret_cast<const unsigned long long*>(st + kUfDirectory)[r + 1] : total_bits;
      if (!bad && pos != next) bad = 1;
    }
    bad = __shfl_sync(kFull, bad, 0) | bad;
    if (__any_sync(kFull, bad)) {
      if (lane == 0) set_status(status, CVLC_ERR_BAD_STREAM);
      continue;
    }
    __syncwarp();
    const bool qsgd = quantizer == CVLC_QUANT_QSGD;
    const uint32_t level_mask = qsgd ? (uint32_t)((1ull << (y - 1)) - 1ull) : 0u;
    const double dlo = qsgd ? 0.0 : (double)lo;
    const double step = qsgd ? __ddiv_rn((double)lo, (double)level_mask)
                             : ((hi == lo) ? 0.0 : __ddiv_rn(__dsub_rn((double)hi, dlo), (double)((1ull << y) - 1ull)));
    const float cf = coef[c];
    for (uint32_t j = lane; j < P; j += 32) {
      const uint32_t code = s_cid[j];
      float v;
      if (qsgd) {
        const float mag = (float)__dmul_rn((double)(code & level_mask), step);
        v = ((code >> (y - 1)) & 1u) ? -mag : mag;
      } else {
        v = (float)__dadd_rn(dlo, __dmul_rn((double)code, step));
      }
      atomicAdd(out + s_pid[j], cf * v);
    }
  }
}

cudaError_t launch_decode_unframed(const uint8_t* const* streams, const uint64_t* stream_bytes, const float* weights,
                                   uint32_t n, double weight_total, uint64_t d, uint32_t s, float* out, int accumulate,
                                   void* ws, cudaStream_t st) {
  static bool attr_done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && !attr_done[dev]) {
    e = cudaFuncSetAttribute(k_decode_unframed, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  unsigned char* w = static_cast<unsigned char*>(ws);
  {
    LaunchScope ls(kKDecodePrepare, st);
    k_uf_decode_prepare<<<1, kUfPrepThreads, 0, st>>>(streams, stream_bytes, weights, n, weight_total, d, s, w);
  }
  if (!accumulate) {
    e = launch_fill_zero(out, d, st);
    if (e != cudaSuccess) return e;
  }
  {
    LaunchScope ls(kKDecodeUnframed, st);
    const size_t smem = ((size_t)n + 1) * 4 + (size_t)(kUfDecThreads / 32) * 2 * kUfMaxRecords * 4;
    k_decode_unframed<<<4 * kNumSM, kUfDecThreads, smem, st>>>(streams, n, d, out, w);
  }
  return cudaGetLastError();
}

}  // namespace cvlc
