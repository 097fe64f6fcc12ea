// Parameter-server side (Section III, step 3): decode every client's packets
// (Fig. 2), dequantize, scale by weight_i / (W * B_i) and accumulate into the dense
// averaged update.  One warp per packet; scatter-accumulate with fp32 reductions.
#include "cvlc_common.cuh"

namespace cvlc {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kPrepThreads = 1024;
constexpr int kDecodeThreads = 256;
constexpr uint32_t kDecStageWords = 512;  // packets up to 2 KB are staged in shared memory
constexpr uint64_t kDecodeWindow = 24ull << 20;  // coordinates of the accumulator filled per decode launch (96 MB: inside the L2)

struct StreamHead {
  uint32_t magic, ver_q_s, d_lo, d_hi, R, packet_bits, header_bits, client_id, seed_lo, seed_hi, round, zero, B_lo, B_hi, k_lo, k_hi;
};

// K7a  validate the global headers, derive per-client coefficients and the packet prefix
__global__ void __launch_bounds__(kPrepThreads)
k_decode_prepare(const uint8_t* const* __restrict__ streams, const uint64_t* __restrict__ stream_bytes,
                 const float* __restrict__ weights, uint32_t n, double weight_total, uint64_t d, uint32_t s,
                 unsigned char* ws) {
  __shared__ double s_part[kPrepThreads / 32];
  __shared__ uint32_t s_cnt[kPrepThreads / 32];
  __shared__ double s_W;
  __shared__ uint32_t s_carry;
  int32_t* status = reinterpret_cast<int32_t*>(ws + kDecWsStatus);
  uint32_t* total_pkts = reinterpret_cast<uint32_t*>(ws + kDecWsTotalPkts);
  float* coef = reinterpret_cast<float*>(ws + kDecWsCoef);
  uint32_t* prefix = reinterpret_cast<uint32_t*>(ws + dec_off_prefix(n));
  uint32_t* meta = reinterpret_cast<uint32_t*>(ws + dec_off_meta(n));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    *status = 0;
    s_carry = 0;
  }
  // total weight
  double wsum = 0.0;
  for (uint32_t i = tid; i < n; i += kPrepThreads) wsum += (double)weights[i];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) wsum += __shfl_xor_sync(kFull, wsum, off);
  if (lane == 0) s_part[warp] = wsum;
  __syncthreads();
  if (tid == 0) {
    double W = 0.0;
    for (int w = 0; w < kPrepThreads / 32; ++w) W += s_part[w];
    s_W = (weight_total != 0.0) ? weight_total : W;
  }
  __syncthreads();
  const double W = s_W;
  if (tid == 0 && !(W > 0.0)) set_status(status, CVLC_ERR_INVALID_ARG);

  // headers, in chunks of kPrepThreads clients; prefix of packet counts in client order
  for (uint32_t base = 0; base < n; base += kPrepThreads) {
    const uint32_t i = base + tid;
    uint32_t R = 0;
    if (i < n) {
      const uint8_t* st = streams[i];
      const uint64_t nbytes = stream_bytes[i];
      bool ok = (st != nullptr) && ((reinterpret_cast<uintptr_t>(st) & 15) == 0) && nbytes >= CVLC_STREAM_HEADER_BYTES;
      if (ok) {
        const uint4* hv = reinterpret_cast<const uint4*>(st);
        const uint4 h0 = __ldg(hv), h1 = __ldg(hv + 1), h3 = __ldg(hv + 3);
        const uint32_t magic = h0.x, ver_q_s = h0.y;
        const uint64_t sd = (uint64_t)h0.z | ((uint64_t)h0.w << 32);
        const uint32_t sR = h1.x, pb = h1.y, hb = h1.z;
        const double B = __longlong_as_double((long long)((uint64_t)h3.x | ((uint64_t)h3.y << 32)));
        ok = (magic == CVLC_STREAM_MAGIC) && ((ver_q_s & 0xFFFF) == 1) && (((ver_q_s >> 16) & 0xFF) <= CVLC_QUANT_QSGD) &&
             ((ver_q_s >> 24) == s) && (sd == d) && (pb != 0) && ((pb & 31) == 0) && (hb >= 80) && (hb < pb) &&
             (B >= 1.0) && (B < 1e300);
        if (ok) ok = ((uint64_t)CVLC_STREAM_HEADER_BYTES + (uint64_t)sR * (pb / 8) == nbytes);
        if (ok) {
          R = sR;
          const float wi = weights[i];
          if (!(wi > 0.0f) || __float_as_uint(wi) >= 0x7F800000u) set_status(status, CVLC_ERR_INVALID_ARG);  // weights are finite and positive
          coef[i] = (float)((double)wi / (W * B));
          meta[2 * i] = pb | ((ver_q_s >> 16) & 0xFF);  // packet bits are a multiple of 32: the quantizer rides below
          meta[2 * i + 1] = hb;
        }
      }
      if (!ok) {
        set_status(status, CVLC_ERR_BAD_STREAM);
        coef[i] = 0.0f;
        meta[2 * i] = 32;
        meta[2 * i + 1] = 0;
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
    if (tid == kPrepThreads - 1) s_carry = below + incl;
    __syncthreads();
  }
  if (tid == 0) {
    prefix[n] = s_carry;
    *total_pkts = s_carry;
  }
}

// K7b  out = 0 (when not accumulating): 4 bytes written per coordinate
__global__ void __launch_bounds__(256)
k_fill_zero(float* __restrict__ out, uint64_t d) {
  const uint64_t nvec = d >> 2;
  float4* ov = reinterpret_cast<float4*>(out);
  const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
  for (uint64_t v = (uint64_t)blockIdx.x * 256 + threadIdx.x; v < nvec; v += (uint64_t)gridDim.x * 256) ov[v] = z;
  if (blockIdx.x == 0 && threadIdx.x < (d & 3)) out[(nvec << 2) + threadIdx.x] = 0.f;
}

// A stream word is read once per window pass and should not push the accumulator's window out of the L2.
__device__ __forceinline__ uint64_t stream_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint32_t ld_stream(const uint32_t* p, uint64_t pol) {
  uint32_t v;
  asm volatile("ld.global.nc.L2::cache_hint.u32 %0, [%1], %2;" : "=r"(v) : "l"(p), "l"(pol));
  return v;
}

// asks for n floats into the L2, one request per 128-byte line
__global__ void __launch_bounds__(256)
k_prefetch_l2(const float* __restrict__ p, uint64_t n) {
  const uint64_t lines = (n * 4 + 127) / 128;
  const char* base = reinterpret_cast<const char*>(p);
  for (uint64_t l = (uint64_t)blockIdx.x * 256 + threadIdx.x; l < lines; l += (uint64_t)gridDim.x * 256)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(base + l * 128));
}

// The records of one staged packet whose width s + y is at most 32 bits: record j starts at bit H + j (s + y), so it
// lies in the words wi, wi + 1 of the packet and one funnel shift cuts it out.  WHOLE: the accumulator is one window.
template <bool QSGD, bool WHOLE>
__device__ __forceinline__ void decode_narrow(const uint32_t* __restrict__ sp, uint32_t P, uint32_t H, uint32_t wd, uint32_t s,
                                              uint32_t y, uint64_t d, uint64_t win_lo, uint64_t win_hi, double dlo, double step,
                                              float cf, float* __restrict__ out, int32_t* status, int lane) {
  const uint32_t rmask = (wd == 32) ? 0xFFFFFFFFu : ((1u << wd) - 1u);
  const uint32_t pmask = (1u << s) - 1u;  // s + y <= 32 and y >= 1: s <= 31
  const uint32_t level_mask = QSGD ? ((1u << (y - 1)) - 1u) : 0u;
  const uint32_t d32 = (d > 0xFFFFFFFFull) ? 0xFFFFFFFFu : (uint32_t)d;  // d <= 2^31
  for (uint32_t j = lane; j < P; j += 32) {
    const uint32_t bit = H + j * wd;
    const uint32_t wi = bit >> 5;
    const uint32_t rec = __funnelshift_r(sp[wi], sp[wi + 1], bit & 31u) & rmask;
    const uint32_t pid = rec & pmask, code = rec >> s;
    if (pid >= d32) {
      set_status(status, CVLC_ERR_BAD_STREAM);
      continue;
    }
    if (!WHOLE && (pid < win_lo || pid >= win_hi)) continue;
    float v;
    if (QSGD) {
      const float mag = (float)__dmul_rn((double)(code & level_mask), step);
      v = ((code >> (y - 1)) & 1u) ? -mag : mag;
    } else {
      v = (float)__dadd_rn(dlo, __dmul_rn((double)code, step));
    }
    atomicAdd(out + pid, cf * v);
  }
}

// K6  decode + dequantize + weighted scatter-accumulate, one warp per packet.  Only the records whose
// position lies in [win_lo, win_hi) are accumulated: an accumulator larger than the L2 is filled window by
// window (one launch each), so that the reductions stay in the L2 instead of becoming DRAM read-modify-writes.
__global__ void __launch_bounds__(kDecodeThreads)
k_decode(const uint8_t* const* __restrict__ streams, uint32_t n, uint64_t d, uint32_t s, float* __restrict__ out,
         unsigned char* ws, uint64_t win_lo, uint64_t win_hi) {
  extern __shared__ uint32_t s_prefix[];  // [n + 1]
  // a packet of up to kDecStageWords words is first copied to the warp's own shared-memory buffer with
  // coalesced, independent loads; the records are then cut out of shared memory (larger packets: out of global)
  __shared__ uint32_t s_pkt[kDecodeThreads / 32][kDecStageWords + 1];  // one word of slack: the narrow path reads word wi + 1
  uint32_t* sp = s_pkt[threadIdx.x >> 5];
  int32_t* status = reinterpret_cast<int32_t*>(ws + kDecWsStatus);
  const float* coef = reinterpret_cast<const float*>(ws + kDecWsCoef);
  const uint32_t* prefix = reinterpret_cast<const uint32_t*>(ws + dec_off_prefix(n));
  const uint32_t* meta = reinterpret_cast<const uint32_t*>(ws + dec_off_meta(n));
  // blocks that run later may see an error set by earlier ones: one thread reads the word, the whole block follows it
  __shared__ int s_err;
  if (threadIdx.x == 0) s_err = *reinterpret_cast<const volatile int32_t*>(status);
  for (uint32_t i = threadIdx.x; i <= n; i += kDecodeThreads) s_prefix[i] = prefix[i];
  __syncthreads();
  if (s_err != 0) return;
  const uint32_t total = s_prefix[n];
  const int lane = threadIdx.x & 31;
  const uint32_t warps_total = gridDim.x * (kDecodeThreads / 32);
  const unsigned long long pid_mask = (1ull << s) - 1ull;
  const uint64_t pol = stream_policy();

  for (uint32_t g = blockIdx.x * (kDecodeThreads / 32) + (threadIdx.x >> 5); g < total; g += warps_total) {
    // client of packet g: last c with prefix[c] <= g
    uint32_t lo_c = 0, hi_c = n;
    while (hi_c - lo_c > 1) {
      const uint32_t mid = (lo_c + hi_c) >> 1;
      if (s_prefix[mid] <= g) lo_c = mid; else hi_c = mid;
    }
    const uint32_t c = lo_c, r = g - s_prefix[c];
    const uint32_t pb = meta[2 * c] & ~31u, quantizer = meta[2 * c] & 31u, H = meta[2 * c + 1];
    const uint32_t n_words = pb >> 5;
    const uint32_t* pkt = reinterpret_cast<const uint32_t*>(streams[c] + CVLC_STREAM_HEADER_BYTES) + (size_t)r * n_words;
    const bool staged = n_words <= kDecStageWords;
    uint32_t y_prev = CVLC_MAX_CODE_BITS;
    if (r > 0) y_prev = (ld_stream(pkt - n_words, pol) >> 8) & 0xFF;
    __syncwarp();  // the previous packet's records have been read
    if (staged) {
      for (uint32_t w = lane; w < n_words; w += 32) sp[w] = ld_stream(pkt + w, pol);
      __syncwarp();
    }
    auto word = [&](uint32_t i) -> uint32_t { return staged ? sp[i] : ld_stream(pkt + i, pol); };
    const uint32_t w0 = word(0), w1 = word(1), w2 = word(2);
    const uint32_t ps = w0 & 0xFF, y = (w0 >> 8) & 0xFF;
    if (ps != s || y < 1 || y > CVLC_MAX_CODE_BITS || y > y_prev) {  // lengths never increase along a stream
      if (lane == 0) set_status(status, CVLC_ERR_BAD_STREAM);
      continue;
    }
    const float lo = __uint_as_float((w0 >> 16) | (w1 << 16));
    const float hi = __uint_as_float((w1 >> 16) | (w2 << 16));
    const uint32_t wd = s + y;
    const uint32_t P = (pb - H) / wd;
    const bool qsgd = quantizer == CVLC_QUANT_QSGD;
    // QSGD: the first centroid field is the packet's l2-norm (finite, not negative); a code is the sign
    // bit above a level of 2^(y-1) - 1 steps, so one bit is not a code
    if (qsgd && (y < 2 || __float_as_uint(lo) >= 0x7F800000u)) {
      if (lane == 0) set_status(status, CVLC_ERR_BAD_STREAM);
      continue;
    }
    // PQ: minimum and maximum are finite and ordered
    if (!qsgd && ((__float_as_uint(lo) & 0x7FFFFFFFu) >= 0x7F800000u || (__float_as_uint(hi) & 0x7FFFFFFFu) >= 0x7F800000u || lo > hi)) {
      if (lane == 0) set_status(status, CVLC_ERR_BAD_STREAM);
      continue;
    }
    const uint32_t level_mask = qsgd ? (uint32_t)((1ull << (y - 1)) - 1ull) : 0u;
    const double dlo = qsgd ? 0.0 : (double)lo;
    const double step = qsgd ? __ddiv_rn((double)lo, (double)level_mask)
                             : ((hi == lo) ? 0.0 : __ddiv_rn(__dsub_rn((double)hi, dlo), (double)((1ull << y) - 1ull)));
    const float cf = coef[c];
    const unsigned long long code_mask = (1ull << y) - 1ull;
    if (staged && wd <= 32) {
      // the usual case: a record fits one 32-bit funnel shift of two staged words
      const bool whole = (win_lo == 0 && win_hi >= d);
      if (qsgd)
        whole ? decode_narrow<true, true>(sp, P, H, wd, s, y, d, win_lo, win_hi, dlo, step, cf, out, status, lane)
              : decode_narrow<true, false>(sp, P, H, wd, s, y, d, win_lo, win_hi, dlo, step, cf, out, status, lane);
      else
        whole ? decode_narrow<false, true>(sp, P, H, wd, s, y, d, win_lo, win_hi, dlo, step, cf, out, status, lane)
              : decode_narrow<false, false>(sp, P, H, wd, s, y, d, win_lo, win_hi, dlo, step, cf, out, status, lane);
      continue;
    }
    for (uint32_t j = lane; j < P; j += 32) {
      const uint32_t bit = H + j * wd;
      const uint32_t wi = bit >> 5, sh = bit & 31;
      // a record of up to 63 bits starting at bit sh of word wi spans at most three words
      const unsigned long long a = word(wi);
      const unsigned long long b = (wi + 1 < n_words) ? word(wi + 1) : 0u;
      unsigned long long rec = (a | (b << 32)) >> sh;
      if (sh + wd > 64) {
        const unsigned long long c2 = (wi + 2 < n_words) ? word(wi + 2) : 0u;
        rec |= c2 << (64 - sh);
      }
      const unsigned long long pid = rec & pid_mask;
      const uint32_t code = (uint32_t)((rec >> s) & code_mask);
      if (pid >= d) {
        set_status(status, CVLC_ERR_BAD_STREAM);
        continue;
      }
      if (pid < win_lo || pid >= win_hi) continue;
      float v;
      if (qsgd) {
        const float mag = (float)__dmul_rn((double)(code & level_mask), step);
        v = ((code >> (y - 1)) & 1u) ? -mag : mag;
      } else {
        v = (float)__dadd_rn(dlo, __dmul_rn((double)code, step));
      }
      atomicAdd(out + pid, cf * v);
    }
  }
}

cudaError_t launch_decode(const uint8_t* const* streams, const uint64_t* stream_bytes, const float* weights,
                          uint32_t n, double weight_total, uint64_t d, uint32_t s, float* out, int accumulate,
                          void* ws, cudaStream_t st) {
  unsigned char* w = static_cast<unsigned char*>(ws);
  { LaunchScope ls(kKDecodePrepare, st); k_decode_prepare<<<1, kPrepThreads, 0, st>>>(streams, stream_bytes, weights, n, weight_total, d, s, w); }
  // Windows of equal size (a multiple of 1024 coordinates), none above kDecodeWindow.  Each window is brought
  // into the L2 right before its decode launch, by the zero fill or, when accumulating, by a prefetch: a
  // reduction that misses the L2 is a DRAM read-modify-write.
  const uint64_t n_win = (d + kDecodeWindow - 1) / kDecodeWindow;
  const uint64_t win = (((d + n_win - 1) / n_win) + 1023) & ~(uint64_t)1023;
  for (uint64_t lo = 0; lo < d; lo += win) {
    const uint64_t hi = lo + win < d ? lo + win : d;
    const uint64_t want = ((hi - lo) / 4 + 255) / 256;
    const int grid = (int)(want < (uint64_t)(8 * kNumSM) ? (want ? want : 1) : 8 * kNumSM);
    if (!accumulate) {
      LaunchScope ls(kKFillZero, st);
      k_fill_zero<<<grid, 256, 0, st>>>(out + lo, hi - lo);
    } else if (n_win > 1) {
      LaunchScope ls(kKPrefetchL2, st);
      k_prefetch_l2<<<grid, 256, 0, st>>>(out + lo, hi - lo);
    }
    LaunchScope ls(kKDecode, st);
    k_decode<<<8 * kNumSM, kDecodeThreads, ((size_t)n + 1) * 4, st>>>(streams, n, d, s, out, w, lo, hi);
  }
  return cudaGetLastError();
}

cudaError_t launch_fill_zero(float* out, uint64_t d, cudaStream_t st) {
  const uint64_t want = (d / 4 + 255) / 256;
  const int grid = (int)(want < (uint64_t)(8 * kNumSM) ? (want ? want : 1) : 8 * kNumSM);
  LaunchScope ls(kKFillZero, st);
  k_fill_zero<<<grid, 256, 0, st>>>(out, d);
  return cudaGetLastError();
}

// K8  model <- model - aggregate (Section III, step 3); nothing is touched after a decode error
__global__ void __launch_bounds__(256)
k_apply(float* __restrict__ model, const float* __restrict__ agg, uint64_t d, const unsigned char* dec_ws) {
  if (*reinterpret_cast<const int32_t*>(dec_ws + kDecWsStatus) != 0) return;
  const uint64_t nvec = d >> 2;
  float4* mv = reinterpret_cast<float4*>(model);
  const float4* av = reinterpret_cast<const float4*>(agg);
  for (uint64_t v = (uint64_t)blockIdx.x * 256 + threadIdx.x; v < nvec; v += (uint64_t)gridDim.x * 256) {
    float4 m = mv[v];
    const float4 a = av[v];
    m.x = __fsub_rn(m.x, a.x);
    m.y = __fsub_rn(m.y, a.y);
    m.z = __fsub_rn(m.z, a.z);
    m.w = __fsub_rn(m.w, a.w);
    mv[v] = m;
  }
  if (blockIdx.x == 0 && threadIdx.x < (d & 3)) {
    const uint64_t i = (nvec << 2) + threadIdx.x;
    model[i] = __fsub_rn(model[i], agg[i]);
  }
}

cudaError_t launch_apply(float* model, const float* agg, uint64_t d, const void* dec_ws, cudaStream_t st) {
  const uint64_t nvec = d >> 2;
  const uint64_t want = (nvec + 255) / 256;
  const int grid = (int)(want < (uint64_t)(8 * kNumSM) ? (want ? want : 1) : 8 * kNumSM);
  LaunchScope ls(kKApply, st);
  k_apply<<<grid, 256, 0, st>>>(model, agg, d, static_cast<const unsigned char*>(dec_ws));
  return cudaGetLastError();
}

}  // namespace cvlc

// ===================================================================================
// Decode-aggregate for callers that cannot allocate device memory
// ===================================================================================

namespace cvlc {

// Scratch of cvlc_decode_aggregate_noalloc: the decode workspace for up to
// CVLC_NOALLOC_MAX_CLIENTS clients (a few KB), resident in every GPU that loads the
// library until the process exits.
constexpr size_t kNoAllocScratchBytes = dec_ws_bytes(CVLC_NOALLOC_MAX_CLIENTS);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// copies the status word of the scratch to the caller's word (device code names the array directly)
__global__ void k_noalloc_publish_status(int32_t* status_out) {
  *status_out = *reinterpret_cast<const int32_t*>(g_noalloc_scratch + kDecWsStatus);
}

// Device address of the scratch on the current device.  In host code the array's name is only a
// handle for the runtime, so the address is asked for once per device and cached.
static cudaError_t noalloc_scratch_address(void** out) {
  static void* cached[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!cached[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    cached[dev] = ptr;
  }
  *out = cached[dev];
  return cudaSuccess;
}

}  // namespace cvlc

extern "C" int cvlc_decode_aggregate_noalloc(const uint8_t* const* streams_dev, const uint64_t* stream_bytes_dev,
                                             const float* weights_dev, uint32_t n_clients, double weight_total,
                                             uint64_t d, float* out_dev, int accumulate, int32_t* status_dev,
                                             void* cuda_stream) {
  using namespace cvlc;
  if (n_clients == 0) return CVLC_ERR_INVALID_ARG;
  if (n_clients > CVLC_NOALLOC_MAX_CLIENTS) return CVLC_ERR_WORKSPACE_TOO_SMALL;  // beyond the built-in scratch
  if (d < 2 || d > (1ull << 31)) return CVLC_ERR_INVALID_ARG;
  if (!(weight_total >= 0.0) || !(weight_total < 1e300)) return CVLC_ERR_INVALID_ARG;
  auto aligned = [](const void* p, size_t a) { return p && (reinterpret_cast<uintptr_t>(p) % a) == 0; };
  if (!aligned(streams_dev, 8) || !aligned(stream_bytes_dev, 8) || !aligned(weights_dev, 4) || !aligned(out_dev, 16) ||
      !aligned(status_dev, 4))
    return CVLC_ERR_INVALID_ARG;
  void* scratch = nullptr;
  if (noalloc_scratch_address(&scratch) != cudaSuccess) return CVLC_ERR_CUDA;
  uint32_t s = 1;
  while ((1ull << s) < d) ++s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // k_decode_prepare resets the status word and rewrites every table entry it later reads,
  // so nothing of the previous call's contents is used
  if (launch_decode(streams_dev, stream_bytes_dev, weights_dev, n_clients, weight_total, d, s, out_dev,
                    accumulate ? 1 : 0, scratch, st) != cudaSuccess)
    return CVLC_ERR_CUDA;
  {
    LaunchScope ls(kKNoallocStatus, st);
    k_noalloc_publish_status<<<1, 1, 0, st>>>(status_dev);
  }
  return cudaGetLastError() == cudaSuccess ? CVLC_OK : CVLC_ERR_CUDA;
}

