// Encoding kernels (Algorithm 1, steps 15-17): top-k candidate selection by the
// plan's histogram threshold, stable LSD radix ranking of the candidates by |x|,
// per-packet minimum/maximum, PQ stochastic quantization with Philox4x32-10 and
// bit packing of (position ID, centroid ID) pairs into fixed-size packets (Fig. 2).
#include "cvlc_common.cuh"

namespace cvlc {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr unsigned long long kFlagAgg = 1ull << 62;     // tile aggregate published
constexpr unsigned long long kFlagPrefix = 2ull << 62;  // inclusive prefix published
constexpr unsigned long long kFlagMask = 3ull << 62;
constexpr unsigned long long kValMask = ~kFlagMask;
constexpr int kMaxPolls = 1 << 20;  // bounded wait of the look-back; then DEVICE_TIMEOUT

__device__ __forceinline__ unsigned long long ld_relaxed(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Waits (bounded) until a look-back state word carries a flag.  Returns 0 after a timeout.
__device__ __forceinline__ unsigned long long wait_state(const unsigned long long* p, int32_t* status) {
  unsigned long long v = ld_relaxed(p);
  int polls = 0;
  while ((v & kFlagMask) == 0) {
    if (++polls > kMaxPolls) {
      set_status(status, CVLC_ERR_DEVICE_TIMEOUT);
      return 0;
    }
    if (polls > 64) __nanosleep(64);
    v = ld_relaxed(p);
  }
  return v;
}

// ===================================================================================
// K0  workspace reset + plan validation
// ===================================================================================

__global__ void k_encode_init(unsigned char* ws, const cvlc_plan_t* __restrict__ plan, EncLayout L, uint64_t d,
                              uint32_t s, uint32_t R) {
  const size_t gtid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t gstride = (size_t)gridDim.x * blockDim.x;
  unsigned long long* w64 = reinterpret_cast<unsigned long long*>(ws);
  const size_t n_head = L.off_sort_state / 8;  // header, digit histograms, selection tile states
  for (size_t i = gtid; i < n_head; i += gstride) w64[i] = 0ull;
  unsigned long long nc = plan->n_candidates;
  if (nc > d) nc = d;
  const size_t tiles = (size_t)((nc + kSortTile - 1) / kSortTile);
  const size_t per_pass = tiles * 256;
  for (int p = 0; p < kSortPasses; ++p) {
    unsigned long long* st = reinterpret_cast<unsigned long long*>(ws + L.off_sort_state) + (size_t)p * L.max_sort_tiles * 256;
    for (size_t i = gtid; i < per_pass; i += gstride) st[i] = 0ull;
  }
  if (gtid == 0) {
    // the plan must belong to these parameters (status is written after the zeroing above
    // by the same thread, so it survives)
    int32_t bad = 0;
    if (plan->status != CVLC_OK) bad = plan->status;
    unsigned long long k = 0, nsum = 0;
    for (int y = 1; y <= CVLC_MAX_CODE_BITS; ++y) {
      k += (unsigned long long)plan->n_y[y] * plan->cap[y];
      nsum += plan->n_y[y];
    }
    if (!bad && (plan->s != s || plan->R != R || nsum != R || k != plan->k || k == 0 || k > plan->n_candidates ||
                 plan->n_candidates > d || plan->thresh_bin >= CVLC_HIST_BINS))
      bad = CVLC_ERR_PLAN_MISMATCH;
    if (bad) reinterpret_cast<EncHeader*>(ws)->status = bad;
  }
}

// ===================================================================================
// K3  threshold selection + order-preserving compaction (single pass, decoupled look-back)
// ===================================================================================
// Emits (key << 32 | sign << 31 | index) for every coordinate whose histogram bin is at or
// above the plan's threshold bin, in ascending index order.  4 bytes read per coordinate.

__global__ void __launch_bounds__(kSelectThreads)
k_select(const float* __restrict__ x, uint64_t d, const cvlc_plan_t* __restrict__ plan, EncHeader* hdr,
         unsigned long long* tile_state, uint64_t n_tiles, unsigned long long* __restrict__ out, uint64_t out_capacity) {
  __shared__ uint32_t s_tile;
  __shared__ unsigned long long s_warp_incl[kSelectThreads / 32];
  __shared__ unsigned long long s_tile_excl;
  if (hdr->status != 0) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t thresh = plan->thresh_bin << 19;
  const float4* xv = reinterpret_cast<const float4*>(x);

  while (true) {
    if (tid == 0) s_tile = atomicAdd(&hdr->select_ticket, 1u);
    __syncthreads();
    const uint64_t tile = s_tile;
    if (tile >= n_tiles) break;
    const uint64_t base_vec = tile * (uint64_t)(kSelectThreads * kSelectVecPerThread);

    uint32_t bits[kSelectVecPerThread][4];
    uint32_t mask[kSelectVecPerThread];
#pragma unroll
    for (int v = 0; v < kSelectVecPerThread; ++v) {
      const uint64_t vi = base_vec + (uint64_t)v * kSelectThreads + tid;
      const uint64_t e0 = vi * 4;
      uint32_t valid = 0;
      if (e0 + 3 < d) {
        const float4 f = __ldg(xv + vi);
        bits[v][0] = __float_as_uint(f.x);
        bits[v][1] = __float_as_uint(f.y);
        bits[v][2] = __float_as_uint(f.z);
        bits[v][3] = __float_as_uint(f.w);
        valid = 0xF;
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          bits[v][c] = 0;
          if (e0 + c < d) {
            bits[v][c] = __float_as_uint(x[e0 + c]);
            valid |= 1u << c;
          }
        }
      }
      uint32_t m = 0;
#pragma unroll
      for (int c = 0; c < 4; ++c) m |= (((bits[v][c] & 0x7FFFFFFFu) >= thresh) ? 1u : 0u) << c;
      mask[v] = m & valid;
    }
    // block scan of the four per-vector counts, packed 16 bits each (tile totals <= 1024)
    unsigned long long packed = 0;
#pragma unroll
    for (int v = 0; v < kSelectVecPerThread; ++v) packed |= (unsigned long long)__popc(mask[v]) << (16 * v);
    unsigned long long incl = packed;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned long long o = __shfl_up_sync(kFull, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) s_warp_incl[warp] = incl;
    __syncthreads();
    unsigned long long below = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kSelectThreads / 32; ++w) {
      const unsigned long long t = s_warp_incl[w];
      if (w < warp) below += t;
      tot += t;
    }
    const unsigned long long excl = below + incl - packed;  // per-vector exclusive counts over threads
    const uint32_t tile_total = (uint32_t)((tot & 0xFFFF) + ((tot >> 16) & 0xFFFF) + ((tot >> 32) & 0xFFFF) + (tot >> 48));

    // decoupled look-back over the preceding tiles (warp 0, 32 tiles per step)
    if (warp == 0) {
      if (lane == 0) st_relaxed(tile_state + tile, (tile == 0 ? kFlagPrefix : kFlagAgg) | tile_total);
      unsigned long long run = 0;
      if (tile > 0) {
        long long base = (long long)tile - 1;
        while (true) {
          const long long idx = base - lane;
          unsigned long long sv = kFlagPrefix;  // before tile 0: empty prefix
          if (idx >= 0) sv = wait_state(tile_state + idx, &hdr->status);
          const unsigned timed_out = __ballot_sync(kFull, sv == 0);
          const unsigned is_prefix = __ballot_sync(kFull, (sv & kFlagMask) == kFlagPrefix);
          if (timed_out) break;
          unsigned long long val = sv & kValMask;
          if (is_prefix) {
            const int firstp = __ffs(is_prefix) - 1;
            if (lane > firstp) val = 0;
          }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) val += __shfl_xor_sync(kFull, val, off);
          run += val;
          if (is_prefix) break;
          base -= 32;
        }
        if (lane == 0) st_relaxed(tile_state + tile, kFlagPrefix | (run + tile_total));
      }
      if (lane == 0) {
        s_tile_excl = run;
        if (tile == n_tiles - 1) {
          hdr->n_selected = run + tile_total;
          if (run + tile_total != plan->n_candidates) set_status(&hdr->status, CVLC_ERR_PLAN_MISMATCH);
        }
      }
    }
    __syncthreads();
    unsigned long long pos = s_tile_excl;
    unsigned long long vec_base = 0;
#pragma unroll
    for (int v = 0; v < kSelectVecPerThread; ++v) {
      unsigned long long o = pos + vec_base + ((excl >> (16 * v)) & 0xFFFF);
      const uint64_t e0 = (base_vec + (uint64_t)v * kSelectThreads + tid) * 4;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (mask[v] & (1u << c)) {
          const uint32_t b = bits[v][c];
          const unsigned long long pair = ((unsigned long long)(b & 0x7FFFFFFFu) << 32) | (unsigned long long)(b & 0x80000000u) |
                                          (unsigned long long)(e0 + c);
          if (o < out_capacity) out[o] = pair;
          ++o;
        }
      }
      vec_base += (tot >> (16 * v)) & 0xFFFF;
    }
    __syncthreads();  // s_tile / s_tile_excl are reused by the next tile
  }
}

// ===================================================================================
// K4  stable LSD radix ranking of the candidates, |x| descending (ties keep ascending index)
// ===================================================================================
// Key digit = digit of (0x7FFFFFFF - key): 8, 8, 8, 7 bits.  One histogram kernel for all
// four digits, then one single-pass kernel per digit (decoupled look-back per digit value).
// A pass whose digit is the same for every candidate is skipped; which buffer holds the
// data after pass q therefore follows from the digit histograms alone.

__device__ __forceinline__ uint32_t sort_digit(unsigned long long pair, int pass) {
  const uint32_t inv = 0x7FFFFFFFu - (uint32_t)(pair >> 32);
  return (inv >> (8 * pass)) & 0xFFu;
}

__global__ void __launch_bounds__(256)
k_sort_hist(const unsigned long long* __restrict__ in, const cvlc_plan_t* __restrict__ plan, const EncHeader* hdr,
            unsigned long long* __restrict__ ghist) {
  __shared__ uint32_t sh[kSortPasses * 256];
  if (hdr->status != 0) return;
  for (int i = threadIdx.x; i < kSortPasses * 256; i += 256) sh[i] = 0;
  __syncthreads();
  const unsigned long long n = plan->n_candidates;
  for (unsigned long long i = (unsigned long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (unsigned long long)gridDim.x * 256) {
    const unsigned long long pair = in[i];
#pragma unroll
    for (int p = 0; p < kSortPasses; ++p) atomicAdd(&sh[p * 256 + sort_digit(pair, p)], 1u);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kSortPasses * 256; i += 256)
    if (sh[i]) atomicAdd(ghist + i, (unsigned long long)sh[i]);
}

// number of passes before `pass` that moved data, and whether `pass` itself is skipped
__device__ __forceinline__ void sort_pass_parity(const unsigned long long* ghist, unsigned long long n, int pass, int* flips,
                                                 bool* skip) {
  int f = 0;
  bool sk = false;
  for (int q = 0; q <= pass; ++q) {
    int hit = 0;
    for (int b = threadIdx.x; b < 256; b += blockDim.x) hit |= (ghist[q * 256 + b] == n);
    const int trivial = __syncthreads_or(hit);
    if (q < pass)
      f += trivial ? 0 : 1;
    else
      sk = trivial != 0;
  }
  *flips = f;
  *skip = sk;
}

__global__ void __launch_bounds__(kSortThreads)
k_sort_pass(int pass, unsigned long long* buf_a, unsigned long long* buf_b, const cvlc_plan_t* __restrict__ plan, EncHeader* hdr,
            const unsigned long long* __restrict__ ghist, unsigned long long* state /* [tiles][256] */) {
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_wc[kSortThreads / 32][256];  // per-warp digit counters -> per-warp offsets
  __shared__ unsigned long long s_base[256];         // global position of this tile's first item per digit
  __shared__ unsigned long long s_scan[256];
  if (hdr->status != 0) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned long long n = plan->n_candidates;
  const unsigned long long n_tiles = (n + kSortTile - 1) / kSortTile;
  int flips;
  bool skip;
  sort_pass_parity(ghist, n, pass, &flips, &skip);
  if (skip) return;
  const unsigned long long* src = (flips & 1) ? buf_b : buf_a;
  unsigned long long* dst = (flips & 1) ? buf_a : buf_b;

  // exclusive scan of this digit's histogram: first position of every digit value
  {
    const unsigned long long c = ghist[pass * 256 + tid];
    unsigned long long incl = c;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned long long o = __shfl_up_sync(kFull, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    unsigned long long below = 0;
    for (int w = 0; w < warp; ++w) below += s_scan[w];
    __syncthreads();
    s_scan[tid] = below + incl - c;
  }
  __syncthreads();
  const unsigned long long gbase = s_scan[tid];
  const unsigned lanemask_lt = (1u << lane) - 1u;

  while (true) {
    if (tid == 0) s_tile = atomicAdd(&hdr->sort_ticket[pass], 1u);
    for (int w = 0; w < kSortThreads / 32; ++w) s_wc[w][tid] = 0;
    __syncthreads();
    const unsigned long long tile = s_tile;
    if (tile >= n_tiles) break;

    unsigned long long item[kSortItemsPerThread];
    uint32_t rank[kSortItemsPerThread];
    const unsigned long long first = tile * kSortTile + (unsigned long long)warp * (32 * kSortItemsPerThread);
#pragma unroll
    for (int i = 0; i < kSortItemsPerThread; ++i) {
      const unsigned long long idx = first + i * 32 + lane;
      item[i] = (idx < n) ? src[idx] : ~0ull;
    }
    // stable rank inside the warp: items in (i, lane) order
#pragma unroll
    for (int i = 0; i < kSortItemsPerThread; ++i) {
      const bool valid = (first + i * 32 + lane) < n;
      const uint32_t dig = valid ? sort_digit(item[i], pass) : 0xFFFFFFFFu;
      const unsigned peers = __match_any_sync(kFull, dig);
      const int leader = __ffs(peers) - 1;
      uint32_t pre = 0;
      if (valid && lane == leader) pre = s_wc[warp][dig];
      pre = __shfl_sync(kFull, pre, leader);
      rank[i] = pre + __popc(peers & lanemask_lt);
      if (valid && lane == leader) s_wc[warp][dig] = pre + __popc(peers);
      __syncwarp();
    }
    __syncthreads();
    // thread = digit value: offsets of the warps inside the tile, tile count, look-back
    {
      uint32_t tot = 0;
#pragma unroll
      for (int w = 0; w < kSortThreads / 32; ++w) {
        const uint32_t c = s_wc[w][tid];
        s_wc[w][tid] = tot;
        tot += c;
      }
      unsigned long long* my_state = state + tile * 256 + tid;
      st_relaxed(my_state, (tile == 0 ? kFlagPrefix : kFlagAgg) | tot);
      unsigned long long run = 0;
      if (tile > 0) {
        for (long long t = (long long)tile - 1; t >= 0; --t) {
          const unsigned long long sv = wait_state(state + (unsigned long long)t * 256 + tid, &hdr->status);
          if (sv == 0) break;  // timed out: status is set, results are void
          run += sv & kValMask;
          if ((sv & kFlagMask) == kFlagPrefix) break;
        }
        st_relaxed(my_state, kFlagPrefix | (run + tot));
      }
      s_base[tid] = gbase + run;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kSortItemsPerThread; ++i) {
      if ((first + i * 32 + lane) < n) {
        const uint32_t dig = sort_digit(item[i], pass);
        const unsigned long long o = s_base[dig] + s_wc[warp][dig] + rank[i];
        if (o < n) dst[o] = item[i];
      }
    }
    __syncthreads();
  }
}

// ===================================================================================
// K5  per-packet min/max, PQ stochastic quantization, bit packing
// ===================================================================================
// One CTA per packet.  Packet r (longest codes first) holds ranks [Z, Z + cap(y_r)).

constexpr int kPackThreads = 128;

__global__ void __launch_bounds__(kPackThreads)
k_pack(const unsigned long long* __restrict__ buf_a, const unsigned long long* __restrict__ buf_b,
       const cvlc_plan_t* __restrict__ plan, const EncHeader* hdr, const unsigned long long* __restrict__ ghist,
       const __grid_constant__ cvlc_params prm, uint32_t s, uint32_t R, uint32_t* __restrict__ stream_words) {
  extern __shared__ unsigned long long recs[];  // [cap(1)]
  __shared__ float s_red[2][kPackThreads / 32];
  __shared__ uint32_t s_y;
  __shared__ unsigned long long s_Z;
  if (hdr->status != 0) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t r = blockIdx.x;

  int flips;
  bool skip;
  sort_pass_parity(ghist, plan->n_candidates, kSortPasses - 1, &flips, &skip);
  if (!skip) flips += 1;
  const unsigned long long* sorted = (flips & 1) ? buf_b : buf_a;

  if (tid == 0) {
    unsigned long long cum = 0, Z = 0;
    uint32_t yy = 0;
    for (int y = CVLC_MAX_CODE_BITS; y >= 1; --y) {
      const unsigned long long ny = plan->n_y[y];
      if (r < cum + ny) {
        yy = (uint32_t)y;
        Z += (r - cum) * plan->cap[y];
        break;
      }
      cum += ny;
      Z += ny * plan->cap[y];
    }
    s_y = yy;
    s_Z = Z;
  }
  __syncthreads();
  const uint32_t y = s_y;
  if (y == 0) return;
  const unsigned long long Z = s_Z;
  const uint32_t P = plan->cap[y];
  const uint32_t wd = s + y;

  // minimum / maximum of the packet's signed values (the centroid distribution of PQ)
  float vmin = CUDART_INF_F, vmax = -CUDART_INF_F;
  for (uint32_t j = tid; j < P; j += kPackThreads) {
    const unsigned long long pair = sorted[Z + j];
    recs[j] = pair;
    const uint32_t key = (uint32_t)(pair >> 32);
    const uint32_t b = key ? (key | ((uint32_t)pair & 0x80000000u)) : 0u;  // -0 is stored as +0
    const float v = __uint_as_float(b);
    vmin = fminf(vmin, v);
    vmax = fmaxf(vmax, v);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    vmin = fminf(vmin, __shfl_xor_sync(kFull, vmin, off));
    vmax = fmaxf(vmax, __shfl_xor_sync(kFull, vmax, off));
  }
  if (lane == 0) {
    s_red[0][warp] = vmin;
    s_red[1][warp] = vmax;
  }
  __syncthreads();
  float lo = s_red[0][0], hi = s_red[1][0];
#pragma unroll
  for (int w = 1; w < kPackThreads / 32; ++w) {
    lo = fminf(lo, s_red[0][w]);
    hi = fmaxf(hi, s_red[1][w]);
  }

  // stochastic rounding onto the 2^y uniform centroids of [lo, hi]
  const double L = (double)((1ull << y) - 1ull);
  const double dlo = (double)lo;
  const double den = __dsub_rn((double)hi, dlo);
  for (uint32_t j = tid; j < P; j += kPackThreads) {
    const unsigned long long pair = recs[j];
    const uint32_t key = (uint32_t)(pair >> 32);
    const uint32_t pid = (uint32_t)pair & 0x7FFFFFFFu;
    const uint32_t b = key ? (key | ((uint32_t)pair & 0x80000000u)) : 0u;
    uint32_t code = 0;
    if (hi != lo) {
      const double t = __dmul_rn(__ddiv_rn(__dsub_rn((double)__uint_as_float(b), dlo), den), L);
      double j0 = floor(t);
      if (j0 > L) j0 = L;
      const double frac = __dsub_rn(t, j0);
      const double u = __dmul_rn((double)philox_coord(prm.seed, prm.client_id, prm.round, pid), 1.0 / 4294967296.0);
      code = __double2uint_rz(j0) + ((u < frac) ? 1u : 0u);
    }
    recs[j] = (unsigned long long)pid | ((unsigned long long)code << s);
  }
  __syncthreads();

  // gather the packet's 32-bit words: header {s, y, lo, hi}, then records of wd bits from bit H
  const uint32_t H = prm.header_bits;
  const uint32_t n_words = prm.packet_bits / 32;
  uint32_t* pkt = stream_words + CVLC_STREAM_HEADER_BYTES / 4 + (size_t)r * n_words;
  const uint32_t blo = __float_as_uint(lo), bhi = __float_as_uint(hi);
  const uint32_t payload_end = H + P * wd;
  for (uint32_t w = tid; w < n_words; w += kPackThreads) {
    const uint32_t bit0 = w * 32;
    uint32_t val = 0;
    if (w == 0) val = s | (y << 8) | (blo << 16);
    if (w == 1) val = (blo >> 16) | (bhi << 16);
    if (w == 2) val = bhi >> 16;
    if (bit0 + 32 > H && bit0 < payload_end) {
      uint32_t j = (bit0 > H) ? (bit0 - H) / wd : 0u;
      for (; j < P; ++j) {
        const int shift = (int)(H + j * wd) - (int)bit0;  // position of the record's bit 0 in this word
        if (shift >= 32) break;
        const unsigned long long rec = recs[j];
        val |= (shift >= 0) ? (uint32_t)(rec << shift) : (uint32_t)(rec >> (-shift));
      }
    }
    pkt[w] = val;
  }

  // global header (64 bytes), written once
  if (r == 0 && tid < 16) {
    uint32_t v = 0;
    const unsigned long long Bbits = (unsigned long long)__double_as_longlong(prm.scale_B);
    const unsigned long long k = plan->k;
    switch (tid) {
      case 0: v = CVLC_STREAM_MAGIC; break;
      case 1: v = 1u | (prm.quantizer << 16) | (s << 24); break;
      case 2: v = (uint32_t)prm.d; break;
      case 3: v = (uint32_t)(prm.d >> 32); break;
      case 4: v = R; break;
      case 5: v = prm.packet_bits; break;
      case 6: v = prm.header_bits; break;
      case 7: v = prm.client_id; break;
      case 8: v = (uint32_t)prm.seed; break;
      case 9: v = (uint32_t)(prm.seed >> 32); break;
      case 10: v = prm.round; break;
      case 11: v = 0; break;
      case 12: v = (uint32_t)Bbits; break;
      case 13: v = (uint32_t)(Bbits >> 32); break;
      case 14: v = (uint32_t)k; break;
      default: v = (uint32_t)(k >> 32); break;
    }
    stream_words[tid] = v;
  }
}

// ===================================================================================
// launcher
// ===================================================================================

cudaError_t launch_encode(const float* x, const cvlc_params& p, uint32_t s, uint32_t R, uint32_t max_cap,
                          const cvlc_plan_t* plan, uint8_t* stream, void* ws, cudaStream_t st) {
  static bool attr_done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const size_t pack_smem = (size_t)max_cap * 8;
  if (dev >= 0 && dev < 64 && !attr_done[dev]) {
    e = cudaFuncSetAttribute(k_pack, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  const EncLayout L = enc_layout(p.d);
  unsigned char* w = static_cast<unsigned char*>(ws);
  EncHeader* hdr = reinterpret_cast<EncHeader*>(w);
  unsigned long long* ghist = reinterpret_cast<unsigned long long*>(w + kEncWsSortHist);
  unsigned long long* sel_state = reinterpret_cast<unsigned long long*>(w + L.off_select_state);
  unsigned long long* sort_state = reinterpret_cast<unsigned long long*>(w + L.off_sort_state);
  unsigned long long* buf_a = reinterpret_cast<unsigned long long*>(w + L.off_buf_a);
  unsigned long long* buf_b = reinterpret_cast<unsigned long long*>(w + L.off_buf_b);

  { LaunchScope ls(kKEncodeInit, st); k_encode_init<<<2 * kNumSM, 256, 0, st>>>(w, plan, L, p.d, s, R); }
  {
    const uint64_t want = L.n_select_tiles;
    const int grid = (int)(want < (uint64_t)(8 * kNumSM) ? want : 8 * kNumSM);
    LaunchScope ls(kKSelect, st);
    k_select<<<grid, kSelectThreads, 0, st>>>(x, p.d, plan, hdr, sel_state, L.n_select_tiles, buf_a, p.d);
  }
  {
    const uint64_t want = L.max_sort_tiles;
    const int grid = (int)(want < (uint64_t)(4 * kNumSM) ? want : 4 * kNumSM);
    { LaunchScope ls(kKSortHist, st); k_sort_hist<<<grid, 256, 0, st>>>(buf_a, plan, hdr, ghist); }
    for (int pass = 0; pass < kSortPasses; ++pass) {
      LaunchScope ls(kKSortPass, st);
      k_sort_pass<<<grid, kSortThreads, 0, st>>>(pass, buf_a, buf_b, plan, hdr, ghist,
                                                 sort_state + (size_t)pass * L.max_sort_tiles * 256);
    }
  }
  { LaunchScope ls(kKPack, st); k_pack<<<R, kPackThreads, pack_smem, st>>>(buf_a, buf_b, plan, hdr, ghist, p, s, R, reinterpret_cast<uint32_t*>(stream)); }
  return cudaGetLastError();
}

}  // namespace cvlc
