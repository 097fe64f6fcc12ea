// Planning kernels: magnitude histogram (Algorithm 1, step 1), the exponent fit of Definition 1 with the
// selection threshold, and the code-length tuning by atomic operations on Eq. (5) (Algorithm 1 steps 2-14),
// one CTA per client, run once per distinct (exponent, scale) of a batch.
//
// The planner's floating point is IEEE binary64 with every multiply and add
// rounded separately (the *_rn intrinsics keep the compiler from contracting
// them), in a fixed order, so that its decisions do not depend on the machine.
#include "cvlc_common.cuh"

namespace cvlc {

// ===================================================================================
// K1  magnitude histogram: h[key >> 19], key = bits(|x|); HBM-bound, 4 bytes / coordinate
// ===================================================================================

constexpr int kHistThreads = kStreamThreads;
constexpr int kHistSub = 4;  // shared sub-histograms per block (64 KB)

// The clients' updates are treated as one concatenated array of units (a unit = one float4,
// plus one ragged-tail unit per client) that is cut into equal contiguous chunks, one per
// block, so the load is even whatever the number of clients; a block that crosses a client
// boundary merges its shared histogram into that client's global one and starts afresh.

// counts the four magnitude keys of a float4; returns the largest of them
__device__ __forceinline__ uint32_t hist_add4(uint32_t* my, const float4 a) {
  const uint32_t k0 = __float_as_uint(a.x) & 0x7FFFFFFFu, k1 = __float_as_uint(a.y) & 0x7FFFFFFFu;
  const uint32_t k2 = __float_as_uint(a.z) & 0x7FFFFFFFu, k3 = __float_as_uint(a.w) & 0x7FFFFFFFu;
  atomicAdd(my + (k0 >> 19), 1u);
  atomicAdd(my + (k1 >> 19), 1u);
  atomicAdd(my + (k2 >> 19), 1u);
  atomicAdd(my + (k3 >> 19), 1u);
  const uint32_t m01 = k0 > k1 ? k0 : k1, m23 = k2 > k3 ? k2 : k3;
  return m01 > m23 ? m01 : m23;
}

template <int CAP>
__global__ void __launch_bounds__(kHistThreads, 2)
k_hist(const __grid_constant__ BatchDesc<CAP> batch, uint64_t d, const __grid_constant__ Partition part,
       unsigned long long* __restrict__ hist_all, uint32_t* __restrict__ nonfinite_all, uint32_t* __restrict__ seg_hist_all,
       uint32_t* __restrict__ row_max_all) {
  extern __shared__ uint32_t sh_hist[];  // [kHistSub][4096]
  for (int i = threadIdx.x; i < kHistSub * CVLC_HIST_BINS; i += kHistThreads) sh_hist[i] = 0;
  __syncthreads();
  uint32_t* my = sh_hist + ((threadIdx.x >> 5) & (kHistSub - 1)) * CVLC_HIST_BINS;
  const int lane = threadIdx.x & 31;

  const uint64_t nvec = d >> 2;
  const uint64_t units = part.units;  // per client: nvec float4 units and one tail unit
  for (uint32_t q = blockIdx.x; q < part.n_chunks; q += gridDim.x) {
  uint64_t pos = (uint64_t)q * part.chunk;
  const uint64_t end = (pos + part.chunk < part.total) ? pos + part.chunk : part.total;

  while (pos < end) {
    const uint64_t c = pos / units;
    const uint64_t seg_end = ((c + 1) * units < end) ? (c + 1) * units : end;
    const uint64_t u0 = pos - c * units, u1 = seg_end - c * units;
    const float* __restrict__ x = batch.c[c].x;
    const float4* xv = reinterpret_cast<const float4*>(x);
    const uint64_t v1 = (u1 < nvec) ? u1 : nvec;  // float4 units of this segment: [u0, v1)
    // largest key of every row (kRowUnits consecutive units from u0 on: a warp-wide load covers 32 / kRowUnits rows);
    // one whole-warp reduction per row of a load, each seeing that row's keys only
    uint32_t* __restrict__ row_max = row_max_all + seg_first_tile(pos, (uint32_t)(q + c)) * kTileRows;
    static_assert(32 % kRowUnits == 0, "a warp-wide load covers whole rows");
    constexpr int kRowsPerLoad = 32 / kRowUnits;
    const int my_group = lane / kRowUnits;
    auto row_maxima = [&](uint32_t mk) -> uint32_t {  // the largest key among the lanes of this lane's row
      if constexpr (kRowsPerLoad <= 2) {  // few rows per load: one whole-warp reduction per row, each seeing that row's keys only
        uint32_t mine = 0;
#pragma unroll
        for (int g = 0; g < kRowsPerLoad; ++g) {
          const uint32_t mg = __reduce_max_sync(0xFFFFFFFFu, my_group == g ? mk : 0u);
          if (my_group == g) mine = mg;
        }
        return mine;
      } else {  // more rows per load: a butterfly inside the row's lanes
#pragma unroll
        for (int off = 1; off < kRowUnits; off <<= 1) {
          const uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, mk, off);
          mk = o > mk ? o : mk;
        }
        return mk;
      }
    };
    uint32_t top = 0;
    uint64_t v = u0 + threadIdx.x;
    // four independent 128-bit loads in flight per thread; the loop condition is the same for the lanes of a warp
    for (; (v - lane) + 31 + 3 * kHistThreads < v1; v += 4 * kHistThreads) {
      float4 a[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) a[u] = __ldg(xv + v + u * kHistThreads);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t m = row_maxima(hist_add4(my, a[u]));
        top = m > top ? m : top;
        if (lane % kRowUnits == 0) row_max[(v - u0 + u * kHistThreads) / kRowUnits] = m;
      }
    }
    for (; v - lane < v1; v += kHistThreads) {  // rows that may end inside the warp
      const bool on = v < v1;
      const uint32_t m = row_maxima(on ? hist_add4(my, __ldg(xv + v)) : 0u);
      top = m > top ? m : top;
      if (lane % kRowUnits == 0 && on) row_max[(v - u0) / kRowUnits] = m;
    }
    // ragged tail of the client (d not a multiple of 4)
    if (u1 == units && threadIdx.x < (d & 3)) {
      const uint32_t k0 = __float_as_uint(x[(nvec << 2) + threadIdx.x]) & 0x7FFFFFFFu;
      top = k0 > top ? k0 : top;
      atomicAdd(my + (k0 >> 19), 1u);
    }
    if (top >= 0x7F800000u) atomicOr(nonfinite_all + c, 1u);  // a key of exponent 255: Inf or NaN
    __syncthreads();
    // merge into the client's histogram and keep this segment's own counts (segment = chunk + client):
    // the selection kernel derives its output offsets from them
    unsigned long long* __restrict__ hist = hist_all + (size_t)c * CVLC_HIST_BINS;
    uint32_t* __restrict__ seg_hist = seg_hist_all + ((size_t)q + c) * CVLC_HIST_BINS;
    for (int b = threadIdx.x; b < CVLC_HIST_BINS; b += kHistThreads) {
      uint32_t cnt = 0;
#pragma unroll
      for (int sub = 0; sub < kHistSub; ++sub) {
        cnt += sh_hist[sub * CVLC_HIST_BINS + b];
        sh_hist[sub * CVLC_HIST_BINS + b] = 0;
      }
      seg_hist[b] = cnt;
      if (cnt) atomicAdd(hist + b, (unsigned long long)cnt);
    }
    __syncthreads();
    pos = seg_end;
  }
  }
}

__global__ void k_zero_words(uint32_t* p, size_t n_words) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += (size_t)gridDim.x * blockDim.x) p[i] = 0;
}

// ===================================================================================
// Series arithmetic of the planner
// ===================================================================================

// log2 of a positive normal double: v = m 2^e, m folded into (sqrt(1/2), sqrt(2)],
// ln m = 2 atanh(t) with t = (m-1)/(m+1), odd series up to t^25.
__device__ __forceinline__ double series_log2(double v) {
  const unsigned long long bits = (unsigned long long)__double_as_longlong(v);
  int e = (int)((bits >> 52) & 0x7FF) - 1023;
  double m = __longlong_as_double((long long)((bits & 0x000FFFFFFFFFFFFFull) | 0x3FF0000000000000ull));
  if (m > 1.4142135623730951) {
    m = __dmul_rn(m, 0.5);
    e += 1;
  }
  const double t = __ddiv_rn(__dsub_rn(m, 1.0), __dadd_rn(m, 1.0));
  const double q = __dmul_rn(t, t);
  double p = 1.0 / 25.0;
#pragma unroll
  for (int j = 11; j >= 0; --j) p = __dadd_rn(__dmul_rn(p, q), 1.0 / (double)(2 * j + 1));
  const double ln_m = __dmul_rn(__dmul_rn(2.0, t), p);
  return __dadd_rn((double)e, __dmul_rn(ln_m, 1.4426950408889634));
}

// u / j for a small positive integer j, correctly rounded, from the rounded reciprocal:
// q0 = RN(u * rcp), r = u - j*q0 (exact in one fused operation: it is a small multiple
// of ulp(q0)), q1 = RN(q0 + r*rcp).  q0 + r*rcp differs from u/j by less than 2^-52 ulp,
// while u/j, a quotient by an integer below 2^5, is either representable or at least
// 1/(2j) ulp away from every rounding boundary, so q1 = RN(u/j).
__device__ __forceinline__ double div_small_int(double u, int j) {
  const double rcp = 1.0 / (double)j;  // folded at compile time when j is constant
  const double q0 = __dmul_rn(u, rcp);
  const double r = __fma_rn(-(double)j, q0, u);
  return __fma_rn(r, rcp, q0);
}

// 2^v for |v| <= 1000: v = n + r with |r| <= 1/2, e^(r ln 2) as the degree-20 Taylor
// polynomial in Horner form p = 1 + (u/j) p, then n added to the exponent field.
__device__ __forceinline__ double series_exp2(double v) {
  const double n = floor(__dadd_rn(v, 0.5));
  const double r = __dsub_rn(v, n);
  const double u = __dmul_rn(r, 0.6931471805599453);
  // u / j for j = 1 .. 20: a division by an odd j is done once, the even ones are its exact halvings
  // (RN(u / 2j) = RN(u / j) / 2: scaling by two commutes with rounding; u is zero or far above the subnormals)
  double uj[21];
  uj[1] = u;
#pragma unroll
  for (int j = 3; j <= 19; j += 2) uj[j] = div_small_int(u, j);
#pragma unroll
  for (int j = 2; j <= 20; j += 2) uj[j] = __dmul_rn(uj[j / 2], 0.5);
  double p = 1.0;
#pragma unroll
  for (int j = 20; j >= 1; --j) p = __dadd_rn(1.0, __dmul_rn(uj[j], p));
  const long long ni = (long long)n;
  return __longlong_as_double(__double_as_longlong(p) + ni * (1ll << 52));
}

__device__ __forceinline__ double series_powr(double a, double beta) { return series_exp2(__dmul_rn(beta, series_log2(a))); }

// share of ||U||^2 in the top Z ranks under Definition 1: ((Z+1)^beta - 1) / (d^beta - 1)
__device__ __forceinline__ double energy_E(uint64_t Z, double beta, double D) {
  return __ddiv_rn(__dsub_rn(series_powr((double)(Z + 1), beta), 1.0), D);
}

// ===================================================================================
// K2  planner: per client a fit kernel (one CTA of 1024 threads), a tuning kernel and a small copy kernel
// ===================================================================================

constexpr int kPlanThreads = 1024;  // the fit kernel: one thread per four histogram bins
// The tuning kernel evaluates up to kPlanItems (evaluation, length) items per round with kTuneThreads threads (an item
// is a chain of about 175 dependent FP64 operations) and leaves most of its SM to the kernels that run next to it:
// measured on the 100-client benchmark, 256 threads take 0.84 ms instead of 0.62 ms with 512 or 1024, all of it hidden
// behind selection and ranking, and slow those down the least.
constexpr int kTuneThreads = 256;
constexpr int kPlanItems = 1024;
constexpr int kPairSlots = (496 + kTuneThreads - 1) / kTuneThreads;  // pairs of a sweep a thread looks at
constexpr unsigned kFull = 0xFFFFFFFFu;

// scratch of the length-tuning loop (the tuning kernel's dynamic shared memory)
constexpr int kMaxBatchOps = 32;  // atomic operations evaluated together
struct PlanOp {                   // one atomic operation of a batch
  int i, j;                       // candidate indices, i > j
  uint32_t X, na0;                // packets shared by the pair; current count of length i
  uint32_t lo, hi;                // bisection interval
  int m;                          // lengths a trial must evaluate (used lengths <= i, plus i and j)
  int levels;                     // bisection levels evaluated in this round (0: waits)
  int item_base, eval_base;       // first (evaluation, slot) item / first evaluation of this operation
  double F_final;                 // F at the end of the bisection
  unsigned char slot_lane[32];    // those lengths, longest first
};
struct PlanSolver {
  double Ecur[32];                // E(W_l) of the current counts
  double Fpre[33];                // running sum of F after length l (index 32: nothing yet)
  double Eab[33];                 // energy of the nearest used length at or above l
  unsigned long long Wc[32];      // ranks covered by lengths >= l, current counts
  unsigned used;                  // lengths with a positive count
  double Ev[kPlanItems];          // trial energies, one per item
  double Fv[kPlanItems];          // trial objective values, one per evaluation
  uint32_t tv[kPlanItems];        // trial split of every evaluation (0xFFFFFFFF: not needed)
  PlanOp op[kMaxBatchOps];
  int item_end[kMaxBatchOps];     // exclusive end of every operation's items / evaluations in this round
  int eval_end[kMaxBatchOps];
  int n_ops, n_items, n_evals, unfinished;
  int next_i, next_j, moved;      // where the sweep resumes after the batch
  uint32_t col_warp[32];          // batch collection: warp totals of the (operations, items) scan
  int col_nops, col_last, col_first_left;  // operations taken; thread of the last one; thread of the first one left over
  unsigned char ea[kPlanItems];   // operation of every evaluation
};

struct PlanShared {
  double Fv[32];
  uint32_t n[32];
  double beta, D, alpha, alpha_q;
  unsigned long long warp_tot[32];
  unsigned long long carry;
  uint32_t warp_cnt[32];
  uint32_t n_points;
};

// candidate lengths of one client and their coefficients (Eq. (5)), built by warp 0
struct PlanTab {
  uint64_t d;
  uint32_t s, R, nY, y_min, fixed_y;
  uint32_t Y[32];     // candidate lengths, ascending
  uint32_t capY[32];  // cap(Y[i])
  double gY[32];      // g(Y[i]) = 1 - (Q/B^2 + (1 - 1/B)^2)
  double QY[32];      // PQ error factor Q(Y[i]) = cap / (2^y - 1)^2
};

// candidate lengths: g(y) > 0 (the paper's B > (Q+1)/2) and not dominated; called by one full warp
__device__ __forceinline__ void build_plan_tab(PlanTab& T, const Shape& shape, double B_in, int lane) {
  const uint32_t y = lane + 1;
  const double B = B_in;
  const bool in_range = y <= shape.max_code_bits;
  const uint32_t cap_y = in_range ? shape.cap[y] : 0u;
  double Q;  // error factor of cap(y) values at y bits (Appendix, case study)
  if (shape.quantizer == CVLC_QUANT_QSGD) {
    // min(P / s_q^2, sqrt(P) / s_q), s_q = 2^(y-1) - 1 levels beside the sign bit; one bit holds no level
    const double sq = (double)((1ull << (y - 1)) - 1ull);
    const double Q1 = __ddiv_rn((double)cap_y, __dmul_rn(sq, sq));
    const double Q2 = __ddiv_rn(__dsqrt_rn((double)cap_y), sq);
    Q = (y < 2) ? CUDART_INF : ((Q1 < Q2) ? Q1 : Q2);
  } else {
    const double L = (double)((1ull << y) - 1ull);  // PQ: P / (2^y - 1)^2
    Q = __ddiv_rn((double)cap_y, __dmul_rn(L, L));
  }
  const double one_m = __dsub_rn(1.0, __ddiv_rn(1.0, B));
  const double g = __dsub_rn(1.0, __dadd_rn(__ddiv_rn(Q, __dmul_rn(B, B)), __dmul_rn(one_m, one_m)));
  unsigned member;
  uint32_t y_min;
  if (shape.fixed_y) {
    y_min = shape.fixed_y;
    member = 1u << (shape.fixed_y - 1);
  } else {
    const unsigned pos = __ballot_sync(kFull, in_range && g > 0.0);
    y_min = pos ? (uint32_t)__ffs(pos) : 1u;  // the host has checked that one exists
    const uint32_t cap_next = __shfl_down_sync(kFull, cap_y, 1);
    const bool keep = in_range && y >= y_min && (y == shape.max_code_bits || cap_y > cap_next);
    member = __ballot_sync(kFull, keep);
  }
  if (member & (1u << lane)) {
    const int i = __popc(member & ((1u << lane) - 1u));
    T.Y[i] = y;
    T.capY[i] = cap_y;
    T.gY[i] = g;
    T.QY[i] = Q;
  }
  if (lane == 0) {
    T.d = shape.d;
    T.s = shape.s;
    T.R = shape.R;
    T.nY = (uint32_t)__popc(member);
    T.y_min = y_min;
    T.fixed_y = shape.fixed_y;
  }
}

// K2a  per client: survival counts, exponent fit, the threshold bin of the selection and the candidates per segment.
// Everything here depends on the histogram alone.  The number of transmitted coordinates k is not known before the
// lengths are tuned, but it never exceeds k_sel = R * cap(shortest candidate length) (every packet at the shortest
// code; with a fixed length, exactly R * cap(y)), so the selection keeps every coordinate down to the bin that holds
// rank min(k_sel, d): a superset of the top k whose first k ranks are the top k.
template <int CAP>
__global__ void __launch_bounds__(kPlanThreads, 1)
k_plan_fit(const unsigned long long* __restrict__ hist_all, const uint32_t* __restrict__ nonfinite_all,
           const __grid_constant__ BatchDesc<CAP> batch, const __grid_constant__ Shape shape,
           const __grid_constant__ Partition part, unsigned char* ws, int have_segments) {
  extern __shared__ unsigned char smem_raw[];
  unsigned long long* Nsuf = reinterpret_cast<unsigned long long*>(smem_raw);  // [4096] survival counts
  double* ptX = reinterpret_cast<double*>(smem_raw + 4096 * 8);                // fit points, ascending bin
  double* ptY = ptX + 4096;
  __shared__ PlanShared S;
  __shared__ PlanTab T;
  __shared__ uint32_t s_thresh_bin, s_top_bin;
  int32_t* ws_status = reinterpret_cast<int32_t*>(ws);

  // blockIdx.x = client
  const unsigned long long* __restrict__ hist = hist_all + (size_t)blockIdx.x * CVLC_HIST_BINS;
  const uint32_t nonfinite = nonfinite_all[blockIdx.x];
  cvlc_plan_t* __restrict__ plan = batch.c[blockIdx.x].plan;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (nonfinite & 2u) {  // a histogram from outside whose counts do not add up to d (its tuning key stays zero: no tuning)
    if (tid == 0) {
      plan->status = CVLC_ERR_INVALID_ARG;
      set_status(ws_status, CVLC_ERR_INVALID_ARG);
    }
    return;
  }

  if (warp == 0) build_plan_tab(T, shape, batch.c[blockIdx.x].scale_B, lane);
  __syncthreads();

  // ---- survival counts N_j = #{bin >= j} ------------------------------------------

  // ---- survival counts N_j = #{bin >= j} ------------------------------------------
  unsigned long long h[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) h[i] = hist[4 * tid + i];
  {
    unsigned long long tot = h[0] + h[1] + h[2] + h[3];
    // inclusive scan from the top bin down: reverse thread order
    unsigned long long v = tot;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned long long o = __shfl_down_sync(kFull, v, off);
      if (lane + off < 32) v += o;
    }
    if (lane == 0) S.warp_tot[warp] = v;
    __syncthreads();
    unsigned long long above = 0;
    for (int w = warp + 1; w < 32; ++w) above += S.warp_tot[w];
    const unsigned long long incl = v + above;  // sum over threads >= tid
    unsigned long long run = incl - tot;        // sum over threads > tid
#pragma unroll
    for (int i = 3; i >= 0; --i) {
      run += h[i];
      Nsuf[4 * tid + i] = run;
    }
  }
  __syncthreads();

  if (T.fixed_y == 0) {
    // ---- fit points: non-empty normal bins in the upper half of the ranks ----------
    uint32_t flags = 0, cnt = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int j = 4 * tid + i;
      const unsigned long long N = Nsuf[j];
      const bool ok = (j >= 16) && (j <= 4079) && (h[i] > 0) && (N >= 1) && (N <= T.d / 2);
      flags |= (ok ? 1u : 0u) << i;
      cnt += ok;
    }
    uint32_t v = cnt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t o = __shfl_up_sync(kFull, v, off);
      if (lane >= off) v += o;
    }
    if (lane == 31) S.warp_cnt[warp] = v;
    __syncthreads();
    uint32_t below = 0;
    for (int w = 0; w < warp; ++w) below += S.warp_cnt[w];
    uint32_t pos = below + v - cnt;
    if (tid == kPlanThreads - 1) S.n_points = below + v;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (flags & (1u << i)) {
        const int j = 4 * tid + i;
        ptX[pos] = series_log2((double)Nsuf[j]);
        ptY[pos] = __dadd_rn((double)((j >> 4) - 127), series_log2(__dadd_rn(1.0, (double)(j & 15) / 16.0)));
        ++pos;
      }
    }
    __syncthreads();
    // ---- least squares of log2|U{l}| on log2 l, sums in ascending bin order ----------
    if (tid == 0) {
      double n = 0.0, Sx = 0.0, Sy = 0.0, Sxx = 0.0, Sxy = 0.0;
      const uint32_t np = S.n_points;
      for (uint32_t i = 0; i < np; ++i) {
        const double X = ptX[i], Y = ptY[i];
        n = __dadd_rn(n, 1.0);
        Sx = __dadd_rn(Sx, X);
        Sy = __dadd_rn(Sy, Y);
        Sxx = __dadd_rn(Sxx, __dmul_rn(X, X));
        Sxy = __dadd_rn(Sxy, __dmul_rn(X, Y));
      }
      const double den = __dsub_rn(__dmul_rn(n, Sxx), __dmul_rn(Sx, Sx));
      double a;
      if (n < 2.0 || !(den > 0.0))
        a = -1.0;
      else
        a = __ddiv_rn(__dsub_rn(__dmul_rn(n, Sxy), __dmul_rn(Sx, Sy)), den);
      double aq = __dmul_rn(floor(__dadd_rn(__dmul_rn(a, 256.0), 0.5)), 1.0 / 256.0);
      if (aq < -4.0) aq = -4.0;
      if (aq > -1.0 / 256.0) aq = -1.0 / 256.0;
      if (aq == -0.5) aq = -0.5 - 1.0 / 256.0;  // beta = 0 would make d^beta - 1 vanish
      S.alpha = a;
      S.alpha_q = aq;
    }
  } else if (tid == 0) {
    S.alpha = -1.0;
    S.alpha_q = -1.0;
  }
  __syncthreads();

  // ---- selection threshold: the bin that holds rank min(k_sel, d) (1-based), how many coordinates sit in it
  // or above, and the highest non-empty bin
  unsigned long long k_sel = (unsigned long long)T.R * T.capY[0];
  if (k_sel > T.d) k_sel = T.d;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int j = 4 * tid + i;
    const unsigned long long N = Nsuf[j];
    const unsigned long long Nn = (j == CVLC_HIST_BINS - 1) ? 0ull : Nsuf[j + 1];
    if (N >= k_sel && Nn < k_sel) {
      plan->thresh_bin = (uint32_t)j;
      plan->n_candidates = N;
      s_thresh_bin = (uint32_t)j;
    }
    if (N > 0 && Nn == 0) {
      plan->top_bin = (uint32_t)j;
      s_top_bin = (uint32_t)j;
    }
  }
  if (tid == 0) {
    const double aq = S.alpha_q;
    plan->status = nonfinite ? CVLC_ERR_NONFINITE_INPUT : CVLC_OK;
    if (nonfinite) set_status(ws_status, CVLC_ERR_NONFINITE_INPUT);
    plan->s = T.s;
    plan->R = T.R;
    plan->y_min = T.y_min;
    plan->n_lengths = T.nY;
    plan->k = 0;
    plan->alpha = S.alpha;
    plan->alpha_q = aq;
    plan->beta = __dadd_rn(__dmul_rn(2.0, aq), 1.0);
    plan->gamma = 0.0;
    plan->B_next = 0.0;
    for (int y = 0; y <= CVLC_MAX_CODE_BITS; ++y) {
      plan->n_y[y] = 0;
      plan->cap[y] = shape.cap[y];
    }
    // clients with the same quantised exponent and the same scale get the same lengths
    unsigned long long* key = reinterpret_cast<unsigned long long*>(ws + plan_off_keys(batch.n)) + 2 * (size_t)blockIdx.x;
    key[0] = (unsigned long long)__double_as_longlong(aq);
    key[1] = (unsigned long long)__double_as_longlong(batch.c[blockIdx.x].scale_B);
  }
  __syncthreads();

  // candidates per segment of this client (segment = part of the client inside one block's chunk of
  // the histogram / selection kernels) and their exclusive prefix: the selection kernel's offsets.
  // A plan made from a histogram alone has no segments; its workspace header stays unmarked.

  if (have_segments) {
    const uint32_t c = blockIdx.x;
    const uint32_t S = part.max_segments;
    uint32_t* seg_count = reinterpret_cast<uint32_t*>(ws + plan_off_seg_count(batch.n));
    unsigned long long* seg_prefix = reinterpret_cast<unsigned long long*>(ws + plan_off_seg_prefix(batch.n, S));
    const uint64_t row_tiles = row_tiles_total(part);
    const uint32_t* seg_hist = reinterpret_cast<const uint32_t*>(ws + plan_off_seg_hist(batch.n, S, row_tiles));
    const uint64_t first = (uint64_t)c * part.units, last = first + part.units - 1;
    const uint32_t b0 = (uint32_t)(first / part.chunk), b1 = (uint32_t)(last / part.chunk);
    const uint32_t jt = s_thresh_bin, jtop = s_top_bin;  // nothing above the client's highest non-empty bin
    for (uint32_t b = b0 + warp; b <= b1; b += kPlanThreads / 32) {
      const uint32_t* hsrc = seg_hist + ((size_t)b + c) * CVLC_HIST_BINS;
      uint32_t sum = 0;
      for (uint32_t j = jt + lane; j <= jtop; j += 32) sum += hsrc[j];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(kFull, sum, off);
      if (lane == 0) seg_count[b + c] = sum;
    }
    // the rows of 128 coordinates that hold a candidate (a key at or above the threshold), listed per segment in
    // ascending order: one warp per segment walks its rows 32 at a time, eight loads in flight
    {
      const uint32_t* row_max = reinterpret_cast<const uint32_t*>(ws + plan_off_row_max(batch.n, S));
      uint32_t* row_list = reinterpret_cast<uint32_t*>(ws + plan_off_row_list(batch.n, S, row_tiles));
      uint32_t* seg_rows = reinterpret_cast<uint32_t*>(ws + plan_off_seg_rows(batch.n, S));
      const uint32_t thresh_key = jt << 19;
      const uint64_t nvec = shape.d >> 2;
      const unsigned lt = (1u << lane) - 1u;
      for (uint32_t b = b0 + warp; b <= b1; b += kPlanThreads / 32) {
        const uint64_t p0 = (first > (uint64_t)b * part.chunk) ? first : (uint64_t)b * part.chunk;
        uint64_t p1 = ((uint64_t)(b + 1) * part.chunk < first + part.units) ? (uint64_t)(b + 1) * part.chunk : first + part.units;
        if (p1 > first + nvec) p1 = first + nvec;  // the client's last unit is its ragged tail, not a float4
        const uint64_t n_units = p1 > p0 ? p1 - p0 : 0;
        const uint64_t n_rows = (n_units + kRowUnits - 1) / kRowUnits;
        const uint64_t base = seg_first_tile(p0, b + c) * kTileRows;
        uint32_t listed = 0;
        for (uint64_t r0 = 0; r0 < n_rows; r0 += 256) {
          uint32_t mx[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint64_t r = r0 + (uint64_t)j * 32 + lane;
            mx[j] = (r < n_rows) ? row_max[base + r] : 0u;
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint64_t r = r0 + (uint64_t)j * 32 + lane;
            const bool on = (r < n_rows) && mx[j] >= thresh_key;
            const unsigned bits = __ballot_sync(kFull, on);
            if (on) row_list[base + listed + __popc(bits & lt)] = (uint32_t)r;
            listed += __popc(bits);
          }
        }
        if (lane == 0) seg_rows[b + c] = listed;
      }
    }
    __syncthreads();
    if (tid == 0) {
      unsigned long long run = 0;
      for (uint32_t b = b0; b <= b1; ++b) {
        seg_prefix[b + c] = run;
        run += seg_count[b + c];
      }
      if (c == 0) {
        PlanWsHeader* hdr = reinterpret_cast<PlanWsHeader*>(ws);
        hdr->n = batch.n;
        hdr->d = shape.d;
        hdr->n_chunks = part.n_chunks;
        hdr->magic = kPlanWsMagic;
      }
    }
  }
}

// K2b  code-length tuning, one CTA per client; only the first client of every tuning key does the work
template <int CAP>
__global__ void __launch_bounds__(kTuneThreads, 1)
k_plan_tune(const __grid_constant__ BatchDesc<CAP> batch, const __grid_constant__ Shape shape, unsigned char* ws) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ PlanShared S;
  __shared__ PlanTab T;
  __shared__ uint32_t s_leader;
  const uint32_t c = blockIdx.x;
  cvlc_plan_t* __restrict__ plan = batch.c[c].plan;
  uint32_t* leader = reinterpret_cast<uint32_t*>(ws + plan_off_leader(batch.n));
  const unsigned long long* keys = reinterpret_cast<const unsigned long long*>(ws + plan_off_keys(batch.n));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  const unsigned long long key0 = keys[2 * (size_t)c], key1 = keys[2 * (size_t)c + 1];
  if (tid == 0) s_leader = c;
  __syncthreads();
  if (key1 == 0ull) {  // no key: the fit refused this client's histogram
    if (tid == 0) leader[c] = 0xFFFFFFFFu;
    return;
  }
  for (uint32_t i = tid; i < c; i += kTuneThreads)
    if (keys[2 * (size_t)i] == key0 && keys[2 * (size_t)i + 1] == key1) atomicMin(&s_leader, i);
  __syncthreads();
  if (tid == 0) leader[c] = s_leader;
  if (s_leader != c) return;  // an earlier client of the batch tunes for this key; k_plan_finish copies its result

  if (warp == 0) build_plan_tab(T, shape, batch.c[c].scale_B, lane);
  if (tid == 0) {
    const double aq = __longlong_as_double((long long)key0);
    const double beta = __dadd_rn(__dmul_rn(2.0, aq), 1.0);
    S.alpha_q = aq;
    S.beta = beta;
    S.D = __dsub_rn(series_powr((double)shape.d, beta), 1.0);
  }
  if (tid < 32) S.n[tid] = 0;
  __syncthreads();
  const double beta = S.beta, D = S.D;
  const int nY = (int)T.nY;
  const uint32_t my_cap = (lane < nY) ? T.capY[lane] : 0u;
  double* ptX = reinterpret_cast<double*>(smem_raw);  // the solver's scratch


  // ---- objective bookkeeping -----------------------------------------------------------
  // F(n) = 1 - gamma of Eq. (5) is a running sum over the used lengths, longest first:
  // F += g_l * (E(W_l) - E(W_prev)), W_l = ranks covered down to and including length l.
  // For the current counts the kernel keeps, per candidate index l: the energy E(W_l)
  // (Q.Ecur), the running sum after length l (Q.Fpre) and the energy of the nearest used
  // length at or above l (Q.Eab).  An atomic operation on the lengths i > j leaves everything
  // above i untouched, so a trial split only needs E for the used lengths at or below i and
  // continues the running sum from Q.Fpre[i + 1]: the same operations in the same order as a
  // full evaluation, on a fraction of the lanes.
  PlanSolver& Q = *reinterpret_cast<PlanSolver*>(ptX);  // the fit points are no longer needed

  auto refresh_state = [&]() {  // all threads; ends with a barrier
    if (warp == 0) {
      const uint32_t my_n = (lane < nY) ? S.n[lane] : 0u;
      uint64_t W = (uint64_t)my_n * my_cap;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint64_t o = __shfl_down_sync(kFull, W, off);
        if (lane + off < 32) W += o;
      }
      Q.Ecur[lane] = (my_n > 0) ? energy_E(W, beta, D) : 0.0;
      Q.Wc[lane] = W;
      const unsigned used = __ballot_sync(kFull, my_n > 0);
      if (lane == 0) Q.used = used;
      __syncwarp();
      if (lane == 0) {
        double F = 0.0, Eprev = 0.0;
        Q.Fpre[32] = 0.0;
        Q.Eab[32] = 0.0;
        for (int l = 31; l >= 0; --l) {
          if (l < nY && S.n[l] > 0) {
            const double Ec = Q.Ecur[l];
            F = __dadd_rn(F, __dmul_rn(T.gY[l], __dsub_rn(Ec, Eprev)));
            Eprev = Ec;
          }
          Q.Fpre[l] = F;
          Q.Eab[l] = Eprev;
        }
      }
    }
    __syncthreads();
  };

  if (T.fixed_y != 0) {
    if (tid == 0) S.n[0] = T.R;
    __syncthreads();
    refresh_state();
  } else {
    // ---- equal packets: best admissible single-length plan, ties to the longer code ----
    if (tid < nY) {
      const uint64_t W = (uint64_t)T.R * T.capY[tid];
      // one term: F = 0 + g * (E - 0)
      S.Fv[tid] = (W > T.d) ? -CUDART_INF : __dmul_rn(T.gY[tid], energy_E(W, beta, D));
    }
    __syncthreads();
    if (tid == 0) {
      int best = -1;
      double bestF = -CUDART_INF;
      for (int i = 0; i < nY; ++i) {
        const double F = S.Fv[i];
        if (F == -CUDART_INF) continue;
        if (best < 0 || F >= bestF) {
          best = i;
          bestF = F;
        }
      }
      S.n[best < 0 ? 0 : best] = T.R;  // the host has checked that a plan is admissible
    }
    __syncthreads();
    refresh_state();

    // ---- atomic operations (Section IV-C) on pairs of lengths until nothing moves ----
    // An atomic operation bisects the split of X = n_i + n_j packets between the lengths i > j
    // for the first t with F(t+1) <= F(t) and moves there if that is strictly better.  Most
    // operations of a sweep change nothing, so consecutive operations are evaluated together as
    // if none of them moved; the first one (in sweep order) that does move is applied, the later
    // ones of the batch are dropped and the sweep resumes right after it: exactly the sequential
    // result.  Per round every unfinished operation gets as many bisection levels as the block's
    // 1024 (evaluation, length) items allow: evaluation e = 2q, 2q+1 of an operation is
    // F(mid+1), F(mid) of node q+1 of its decision tree (heap order: child 2h after
    // "F(mid+1) <= F(mid)", child 2h+1 after "F(mid+1) > F(mid)").
    auto next_pair = [&](int phase, int& i, int& j) {  // sweep order; i = 0 marks the end
      if (phase == 0) {
        --i;
        j = i - 1;
      } else if (j > 0) {
        --j;
      } else {
        --i;
        j = i - 1;
      }
    };
    for (int round = 0; round < 64; ++round) {
      int movedB = 0;
      for (int phase = 0; phase < 2; ++phase) {  // 0: neighbouring lengths until quiet; 1: every pair once
        const int max_sweeps = (phase == 0) ? 256 : 1;
        for (int sweep = 0; sweep < max_sweeps; ++sweep) {
          int moved = 0;
          int ci = nY - 1, cj = nY - 2;  // cursor of the sweep
          while (ci >= 1) {
            // ---- collect a batch: thread t looks at the t-th pair of the sweep from the cursor on (at most
            // 31 + 465 pairs).  The batch is the first pairs, in sweep order, that share packets (X > 0), up to
            // kMaxBatchOps of them and as long as two evaluations of each fit the block: a prefix of the flagged
            // pairs, found with one block scan of (operations, items) packed in a word.
            {
              auto pair_at = [&](int t, int& i, int& j) -> bool {
                if (t < 0) return false;
                if (phase == 0) {
                  i = ci - t;
                  j = i - 1;
                  return i >= 1;
                }
                const int first = cj + 1;  // rest of the cursor's row: j = cj .. 0
                if (t < first) {
                  i = ci;
                  j = cj - t;
                  return true;
                }
                const int rest = (ci - 1) * ci / 2;  // rows ci - 1 .. 1, row r holding the pairs (r, r-1) .. (r, 0)
                const int tp = t - first;
                if (tp >= rest) return false;
                const int u = rest - 1 - tp;  // counted upwards from pair (1, 0)
                int r = 1;
                while ((r * (r + 1)) / 2 <= u) ++r;
                i = r;
                j = u - (r - 1) * r / 2;
                return true;
              };
              // a thread looks at the pairs t = tid, tid + kTuneThreads, ...; the scan runs over t in order
              const unsigned used = Q.used;
              if (tid == 0) {
                Q.col_nops = 0;
                Q.col_last = -1;
                Q.col_first_left = 0x7FFFFFFF;
              }
              uint32_t carry = 0;
#pragma unroll
              for (int slot = 0; slot < kPairSlots; ++slot) {
                const int t = slot * kTuneThreads + tid;
                int pi = 0, pj = 0;
                const bool valid = pair_at(t, pi, pj);
                uint32_t X = 0;
                unsigned need = 0;
                int m = 0;
                if (valid) {
                  X = S.n[pi] + S.n[pj];
                  if (X > 0) {
                    need = (used | (1u << pi) | (1u << pj)) & (0xFFFFFFFFu >> (31 - pi));
                    m = __popc(need);
                  }
                }
                const bool flag = valid && X > 0;
                uint32_t incl = flag ? ((1u << 16) | (uint32_t)(2 * m)) : 0u;  // items stay below 2^16: 496 pairs of at most 64
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                  const uint32_t o = __shfl_up_sync(kFull, incl, off);
                  if (lane >= off) incl += o;
                }
                if (lane == 31) Q.col_warp[warp] = incl;
                __syncthreads();
                {
                  const uint32_t wt = (lane < kTuneThreads / 32) ? Q.col_warp[lane] : 0u;
                  uint32_t wi = wt;
#pragma unroll
                  for (int off = 1; off < 32; off <<= 1) {
                    const uint32_t o = __shfl_up_sync(kFull, wi, off);
                    if (lane >= off) wi += o;
                  }
                  incl += carry + __shfl_sync(kFull, wi - wt, warp);
                  carry += __shfl_sync(kFull, wi, 31);
                }
                const int rank = (int)(incl >> 16) - 1;
                const bool taken = flag && rank < kMaxBatchOps && (incl & 0xFFFFu) <= (uint32_t)kPlanItems;
                if (taken) {
                  PlanOp& o = Q.op[rank];
                  o.i = pi; o.j = pj; o.X = X; o.na0 = S.n[pi]; o.lo = 0; o.hi = X; o.m = m; o.F_final = 0.0;
                  for (unsigned rest_bits = need; rest_bits;) {  // the lengths a trial evaluates, longest first
                    const int l = 31 - __clz(rest_bits);
                    rest_bits ^= 1u << l;
                    o.slot_lane[l == 31 ? 0 : __popc(need >> (l + 1))] = (unsigned char)l;
                  }
                  atomicMax(&Q.col_nops, rank + 1);
                  atomicMax(&Q.col_last, t);
                } else if (flag) {
                  atomicMin(&Q.col_first_left, t);
                }
                if (slot + 1 < kPairSlots) __syncthreads();  // the warp totals are reused by the next slot
              }
              __syncthreads();
              const int n_ops = Q.col_nops;
              // the sweep resumes after the last operation of a full batch, else at the first pair left over
              const int resume = (n_ops == kMaxBatchOps) ? Q.col_last + 1
                                                         : (Q.col_first_left != 0x7FFFFFFF ? Q.col_first_left : -1);
              int bi = 0, bj = 0;
              if (!pair_at(resume, bi, bj)) bi = bj = 0;
              if (tid == 0) {
                Q.n_ops = n_ops;
                Q.next_i = bi;
                Q.next_j = bj;
                Q.moved = 0;
                Q.unfinished = n_ops;
              }
              ci = bi;
              cj = bj;
              if (n_ops == 0) {  // the rest of the sweep had nothing to split
                __syncthreads();  // the collection's scratch is reset by the next one
                continue;
              }
            }
            __syncthreads();
            const int n_ops = Q.n_ops;
            const double F_cur = Q.Fpre[0];
            // ---- rounds until every operation of the batch has finished its bisection
            // level assignment (warp 0, lane = operation), before the first round and right after every tree walk:
            // the planner is bound by the FP64 throughput
            // of its SM, and every extra level evaluated ahead doubles the work, so all operations get
            // the same small depth: the largest one whose items fit the block
            auto assign_levels = [&]() {
                const bool mine = lane < n_ops;
                const uint32_t span = (mine && Q.op[lane].lo < Q.op[lane].hi) ? Q.op[lane].hi - Q.op[lane].lo : 0u;
                const int need_levels = span ? 32 - __clz(span) : 0;  // a bisection of s points takes at most floor(log2 s) + 1 steps
                const int m_op = mine ? Q.op[lane].m : 0;
                // items of the whole batch at every candidate depth: nine reductions side by side (one after the
                // other they are nine chains of five dependent shuffles, as long as the energy evaluation itself)
                int items_at[9];
#pragma unroll
                for (int cand = 1; cand <= 9; ++cand) {
                  const int lvc = need_levels < cand ? need_levels : cand;
                  items_at[cand - 1] = lvc ? 2 * ((1 << lvc) - 1) * m_op : 0;
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
                  for (int q = 0; q < 9; ++q) items_at[q] += __shfl_xor_sync(kFull, items_at[q], off);
                }
                int depth = 0;
#pragma unroll
                for (int q = 0; q < 9; ++q) {
                  if (items_at[q] <= kPlanItems && depth == q) depth = q + 1;  // the sums grow with the depth
                }
                const int lv = need_levels < depth ? need_levels : depth;
                const int ne = lv ? 2 * ((1 << lv) - 1) : 0;
                int items_incl = ne * m_op, evals_incl = ne;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                  const int a1 = __shfl_up_sync(kFull, items_incl, off), a2 = __shfl_up_sync(kFull, evals_incl, off);
                  if (lane >= off) {
                    items_incl += a1;
                    evals_incl += a2;
                  }
                }
                if (mine) {
                  Q.op[lane].levels = lv;
                  Q.op[lane].item_base = items_incl - ne * m_op;
                  Q.op[lane].eval_base = evals_incl - ne;
                }
                Q.item_end[lane] = items_incl;
                Q.eval_end[lane] = evals_incl;
                const unsigned unfinished = __ballot_sync(kFull, need_levels > 0);
                if (lane == 31) {
                  Q.n_items = items_incl;
                  Q.n_evals = evals_incl;
                  Q.unfinished = __popc(unfinished);
                }
                          };
            if (warp == 0) assign_levels();
            while (true) {
              __syncthreads();
              if (Q.unfinished == 0) break;
              // phase 1: energies, one thread per (operation, evaluation, slot)
              for (int vt = tid; vt < Q.n_items; vt += kTuneThreads) {
                int a = -1, e = 0, sl = 0;
                uint32_t t = 0xFFFFFFFFu;
                // the operation whose item range holds this item: first a with vt < item_end[a]
                int lo_a = 0, hi_a = 31;
                while (lo_a < hi_a) {
                  const int mid = (lo_a + hi_a) >> 1;
                  if (vt < Q.item_end[mid]) hi_a = mid; else lo_a = mid + 1;
                }
                a = lo_a;
                const PlanOp& o = Q.op[a];
                const int rel = vt - o.item_base;
                e = rel / o.m;
                sl = rel - e * o.m;
                const int hnode = (e >> 1) + 1;
                const int depth = 31 - __clz(hnode);
                uint32_t l3 = o.lo, h3 = o.hi;
                bool open = true;
                for (int b = depth - 1; b >= 0; --b) {
                  if (!(l3 < h3)) { open = false; break; }
                  const uint32_t mid = l3 + (h3 - l3) / 2;
                  if ((hnode >> b) & 1) l3 = mid + 1; else h3 = mid;
                }
                if (open && l3 < h3) {
                  t = l3 + (h3 - l3) / 2 + ((e & 1) ? 0u : 1u);
                  const int l = o.slot_lane[sl];
                  // ranks down to length l with the pair's packets re-split: the current cover, minus the
                  // pair's current share, plus the trial's
                  uint64_t W = Q.Wc[l] - (uint64_t)S.n[o.i] * T.capY[o.i] + (uint64_t)t * T.capY[o.i];
                  if (l <= o.j) W = W - (uint64_t)S.n[o.j] * T.capY[o.j] + (uint64_t)(o.X - t) * T.capY[o.j];
                  Q.Ev[vt] = energy_E(W, beta, D);
                }
                if (sl == 0) {
                  Q.tv[o.eval_base + e] = t;
                  Q.ea[o.eval_base + e] = (unsigned char)a;
                }
              }
              __syncthreads();
              // phase 2: one thread per evaluation continues the running sum below length i with the terms
              // g_l * (E_l - E_prev) in the order of the lengths; only the lengths i and j can be unused in a trial
              // (no term, and the next term's E_prev skips them).  The terms do not depend on the sum, so they are
              // worked out four at a time ahead of the ordered additions.
              for (int vt = tid; vt < Q.n_evals; vt += kTuneThreads) {
                const PlanOp& o = Q.op[Q.ea[vt]];
                const uint32_t tt = Q.tv[vt];
                if (tt != 0xFFFFFFFFu) {
                  const int ee = vt - o.eval_base;
                  const double* Ez = Q.Ev + o.item_base + ee * o.m;
                  double F = Q.Fpre[o.i + 1];
                  double Eprev = Q.Eab[o.i + 1];
                  for (int z0 = 0; z0 < o.m; z0 += 4) {
                    double term4[4];
                    bool on4[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                      const int z = z0 + q;
                      on4[q] = false;
                      term4[q] = 0.0;
                      if (z < o.m) {
                        const int l = o.slot_lane[z];
                        const uint32_t nn = (l == o.i) ? tt : (l == o.j) ? (o.X - tt) : 1u;
                        if (nn > 0) {
                          const double Ec = Ez[z];
                          on4[q] = true;
                          term4[q] = __dmul_rn(T.gY[l], __dsub_rn(Ec, Eprev));
                          Eprev = Ec;
                        }
                      }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                      if (on4[q]) F = __dadd_rn(F, term4[q]);
                  }
                  const uint64_t Wtot = Q.Wc[0] - (uint64_t)S.n[o.i] * T.capY[o.i] - (uint64_t)S.n[o.j] * T.capY[o.j] +
                                        (uint64_t)tt * T.capY[o.i] + (uint64_t)(o.X - tt) * T.capY[o.j];
                  Q.Fv[vt] = (Wtot > T.d) ? -CUDART_INF : F;
                }
              }
              __syncthreads();
              // phase 4: one thread per operation walks its decision tree
              if (tid < n_ops) {
                PlanOp& o = Q.op[tid];
                if (o.levels > 0) {
                  uint32_t lo = o.lo, hi = o.hi;
                  double Ff = o.F_final;
                  int hnode = 1;
                  for (int level = 0; level < o.levels && lo < hi; ++level) {
                    const uint32_t mid = lo + (hi - lo) / 2;
                    const double F1 = Q.Fv[o.eval_base + 2 * (hnode - 1)], F0 = Q.Fv[o.eval_base + 2 * (hnode - 1) + 1];
                    if (F1 > F0) {
                      lo = mid + 1;
                      Ff = F1;
                      hnode = 2 * hnode + 1;
                    } else {
                      hi = mid;
                      Ff = F0;
                      hnode = 2 * hnode;
                    }
                  }
                  o.lo = lo;
                  o.hi = hi;
                  o.F_final = Ff;
                }
              }
              if (warp == 0) {  // the lanes that walked the trees own the same operations in the level assignment
                __syncwarp();
                assign_levels();
              }
            }
            // ---- the first operation of the batch that improves F is applied; the sweep resumes after it
            if (tid == 0) {
              for (int a = 0; a < n_ops; ++a) {
                const PlanOp& o = Q.op[a];
                if (o.lo != o.na0 && o.F_final > F_cur) {
                  S.n[o.i] = o.lo;
                  S.n[o.j] = o.X - o.lo;
                  int ri = o.i, rj = o.j;
                  next_pair(phase, ri, rj);
                  Q.next_i = ri;
                  Q.next_j = rj;
                  Q.moved = 1;
                  break;
                }
              }
            }
            __syncthreads();
            ci = Q.next_i;
            cj = Q.next_j;
            if (Q.moved) {
              moved = 1;
              refresh_state();
            } else {
              __syncthreads();
            }
          }
          if (phase == 1) movedB = moved;
          if (!moved) break;
        }
      }
      if (!movedB) break;
    }
  }

  // ---- outputs ---------------------------------------------------------------------
  if (tid == 0) {
    unsigned long long k = 0;
    double Qmax = 0.0;
    for (int i = 0; i < nY; ++i) {
      k += (unsigned long long)S.n[i] * T.capY[i];
      if (S.n[i] > 0 && T.QY[i] > Qmax) Qmax = T.QY[i];
    }
    plan->k = k;
    plan->gamma = __dsub_rn(1.0, Q.Fpre[0]);
    plan->B_next = __dadd_rn(1.0, Qmax);
    for (int i = 0; i < nY; ++i) plan->n_y[T.Y[i]] = S.n[i];
  }
}

// K2c  the clients that share a tuning key take the lengths of the client that tuned for it
template <int CAP>
__global__ void __launch_bounds__(256)
k_plan_finish(const __grid_constant__ BatchDesc<CAP> batch, const unsigned char* ws) {
  const uint32_t c = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (c >= batch.n) return;
  const uint32_t l = reinterpret_cast<const uint32_t*>(ws + plan_off_leader(batch.n))[c];
  if (l == 0xFFFFFFFFu || l == c || l >= batch.n) return;
  cvlc_plan_t* dst = batch.c[c].plan;
  const cvlc_plan_t* src = batch.c[l].plan;
  dst->n_y[lane] = src->n_y[lane];
  if (lane == 0) {
    dst->n_y[CVLC_MAX_CODE_BITS] = src->n_y[CVLC_MAX_CODE_BITS];
    dst->k = src->k;
    dst->gamma = src->gamma;
    dst->B_next = src->B_next;
  }
}

// ===================================================================================
// launchers
// ===================================================================================

constexpr size_t kFitSmem = 3 * 4096 * 8;  // survival counts and the fit points
constexpr size_t kTuneSmem = (sizeof(PlanSolver) + 255) & ~(size_t)255;

template <int CAP>
static cudaError_t plan_attributes() {
  static bool attr_done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && !attr_done[dev]) {
    e = cudaFuncSetAttribute(k_hist<CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kHistSub * CVLC_HIST_BINS * 4);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_plan_fit<CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFitSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_plan_tune<CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTuneSmem);
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  return cudaSuccess;
}

template <int CAP>
static void fill_batch(BatchDesc<CAP>& batch, const ClientDesc* clients, uint32_t n) {
  batch.n = n;
  batch.pad = 0;
  for (uint32_t i = 0; i < n; ++i) batch.c[i] = clients[i];
}

// histogram of every client, then (unless only the histograms are wanted) fit, threshold and segment tables
template <int CAP>
static cudaError_t launch_plan_front_t(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws,
                                       unsigned long long* hist_out, cudaStream_t st) {
  cudaError_t e = plan_attributes<CAP>();
  if (e != cudaSuccess) return e;
  BatchDesc<CAP> batch;
  fill_batch(batch, clients, n);
  unsigned char* w = static_cast<unsigned char*>(ws);
  unsigned long long* hist = reinterpret_cast<unsigned long long*>(w + kPlanWsHist);
  uint32_t* flags = reinterpret_cast<uint32_t*>(w + plan_off_flags(n));
  const Partition part = make_partition(shape.d, n);
  const uint64_t row_tiles = row_tiles_total(part);
  uint32_t* seg_hist = reinterpret_cast<uint32_t*>(w + plan_off_seg_hist(n, part.max_segments, row_tiles));
  uint32_t* row_max = reinterpret_cast<uint32_t*>(w + plan_off_row_max(n, part.max_segments));
  {
    // header, histograms, flags, tuning keys and segment tables start at zero; the per-segment histograms and the
    // rows' maxima are written in full by the histogram kernel
    LaunchScope ls(kKZeroWords, st);
    k_zero_words<<<2 * kNumSM, 1024, 0, st>>>(reinterpret_cast<uint32_t*>(w), plan_off_row_max(n, part.max_segments) / 4);
  }
  {
    // two resident blocks per SM share the concatenated updates evenly
    LaunchScope ls(kKHist, st);
    k_hist<CAP><<<part.grid, kHistThreads, kHistSub * CVLC_HIST_BINS * 4, st>>>(batch, shape.d, part, hist, flags, seg_hist, row_max);
  }
  if (hist_out) {
    // the histograms alone: what a client sends when the parameter server plans for it.  The workspace
    // header stays unmarked, so an encode call cannot take it for one that holds a plan's segment tables.
    const cudaError_t e2 = cudaGetLastError();
    if (e2 != cudaSuccess) return e2;
    return cudaMemcpyAsync(hist_out, hist, (size_t)n * CVLC_HIST_BINS * 8, cudaMemcpyDeviceToDevice, st);
  }
  {
    LaunchScope ls(kKPlanFit, st);
    k_plan_fit<CAP><<<n, kPlanThreads, kFitSmem, st>>>(hist, flags, batch, shape, part, w, 1);
  }
  return cudaGetLastError();
}

template <int CAP>
static cudaError_t launch_plan_back_t(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws, cudaStream_t st) {
  cudaError_t e = plan_attributes<CAP>();
  if (e != cudaSuccess) return e;
  BatchDesc<CAP> batch;
  fill_batch(batch, clients, n);
  unsigned char* w = static_cast<unsigned char*>(ws);
  {
    LaunchScope ls(kKPlanTune, st);
    k_plan_tune<CAP><<<n, kTuneThreads, kTuneSmem, st>>>(batch, shape, w);
  }
  {
    LaunchScope ls(kKPlanFinish, st);
    k_plan_finish<CAP><<<(n + 7) / 8, 256, 0, st>>>(batch, w);
  }
  return cudaGetLastError();
}

cudaError_t launch_plan_front(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws, cudaStream_t st) {
  if (n <= (uint32_t)kSmallBatch) return launch_plan_front_t<kSmallBatch>(clients, n, shape, ws, nullptr, st);
  return launch_plan_front_t<kLargeBatch>(clients, n, shape, ws, nullptr, st);
}

cudaError_t launch_plan_back(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws, cudaStream_t st) {
  if (n <= (uint32_t)kSmallBatch) return launch_plan_back_t<kSmallBatch>(clients, n, shape, ws, st);
  return launch_plan_back_t<kLargeBatch>(clients, n, shape, ws, st);
}

cudaError_t launch_plan(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws, cudaStream_t st) {
  const cudaError_t e = launch_plan_front(clients, n, shape, ws, st);
  if (e != cudaSuccess) return e;
  return launch_plan_back(clients, n, shape, ws, st);
}

cudaError_t launch_histogram(const ClientDesc* clients, uint32_t n, const Shape& shape, void* ws,
                             unsigned long long* hist_out, cudaStream_t st) {
  if (n <= (uint32_t)kSmallBatch) return launch_plan_front_t<kSmallBatch>(clients, n, shape, ws, hist_out, st);
  return launch_plan_front_t<kLargeBatch>(clients, n, shape, ws, hist_out, st);
}

// Checks histograms that come from outside: flag bit 0 = a value of exponent 255 (Inf, NaN),
// bit 1 = the counts do not add up to d.
__global__ void __launch_bounds__(256)
k_hist_check(const unsigned long long* __restrict__ hist_all, uint64_t d, uint32_t* __restrict__ flags) {
  __shared__ unsigned long long s_sum[8];
  __shared__ uint32_t s_nonfinite;
  const unsigned long long* hist = hist_all + (size_t)blockIdx.x * CVLC_HIST_BINS;
  if (threadIdx.x == 0) s_nonfinite = 0;
  __syncthreads();
  unsigned long long sum = 0;
  for (int j = threadIdx.x; j < CVLC_HIST_BINS; j += 256) {
    const unsigned long long h = hist[j];
    sum += h;
    if (j >= (int)(0x7F800000u >> 19) && h != 0) s_nonfinite = 1u;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(kFull, sum, off);
  if ((threadIdx.x & 31) == 0) s_sum[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long tot = 0;
    for (int w = 0; w < 8; ++w) tot += s_sum[w];
    flags[blockIdx.x] = s_nonfinite | ((tot != d) ? 2u : 0u);
  }
}

template <int CAP>
static cudaError_t launch_plan_from_hist_t(const ClientDesc* clients, uint32_t n, const Shape& shape,
                                           const unsigned long long* hist, void* ws, cudaStream_t st) {
  cudaError_t e = plan_attributes<CAP>();
  if (e != cudaSuccess) return e;
  BatchDesc<CAP> batch;
  fill_batch(batch, clients, n);
  unsigned char* w = static_cast<unsigned char*>(ws);
  uint32_t* flags = reinterpret_cast<uint32_t*>(w + plan_off_flags(n));
  const Partition part = make_partition(shape.d, n);
  {
    // status word, header, tuning keys and leaders start at zero: the header stays unmarked, so an encode call
    // cannot take this workspace for one that holds segment tables
    LaunchScope ls(kKZeroWords, st);
    k_zero_words<<<1, 64, 0, st>>>(reinterpret_cast<uint32_t*>(w), kPlanWsHist / 4);
  }
  {
    LaunchScope ls(kKZeroWords, st);
    k_zero_words<<<8, 256, 0, st>>>(reinterpret_cast<uint32_t*>(w + plan_off_keys(n)), (plan_off_seg_count(n) - plan_off_keys(n)) / 4);
  }
  {
    LaunchScope ls(kKHistCheck, st);
    k_hist_check<<<n, 256, 0, st>>>(hist, shape.d, flags);
  }
  {
    LaunchScope ls(kKPlanFit, st);
    k_plan_fit<CAP><<<n, kPlanThreads, kFitSmem, st>>>(hist, flags, batch, shape, part, w, 0);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return launch_plan_back_t<CAP>(clients, n, shape, ws, st);
}

cudaError_t launch_plan_from_hist(const ClientDesc* clients, uint32_t n, const Shape& shape,
                                  const unsigned long long* hist, void* ws, cudaStream_t st) {
  if (n <= (uint32_t)kSmallBatch) return launch_plan_from_hist_t<kSmallBatch>(clients, n, shape, hist, ws, st);
  return launch_plan_from_hist_t<kLargeBatch>(clients, n, shape, hist, ws, st);
}

// ===================================================================================
// Problem P2 with real-valued packet sizes (Section IV-C; Algorithm 1 steps 2-14 with the equidistant
// search over k of Section IV-D): a plan only, for comparing its error bound with the integer-length rule
// ===================================================================================
// One warp per value of k.  For that k the packets start equal and are re-split two consecutive ones at a time,
// r = 2 .. R in order (each re-split sees the previous one: the sweep is sequential by definition); a re-split
// minimises Eq. (7), strongly convex in the split (Lemma 2), by bracketing: the 32 lanes evaluate 32 equidistant
// splits of the bracket, the bracket shrinks to the neighbours of the best one, eight times.  All arithmetic is
// binary64 with separately rounded operations in a fixed order, so the result does not depend on the machine.

struct LiteralArgs {
  double bH, s, B, P_min, P_max, tol, alpha_q;
  unsigned long long k_lo, k_hi, d;
  uint32_t R, n_k, max_sweeps, quantizer;
};

// the bracket of Eq. (5) for a packet of P records at the length the packet constraint leaves: y = (b - H) / P - s
__device__ __forceinline__ double literal_cost(double P, const LiteralArgs& a) {
  const double y = __dsub_rn(__ddiv_rn(a.bH, P), a.s);
  double Q;
  if (a.quantizer == CVLC_QUANT_QSGD) {
    const double sq = __dsub_rn(series_exp2(__dsub_rn(y, 1.0)), 1.0);
    const double Q1 = __ddiv_rn(P, __dmul_rn(sq, sq));
    const double Q2 = __ddiv_rn(__dsqrt_rn(P), sq);
    Q = (Q1 < Q2) ? Q1 : Q2;
  } else {
    const double L = __dsub_rn(series_exp2(y), 1.0);
    Q = __ddiv_rn(P, __dmul_rn(L, L));
  }
  const double one_m = __dsub_rn(1.0, __ddiv_rn(1.0, a.B));
  return __dadd_rn(__ddiv_rn(Q, __dmul_rn(a.B, a.B)), __dmul_rn(one_m, one_m));
}

__device__ __forceinline__ double literal_energy(double Z, double beta, double D) {
  return __ddiv_rn(__dsub_rn(series_powr(__dadd_rn(Z, 1.0), beta), 1.0), D);
}

// Eq. (7) as a function of p = P_r: X = P_{r-1} + P_r, Z0 = Z_{r-2}, Z2 = Z_r
__device__ __forceinline__ double literal_pair_f(double p, double X, double Z0, double Z2, const LiteralArgs& a, double beta, double D) {
  const double Em = literal_energy(__dadd_rn(Z0, __dsub_rn(X, p)), beta, D);
  const double hi_part = __dmul_rn(literal_cost(p, a), __dsub_rn(literal_energy(Z2, beta, D), Em));
  const double lo_part = __dmul_rn(literal_cost(__dsub_rn(X, p), a), __dsub_rn(Em, literal_energy(Z0, beta, D)));
  return __dadd_rn(hi_part, lo_part);
}

__global__ void __launch_bounds__(32)
k_plan_literal(const __grid_constant__ LiteralArgs a, unsigned long long* __restrict__ k_grid, double* __restrict__ gamma_of_k,
               uint32_t* __restrict__ sweeps_of_k, double* __restrict__ P_all) {
  extern __shared__ double lit_smem[];  // P[R], Z[R + 1]
  double* P = lit_smem;
  double* Z = lit_smem + a.R;
  const int lane = threadIdx.x;
  const uint32_t ik = blockIdx.x, R = a.R;
  const double beta = __dadd_rn(__dmul_rn(2.0, a.alpha_q), 1.0);
  const double D = __dsub_rn(series_powr((double)a.d, beta), 1.0);
  // equidistant values of k; the product stays below 2^64 (n_k <= 4096, k <= 2^31 * 2^31 is never reached: k <= d)
  const unsigned long long k = (a.n_k == 1) ? a.k_lo : a.k_lo + ((unsigned long long)ik * (a.k_hi - a.k_lo)) / (a.n_k - 1);
  const double P0 = __ddiv_rn((double)k, (double)R);
  for (uint32_t r = lane; r < R; r += 32) P[r] = P0;
  __syncwarp();
  uint32_t sweep = 0;
  for (; sweep < a.max_sweeps; ++sweep) {
    if (lane == 0) {
      double z = 0.0;
      Z[0] = 0.0;
      for (uint32_t r = 0; r < R; ++r) {
        z = __dadd_rn(z, P[r]);
        Z[r + 1] = z;
      }
    }
    __syncwarp();
    double moved = 0.0;
    for (uint32_t r = 1; r < R; ++r) {
      const double Pr = P[r];
      const double X = __dadd_rn(P[r - 1], Pr), Z0 = Z[r - 1], Z2 = Z[r + 1];
      double lo = __ddiv_rn(X, 2.0), hi = __dsub_rn(X, a.P_min);
      if (lo < a.P_min) lo = a.P_min;
      const double lo2 = __dsub_rn(X, a.P_max);
      if (lo < lo2) lo = lo2;
      if (hi > a.P_max) hi = a.P_max;
      if (!(lo < hi)) continue;
      double best_x = lo;
      for (int round = 0; round < 8; ++round) {
        const double step = __ddiv_rn(__dsub_rn(hi, lo), 31.0);
        const double xj = (lane == 31) ? hi : __dadd_rn(lo, __dmul_rn((double)lane, step));
        double f = literal_pair_f(xj, X, Z0, Z2, a, beta, D);
        int j = lane;
        // the first of the smallest values
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          const double fo = __shfl_xor_sync(kFull, f, off);
          const int jo = __shfl_xor_sync(kFull, j, off);
          if (fo < f || (fo == f && jo < j)) {
            f = fo;
            j = jo;
          }
        }
        const double nlo = (j == 0) ? lo : __dadd_rn(lo, __dmul_rn((double)(j - 1), step));
        const double nhi = (j >= 30) ? hi : __dadd_rn(lo, __dmul_rn((double)(j + 1), step));
        best_x = (j == 31) ? hi : __dadd_rn(lo, __dmul_rn((double)j, step));
        lo = nlo;
        hi = nhi;
      }
      // lanes 0 and 1 evaluate the new and the current split
      const double fe = literal_pair_f(lane == 0 ? best_x : Pr, X, Z0, Z2, a, beta, D);
      const double f_new = __shfl_sync(kFull, fe, 0), f_old = __shfl_sync(kFull, fe, 1);
      if (f_new < f_old) {
        const double delta = fabs(__dsub_rn(best_x, Pr));
        if (delta > moved) moved = delta;
        if (lane == 0) {
          const double Pm = __dsub_rn(X, best_x);
          P[r - 1] = Pm;
          P[r] = best_x;
          Z[r] = __dadd_rn(Z0, Pm);
        }
      }
      __syncwarp();
    }
    if (!(moved > a.tol)) {
      ++sweep;
      break;
    }
  }
  // Eq. (5) at these packet sizes: the terms side by side, their sum in packet order
  if (lane == 0) {
    double z = 0.0;
    Z[0] = 0.0;
    for (uint32_t r = 0; r < R; ++r) {
      z = __dadd_rn(z, P[r]);
      Z[r + 1] = z;
    }
  }
  __syncwarp();
  double* P_out = P_all + (size_t)ik * R;
  double* term = P_out;  // the terms borrow the output slots; the packet sizes follow once the sum is taken
  for (uint32_t r = lane; r < R; r += 32) {
    const double Eprev = (r == 0) ? 0.0 : literal_energy(Z[r], beta, D);
    const double Ecur = literal_energy(Z[r + 1], beta, D);
    term[r] = __dmul_rn(literal_cost(P[r], a), __dsub_rn(Ecur, Eprev));
  }
  __syncwarp();
  if (lane == 0) {
    double gamma = __dsub_rn(1.0, literal_energy(Z[R], beta, D));
    for (uint32_t r = 0; r < R; ++r) gamma = __dadd_rn(gamma, term[r]);
    gamma_of_k[ik] = gamma;
    k_grid[ik] = k;
    sweeps_of_k[ik] = sweep;
  }
  __syncwarp();
  for (uint32_t r = lane; r < R; r += 32) P_out[r] = P[r];
}

// the value of k with the smallest error bound (the first one on ties) and its packet sizes
__global__ void __launch_bounds__(256)
k_plan_literal_pick(const __grid_constant__ LiteralArgs a, const unsigned long long* __restrict__ k_grid,
                    const double* __restrict__ gamma_of_k, const uint32_t* __restrict__ sweeps_of_k,
                    const double* __restrict__ P_all, cvlc_literal_plan_t* __restrict__ out, double* __restrict__ P_star) {
  __shared__ uint32_t s_best;
  if (threadIdx.x == 0) {
    uint32_t best = 0;
    for (uint32_t i = 1; i < a.n_k; ++i)
      if (gamma_of_k[i] < gamma_of_k[best]) best = i;
    s_best = best;
    out->status = CVLC_OK;
    out->R = a.R;
    out->n_k = a.n_k;
    out->sweeps = sweeps_of_k[best];
    out->k_star = k_grid[best];
    out->gamma_star = gamma_of_k[best];
    out->alpha_q = a.alpha_q;
    out->beta = __dadd_rn(__dmul_rn(2.0, a.alpha_q), 1.0);
  }
  __syncthreads();
  if (P_star)
    for (uint32_t r = threadIdx.x; r < a.R; r += 256) P_star[r] = P_all[(size_t)s_best * a.R + r];
}

cudaError_t launch_plan_literal(const cvlc_params& p, double alpha_q, uint32_t s, uint32_t R, uint32_t n_k, uint32_t max_sweeps,
                                unsigned long long k_lo, unsigned long long k_hi, double P_min, double P_max, double tol,
                                cvlc_literal_plan_t* out, double* P_star, void* ws, cudaStream_t st) {
  LiteralArgs a;
  a.bH = (double)(p.packet_bits - p.header_bits);
  a.s = (double)s;
  a.B = p.scale_B;
  a.P_min = P_min;
  a.P_max = P_max;
  a.tol = tol;
  a.alpha_q = alpha_q;
  a.k_lo = k_lo;
  a.k_hi = k_hi;
  a.d = p.d;
  a.R = R;
  a.n_k = n_k;
  a.max_sweeps = max_sweeps;
  a.quantizer = p.quantizer;
  unsigned char* w = static_cast<unsigned char*>(ws);
  unsigned long long* k_grid = reinterpret_cast<unsigned long long*>(w + literal_off_k(n_k));
  double* gamma_of_k = reinterpret_cast<double*>(w + literal_off_gamma(n_k));
  uint32_t* sweeps_of_k = reinterpret_cast<uint32_t*>(w + literal_off_sweeps(n_k));
  double* P_all = reinterpret_cast<double*>(w + literal_off_P(n_k));
  {
    LaunchScope ls(kKPlanLiteral, st);
    k_plan_literal<<<n_k, 32, (2 * (size_t)R + 1) * 8, st>>>(a, k_grid, gamma_of_k, sweeps_of_k, P_all);
  }
  {
    LaunchScope ls(kKPlanLiteral, st);
    k_plan_literal_pick<<<1, 256, 0, st>>>(a, k_grid, gamma_of_k, sweeps_of_k, P_all, out, P_star);
  }
  return cudaGetLastError();
}

// ---- diagnostics ---------------------------------------------------------------------

__global__ void k_selftest_philox(uint64_t seed, uint32_t client_id, uint32_t round, uint64_t first, uint64_t n, uint32_t* out) {
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t c = first + i;
    const uint4 r = philox4x32_10(make_uint4((uint32_t)c, (uint32_t)(c >> 32), client_id, round),
                                  make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
    out[4 * i + 0] = r.x;
    out[4 * i + 1] = r.y;
    out[4 * i + 2] = r.z;
    out[4 * i + 3] = r.w;
  }
}

__global__ void k_selftest_math(const double* in, uint64_t n, double* l2, double* e2, double* dv, double* dr) {
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const double v = in[i];
    if (l2) l2[i] = (v > 0.0) ? series_log2(v) : 0.0;
    if (e2) e2[i] = (fabs(v) <= 1000.0) ? series_exp2(v) : 0.0;
    if (dv && dr) {
      for (int j = 1; j <= 20; ++j) {
        dv[i * 20 + j - 1] = div_small_int(v, j);
        dr[i * 20 + j - 1] = __ddiv_rn(v, (double)j);
      }
    }
  }
}

cudaError_t launch_selftest_philox(uint64_t seed, uint32_t client_id, uint32_t round, uint64_t first, uint64_t n,
                                   uint32_t* out, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  { LaunchScope ls(kKSelftest, st); k_selftest_philox<<<kNumSM, 256, 0, st>>>(seed, client_id, round, first, n, out); }
  return cudaGetLastError();
}

cudaError_t launch_selftest_math(const double* in, uint64_t n, double* l2, double* e2, double* dv, double* dr,
                                 cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  { LaunchScope ls(kKSelftest, st); k_selftest_math<<<kNumSM, 256, 0, st>>>(in, n, l2, e2, dv, dr); }
  return cudaGetLastError();
}

}  // namespace cvlc
