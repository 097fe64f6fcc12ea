// Encoding kernels (Algorithm 1, steps 15-17), batched over clients: top-k candidate
// selection by the plan's histogram threshold, stable LSD radix ranking of the candidates
// by |x|, the per-packet centroid distribution (PQ: minimum and maximum; QSGD: l2-norm),
// stochastic quantization with Philox4x32-10 (PQ or QSGD) and bit packing of
// (position ID, centroid ID) pairs into fixed-size packets (Fig. 2).
#include "cvlc_common.cuh"
#include "cvlc_lookback.cuh"
#include "cvlc_quant.cuh"

namespace cvlc {

constexpr unsigned kFull = 0xFFFFFFFFu;
// Whether an earlier kernel of the call has reported an error.  Other blocks may set the word while this kernel
// runs, so one thread reads it and the whole block takes the same branch.
__device__ __forceinline__ bool block_sees_error(const int32_t* status) {
  __shared__ int s_err;
  if (threadIdx.x == 0) s_err = *reinterpret_cast<const volatile int32_t*>(status);
  __syncthreads();
  return s_err != 0;
}

__device__ __forceinline__ uint32_t sort_tiles_of(unsigned long long n_candidates, unsigned long long capacity) {
  const unsigned long long nc = n_candidates < capacity ? n_candidates : capacity;
  return (uint32_t)((nc + kSortTile - 1) / kSortTile);
}

// ===================================================================================
// K0  workspace reset, plan validation, sort-tile prefix over the clients
// ===================================================================================
// The grid zeroes the per-client counters, digit histograms and look-back states; block 0
// alone owns the 256-byte header and the sort-tile prefix (nobody else writes them).

template <int CAP>
__global__ void __launch_bounds__(256)
k_encode_init(unsigned char* ws, const __grid_constant__ BatchDesc<CAP> batch, const __grid_constant__ Shape shape,
              const __grid_constant__ EncLayout L, const unsigned char* plan_ws, const __grid_constant__ Partition part) {
  __shared__ unsigned long long s_total;
  __shared__ int s_bad, s_pass3;
  __shared__ uint32_t s_tiles[CVLC_MAX_BATCH];  // sort tiles of every client
  const uint32_t n = batch.n;
  if (threadIdx.x == 0) {
    s_total = 0;
    s_bad = 0;
    s_pass3 = 0;
  }
  __syncthreads();
  {
    unsigned long long t = 0;
    int pass3 = 0;
    for (uint32_t c = threadIdx.x; c < n; c += blockDim.x) {  // the plans are read side by side, not one after the other
      const cvlc_plan_t* plan = batch.c[c].plan;
      const uint32_t tiles = sort_tiles_of(plan->n_candidates, L.capacity);
      s_tiles[c] = tiles;
      t += tiles;
      if (plan->top_bin + 1u - plan->thresh_bin > 256u) pass3 = 1;  // see top_digit_is_zero
    }
    if (t) atomicAdd(&s_total, t);
    if (pass3) atomicOr(&s_pass3, 1);
  }
  __syncthreads();
  const size_t gtid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t gstride = (size_t)gridDim.x * blockDim.x;
  {
    unsigned long long* a = reinterpret_cast<unsigned long long*>(ws + L.off_n_selected);
    for (size_t i = gtid; i < n; i += gstride) a[i] = 0ull;
    unsigned long long* b = reinterpret_cast<unsigned long long*>(ws + L.off_ghist);
    const size_t nb = (L.off_sort_state - L.off_ghist) / 8;  // digit histograms, their scans, selection tile states
    for (size_t i = gtid; i < nb; i += gstride) b[i] = 0ull;
  }
  // look-back states of the digit passes that will run (the fourth only if some client's keys span more than 2^27)
  const size_t per_pass = (size_t)s_total * kDigits;
  const int n_passes = s_pass3 ? kSortPasses : kSortPasses - 1;
  for (int p = 0; p < n_passes; ++p) {
    ulonglong2* st = reinterpret_cast<ulonglong2*>(reinterpret_cast<unsigned long long*>(ws + L.off_sort_state) +
                                                   (size_t)p * n * L.sort_tiles_max * kDigits);
    for (size_t i = gtid; i < per_pass / 2; i += gstride) st[i] = make_ulonglong2(0ull, 0ull);
  }
  if (blockIdx.x != 0) return;

  EncHeader* hdr = reinterpret_cast<EncHeader*>(ws);
  uint32_t* prefix = reinterpret_cast<uint32_t*>(ws + L.off_sort_prefix);
  for (uint32_t c = threadIdx.x; c < n; c += blockDim.x) {
    // Only what selection and ranking use is checked here (the code lengths may still be on their way on
    // another stream); the packing kernel checks the lengths.
    const cvlc_plan_t* plan = batch.c[c].plan;
    int bad = 0;
    if (plan->status != CVLC_OK)
      bad = plan->status;
    else if (plan->s != shape.s || plan->R != shape.R || plan->n_candidates == 0 || plan->n_candidates > shape.d ||
             plan->thresh_bin >= CVLC_HIST_BINS || plan->top_bin >= CVLC_HIST_BINS || plan->top_bin < plan->thresh_bin)
      bad = CVLC_ERR_PLAN_MISMATCH;
    else if (plan->n_candidates > L.capacity)
      bad = CVLC_ERR_WORKSPACE_TOO_SMALL;
    if (bad) atomicCAS(&s_bad, 0, bad);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t run = 0, mx = 0;
    for (uint32_t c = 0; c < n; ++c) {
      prefix[c] = run;
      const uint32_t t = s_tiles[c];
      run += t;
      if (t > mx) mx = t;
    }
    prefix[n] = run;
    if (plan_ws && !s_bad) {
      // the segment tables must have been made for this very batch
      const PlanWsHeader* ph = reinterpret_cast<const PlanWsHeader*>(plan_ws);
      if (ph->magic != kPlanWsMagic || ph->n != n || ph->d != shape.d || ph->n_chunks != part.n_chunks) s_bad = CVLC_ERR_PLAN_MISMATCH;
    }
    hdr->max_sort_tiles = mx;
    hdr->status = s_bad;
    hdr->select_ticket = 0;
    for (int p = 0; p < kSortPasses; ++p) hdr->sort_ticket[p] = 0;
    hdr->total_sort_tiles = run;
  }
}

// ===================================================================================
// K3  threshold selection + order-preserving compaction (single pass, decoupled look-back)
// ===================================================================================
// Emits (key << 32 | sign << 31 | index) for every coordinate whose histogram bin is at or
// above the plan's threshold bin, in ascending index order.  4 bytes read per coordinate.
// Tiles of 8192 coordinates are handed out by an atomic ticket (tile-major, clients interleaved:
// the tiles in flight at any time are a few consecutive tiles of every client), so every
// predecessor of a tile is running or done; the look-back reads 512 predecessors per step.
// Used when the plan's workspace (and with it the per-segment counts) is not available.

template <int CAP>
__global__ void __launch_bounds__(kSelectThreads)
k_select_lookback(const __grid_constant__ BatchDesc<CAP> batch, uint64_t d, unsigned char* ws, const __grid_constant__ EncLayout L) {
  __shared__ uint32_t s_tile;
  __shared__ unsigned long long s_warp_incl[kSelectThreads / 32];
  __shared__ unsigned long long s_look_sum[kSelectThreads / 32];
  __shared__ uint32_t s_look_flag[kSelectThreads / 32];
  EncHeader* hdr = reinterpret_cast<EncHeader*>(ws);
  if (block_sees_error(&hdr->status)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint64_t tiles_per_client = L.select_tiles;
  const uint64_t total_tiles = tiles_per_client * batch.n;
  unsigned long long* n_selected = reinterpret_cast<unsigned long long*>(ws + L.off_n_selected);

  while (true) {
    if (tid == 0) s_tile = atomicAdd(&hdr->select_ticket, 1u);
    __syncthreads();
    const uint64_t gt = s_tile;
    if (gt >= total_tiles) break;
    const uint64_t tile = gt / batch.n;
    const uint32_t c = (uint32_t)(gt - tile * batch.n);
    const float* __restrict__ x = batch.c[c].x;
    const cvlc_plan_t* __restrict__ plan = batch.c[c].plan;
    const float4* xv = reinterpret_cast<const float4*>(x);
    const uint32_t thresh = plan->thresh_bin << 19;
    unsigned long long* tile_state = reinterpret_cast<unsigned long long*>(ws + L.off_select_state) + (size_t)c * tiles_per_client;
    unsigned long long* __restrict__ out = reinterpret_cast<unsigned long long*>(ws + L.off_buf_a) + (size_t)c * L.capacity;
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
        for (int cc = 0; cc < 4; ++cc) {
          bits[v][cc] = 0;
          if (e0 + cc < d) {
            bits[v][cc] = __float_as_uint(x[e0 + cc]);
            valid |= 1u << cc;
          }
        }
      }
      uint32_t m = 0;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) m |= (((bits[v][cc] & 0x7FFFFFFFu) >= thresh) ? 1u : 0u) << cc;
      mask[v] = m & valid;
    }
    // block scan of the four per-vector counts, packed 16 bits each (tile totals <= 2048)
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

    // decoupled look-back: thread i inspects predecessor (tile - 1 - i) of this client
    if (tid == 0) st_relaxed(tile_state + tile, (tile == 0 ? kFlagPrefix : kFlagAgg) | tile_total);
    unsigned long long run = 0;
    if (tile > 0) {
      long long base = (long long)tile - 1;
      while (true) {
        const long long idx = base - tid;
        unsigned long long sv = kFlagPrefix;  // before tile 0: empty prefix
        if (idx >= 0) sv = wait_state(tile_state + idx, &hdr->status);
        const bool to = (sv == 0);
        const unsigned is_prefix = __ballot_sync(kFull, (sv & kFlagMask) == kFlagPrefix);
        unsigned long long val = sv & kValMask;
        if (is_prefix) {
          const int firstp = __ffs(is_prefix) - 1;
          if (lane > firstp) val = 0;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) val += __shfl_xor_sync(kFull, val, off);
        if (lane == 0) {
          s_look_sum[warp] = val;
          s_look_flag[warp] = is_prefix ? 1u : 0u;
        }
        const int any_to = __syncthreads_or(to);
        // the nearest warp (smallest distance) that saw a prefix ends the walk
        bool found = false;
        unsigned long long add = 0;
#pragma unroll
        for (int w = 0; w < kSelectThreads / 32; ++w) {
          if (!found) {
            add += s_look_sum[w];
            found = s_look_flag[w] != 0;
          }
        }
        run += add;
        __syncthreads();
        if (any_to || found) break;  // after a timeout the status is set and the results are void
        base -= kSelectThreads;
      }
      if (tid == 0) st_relaxed(tile_state + tile, kFlagPrefix | (run + tile_total));
    }
    if (tid == 0 && tile == tiles_per_client - 1) {
      n_selected[c] = run + tile_total;
      if (run + tile_total != plan->n_candidates) set_status(&hdr->status, CVLC_ERR_PLAN_MISMATCH);
    }
    unsigned long long vec_base = 0;
#pragma unroll
    for (int v = 0; v < kSelectVecPerThread; ++v) {
      unsigned long long o = run + vec_base + ((excl >> (16 * v)) & 0xFFFF);
      const uint64_t e0 = (base_vec + (uint64_t)v * kSelectThreads + tid) * 4;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        if (mask[v] & (1u << cc)) {
          const uint32_t b = bits[v][cc];
          const unsigned long long pair = ((unsigned long long)(b & 0x7FFFFFFFu) << 32) | (unsigned long long)(b & 0x80000000u) |
                                          (unsigned long long)(e0 + cc);
          if (o < L.capacity) out[o] = pair;
          ++o;
        }
      }
      vec_base += (tot >> (16 * v)) & 0xFFFF;
    }
    __syncthreads();  // s_tile and the look-back scratch are reused by the next tile
  }
}

// ===================================================================================
// K3' threshold selection with offsets known in advance (no exchange between blocks)
// ===================================================================================
// Same chunking of the concatenated updates as the histogram kernel: block b streams its chunk
// once with 128-bit loads, one tile (8192 coordinates) ahead of the compaction.  The number of
// candidates in every earlier segment of the client is known from the per-segment histograms
// (seg_prefix, written by the planner), so the output position of a candidate is
// seg_prefix + its rank inside the block's segment: a block-level scan per tile and nothing else.

constexpr int kSelStages = 3;  // tiles in flight per block (cp.async groups)
constexpr size_t kSelStageBytes = (size_t)kSelectThreads * kSelectVecPerThread * 16;  // 32 KB

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// sort key digits (see the ranking kernels below); the selection kernel already counts them
__device__ __forceinline__ uint32_t sort_keytop(const cvlc_plan_t* plan) { return ((plan->top_bin + 1u) << 19) - 1u; }
// With at most 256 histogram bins between the threshold and the top, keytop - key stays below 2^27 for every
// candidate: the fourth digit is zero throughout and neither counted nor ranked.
__device__ __forceinline__ bool top_digit_is_zero(const cvlc_plan_t* plan) { return plan->top_bin + 1u - plan->thresh_bin <= 256u; }

__device__ __forceinline__ uint32_t sort_digit(unsigned long long pair, int pass, uint32_t keytop) {
  const uint32_t key = (uint32_t)(pair >> 32);
  const uint32_t inv = key > keytop ? 0u : keytop - key;  // key > keytop only if the plan is not of this update
  return (inv >> (kDigitBits * pass)) & (kDigits - 1);
}

// Staging layout: float4 unit g of a tile (g = 0 .. 2047, in memory order) sits in slot
// g ^ ((g >> 3) & 3).  The copies of a warp (consecutive g) and the reads of a warp (thread t
// reads its own four consecutive units 4t .. 4t+3) are then both free of bank conflicts.
constexpr int kSelThreads = 512;                      // threads of the selection kernel
constexpr int kSelVec = 4;                            // float4 units (16 coordinates) per thread and tile
constexpr uint32_t kSelTileVec = kSelThreads * kSelVec;  // 2048 float4 = 8192 coordinates = 32 KB
static_assert(kSelTileVec * 16 == kSelStageBytes, "stage size");
__device__ __forceinline__ uint32_t sel_slot(uint32_t g) { return g ^ ((g >> 3) & (uint32_t)(kSelVec - 1)); }

template <int CAP>
__global__ void __launch_bounds__(kSelThreads, 2)
k_select(const __grid_constant__ BatchDesc<CAP> batch, uint64_t d, const __grid_constant__ Partition part,
         const unsigned char* __restrict__ plan_ws, unsigned char* ws, const __grid_constant__ EncLayout L) {
  extern __shared__ float4 s_stage[];  // [kSelStages][2048 float4]
  __shared__ uint32_t s_warp_incl[2][kSelThreads / 32];
  __shared__ uint32_t s_dhist[kSortPasses * kDigits];  // digit histograms of the segment's candidates (for the ranking passes)
  for (int i = threadIdx.x; i < kSortPasses * kDigits; i += kSelThreads) s_dhist[i] = 0;
  __syncthreads();
  EncHeader* hdr = reinterpret_cast<EncHeader*>(ws);
  if (block_sees_error(&hdr->status)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t S = part.max_segments;
  const uint32_t* seg_count = reinterpret_cast<const uint32_t*>(plan_ws + plan_off_seg_count(batch.n));
  const unsigned long long* seg_prefix = reinterpret_cast<const unsigned long long*>(plan_ws + plan_off_seg_prefix(batch.n, S));
  // per segment, the rows of 32 units that hold a candidate, in ascending order (from the planner)
  const uint32_t* row_list = reinterpret_cast<const uint32_t*>(plan_ws + plan_off_row_list(batch.n, S, row_tiles_total(part)));
  const uint32_t* seg_rows = reinterpret_cast<const uint32_t*>(plan_ws + plan_off_seg_rows(batch.n, S));
  unsigned long long* n_selected = reinterpret_cast<unsigned long long*>(ws + L.off_n_selected);
  const uint64_t nvec = d >> 2;
  const uint64_t units = part.units;
  constexpr uint32_t kTileVec = kSelTileVec;
  static_assert(kSelTileVec == kTileUnits && kSelVec == 4 && kRowUnits % kSelVec == 0 && 32 % kRowUnits == 0,
                "a warp stages whole rows of a tile, a thread's four units lie in one row");
  int parity = 0;
  __shared__ uint32_t s_chunk;

  while (true) {
  // chunks by ticket: a chunk full of candidates costs several times one without
  if (tid == 0) s_chunk = atomicAdd(&hdr->select_ticket, 1u);
  __syncthreads();
  const uint32_t q = s_chunk;
  if (q >= part.n_chunks) break;
  uint64_t pos = (uint64_t)q * part.chunk;
  const uint64_t end = (pos + part.chunk < part.total) ? pos + part.chunk : part.total;

  while (pos < end) {
    const uint32_t c = (uint32_t)(pos / units);
    const uint64_t seg_end = ((c + 1) * units < end) ? (c + 1) * units : end;
    const uint64_t u0 = pos - c * units, u1 = seg_end - c * units;  // units [u0, u1) of client c
    const bool with_tail = (u1 == units);                            // the segment ends with the client's tail unit
    const uint64_t v_end = with_tail ? nvec : u1;                    // float4 units [u0, v_end)
    const float* __restrict__ x = batch.c[c].x;
    const float4* __restrict__ xseg = reinterpret_cast<const float4*>(x) + u0;
    const cvlc_plan_t* __restrict__ plan = batch.c[c].plan;
    const uint32_t thresh = plan->thresh_bin << 19;
    // finite inputs: key >= thresh <=> |x| > the float just below thresh <=> (that float) - |x| is negative.  The
    // difference of two distinct floats never rounds to zero, so its sign bit is the candidate flag: one
    // subtraction and one funnel shift per coordinate.  thresh == 0: every coordinate is a candidate.
    const float below_thresh_f = __uint_as_float(thresh ? thresh - 1u : 0u);
    const uint32_t cap32 = (uint32_t)L.capacity;  // <= d <= 2^31
    const uint32_t keytop = sort_keytop(plan);
    const bool count_top = !top_digit_is_zero(plan);
    const uint32_t seg = q + c;
    unsigned long long* __restrict__ out = reinterpret_cast<unsigned long long*>(ws + L.off_buf_a) + (size_t)c * L.capacity;
    unsigned long long run = seg_prefix[seg];
    const unsigned long long run0 = run;
    const uint64_t n_vec = (v_end > u0) ? v_end - u0 : 0;        // float4 units of the segment
    // The segment's rows with candidates, a tile (kTileRows of them) at a time: tile t of the staging buffers holds the
    // rows kTileRows t .. of the list, warp w the next kRowsPerWarp of them (ascending rows in ascending lanes: index
    // order is kept).
    constexpr uint32_t kRowsPerWarp = 32 * kSelVec / kRowUnits;
    const uint32_t n_vec32 = (uint32_t)n_vec;  // a segment is at most one chunk: far below 2^32 units
    const uint32_t n_listed = seg_rows[seg];
    const uint32_t n_tiles = (n_listed + kTileRows - 1) / kTileRows;
    const uint32_t* __restrict__ list = row_list + seg_first_tile(pos, seg) * kTileRows;
    constexpr uint32_t kNoRow = 0xFFFFFFFFu;
    auto row_at = [&](uint32_t t, uint32_t slot) -> uint32_t {  // the row in slot `slot` of this warp's part of tile t
      const uint32_t idx = t * (uint32_t)kTileRows + (uint32_t)warp * kRowsPerWarp + slot;
      return (idx < n_listed) ? __ldg(list + idx) : kNoRow;
    };

    // A warp stages exactly the 128 units (512 coordinates) its own lanes will read: four copies of 32 float4s each,
    // 32 / kRowUnits rows per copy.  Waiting for a tile and reusing a staging slot are then a matter between the lanes of one
    // warp, and the block meets only once per tile, for the scan.
    struct CopyRows { uint32_t r[kSelVec]; };
    auto copy_rows_of = [&](uint32_t t) -> CopyRows {  // the rows this lane copies from in tile t, one per copy
      CopyRows cr;
#pragma unroll
      for (int v = 0; v < kSelVec; ++v) cr.r[v] = row_at(t, ((uint32_t)v * 32u + (uint32_t)lane) / kRowUnits);
      return cr;
    };
    uint32_t istage = 0;
    auto issue = [&](const CopyRows& cr) {
      float4* dst = s_stage + (size_t)istage * kTileVec;
#pragma unroll
      for (int v = 0; v < kSelVec; ++v) {
        const uint32_t g = (uint32_t)(warp * (32 * kSelVec) + v * 32 + lane);
        const uint32_t unit = cr.r[v] * (uint32_t)kRowUnits + (uint32_t)lane % kRowUnits;
        if (cr.r[v] != kNoRow && unit < n_vec32) cp_async16(dst + sel_slot(g), xseg + unit);
      }
      istage = (istage + 1 == kSelStages) ? 0u : istage + 1;
      cp_async_commit();  // one group per tile slot, empty past the end, keeps the group count uniform
    };

    static_assert(kSelStages == 3, "row indices are carried two tiles (copies) and one tile (own row) ahead");
    issue(copy_rows_of(0));
    issue(copy_rows_of(1));
    CopyRows ahead = copy_rows_of(2);                 // for the copies of tile t + 2
    const uint32_t my_slot = (uint32_t)lane * kSelVec / kRowUnits;  // the slot of the row this thread's four units lie in
    uint32_t mine = row_at(0, my_slot);                              // the row this thread reads in tile t
    uint32_t mine_next = row_at(1, my_slot);
    uint32_t stage = 0;
    for (uint32_t t = 0; t < n_tiles; ++t) {
      const CopyRows ahead2 = copy_rows_of(t + 3);    // asked for one tile before they are needed
      const uint32_t mine_next2 = row_at(t + 2, my_slot);
      cp_async_wait<kSelStages - 2>();  // this lane's copies of tile t have landed
      __syncwarp();                     // ... and the other lanes'; and the warp is done with its part of tile t - 1,
      issue(ahead);                     // whose staging slot the next copies overwrite
      ahead = ahead2;
      const uint32_t my_row = mine;
      mine = mine_next;
      mine_next = mine_next2;
      const float4* src = s_stage + (size_t)stage * kTileVec;
      stage = (stage + 1 == kSelStages) ? 0u : stage + 1;
      // this thread's 16 consecutive coordinates: four units of the row that it reads with its neighbours
      uint32_t m = 0;
      const uint32_t g0 = (uint32_t)kSelVec * tid;
      const uint32_t ct = ((uint32_t)tid >> 1) & (uint32_t)(kSelVec - 1);
      const uint32_t unit0 = my_row * (uint32_t)kRowUnits + ((uint32_t)lane * kSelVec) % kRowUnits;  // first unit of the thread, in the segment
      const uint32_t left = (my_row != kNoRow && unit0 < n_vec32) ? ((n_vec32 - unit0 < (uint32_t)kSelVec) ? n_vec32 - unit0 : (uint32_t)kSelVec) : 0u;
#pragma unroll
      for (int j = 0; j < kSelVec; ++j) {
        if ((uint32_t)j < left) {
          // units 4 tid + j sit in slots 4 tid + (j ^ ct): the swizzle only touches the two low bits
          const float4 f = src[g0 + ((uint32_t)j ^ ct)];
          m = __funnelshift_l(__float_as_uint(__fsub_rn(below_thresh_f, fabsf(f.x))), m, 1);
          m = __funnelshift_l(__float_as_uint(__fsub_rn(below_thresh_f, fabsf(f.y))), m, 1);
          m = __funnelshift_l(__float_as_uint(__fsub_rn(below_thresh_f, fabsf(f.z))), m, 1);
          m = __funnelshift_l(__float_as_uint(__fsub_rn(below_thresh_f, fabsf(f.w))), m, 1);
        } else {
          m <<= 4;
        }
      }
      if (thresh == 0u) m = (left >= (uint32_t)kSelVec) ? 0xFFFFu : (0xFFFFu << (4 * (kSelVec - left))) & 0xFFFFu;
      // coordinate c of the thread (0 .. 15, ascending index) is bit 15 - c of m
      const uint32_t cnt = __popc(m);
      // block scan of the per-thread counts: inside the warp, then over the warp totals
      uint32_t incl = cnt;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(kFull, incl, off);
        if (lane >= off) incl += o;
      }
      if (lane == 31) s_warp_incl[parity][warp] = incl;
      __syncthreads();
      const uint32_t wt = (lane < kSelThreads / 32) ? s_warp_incl[parity][lane] : 0u;
      uint32_t wincl = wt;
#pragma unroll
      for (int off = 1; off < kSelThreads / 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(kFull, wincl, off);
        if (lane >= off) wincl += o;
      }
      const uint32_t tot = __shfl_sync(kFull, wincl, kSelThreads / 32 - 1);
      const uint32_t below = __shfl_sync(kFull, wincl - wt, warp);
      parity ^= 1;
      // emit this thread's candidates (few): values are re-read from the staging buffer
      uint32_t o = (uint32_t)run + below + incl - cnt;  // positions inside a client's buffer fit 32 bits
      const uint32_t* srcw16 = reinterpret_cast<const uint32_t*>(src) + 16 * tid;  // this thread's 16 staged words
      const uint32_t cx = ct << 2;
      const uint32_t e32 = (uint32_t)((u0 + unit0) * 4);  // index of the thread's first coordinate (< 2^31)
      while (m) {
        const int hb = 31 - __clz(m);  // highest flag = lowest index first
        m ^= 1u << hb;
        const uint32_t c16 = 15u - (uint32_t)hb;
        const uint32_t b = srcw16[c16 ^ cx];
        const uint32_t key = b & 0x7FFFFFFFu;
        if (o < cap32) out[o] = ((unsigned long long)key << 32) | (unsigned long long)((b & 0x80000000u) | (e32 + c16));
        const uint32_t inv = keytop - (key < keytop ? key : keytop);
#pragma unroll
        for (int p = 0; p < kSortPasses - 1; ++p) atomicAdd(&s_dhist[p * kDigits + ((inv >> (kDigitBits * p)) & (kDigits - 1))], 1u);
        if (count_top) atomicAdd(&s_dhist[(kSortPasses - 1) * kDigits + (inv >> (kDigitBits * (kSortPasses - 1)))], 1u);
        ++o;
      }
      run += tot;
    }
    cp_async_wait<0>();
    if (with_tail && tid == 0) {
      // the client's ragged tail (d % 4 scalars) follows every float4 unit: one thread appends it
      for (uint64_t e = nvec * 4; e < d; ++e) {
        const uint32_t b = __float_as_uint(x[e]);
        if ((b & 0x7FFFFFFFu) >= thresh) {
          const unsigned long long pair = ((unsigned long long)(b & 0x7FFFFFFFu) << 32) | (unsigned long long)(b & 0x80000000u) | (unsigned long long)e;
          if (run < L.capacity) out[run] = pair;
          for (int p = 0; p < kSortPasses; ++p)
            if (p < kSortPasses - 1 || count_top) atomicAdd(&s_dhist[p * kDigits + sort_digit(pair, p, keytop)], 1u);
          ++run;
        }
      }
    }
    if (tid == 0) {
      // the update must be the one the plan was made from
      if (run - run0 != seg_count[seg]) set_status(&hdr->status, CVLC_ERR_PLAN_MISMATCH);
      if (with_tail) n_selected[c] = run;
    }
    __syncthreads();  // the staging buffers (and the ticket word) are reused by the next segment
    {
      // the segment's digit counts join the client's
      unsigned long long* ghist = reinterpret_cast<unsigned long long*>(ws + L.off_ghist) + (size_t)c * kSortPasses * kDigits;
      for (int i = tid; i < kSortPasses * kDigits; i += kSelThreads) {
        const uint32_t v = s_dhist[i];
        s_dhist[i] = 0;
        if (v) atomicAdd(ghist + i, (unsigned long long)v);
      }
      __syncthreads();
    }
    pos = seg_end;
  }
  }
}

// ===================================================================================
// K4  stable LSD radix ranking of the candidates, |x| descending (ties keep ascending index)
// ===================================================================================
// Sort key = keytop - key, keytop = the largest key of the client's highest non-empty histogram
// bin, so the key only spans the bins between the threshold and the top: 19 + log2(#bins) bits.
// Digits of 9, 9, 9, 4 bits.  One histogram kernel for all four digits and all clients, a small
// scan kernel, then one single-pass kernel per digit (tiles handed out by ticket, tile-major with
// the clients interleaved; decoupled look-back per digit value).  A pass whose digit is the same
// for every candidate of a client (normally the fourth) is skipped for that client; which buffer
// holds its data after pass q follows from the mask of skipped passes.

// The clients' candidate arrays are concatenated in units of sort tiles (kSortTile pairs) and cut
// into equal contiguous chunks, one per block; a block that crosses a client boundary merges
// its shared histograms into that client's and starts afresh.
template <int CAP>
__global__ void __launch_bounds__(256)
k_sort_hist(const __grid_constant__ BatchDesc<CAP> batch, unsigned char* ws, const __grid_constant__ EncLayout L) {
  __shared__ uint32_t sh[kSortPasses * kDigits];
  const EncHeader* hdr = reinterpret_cast<const EncHeader*>(ws);
  if (block_sees_error(&hdr->status)) return;
  const uint32_t* prefix = reinterpret_cast<const uint32_t*>(ws + L.off_sort_prefix);
  unsigned long long* ghist_all = reinterpret_cast<unsigned long long*>(ws + L.off_ghist);
  for (int i = threadIdx.x; i < kSortPasses * kDigits; i += 256) sh[i] = 0;
  __syncthreads();
  const uint32_t total_tiles = prefix[batch.n];
  const uint32_t chunk = (total_tiles + gridDim.x - 1) / gridDim.x;
  uint32_t t = blockIdx.x * chunk;
  const uint32_t t_end = (t + chunk < total_tiles) ? t + chunk : total_tiles;
  uint32_t c = 0;
  while (t < t_end) {
    while (prefix[c + 1] <= t) ++c;  // client of tile t (clients without tiles are passed over)
    const uint32_t seg_end = prefix[c + 1] < t_end ? prefix[c + 1] : t_end;
    const unsigned long long n = batch.c[c].plan->n_candidates;
    const uint32_t keytop = sort_keytop(batch.c[c].plan);
    const int n_count = top_digit_is_zero(batch.c[c].plan) ? kSortPasses - 1 : kSortPasses;
    const unsigned long long* __restrict__ in = reinterpret_cast<const unsigned long long*>(ws + L.off_buf_a) + (size_t)c * L.capacity;
    const unsigned long long i0 = (unsigned long long)(t - prefix[c]) * kSortTile;
    unsigned long long i1 = (unsigned long long)(seg_end - prefix[c]) * kSortTile;
    if (i1 > n) i1 = n;
    for (unsigned long long i = i0 + threadIdx.x; i < i1; i += 256) {
      const unsigned long long pair = in[i];
#pragma unroll
      for (int p = 0; p < kSortPasses; ++p)
        if (p < n_count) atomicAdd(&sh[p * kDigits + sort_digit(pair, p, keytop)], 1u);
    }
    __syncthreads();
    unsigned long long* ghist = ghist_all + (size_t)c * kSortPasses * kDigits;
    for (int i = threadIdx.x; i < kSortPasses * kDigits; i += 256) {
      const uint32_t v = sh[i];
      sh[i] = 0;
      if (v) atomicAdd(ghist + i, (unsigned long long)v);
    }
    __syncthreads();
    t = seg_end;
  }
}

// per client: exclusive scans of the four digit histograms and the mask of constant digits
template <int CAP>
__global__ void __launch_bounds__(kDigits)
k_sort_scan(const __grid_constant__ BatchDesc<CAP> batch, unsigned char* ws, const __grid_constant__ EncLayout L) {
  __shared__ unsigned long long s_scan[kDigits / 32];
  const EncHeader* hdr = reinterpret_cast<const EncHeader*>(ws);
  if (block_sees_error(&hdr->status)) return;
  const uint32_t c = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned long long n = batch.c[c].plan->n_candidates;
  const unsigned long long* ghist = reinterpret_cast<const unsigned long long*>(ws + L.off_ghist) + (size_t)c * kSortPasses * kDigits;
  unsigned long long* gbase = reinterpret_cast<unsigned long long*>(ws + L.off_gbase) + (size_t)c * kSortPasses * kDigits;
  uint32_t mask = top_digit_is_zero(batch.c[c].plan) ? 1u << (kSortPasses - 1) : 0u;  // not counted: known to be constant
  for (int p = 0; p < kSortPasses; ++p) {
    const unsigned long long cnt = ghist[p * kDigits + tid];
    if (__syncthreads_or(cnt == n)) mask |= 1u << p;
    unsigned long long incl = cnt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned long long o = __shfl_up_sync(kFull, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    unsigned long long below = 0;
    for (int w = 0; w < warp; ++w) below += s_scan[w];
    gbase[p * kDigits + tid] = below + incl - cnt;
    __syncthreads();
  }
  if (tid == 0) reinterpret_cast<uint32_t*>(ws + L.off_pass_mask)[c] = mask;
}

// two adjacent look-back words in one 128-bit access (each 64-bit half is its own atomic access)
__device__ __forceinline__ void ld_relaxed2(const unsigned long long* p, unsigned long long& a, unsigned long long& b) {
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_relaxed2(unsigned long long* p, unsigned long long a, unsigned long long b) {
  asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(a), "l"(b) : "memory");
}

struct SortShared {
  uint32_t tile;                                        // ticket of the tile being worked on
  uint32_t next;                                        // the ticket after it (known once the tile's items are requested)
  uint32_t scan_w[kSortThreads / 32];                   // warp totals of the block scan
  __align__(16) uint16_t wc[kSortThreads / 32][kDigits];  // per warp and digit value: the count, then the first slot
                                                          // (lanes index it by digit value: the banks are as random as the digits)
  uint32_t gofs[kDigits];  // per digit value: (position in dst of the tile's first item of that value) - (its slot in the tile)
  uint32_t mm[kSortThreads / 32][kDigits];  // per warp and digit value: lanes of the current row holding it (zero between rows)
};

constexpr size_t kSortSharedBytes = (sizeof(SortShared) + 15) & ~(size_t)15;
constexpr size_t sort_smem_bytes(uint32_t n) { return kSortSharedBytes + (size_t)kSortTile * 8 + (4 * (size_t)n + 1) * 4; }

// One tile of one digit pass.  FULL: the tile holds kSortTile items (no bounds checks in the item loops).
// Thread t < 256 owns the digit values 2t and 2t + 1 in the counting, scan and look-back steps.
template <bool FULL, class Prefetch>
__device__ __forceinline__ void sort_tile(SortShared& sh, unsigned long long* __restrict__ s_items,
                                          const unsigned long long* __restrict__ src, unsigned long long* __restrict__ dst,
                                          unsigned long long* __restrict__ state, const unsigned long long* __restrict__ gbase,
                                          uint32_t tile, uint32_t count, uint32_t n32, uint32_t keytop, int shift,
                                          int32_t* status, uint32_t next, Prefetch&& prefetch_next) {
  constexpr int kWarps = kSortThreads / 32;
  constexpr int IT = kSortItemsPerThread;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned lanemask_lt = (1u << lane) - 1u;
  const uint32_t wbase = (uint32_t)warp * (32 * IT) + lane;  // this thread's first item inside the tile

  unsigned long long item[IT];
  uint32_t rd[IT];  // digit value | rank among the warp's items of that value << 16
  {
    const unsigned long long* __restrict__ p = src + (size_t)tile * kSortTile + wbase;
#pragma unroll
    for (int i = 0; i < IT; ++i) item[i] = (FULL || wbase + i * 32 < count) ? p[i * 32] : ~0ull;
  }
  if (tid == 0) sh.next = next;  // waits for the ticket counter's answer, behind the item requests
  // the look-back needs the digit values' first positions in dst: requested early, used late
  unsigned long long gb0 = 0, gb1 = 0;
  if (tid < kDigits / 2) {
    const ulonglong2 g = *reinterpret_cast<const ulonglong2*>(gbase + 2 * tid);
    gb0 = g.x;
    gb1 = g.y;
  }
  // stable rank inside the warp, items in (i, lane) order.  The lanes of a row that hold the same digit value
  // find each other through a word of shared memory that each of them ORs its lane bit into (nine ballots cost
  // four times the issue slots, a match instruction one step per distinct value in the warp); all of them read
  // the warp's running count of the value, the highest lane then updates it and clears the word.
  uint32_t* mm = &sh.mm[warp][0];
#pragma unroll
  for (int i = 0; i < IT; ++i) {
    const bool valid = FULL || (wbase + i * 32 < count);
    const uint32_t key = (uint32_t)(item[i] >> 32);
    const uint32_t inv = keytop - (key < keytop ? key : keytop);  // key > keytop only if the plan is not of this update
    const uint32_t dig = (inv >> shift) & (kDigits - 1);
    if (valid) atomicOr(mm + dig, 1u << lane);
    __syncwarp();
    unsigned peers = 1u << lane;
    uint32_t pre = 0;
    if (valid) {
      peers = *reinterpret_cast<volatile uint32_t*>(mm + dig);
      pre = *reinterpret_cast<volatile uint16_t*>(&sh.wc[warp][dig]);
    }
    __syncwarp();
    rd[i] = dig | ((pre + __popc(peers & lanemask_lt)) << 16);
    if (valid && (peers >> lane) == 1u) {  // no peer in a higher lane
      sh.wc[warp][dig] = (uint16_t)(pre + __popc(peers));
      mm[dig] = 0u;
    }
    __syncwarp();
  }
  __syncthreads();
  prefetch_next(sh.next);

  // counts of the two digit values in every warp (a 32-bit word holds both), published as the tile's aggregate
  constexpr int kOwners = kDigits / 2;
  const bool owner = tid < kOwners;
  uint32_t* wc32 = reinterpret_cast<uint32_t*>(&sh.wc[0][0]);
  uint32_t tot0 = 0, tot1 = 0, incl = 0;
  unsigned long long* my_state = state + (size_t)tile * kDigits + 2 * (tid & (kOwners - 1));
  if (owner) {
    uint32_t p = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) p += wc32[w * (kDigits / 2) + tid];  // 16-bit lanes: no carry (<= kSortTile)
    tot0 = p & 0xFFFFu;
    tot1 = p >> 16;
    const unsigned long long f = (tile == 0) ? kFlagPrefix : kFlagAgg;
    st_relaxed2(my_state, f | tot0, f | tot1);
    // first slot of every digit value inside the tile: block scan in digit order
    incl = tot0 + tot1;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t o = __shfl_up_sync(kFull, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) sh.scan_w[warp] = incl;
  }
  __syncthreads();
  if (owner) {
    uint32_t below = 0;
#pragma unroll
    for (int w = 0; w < kOwners / 32; ++w) {
      const uint32_t v = sh.scan_w[w];
      if (w < warp) below += v;
    }
    const uint32_t dstart0 = below + incl - (tot0 + tot1);
    const uint32_t dstart1 = dstart0 + tot0;
    // the counters become first slots: slot of (value, warp) = first slot of the value + items of earlier warps
    {
      uint32_t t = dstart0 | (dstart1 << 16);  // both running slots stay below 2^16
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const uint32_t v = wc32[w * (kDigits / 2) + tid];
        wc32[w * (kDigits / 2) + tid] = t;
        t += v;
      }
    }
    // decoupled look-back over the client's earlier tiles, both digit values per step
    unsigned long long run0 = 0, run1 = 0;
    if (tile > 0) {
      constexpr int kWin = 4;  // predecessors requested together: one round trip for all of them
      bool open0 = true, open1 = true;
      for (long long t = (long long)tile - 1; t >= 0 && (open0 || open1); t -= kWin) {
        unsigned long long a[kWin], b[kWin];
#pragma unroll
        for (int j = 0; j < kWin; ++j) {
          a[j] = b[j] = kFlagPrefix;  // before the client's first tile: nothing, chain closed
          if (t - j >= 0) ld_relaxed2(state + (size_t)(t - j) * kDigits + 2 * tid, a[j], b[j]);
        }
#pragma unroll
        for (int j = 0; j < kWin; ++j) {
          if (!(open0 || open1)) break;
          int polls = 0;
          while ((a[j] & kFlagMask) == 0 || (b[j] & kFlagMask) == 0) {
            if (++polls > kMaxPolls) {
              set_status(status, CVLC_ERR_DEVICE_TIMEOUT);
              a[j] = b[j] = kFlagPrefix;  // give up: close both chains
              break;
            }
            if (polls > 64) __nanosleep(64);
            ld_relaxed2(state + (size_t)(t - j) * kDigits + 2 * tid, a[j], b[j]);
          }
          if (open0) {
            run0 += a[j] & kValMask;
            open0 = (a[j] & kFlagMask) != kFlagPrefix;
          }
          if (open1) {
            run1 += b[j] & kValMask;
            open1 = (b[j] & kFlagMask) != kFlagPrefix;
          }
        }
      }
      st_relaxed2(my_state, kFlagPrefix | (run0 + tot0), kFlagPrefix | (run1 + tot1));
    }
    sh.gofs[2 * tid] = (uint32_t)(gb0 + run0) - dstart0;
    sh.gofs[2 * tid + 1] = (uint32_t)(gb1 + run1) - dstart1;
  }
  __syncthreads();
  // the items go to shared memory in digit order, then out in runs of consecutive addresses
#pragma unroll
  for (int i = 0; i < IT; ++i) {
    if (FULL || wbase + i * 32 < count) {
      const uint32_t dig = rd[i] & 0xFFFFu;
      s_items[(uint32_t)sh.wc[warp][dig] + (rd[i] >> 16)] = item[i];
    }
  }
  __syncthreads();
  if (FULL) {
#pragma unroll
    for (int j = 0; j < IT; ++j) {
      const uint32_t k = j * kSortThreads + tid;
      const unsigned long long it = s_items[k];
      const uint32_t key = (uint32_t)(it >> 32);
      const uint32_t inv = keytop - (key < keytop ? key : keytop);
      const uint32_t o = sh.gofs[(inv >> shift) & (kDigits - 1)] + k;
      if (o < n32) dst[o] = it;
    }
  } else {
    for (uint32_t k = tid; k < count; k += kSortThreads) {
      const unsigned long long it = s_items[k];
      const uint32_t key = (uint32_t)(it >> 32);
      const uint32_t inv = keytop - (key < keytop ? key : keytop);
      const uint32_t o = sh.gofs[(inv >> shift) & (kDigits - 1)] + k;
      if (o < n32) dst[o] = it;
    }
  }
}

template <int CAP>
__global__ void __launch_bounds__(kSortThreads, kSortMinBlocks)
k_sort_pass(int pass, const __grid_constant__ BatchDesc<CAP> batch, unsigned char* ws, const __grid_constant__ EncLayout L) {
  static_assert(kSortThreads * 2 >= kDigits && kSortTile <= 0xFFFF, "two digit values per owning thread; 16-bit slots");
  extern __shared__ __align__(16) unsigned char s_raw[];
  SortShared& sh = *reinterpret_cast<SortShared*>(s_raw);
  unsigned long long* s_items = reinterpret_cast<unsigned long long*>(s_raw + kSortSharedBytes);  // [kSortTile] the tile's items in digit order
  uint32_t* s_prefix = reinterpret_cast<uint32_t*>(s_items + kSortTile);                         // [n + 1] first sort tile of every client
  uint32_t* s_ncand = s_prefix + (batch.n + 1);  // [n] candidates of the client
  uint32_t* s_keytop = s_ncand + batch.n;        // [n] top of its key range
  uint32_t* s_mask = s_keytop + batch.n;         // [n] its constant digits
  EncHeader* hdr = reinterpret_cast<EncHeader*>(ws);
  if (block_sees_error(&hdr->status)) return;
  const int tid = threadIdx.x;
  const uint32_t n_clients = batch.n;
  {
    const uint32_t* prefix = reinterpret_cast<const uint32_t*>(ws + L.off_sort_prefix);
    const uint32_t* pass_mask = reinterpret_cast<const uint32_t*>(ws + L.off_pass_mask);
    for (uint32_t i = tid; i <= n_clients; i += kSortThreads) s_prefix[i] = prefix[i];
    for (uint32_t i = tid; i < n_clients; i += kSortThreads) {
      const cvlc_plan_t* plan = batch.c[i].plan;
      s_ncand[i] = (uint32_t)plan->n_candidates;  // <= capacity < 2^32: checked by k_encode_init
      s_keytop[i] = sort_keytop(plan);
      s_mask[i] = pass_mask[i];
    }
  }
  for (int i = tid; i < (kSortThreads / 32) * kDigits; i += kSortThreads) (&sh.mm[0][0])[i] = 0u;
  if (tid == 0) sh.tile = atomicAdd(&hdr->sort_ticket[pass], 1u);
  __syncthreads();
  const uint32_t total_tickets = hdr->max_sort_tiles * n_clients;
  unsigned long long* state_all =
      reinterpret_cast<unsigned long long*>(ws + L.off_sort_state) + (size_t)pass * n_clients * L.sort_tiles_max * kDigits;
  uint4* s_wc4 = reinterpret_cast<uint4*>(&sh.wc[0][0]);
  const int shift = kDigitBits * pass;

  while (true) {
    const uint32_t gt = sh.tile;
    if (gt >= total_tickets) break;
    s_wc4[2 * tid] = make_uint4(0u, 0u, 0u, 0u);
    s_wc4[2 * tid + 1] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();  // everyone has read the ticket; the counters are clear
    // the next ticket is fetched while this tile is worked on
    uint32_t next = 0;
    if (tid == 0) next = atomicAdd(&hdr->sort_ticket[pass], 1u);
    // tile-major tickets with the clients interleaved: the tiles in flight are a few consecutive
    // tiles of every client, which keeps every look-back short
    const uint32_t tile = gt / n_clients;
    const uint32_t c = gt - tile * n_clients;
    const uint32_t mask = s_mask[c];
    auto source = [&](uint32_t cc, uint32_t m) -> unsigned long long* {  // buffer holding client cc's items before this pass
      const int flips = __popc(~m & ((1u << pass) - 1u));
      return reinterpret_cast<unsigned long long*>(ws + ((flips & 1) ? L.off_buf_b : L.off_buf_a)) + (size_t)cc * L.capacity;
    };
    if (tile < s_prefix[c + 1] - s_prefix[c] && !(mask & (1u << pass))) {  // else: no such tile, or a constant digit
      const uint32_t n32 = s_ncand[c];
      const uint32_t keytop = s_keytop[c];
      const int flips = __popc(~mask & ((1u << pass) - 1u));
      const unsigned long long* src = source(c, mask);
      unsigned long long* dst =
          reinterpret_cast<unsigned long long*>(ws + ((flips & 1) ? L.off_buf_a : L.off_buf_b)) + (size_t)c * L.capacity;
      unsigned long long* state = state_all + (size_t)s_prefix[c] * kDigits;
      const unsigned long long* gbase = reinterpret_cast<const unsigned long long*>(ws + L.off_gbase) +
                                        (size_t)c * kSortPasses * kDigits + (size_t)pass * kDigits;
      const uint32_t tile_first = tile * (uint32_t)kSortTile;
      const uint32_t count = (n32 - tile_first < (uint32_t)kSortTile) ? n32 - tile_first : (uint32_t)kSortTile;
      // the next tile's items are asked into L2 while this one is ranked and written
      auto prefetch_next = [&](uint32_t nt) {
        if (nt >= total_tickets) return;
        const uint32_t t2 = nt / n_clients, c2 = nt - t2 * n_clients;
        for (uint32_t l = tid; l < (uint32_t)(kSortTile / 16); l += kSortThreads) {  // 128-byte lines of 16 items
          const uint32_t line = t2 * (uint32_t)(kSortTile / 16) + l;
          if (line * 16u < s_ncand[c2]) {
            const unsigned long long* p = source(c2, s_mask[c2]) + (size_t)line * 16;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
          }
        }
      };
      if (count == (uint32_t)kSortTile)
        sort_tile<true>(sh, s_items, src, dst, state, gbase, tile, count, n32, keytop, shift, &hdr->status, next, prefetch_next);
      else
        sort_tile<false>(sh, s_items, src, dst, state, gbase, tile, count, n32, keytop, shift, &hdr->status, next, prefetch_next);
    }
    if (tid == 0) sh.tile = next;
    __syncthreads();
  }
}

// ===================================================================================
// K5  per-packet centroid distribution (PQ: min/max; QSGD: l2-norm), stochastic quantization, bit packing
// ===================================================================================
// One warp works through kPackGroup consecutive packets of one client, without block-wide barriers.  Packet r
// (longest codes first) holds ranks [Z, Z + cap(y_r)).  The packet is assembled in the warp's shared-memory
// buffer: every record ORs its bits into the (at most three) 32-bit words it touches, then the words go out with
// consecutive addresses.  The ranked pairs are read twice from global memory (statistics, then quantization);
// the second read hits in cache.  A lane quantizes about twelve records of a packet: twelve independent Philox
// chains in flight.

constexpr int kPackThreads = 128;
constexpr int kPackWarps = kPackThreads / 32;
constexpr int kPackGroup = 1;  // packets per warp (more of them amortise the length table but lengthen the tail)

template <int CAP, bool QSGD>
__global__ void __launch_bounds__(kPackThreads)
k_pack(const __grid_constant__ BatchDesc<CAP> batch, const __grid_constant__ Shape shape, unsigned char* ws,
       const __grid_constant__ EncLayout L, uint32_t warp_bytes, int write_residual) {
  extern __shared__ __align__(16) unsigned char s_pack[];  // per warp: packet words; QSGD: then cap(1) squares
  EncHeader* hdr = reinterpret_cast<EncHeader*>(ws);
  if (block_sees_error(&hdr->status)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t c = blockIdx.y;
  const ClientDesc& cd = batch.c[c];
  const cvlc_plan_t* __restrict__ plan = cd.plan;
  const uint32_t s = shape.s;
  const uint32_t H = shape.header_bits;
  const uint32_t n_words = shape.packet_bits / 32;
  unsigned char* s_mine = s_pack + (size_t)warp * warp_bytes;
  uint32_t* words = reinterpret_cast<uint32_t*>(s_mine);
  uint32_t* stream_words = reinterpret_cast<uint32_t*>(cd.stream);
  // error compensation: the encoder's input is memory + update and becomes the new memory, i.e. every sent
  // coordinate gives up what the parameter server will rebuild for it (its centroid value divided by B)
  float* __restrict__ residual = write_residual ? const_cast<float*>(cd.x) : nullptr;
  const PhiloxRoundKeys rk = philox_round_keys(cd.seed);

  const uint32_t mask = reinterpret_cast<const uint32_t*>(ws + L.off_pass_mask)[c];
  const int flips = __popc(~mask & ((1u << kSortPasses) - 1u));
  const unsigned long long* __restrict__ sorted =
      reinterpret_cast<const unsigned long long*>(ws + ((flips & 1) ? L.off_buf_b : L.off_buf_a)) + (size_t)c * L.capacity;

  // packet -> its code length and first rank: lane l holds length 32 - l (longest first) with the
  // inclusive sums of packets and of records up to and including that length
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
    // the code lengths must fill the stream's R packets with k of the selected candidates (every warp of every
    // block of the client sees the same plan and takes the same branch)
    const uint32_t tot_packets = __shfl_sync(kFull, cum, 31);
    const unsigned long long tot_records = __shfl_sync(kFull, zc, 31);
    const bool qsgd_one_bit = QSGD && __shfl_sync(kFull, ny, 31) != 0;  // a one-bit QSGD code holds no level
    if (tot_packets != shape.R || tot_records != plan->k || tot_records == 0 || tot_records > plan->n_candidates || qsgd_one_bit) {
      if (blockIdx.x == 0 && tid == 0) set_status(&hdr->status, CVLC_ERR_PLAN_MISMATCH);
      return;
    }
  }

  for (int g = 0; g < kPackGroup; ++g) {
    const uint32_t r = (blockIdx.x * kPackWarps + warp) * kPackGroup + g;
    if (r >= shape.R) break;
    const unsigned hit = __ballot_sync(kFull, r < cum);
    if (hit == 0) break;
    const int src_lane = __ffs(hit) - 1;
    const uint32_t y = CVLC_MAX_CODE_BITS - (uint32_t)src_lane;
    const unsigned long long Z = __shfl_sync(kFull, (zc - nz) + (unsigned long long)(r - (cum - ny)) * capl, src_lane);
    const uint32_t P = __shfl_sync(kFull, capl, src_lane);
    for (uint32_t w = lane; w < n_words; w += 32) words[w] = 0u;
    __syncwarp();
    const uint32_t wd = s + y;
    const unsigned long long* __restrict__ seg = sorted + Z;
    float lo, hi;  // the header's two centroid fields
    // a record's bits, low bit first from packet bit H + j * wd
    const bool narrow = wd <= 32;  // a record then touches at most two words
    auto put = [&](uint32_t j, unsigned long long rec) {
      const uint32_t bitpos = H + j * wd;
      const uint32_t w = bitpos >> 5, sh = bitpos & 31u;
      if (narrow) {
        const uint32_t r32 = (uint32_t)rec;
        const uint32_t p0 = r32 << sh, p1 = __funnelshift_l(r32, 0u, sh);  // the bits that leave the first word
        if (p0) atomicOr(words + w, p0);
        if (p1) atomicOr(words + w + 1, p1);
        return;
      }
      const unsigned long long lo64 = rec << sh;
      const uint32_t p0 = (uint32_t)lo64, p1 = (uint32_t)(lo64 >> 32);
      const uint32_t p2 = sh ? (uint32_t)(rec >> (64 - sh)) : 0u;
      if (p0) atomicOr(words + w, p0);
      if (p1) atomicOr(words + w + 1, p1);
      if (p2) atomicOr(words + w + 2, p2);
    };

    if constexpr (QSGD) {
      // ---- QSGD: |x| against the packet's l2-norm; code = sign bit above a level of s_q = 2^(y-1) - 1 steps ----
      double* sqv = reinterpret_cast<double*>(s_mine + (((size_t)n_words * 4 + 15) & ~(size_t)15));
      for (uint32_t j = lane; j < P; j += 32) {
        const double a = (double)__uint_as_float((uint32_t)(seg[j] >> 32));
        sqv[j] = __dmul_rn(a, a);  // exact: 24 x 24 bits
      }
      __syncwarp();
      // the norm is defined with the squares added in rank order in double: one lane walks the chain
      float norm = 0.0f;
      if (lane == 0) norm = qsgd_norm_of_squares(sqv, P);
      norm = __shfl_sync(kFull, norm, 0);
      lo = norm;
      hi = 0.0f;
      const uint32_t sq = (uint32_t)((1ull << (y - 1)) - 1ull);  // y >= 2: checked with the plan
      const double sqd = (double)sq;
      const double dn = (double)norm;
      const double scale = (norm > 0.0f) ? __ddiv_rn(sqd, dn) : 0.0;
      for (uint32_t j = lane; j < P; j += 32) {
        const unsigned long long pair = seg[j];
        const uint32_t key = (uint32_t)(pair >> 32);
        const uint32_t pid = (uint32_t)pair & 0x7FFFFFFFu;
        const uint32_t sign = key ? (((uint32_t)pair >> 31) & 1u) : 0u;  // -0 is stored as +0
        uint32_t level = 0;
        if (norm > 0.0f) {
          const double a = (double)__uint_as_float(key);
          const double u = __dmul_rn((double)philox_coord(rk, cd.client_id, cd.round, pid), 1.0 / 4294967296.0);
          level = qsgd_quantize_level(a, dn, sqd, sq, scale, u);
        }
        const uint32_t code = (sign << (y - 1)) | level;
        put(j, (unsigned long long)pid | ((unsigned long long)code << s));
        if (residual) {
          const float mag = (float)__dmul_rn((double)level, __ddiv_rn(dn, sqd));
          const float v = sign ? -mag : mag;
          const float xv = __uint_as_float(key ? (key | ((uint32_t)pair & 0x80000000u)) : 0u);
          residual[pid] = __fsub_rn(xv, (float)__ddiv_rn((double)v, cd.scale_B));
        }
      }
    } else {
      // ---- PQ: minimum / maximum of the packet's signed values (its centroid distribution) ----
      float vmin = CUDART_INF_F, vmax = -CUDART_INF_F;
      for (uint32_t j = lane; j < P; j += 32) {
        const unsigned long long pair = seg[j];
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
      lo = vmin;
      hi = vmax;

      // stochastic rounding onto the 2^y uniform centroids of [lo, hi]
      const double Lc = (double)((1ull << y) - 1ull);
      const double dlo = (double)lo;
      const double den = __dsub_rn((double)hi, dlo);
      const double scale = (hi != lo) ? __ddiv_rn(Lc, den) : 0.0;
      const double cstep = (hi != lo) ? __ddiv_rn(den, Lc) : 0.0;  // distance of two centroids
      for (uint32_t j = lane; j < P; j += 32) {
        const unsigned long long pair = seg[j];
        const uint32_t key = (uint32_t)(pair >> 32);
        const uint32_t pid = (uint32_t)pair & 0x7FFFFFFFu;
        const uint32_t b = key ? (key | ((uint32_t)pair & 0x80000000u)) : 0u;
        uint32_t code = 0;
        if (hi != lo) {
          const double num = __dsub_rn((double)__uint_as_float(b), dlo);
          const double u = __dmul_rn((double)philox_coord(rk, cd.client_id, cd.round, pid), 1.0 / 4294967296.0);
          code = pq_quantize(num, den, Lc, scale, u);
        }
        put(j, (unsigned long long)pid | ((unsigned long long)code << s));
        if (residual) {
          const float v = (hi != lo) ? (float)__dadd_rn(dlo, __dmul_rn((double)code, cstep)) : lo;
          residual[pid] = __fsub_rn(__uint_as_float(b), (float)__ddiv_rn((double)v, cd.scale_B));
        }
      }
    }  // PQ

    // packet header {s, y, lo, hi} in bits 0..79 (bits 80..H-1 stay zero)
    if (lane == 0) {
      const uint32_t blo = __float_as_uint(lo), bhi = __float_as_uint(hi);
      atomicOr(words + 0, s | (y << 8) | (blo << 16));
      atomicOr(words + 1, (blo >> 16) | (bhi << 16));
      atomicOr(words + 2, bhi >> 16);
    }
    __syncwarp();
    uint32_t* pkt = stream_words + CVLC_STREAM_HEADER_BYTES / 4 + (size_t)r * n_words;
    for (uint32_t w = lane; w < n_words; w += 32) pkt[w] = words[w];
    __syncwarp();  // the word buffer is reused by the next packet
  }

  // global header (64 bytes), written once per client
  if (blockIdx.x == 0 && tid < 16) {
    uint32_t v = 0;
    const unsigned long long Bbits = (unsigned long long)__double_as_longlong(cd.scale_B);
    const unsigned long long k = plan->k;
    switch (tid) {
      case 0: v = CVLC_STREAM_MAGIC; break;
      case 1: v = 1u | (shape.quantizer << 16) | (s << 24); break;
      case 2: v = (uint32_t)shape.d; break;
      case 3: v = (uint32_t)(shape.d >> 32); break;
      case 4: v = shape.R; break;
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
    stream_words[tid] = v;
  }
}

// ===================================================================================
// launcher
// ===================================================================================

template <int CAP>
static cudaError_t launch_encode_t(const ClientDesc* clients, uint32_t n, const Shape& shape, uint64_t capacity,
                                   const void* plan_ws, void* ws, cudaStream_t st, cudaEvent_t wait_before_pack,
                                   int write_residual) {
  static bool attr_done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && !attr_done[dev]) {
    e = cudaFuncSetAttribute(k_pack<CAP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_pack<CAP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_select<CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSelStages * kSelStageBytes));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_sort_pass<CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sort_smem_bytes(CVLC_MAX_BATCH));
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  BatchDesc<CAP> batch;
  batch.n = n;
  batch.pad = 0;
  for (uint32_t i = 0; i < n; ++i) batch.c[i] = clients[i];
  const EncLayout L = enc_layout(shape.d, n, capacity);
  unsigned char* w = static_cast<unsigned char*>(ws);
  const bool qsgd = shape.quantizer == CVLC_QUANT_QSGD;
  // packet words; QSGD: and the squares of a packet's values
  const size_t pack_warp = (((size_t)shape.packet_bits / 8 + 15) & ~(size_t)15) + (qsgd ? (size_t)shape.cap[1] * 8 : 0);
  const size_t pack_smem = pack_warp * kPackWarps;
  const unsigned pack_grid = (shape.R + kPackWarps * kPackGroup - 1) / (kPackWarps * kPackGroup);

  const Partition part = make_partition(shape.d, n);
  const unsigned char* pws = static_cast<const unsigned char*>(plan_ws);
  {
    LaunchScope ls(kKEncodeInit, st);
    k_encode_init<CAP><<<2 * kNumSM, 256, 0, st>>>(w, batch, shape, L, pws, part);
  }
  if (pws) {
    LaunchScope ls(kKSelect, st);
    k_select<CAP><<<part.grid, kSelThreads, kSelStages * kSelStageBytes, st>>>(batch, shape.d, part, pws, w, L);
  } else {
    const uint64_t want = L.select_tiles * n;
    const unsigned grid = (unsigned)(want < (uint64_t)(4 * kNumSM) ? want : 4 * kNumSM);
    LaunchScope ls(kKSelectLookback, st);
    k_select_lookback<CAP><<<grid, kSelectThreads, 0, st>>>(batch, shape.d, w, L);
  }
  {
    const uint64_t want = L.sort_tiles_max * n;
    const unsigned grid = (unsigned)(want < (uint64_t)(kSortMinBlocks * kNumSM) ? want : kSortMinBlocks * kNumSM);
    if (!pws) {  // the selection with known offsets has counted the digits already
      LaunchScope ls(kKSortHist, st);
      k_sort_hist<CAP><<<grid, 256, 0, st>>>(batch, w, L);
    }
    {
      LaunchScope ls(kKSortScan, st);
      k_sort_scan<CAP><<<n, kDigits, 0, st>>>(batch, w, L);
    }
    for (int pass = 0; pass < kSortPasses; ++pass) {
      LaunchScope ls(kKSortPass, st);
      k_sort_pass<CAP><<<grid, kSortThreads, sort_smem_bytes(n), st>>>(pass, batch, w, L);
    }
  }
  if (wait_before_pack) {
    const cudaError_t ew = cudaStreamWaitEvent(st, wait_before_pack, 0);
    if (ew != cudaSuccess) return ew;
  }
  if (write_residual == kPackNone) return cudaGetLastError();  // the caller writes the ranked records in a format of its own
  {
    LaunchScope ls(kKPack, st);
    if (qsgd)
      k_pack<CAP, true><<<dim3(pack_grid, n), kPackThreads, pack_smem, st>>>(batch, shape, w, L, (uint32_t)pack_warp, write_residual);
    else
      k_pack<CAP, false><<<dim3(pack_grid, n), kPackThreads, pack_smem, st>>>(batch, shape, w, L, (uint32_t)pack_warp, write_residual);
  }
  return cudaGetLastError();
}

cudaError_t launch_encode(const ClientDesc* clients, uint32_t n, const Shape& shape, uint64_t capacity,
                          const void* plan_ws, void* ws, cudaStream_t st, cudaEvent_t wait_before_pack, int write_residual) {
  if (n <= (uint32_t)kSmallBatch)
    return launch_encode_t<kSmallBatch>(clients, n, shape, capacity, plan_ws, ws, st, wait_before_pack, write_residual);
  return launch_encode_t<kLargeBatch>(clients, n, shape, capacity, plan_ws, ws, st, wait_before_pack, write_residual);
}

// memory <- memory + update in fp32, for every client of a batch (the first step of a round with error compensation)
struct EcPair {
  float* memory;
  const float* update;
};
struct EcBatch {
  uint32_t n, pad;
  EcPair c[CVLC_MAX_BATCH];
};

__global__ void __launch_bounds__(256)
k_ec_accumulate(const __grid_constant__ EcBatch batch, uint64_t d) {
  const uint64_t nvec = d >> 2;
  const uint64_t per_client = nvec + 1;  // float4 units and one unit for the ragged tail
  const uint64_t total = per_client * batch.n;
  for (uint64_t g = (uint64_t)blockIdx.x * 256 + threadIdx.x; g < total; g += (uint64_t)gridDim.x * 256) {
    const uint32_t c = (uint32_t)(g / per_client);
    const uint64_t v = g - (uint64_t)c * per_client;
    float* m = batch.c[c].memory;
    const float* u = batch.c[c].update;
    if (v < nvec) {
      float4 a = reinterpret_cast<float4*>(m)[v];
      const float4 b = __ldg(reinterpret_cast<const float4*>(u) + v);
      a.x = __fadd_rn(a.x, b.x);
      a.y = __fadd_rn(a.y, b.y);
      a.z = __fadd_rn(a.z, b.z);
      a.w = __fadd_rn(a.w, b.w);
      reinterpret_cast<float4*>(m)[v] = a;
    } else {
      for (uint64_t i = nvec << 2; i < d; ++i) m[i] = __fadd_rn(m[i], u[i]);
    }
  }
}

cudaError_t launch_ec_accumulate(float* const* memory, const float* const* update, uint32_t n, uint64_t d, cudaStream_t st) {
  EcBatch batch;
  batch.n = n;
  batch.pad = 0;
  for (uint32_t i = 0; i < n; ++i) {
    batch.c[i].memory = memory[i];
    batch.c[i].update = update[i];
  }
  const uint64_t want = (((d >> 2) + 1) * n + 255) / 256;
  const unsigned grid = (unsigned)(want < (uint64_t)(8 * kNumSM) ? want : 8 * kNumSM);
  { LaunchScope ls(kKEcAccumulate, st); k_ec_accumulate<<<grid, 256, 0, st>>>(batch, d); }
  return cudaGetLastError();
}

// The bounded wait of the look-back scans, run on a word nobody publishes: after max_polls polls it gives up,
// reports DEVICE_TIMEOUT and the kernel returns.
__global__ void k_selftest_wait(const unsigned long long* word, int32_t* status, int max_polls) {
  wait_state(word, status, max_polls);
}

cudaError_t launch_selftest_wait(unsigned long long* word, int32_t* status, uint32_t max_polls, cudaStream_t st) {
  { LaunchScope ls(kKSelftest, st); k_selftest_wait<<<1, 32, 0, st>>>(word, status, (int)max_polls); }
  return cudaGetLastError();
}

}  // namespace cvlc
