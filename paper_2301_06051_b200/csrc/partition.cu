// Integer side of the path: window keys, stable LSD radix sort of (key, voxel id) pairs,
// per-window scans, set table fill (Sec. 3.2, Eq. 1-3).  Everything here is exact int32/uint32/uint64
// arithmetic, so results are bit-reproducible.
#include <limits.h>

#include "dsvt_common.cuh"

namespace {

constexpr int kScanThreads = 1024;
constexpr int kScanItems = 8;                         // per thread
constexpr int kScanTile = kScanThreads * kScanItems;  // per block iteration
constexpr int kSortThreads = 256;
constexpr int kSortRounds = 8;
constexpr int kSortTile = kSortThreads * kSortRounds;  // keys per block per pass
constexpr int kRadixBits = 8;
constexpr int kRadix = 1 << kRadixBits;


__device__ __forceinline__ int warp_incl_scan(int v) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// Exclusive scan of one value per thread over the whole block (blockDim.x <= 1024, multiple of 32).
// warp_tot: shared int[33].  Returns the exclusive prefix; *total = block sum.
__device__ __forceinline__ int block_excl_scan(int v, int* warp_tot, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int incl = warp_incl_scan(v);
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int t = lane < nwarp ? warp_tot[lane] : 0;
    int ti = warp_incl_scan(t);
    warp_tot[lane] = ti - t;
    if (lane == 31) warp_tot[32] = ti;
  }
  __syncthreads();
  const int r = warp_tot[warp] + incl - v;
  *total = warp_tot[32];
  __syncthreads();
  return r;
}

// ---- generic exclusive scan ------------------------------------------------------------------
// Single block, loops over the array carrying the running total.  out has count + 1 entries.
__global__ void __launch_bounds__(kScanThreads) scan_loop_kernel(const int32_t* in, int32_t* out, int64_t count,
                                                                 int32_t* total_out) {
  __shared__ int warp_tot[33];
  pdl_enter();
  int carry = 0;
  for (int64_t base = 0; base < count; base += kScanTile) {
    int v[kScanItems];
    int s = 0;
    const int64_t i0 = base + (int64_t)threadIdx.x * kScanItems;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
      v[k] = (i0 + k < count) ? in[i0 + k] : 0;
      s += v[k];
    }
    int tot;
    int p = carry + block_excl_scan(s, warp_tot, &tot);  // ends with a barrier: all loads precede all stores
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
      if (i0 + k < count) out[i0 + k] = p;
      p += v[k];
    }
    carry += tot;
  }
  if (threadIdx.x == 0) {
    out[count] = carry;
    if (total_out) *total_out = carry;
  }
}

// Multi-block variant: (1) per-block local scan + block sums, (2) scan of block sums, (3) add.
__global__ void __launch_bounds__(kScanThreads) scan_local_kernel(const int32_t* in, int32_t* out, int64_t count,
                                                                  int32_t* block_sums) {
  __shared__ int warp_tot[33];
  pdl_enter();
  int v[kScanItems];
  int s = 0;
  const int64_t i0 = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
#pragma unroll
  for (int k = 0; k < kScanItems; ++k) {
    v[k] = (i0 + k < count) ? in[i0 + k] : 0;
    s += v[k];
  }
  int tot;
  int p = block_excl_scan(s, warp_tot, &tot);
#pragma unroll
  for (int k = 0; k < kScanItems; ++k) {
    if (i0 + k < count) out[i0 + k] = p;
    p += v[k];
  }
  if (threadIdx.x == 0) block_sums[blockIdx.x] = tot;
}

__global__ void __launch_bounds__(kScanThreads) scan_add_kernel(int32_t* out, int64_t count,
                                                                const int32_t* __restrict__ block_offs,
                                                                int64_t nblocks, int32_t* total_out) {
  pdl_enter();
  const int add = block_offs[blockIdx.x];
  const int64_t i0 = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
#pragma unroll
  for (int k = 0; k < kScanItems; ++k)
    if (i0 + k < count) out[i0 + k] += add;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    out[count] = block_offs[nblocks];
    if (total_out) *total_out = block_offs[nblocks];
  }
}

// ---- window keys -----------------------------------------------------------------------------
struct PartGeom {
  int32_t batch, gx, gy, gz, L, W, H, nWx, nWy, nWz, axis;
  int32_t sx, sy, sz;  // displacement of the window cut (hybrid window partition): cell x sits at x + sx
  uint32_t V;
};

__global__ void window_key_kernel(const int4* __restrict__ coords, int32_t n, PartGeom g, uint32_t* __restrict__ keys,
                                  int32_t* __restrict__ vals, int32_t* __restrict__ win_count,
                                  int32_t* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  int4 c = coords[i];  // (b, x, y, z)
  const bool bad =
      c.x < 0 || c.x >= g.batch || c.y < 0 || c.y >= g.gx || c.z < 0 || c.z >= g.gy || c.w < 0 || c.w >= g.gz;
  if (bad) {
    atomicOr(status, DSVT_STATUS_BAD_COORD);
    c.x = min(max(c.x, 0), g.batch - 1);
    c.y = min(max(c.y, 0), g.gx - 1);
    c.z = min(max(c.z, 0), g.gy - 1);
    c.w = min(max(c.w, 0), g.gz - 1);
  }
  const int xs = c.y + g.sx, ys = c.z + g.sy, zs = c.w + g.sz;
  const int wx = xs / g.L, wy = ys / g.W, wz = zs / g.H;
  const int xi = xs - wx * g.L, yi = ys - wy * g.W, zi = zs - wz * g.H;
  const uint32_t win = (uint32_t)(((c.x * g.nWx + wx) * g.nWy + wy) * g.nWz + wz);
  const uint32_t inner =
      g.axis == 0 ? (uint32_t)((xi * g.W + yi) * g.H + zi) : (uint32_t)((yi * g.L + xi) * g.H + zi);
  keys[i] = win * g.V + inner;
  vals[i] = i;
  atomicAdd(&win_count[win], 1);
}

// ---- stable LSD radix sort, 8 bits per pass ----------------------------------------------------
__global__ void __launch_bounds__(kSortThreads) radix_hist_kernel(const uint32_t* __restrict__ keys, int32_t n,
                                                                  int shift, int32_t* __restrict__ hist,
                                                                  int32_t ntiles) {
  __shared__ int h[kRadix];
  h[threadIdx.x] = 0;
  __syncthreads();
  const int base = blockIdx.x * kSortTile;
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    const int i = base + r * kSortThreads + threadIdx.x;
    if (i < n) atomicAdd(&h[(keys[i] >> shift) & (kRadix - 1)], 1);
  }
  __syncthreads();
  hist[threadIdx.x * ntiles + blockIdx.x] = h[threadIdx.x];  // digit-major: scan order = (digit, tile)
}

__global__ void __launch_bounds__(kSortThreads) radix_scatter_kernel(const uint32_t* __restrict__ keys_in,
                                                                     const int32_t* __restrict__ vals_in,
                                                                     uint32_t* __restrict__ keys_out,
                                                                     int32_t* __restrict__ vals_out, int32_t n,
                                                                     int shift, const int32_t* __restrict__ offs,
                                                                     int32_t ntiles) {
  constexpr int kWarps = kSortThreads / 32;
  __shared__ int wcnt[kWarps][kRadix];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int run = offs[threadIdx.x * ntiles + blockIdx.x];  // thread d owns digit d's running output position
  const int base = blockIdx.x * kSortTile;
  for (int r = 0; r < kSortRounds; ++r) {
    if (base + r * kSortThreads >= n) break;  // uniform over the block
#pragma unroll
    for (int w = 0; w < kWarps; ++w) wcnt[w][threadIdx.x] = 0;
    __syncthreads();
    const int i = base + r * kSortThreads + threadIdx.x;
    const bool live = i < n;
    uint32_t key = 0;
    int val = 0, digit = 0, rank = 0;
    if (live) {
      key = keys_in[i];
      val = vals_in[i];
      digit = (key >> shift) & (kRadix - 1);
    }
    const unsigned act = __ballot_sync(0xffffffffu, live);
    if (live) {
      const unsigned peers = __match_any_sync(act, digit);
      rank = __popc(peers & ((1u << lane) - 1u));
      if (rank == 0) wcnt[warp][digit] = __popc(peers);
    }
    __syncthreads();
    {  // thread d: exclusive prefix over the warps for digit d, starting at its running position
      int acc = run;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const int t = wcnt[w][threadIdx.x];
        wcnt[w][threadIdx.x] = acc;
        acc += t;
      }
      run = acc;
    }
    __syncthreads();
    if (live) {
      const int dst = wcnt[warp][digit] + rank;
      keys_out[dst] = key;
      vals_out[dst] = val;
    }
    __syncthreads();
  }
}

// ---- per-window scans (Eq. 2) ------------------------------------------------------------------
// Single block.  win_start = exclusive scan of N_w; win_setoff = exclusive scan of S_w = ceil(N_w / tau).
__device__ __forceinline__ void window_scan_body(const int32_t* __restrict__ win_count, int32_t num_windows,
                                                 int32_t tau, int32_t* win_start, int32_t* win_setoff, int32_t cap_sets,
                                                 int32_t* num_sets0, int32_t* num_sets1, int32_t* status) {
  __shared__ int warp_tot[33];
  int carry_n = 0, carry_s = 0;
  for (int base = 0; base < num_windows; base += kScanTile) {
    int cn[kScanItems], cs[kScanItems];
    int sn = 0, ss = 0;
    const int i0 = base + threadIdx.x * kScanItems;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
      const int N = (i0 + k < num_windows) ? win_count[i0 + k] : 0;
      cn[k] = N;
      cs[k] = N / tau + ((N % tau) > 0 ? 1 : 0);  // Eq. 2
      sn += cn[k];
      ss += cs[k];
    }
    int tn, ts;
    int pn = carry_n + block_excl_scan(sn, warp_tot, &tn);
    int ps = carry_s + block_excl_scan(ss, warp_tot, &ts);
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
      if (i0 + k < num_windows) {
        win_start[i0 + k] = pn;
        win_setoff[i0 + k] = ps;
      }
      pn += cn[k];
      ps += cs[k];
    }
    carry_n += tn;
    carry_s += ts;
  }
  if (threadIdx.x == 0) {
    win_start[num_windows] = carry_n;
    win_setoff[num_windows] = carry_s;
    if (carry_s > cap_sets) {
      atomicOr(status, DSVT_STATUS_TABLE_OVERFLOW);
      carry_s = cap_sets;
    }
    *num_sets0 = carry_s;
    if (num_sets1) *num_sets1 = carry_s;
  }
}

__global__ void __launch_bounds__(kScanThreads) window_scan_kernel(const int32_t* __restrict__ win_count,
                                                                   int32_t num_windows, int32_t tau,
                                                                   int32_t* win_start, int32_t* win_setoff,
                                                                   int32_t cap_sets, int32_t* num_sets,
                                                                   int32_t* status) {
  window_scan_body(win_count, num_windows, tau, win_start, win_setoff, cap_sets, num_sets, nullptr, status);
}

// ---- set table fill (Eq. 3, Eq. 4's rank -> voxel id) -------------------------------------------
// One warp per set; grid row y fills the table of sort axis slot y.
struct FillAxis {
  const int32_t* sorted_vox;
  const int32_t* num_sets;
  int32_t* table;
  int32_t* rowoff;
};
__global__ void table_fill_kernel(FillAxis ax0, FillAxis ax1, const int32_t* __restrict__ win_count,
                                  const int32_t* __restrict__ win_start, const int32_t* __restrict__ win_setoff,
                                  int32_t num_windows, int32_t tau) {
  const FillAxis ax = blockIdx.y ? ax1 : ax0;
  const int lane = threadIdx.x & 31;
  const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int S_all = *ax.num_sets;
  if (s >= S_all) return;
  // last window w with win_setoff[w] <= s; it is non-empty because win_setoff[w + 1] > s
  int lo = 0, hi = num_windows;  // invariant: win_setoff[lo] <= s < win_setoff[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (win_setoff[mid] <= s) lo = mid; else hi = mid;
  }
  const int w = lo;
  const uint64_t N = (uint64_t)win_count[w];
  const uint64_t Sw = (uint64_t)(win_setoff[w + 1] - win_setoff[w]);
  const uint64_t j = (uint64_t)(s - win_setoff[w]);
  const int start = win_start[w];
  const uint64_t den = Sw * (uint64_t)tau;
  for (int k = lane; k < tau; k += 32) {
    const uint64_t q = ((j * (uint64_t)tau + (uint64_t)k) * N) / den;  // Eq. 3, exact integer floor
    ax.table[(size_t)s * tau + k] = ax.sorted_vox[start + (int)q];
  }
  if (ax.rowoff && lane == 0) {
    ax.rowoff[s] = start + (int)((j * N) / Sw);  // first rank of set j (proof of Theorem A.2)
    if (s == S_all - 1) ax.rowoff[S_all] = start + (int)(((j + 1) * N) / Sw);
  }
}

// ---- distinct-member counts of a caller-supplied table ------------------------------------------
// cnt[s] = number of slots k with k == 0 or row[k] != row[k-1]; 0 for s >= *num_sets.  One warp per set.
__global__ void table_unique_count_kernel(const int32_t* __restrict__ table, int32_t cap_sets,
                                          const int32_t* __restrict__ num_sets, int32_t tau,
                                          int32_t* __restrict__ cnt) {
  const int lane = threadIdx.x & 31;
  const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (s >= cap_sets) return;
  int c = 0;
  if (s < *num_sets) {
    const int32_t* row = table + (size_t)s * tau;
    for (int k0 = 0; k0 < tau; k0 += 32) {
      const int k = k0 + lane;
      const bool uniq = k < tau && (k == 0 || row[k] != row[k - 1]);
      c += __popc(__ballot_sync(0xffffffffu, uniq));
    }
  }
  if (lane == 0) cnt[s] = c;
}

// ---- tile plan for the tensor-core layer kernel -------------------------------------------------
// Greedy packing of whole sets, in table order, into tiles of at most max_rows distinct rows:
// plan[0] = number of tiles, plan[1 + t] = first set of tile t, plan[1 + tiles] = number of sets;
// plan[0] = -1 if there are more sets than this kernel handles (the layer kernel then schedules by
// row segments).  The greedy chain 0 -> next(0) -> next(next(0)) ... is found by pointer doubling, all
// sets in parallel: single block, arrays in shared memory.
constexpr int kPlanMaxSets = 24576;
// Scratch of the packed plan behind the three per-set arrays: per-warp bin counts / cursors of the counting sort,
// bin starts, the histogram (later the flags of the tile counts on trial).
constexpr int kPackBins = 132;  // set sizes 1 .. 128, rounded up
struct PackScratch {
  unsigned short whist[32][kPackBins];
  int bin_start[kPackBins], hist[kPackBins];
};
// Dynamic shared memory the plan needs for at most smax sets.
__host__ __device__ constexpr size_t plan_smem_bytes(int smax) {
  return (size_t)(smax + 1) * 8 + (((size_t)smax + 15) & ~(size_t)15) + 16 + sizeof(PackScratch);
}

// Packed plan.  Sets are independent of one another, so a tile may hold any of them: the greedy plan in table
// order leaves a tenth of every tile empty (the next set did not fit), this one deals the sets, sorted by their
// number of rows (descending, ties in table order), out to T tiles in boustrophedon rounds, largest to tile 0 ..
// T - 1, the next T to tile T - 1 .. 0, and so on, which levels the tiles' row counts to within a few rows; T is
// the smallest of a ladder of candidates from ceil(rows / max_rows) upwards for which no tile exceeds max_rows.
// Written behind the plan header: the sets in tile order (order[p]) and the rows before each position (prow[p]);
// tile t covers positions [plan[1 + t], plan[2 + t]).  Returns the number of tiles, or 0 (nothing written) if some set
// has no row or more than max_rows, or no candidate below `limit` tiles fits.
struct PlanWindows {  // optional: the windows behind the sets (sets of a window are consecutive), or win_setoff = NULL
  const int32_t* win_setoff;
  const int32_t* win_count;
  int32_t num_windows;
};
__device__ int packed_plan_body(int32_t* rowoff, int32_t* rowoff_copy, int S, int32_t cap_sets, int32_t smax,
                                 int32_t max_rows, int limit, PlanWindows pw, int* plan_smem, int* warp_tot) {
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
  if (max_rows >= kPackBins || nthr <= max_rows || (nthr & 31) != 0) return 0;
  int* srt = plan_smem;                // set ids, sorted by rows descending
  int* ro = srt + (smax + 1);          // row offsets in table order
  unsigned char* ssz = reinterpret_cast<unsigned char*>(ro + (smax + 1));  // rows of srt[i]
  PackScratch* ps = reinterpret_cast<PackScratch*>(ssz + (((size_t)smax + 15) & ~(size_t)15));
  constexpr int kRowMask = 0xffffff;  // (at most smax * max_rows rows: 24 bits hold them)
  for (int s = tid; s <= S; s += nthr) ro[s] = rowoff[s];
  for (int b = tid; b < kPackBins; b += nthr) ps->hist[b] = 0;
  __syncthreads();
  // Sort key of a set: the rows of its window's largest set, so that the sets of a window (whose sizes differ by
  // at most one) stay neighbours in the sorted order and land in neighbouring tiles.  The same plan serves every
  // layer on these windows, so the voxels a tile reads were written by tiles a few numbers away in the layer
  // before, not by tiles anywhere in it.  Kept in the top byte of the set's row offset; 0 = the set's own rows.
  if (pw.win_setoff && ro[S] <= kRowMask) {
    for (int w = tid; w < pw.num_windows; w += nthr) {
      const int so = pw.win_setoff[w], cnt = pw.win_setoff[w + 1] - so;
      if (cnt <= 0 || so < 0) continue;
      const int key = (pw.win_count[w] + cnt - 1) / cnt;
      if (key < 1 || key > max_rows) continue;
      for (int j = 0; j < cnt && so + j < S; ++j) ro[so + j] |= key << 24;
    }
    __syncthreads();
  }
  auto rows_of = [&](int q) { return (ro[q + 1] & kRowMask) - (ro[q] & kRowMask); };
  auto key_of = [&](int q) { const int k = (int)((unsigned)ro[q] >> 24), c = rows_of(q); return k >= c ? k : c; };
  bool bad = ro[S] > kRowMask;
  for (int s = tid; s < S; s += nthr) {
    const int c = rows_of(s);
    bad |= c < 1 || c > max_rows;
  }
  if (__syncthreads_or(bad)) return 0;
  // stable counting sort: every warp takes a contiguous range of the sets; counts per (warp, bin), their prefixes
  // over the warps, then each warp walks its range again and places its sets
  for (int i = tid; i < 32 * kPackBins; i += nthr) (&ps->whist[0][0])[i] = 0;
  __syncthreads();
  const int per_warp = (S + nwarp - 1) / nwarp;
  const int w0 = min(warp * per_warp, S), w1 = min(w0 + per_warp, S);
  for (int b0 = w0; b0 < w1; b0 += 32) {
    const int s = b0 + lane;
    const int c = s < w1 ? key_of(s) : 0;  // the bin
    const unsigned same = __match_any_sync(0xffffffffu, c);
    if (c && lane == __ffs(same) - 1) ps->whist[warp][c] = (unsigned short)(ps->whist[warp][c] + __popc(same));
    __syncwarp();
  }
  __syncthreads();
  if (tid >= 1 && tid <= max_rows) {  // bin tid: the warps' counts -> exclusive prefixes, and the bin's size
    int run = 0;
    for (int w = 0; w < nwarp; ++w) { const int t = ps->whist[w][tid]; ps->whist[w][tid] = (unsigned short)run; run += t; }
    ps->hist[tid] = run;
  }
  __syncthreads();
  if (warp == 0) {  // the bins in descending order of their key: suffix sums, four bins per lane
    int h[4], mine = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) { const int b = 4 * lane + 1 + k; h[k] = b <= max_rows ? ps->hist[b] : 0; mine += h[k]; }
    int suf = mine;  // this lane's bins and all higher ones
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, suf, off);
      if (lane + off < 32) suf += v;
    }
    int acc = suf - mine;  // sets in bins above this lane's
#pragma unroll
    for (int k = 3; k >= 0; --k) { const int b = 4 * lane + 1 + k; if (b <= max_rows) ps->bin_start[b] = acc; acc += h[k]; }
  }
  __syncthreads();
  for (int b0 = w0; b0 < w1; b0 += 32) {
    const int s = b0 + lane;
    const int c = s < w1 ? key_of(s) : 0;
    const unsigned same = __match_any_sync(0xffffffffu, c);
    const int before = c ? ps->whist[warp][c] : 0;
    if (c) {
      const int pos = ps->bin_start[c] + before + __popc(same & ((1u << lane) - 1u));
      srt[pos] = s;
      ssz[pos] = (unsigned char)rows_of(s);
    }
    __syncwarp();
    if (c && lane == __ffs(same) - 1) ps->whist[warp][c] = (unsigned short)(before + __popc(same));
    __syncwarp();
  }
  __syncthreads();
  // rows of tile t when the sorted sets are dealt out to T tiles
  auto tile_rows = [&](int t, int T) {
    int sum = 0, r = 0;
    for (int i0 = 0; i0 < S; i0 += T, ++r) {
      const int i = i0 + ((r & 1) ? T - 1 - t : t);
      if (i < S) sum += ssz[i];
    }
    return sum;
  };
  const int total = ro[S] & kRowMask;
  const int T0 = (total + max_rows - 1) / max_rows;
  // Tile counts are tried a batch at a time (one barrier per batch): over[j] = some tile of candidate j is too full.
  constexpr int kBatch = 8;
  int* over = ps->hist;  // (the histogram has served)
  int cand[kBatch];
  auto try_batch = [&](int ncand) {
    if (tid < kBatch) over[tid] = 0;
    __syncthreads();
    for (int j = 0; j < ncand; ++j)
      for (int t = tid; t < cand[j]; t += nthr)
        if (tile_rows(t, cand[j]) > max_rows) over[j] = 1;
    __syncthreads();
  };
  const int top = min(S, limit - 1);  // (a plan with as many tiles as `limit` is no gain)
  int T = -1, last = T0 - 1;          // last = the largest count known not to fit
  {
    const int ladder[15] = {0, 1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64, 96, 128};  // 128ths of T0 on top of T0
    for (int j0 = 0; j0 < 15 && T < 0 && last < top; j0 += 5) {
      int nc = 0, prev = last;
      for (int j = j0; j < j0 + 5; ++j) {
        const int Tj = min(top, T0 + (int)(((int64_t)T0 * ladder[j] + 127) / 128));
        if (Tj > prev) { cand[nc++] = Tj; prev = Tj; }
      }
      if (nc == 0) break;
      try_batch(nc);
      for (int j = 0; j < nc && T < 0; ++j) {
        if (!over[j]) T = cand[j];
        else last = cand[j];
      }
      __syncthreads();  // (everyone has read the flags)
    }
  }
  if (T < 0) return 0;
  if (T - last - 1 > T0 / 128) {  // between two rungs, if they are more than a percent apart: evenly spaced counts
    // (fitting is not monotonic in T: any count that fits will do, the smallest found is taken)
    const int gap = T - last - 1, nc = min(gap, kBatch);
    for (int j = 0; j < nc; ++j) cand[j] = last + 1 + (int)(((int64_t)j * gap) / nc);
    try_batch(nc);
    for (int j = 0; j < nc; ++j)
      if (!over[j]) { T = cand[j]; break; }
    __syncthreads();
  }
  // positions: tile t holds the sets of rounds 0 .. full - 1 and, for rem tiles, one of the last round
  const int full = S / T, rem = S % T;
  const bool extra_first = (full & 1) == 0;  // the last, partial round runs forwards: tiles 0 .. rem - 1 get its sets
  auto tile_start = [&](int t) { return t * full + (extra_first ? min(t, rem) : max(0, t - (T - rem))); };
  // rows before each tile: the tiles' row counts (one thread per tile), then a scan over contiguous chunks of them
  int* tbase = ro;  // (the offsets in table order have served: the sorted sizes are in ssz)
  __syncthreads();
  for (int t = tid; t < T; t += nthr) tbase[t] = tile_rows(t, T);
  __syncthreads();
  const int chunk = (T + nthr - 1) / nthr;
  const int t0 = min(tid * chunk, T), t1 = min(t0 + chunk, T);
  int local = 0;
  for (int t = t0; t < t1; ++t) local += tbase[t];
  int tot;
  int rows = block_excl_scan(local, warp_tot, &tot);
  for (int t = t0; t < t1; ++t) { const int c = tbase[t]; tbase[t] = rows; rows += c; }
  __syncthreads();
  int32_t* out[2] = {rowoff, rowoff_copy};
  for (int t = tid; t <= T; t += nthr) {
    const int v = t < T ? tile_start(t) : S;
    for (int q = 0; q < 2; ++q)
      if (out[q]) out[q][cap_sets + 2 + t] = v;
  }
  // one thread per position (neighbouring threads write neighbouring entries): its tile, its round, the rows before it
  for (int p = tid; p < S; p += nthr) {
    int t, r;
    if (extra_first) {
      const int cut = rem * (full + 1);
      if (p < cut) { t = p / (full + 1); r = p - t * (full + 1); }
      else { t = rem + (p - cut) / full; r = (p - cut) - (t - rem) * full; }
    } else {
      const int cut = (T - rem) * full;
      if (p < cut) { t = p / full; r = p - t * full; }
      else { t = (T - rem) + (p - cut) / (full + 1); r = (p - cut) - (t - (T - rem)) * (full + 1); }
    }
    int before = tbase[t];
    for (int k = 0; k < r; ++k) before += ssz[k * T + ((k & 1) ? T - 1 - t : t)];
    const int set = srt[r * T + ((r & 1) ? T - 1 - t : t)];
    for (int q = 0; q < 2; ++q)
      if (out[q]) {
        out[q][2 * (size_t)cap_sets + 3 + p] = set;
        out[q][3 * (size_t)cap_sets + 3 + p] = before;
      }
  }
  if (tid == 0)
    for (int q = 0; q < 2; ++q)
      if (out[q]) {
        out[q][cap_sets + 1] = T | DSVT_PLAN_PACKED;
        out[q][3 * (size_t)cap_sets + 3 + S] = tot;
      }
  return T;
}

// The plan of `rowoff` (its offsets are read, its plan written; a second buffer with the same offsets, e.g. the
// other sort axis of the same windows, receives a copy).  One block, any size up to 1024 threads.
__device__ void tile_plan_body(int32_t* rowoff, int32_t* rowoff_copy, int S, int32_t cap_sets, int32_t smax,
                               int32_t max_rows, PlanWindows pw, int* plan_smem, int* warp_tot) {
  int32_t* plan = rowoff + cap_sets + 1;
  int32_t* plan2 = rowoff_copy ? rowoff_copy + cap_sets + 1 : nullptr;
  int* cur = plan_smem;
  int* nxt = cur + (smax + 1);
  unsigned char* mark = reinterpret_cast<unsigned char*>(nxt + (smax + 1));
  const int tid = threadIdx.x, nthr = blockDim.x;
  if (S > smax) {
    if (tid == 0) { plan[0] = -1; if (plan2) plan2[0] = -1; }
    return;
  }
  if (S <= 0) {
    if (tid == 0) { plan[0] = 0; plan[1] = 0; if (plan2) { plan2[0] = 0; plan2[1] = 0; } }
    return;
  }
  // The packed plan first.  If it comes within an eighth of the fewest tiles there can be, it stands; else the plan
  // in table order is worked out as well and the one with fewer tiles is kept.
  const int packed = packed_plan_body(rowoff, rowoff_copy, S, cap_sets, smax, max_rows, INT_MAX, pw, plan_smem, warp_tot);
  const int fewest = (rowoff[S] + max_rows - 1) / max_rows;
  if (packed > 0 && packed <= fewest + fewest / 8) return;
  __syncthreads();  // (the shared arrays are reused)
  // the offsets once into shared memory (the second pointer array is free until the doubling rounds): every set
  // then finds the end of the tile that would start with it by a binary search there
  int* ro = nxt;
  for (int s = tid; s <= S; s += nthr) ro[s] = rowoff[s];
  __syncthreads();
  for (int s = tid; s < S; s += nthr) {
    const int base = ro[s];
    int e = s + 1;
    const int first = ro[s + 1] - base;
    if (first > 0 && first <= max_rows) {  // last e in (s, S] with rowoff[e] - base <= max_rows
      int lo = s + 1, hi = min(S, s + max_rows);
      while (lo < hi) { const int m = (lo + hi + 1) >> 1; if (ro[m] - base <= max_rows) lo = m; else hi = m - 1; }
      e = lo;
    }
    cur[s] = e;
    mark[s] = (s == 0);
  }
  if (tid == 0) cur[S] = S;
  __syncthreads();
  for (int len = 1; len < S; len <<= 1) {
    // marked sets are tile starts; cur = 'next' applied len times
    for (int s = tid; s < S; s += nthr)
      if (mark[s] && cur[s] < S) mark[cur[s]] = 1;
    for (int s = tid; s <= S; s += nthr) nxt[s] = cur[cur[s]];
    __syncthreads();
    int* t = cur; cur = nxt; nxt = t;
  }
  // ordered compaction of the marks
  const int chunk = (S + nthr - 1) / nthr;
  const int s0 = min(tid * chunk, S), s1 = min(s0 + chunk, S);
  int cnt = 0;
  for (int s = s0; s < s1; ++s) cnt += mark[s];
  int total;
  int off = block_excl_scan(cnt, warp_tot, &total);
  if (packed > 0 && packed < total) return;  // the packed plan has fewer tiles: it stays
  for (int s = s0; s < s1; ++s)
    if (mark[s]) {
      plan[1 + off] = s;
      if (plan2) plan2[1 + off] = s;
      ++off;
    }
  if (tid == 0) {
    plan[0] = total; plan[1 + total] = S;
    if (plan2) { plan2[0] = total; plan2[1 + total] = S; }
  }
}

__global__ void __launch_bounds__(kScanThreads) tile_plan_kernel(int32_t* rowoff0, int32_t* rowoff1,
                                                                 const int32_t* __restrict__ num_sets, int32_t cap_sets,
                                                                 int32_t smax, int32_t max_rows, PlanWindows pw) {
  extern __shared__ int plan_smem[];
  __shared__ int warp_tot[33];
  int32_t* rowoff = blockIdx.x ? rowoff1 : rowoff0;  // one block per buffer: offsets, then the plan
  if (!rowoff) return;
  tile_plan_body(rowoff, nullptr, min(*num_sets, cap_sets), cap_sets, smax, max_rows, pw, plan_smem, warp_tot);
}

// ---- bitmap route: ranks by population count instead of sorting --------------------------------
// When the key space (windows x padded cells per window) fits a bitmap, the inner-window rank of a
// voxel (Eq. 1 followed by the sort) is the number of occupied cells of its window with a smaller
// key: each window owns wpw whole 32-bit words of the bitmap, wordrank holds the exclusive popcount
// prefix of the words inside their window, and a voxel's rank is wordrank[word] plus the set bits
// below its own.  Both sort axes are handled by the same launches (they share windows and counts).
struct BmAxis {
  uint32_t* keys;      // [n] window * Vp + inner-window key
  uint32_t* bitmap;    // [num_windows * wpw], cleared by the caller
  int32_t* wordrank;   // [num_windows * wpw]
  int32_t* sorted;     // [n] voxel ids in (window, inner-window) order
  int32_t axis;        // 0: X main order, 1: Y main order
};
struct BmJob {
  BmAxis ax[2];
  int32_t naxes;
};

__global__ void bm_mark_kernel(const int4* __restrict__ coords, int32_t n_max, const int32_t* __restrict__ n_dev,
                               PartGeom g, uint32_t Vp, BmJob job,
                               int32_t* __restrict__ win_count, int32_t* __restrict__ dup_count,
                               int32_t* __restrict__ dup, int32_t* __restrict__ status) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // (the scan kernel may be set up meanwhile)
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int n = n_dev ? min(max(*n_dev, 0), n_max) : n_max;  // (a count that lives on the device)
  if (i >= n) return;
  int4 c = coords[i];  // (b, x, y, z)
  const bool bad =
      c.x < 0 || c.x >= g.batch || c.y < 0 || c.y >= g.gx || c.z < 0 || c.z >= g.gy || c.w < 0 || c.w >= g.gz;
  if (bad) {
    atomicOr(status, DSVT_STATUS_BAD_COORD);
    c.x = min(max(c.x, 0), g.batch - 1);
    c.y = min(max(c.y, 0), g.gx - 1);
    c.z = min(max(c.z, 0), g.gy - 1);
    c.w = min(max(c.w, 0), g.gz - 1);
  }
  const int xs = c.y + g.sx, ys = c.z + g.sy, zs = c.w + g.sz;
  const int wx = xs / g.L, wy = ys / g.W, wz = zs / g.H;
  const int xi = xs - wx * g.L, yi = ys - wy * g.W, zi = zs - wz * g.H;
  const uint32_t win = (uint32_t)(((c.x * g.nWx + wx) * g.nWy + wy) * g.nWz + wz);
  atomicAdd(&win_count[win], 1);
  int ticket = -1;
#pragma unroll
  for (int a = 0; a < 2; ++a) {
    if (a < job.naxes) {
      const uint32_t inner =
          job.ax[a].axis == 0 ? (uint32_t)((xi * g.W + yi) * g.H + zi) : (uint32_t)((yi * g.L + xi) * g.H + zi);
      const uint32_t key = win * Vp + inner;
      job.ax[a].keys[i] = key;
      const uint32_t bit = 1u << (key & 31);
      const uint32_t old = atomicOr(&job.ax[a].bitmap[key >> 5], bit);
      if (a == 0 && (old & bit)) {  // cell already taken: this voxel goes behind the window's distinct cells
        ticket = atomicAdd(&dup_count[win], 1);
        atomicOr(status, DSVT_STATUS_DUPLICATE_CELL);
      }
    }
  }
  dup[i] = ticket;
}

// Block 0: the per-window scans (Eq. 2) and the sets' row offsets.  Other blocks: wordrank, one warp per (axis,
// window).
__global__ void __launch_bounds__(kScanThreads) bm_scan_kernel(const int32_t* __restrict__ win_count,
                                                               int32_t num_windows, int32_t tau, int32_t* win_start,
                                                               int32_t* win_setoff, int32_t cap_sets,
                                                               int32_t* num_sets0, int32_t* num_sets1, BmJob job,
                                                               int32_t wpw, int32_t* rowoff0, int32_t* rowoff1,
                                                               int32_t* status) {
  pdl_enter();
  if (blockIdx.x == 0) {
    window_scan_body(win_count, num_windows, tau, win_start, win_setoff, cap_sets, num_sets0, num_sets1, status);
    if (!rowoff0 && !rowoff1) return;
    __syncthreads();  // the scans are visible to the whole block
    // row offsets: set j of a window of N voxels in S sets starts at rank floor(j N / S) (proof of Theorem A.2);
    // they depend on the windows only, so both axes get the same ones
    for (int w = threadIdx.x; w < num_windows; w += kScanThreads) {
      const int N = win_count[w];
      if (N == 0) continue;
      const int so = win_setoff[w], S = win_setoff[w + 1] - so, start = win_start[w];
      for (int j = 0; j < S && so + j < cap_sets; ++j) {
        const int v = start + (int)(((int64_t)j * N) / S);
        if (rowoff0) rowoff0[so + j] = v;
        if (rowoff1) rowoff1[so + j] = v;
      }
    }
    if (threadIdx.x == 0) {
      const int S_all = min(win_setoff[num_windows], cap_sets);
      // (with more sets than the caller's capacity the last kept set ends where the first dropped one starts)
      int end = win_start[num_windows];
      if (win_setoff[num_windows] > cap_sets) {
        int lo = 0, hi = num_windows;  // window of set cap_sets
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (win_setoff[mid] <= cap_sets) lo = mid; else hi = mid; }
        const int N = win_count[lo], so = win_setoff[lo], S = win_setoff[lo + 1] - so;
        end = win_start[lo] + (int)(((int64_t)(cap_sets - so) * N) / S);
      }
      if (rowoff0) rowoff0[S_all] = end;
      if (rowoff1) rowoff1[S_all] = end;
    }
    return;
  }
  const int lane = threadIdx.x & 31;
  const int64_t items = (int64_t)job.naxes * num_windows;
  const int64_t stride = (int64_t)(gridDim.x - 1) * (kScanThreads / 32);
  for (int64_t it = (int64_t)(blockIdx.x - 1) * (kScanThreads / 32) + (threadIdx.x >> 5); it < items; it += stride) {
    const int a = it >= num_windows ? 1 : 0;
    const int w = (int)(it - (int64_t)a * num_windows);
    if (win_count[w] == 0) continue;
    const uint32_t* bm = a ? job.ax[1].bitmap : job.ax[0].bitmap;
    int32_t* wr = a ? job.ax[1].wordrank : job.ax[0].wordrank;
    const size_t base = (size_t)w * wpw;
    int carry = 0;
    for (int c0 = 0; c0 < wpw; c0 += 32) {
      const int k = c0 + lane;
      const int v = k < wpw ? __popc(bm[base + k]) : 0;
      const int incl = warp_incl_scan(v);
      if (k < wpw) wr[base + k] = carry + incl - v;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
  }
}

// Rank -> table: a voxel of inner-window rank r in a window of N voxels and S sets fills the slots m = j tau + k of
// the window's table rows with floor(m N / (S tau)) == r (Eq. 3, exact integers), i.e. m in
// [ceil(r S tau / N), ceil((r + 1) S tau / N)): one or two slots as a rule, tau of them for a window of one voxel.
// Block 0 builds the tile plan meanwhile (the row offsets come from the scan kernel).
struct FillOut {
  int32_t* table[2];
  int32_t* perm[2];   // optional: voxel ids in sorted order
  int32_t* rowoff[2]; // optional: offsets are read, the plan is written
};
__global__ void __launch_bounds__(kScanThreads) bm_place_fill_kernel(int32_t n_max, const int32_t* __restrict__ n_dev,
                                                                     BmJob job, int32_t wpw,
                                                            const int32_t* __restrict__ dup,
                                                            const int32_t* __restrict__ win_count,
                                                            const int32_t* __restrict__ win_start,
                                                            const int32_t* __restrict__ win_setoff, int32_t tau,
                                                            int32_t cap_sets, const int32_t* __restrict__ num_sets,
                                                            FillOut out, int32_t smax, int32_t num_windows) {
  extern __shared__ int plan_smem[];
  __shared__ int warp_tot[33];
  pdl_enter();
  if (blockIdx.x == 0) {  // the plan (one for both axes: their row offsets are the same)
    int32_t* r0 = out.rowoff[0] ? out.rowoff[0] : out.rowoff[1];
    int32_t* r1 = out.rowoff[0] ? out.rowoff[1] : nullptr;
    const PlanWindows pw{win_setoff, win_count, num_windows};
    if (r0) tile_plan_body(r0, r1, min(*num_sets, cap_sets), cap_sets, smax, 128, pw, plan_smem, warp_tot);
    return;
  }
  const int i = (blockIdx.x - 1) * blockDim.x + threadIdx.x;
  const int n = n_dev ? min(max(*n_dev, 0), n_max) : n_max;
  if (i >= n) return;
  const int ticket = dup[i];
#pragma unroll
  for (int a = 0; a < 2; ++a) {
    if (a < job.naxes) {
      const uint32_t key = job.ax[a].keys[i];
      const uint32_t word = key >> 5;
      const uint32_t win = word / (uint32_t)wpw;
      int r;
      if (ticket < 0) {
        r = job.ax[a].wordrank[word] + __popc(job.ax[a].bitmap[word] & ((1u << (key & 31)) - 1u));
      } else {
        const size_t last = (size_t)win * wpw + (wpw - 1);
        r = job.ax[a].wordrank[last] + __popc(job.ax[a].bitmap[last]) + ticket;
      }
      const int start = win_start[win];
      if (out.perm[a]) out.perm[a][start + r] = i;
      const uint64_t N = (uint64_t)win_count[win];
      const int so = win_setoff[win];
      const uint64_t St = (uint64_t)(win_setoff[win + 1] - so) * (uint64_t)tau;
      const uint64_t m_lo = ((uint64_t)r * St + N - 1) / N, m_hi = ((uint64_t)(r + 1) * St + N - 1) / N;
      const int64_t room = ((int64_t)cap_sets - so) * tau;  // slots of this window that fit the caller's table
      int32_t* dst = out.table[a] + (size_t)so * tau;
      for (uint64_t m = m_lo; m < m_hi && (int64_t)m < room; ++m) dst[m] = i;
    }
  }
}

}  // namespace

// ---------------------------------------------------------------------------------------------------
int dsvt_launch_scan_i32(dsvt_ctx* ctx, const int32_t* in, int32_t* out, int64_t count, int32_t* total_out) {
  // (the scan kernels wait for their predecessor themselves: their launches may overlap its tail)
  cudaStream_t st = ctx->stream;
  if (count <= 8 * (int64_t)kScanTile) {
    DSVT_CUDA_TRY(ctx, launch_pdl(scan_loop_kernel, dim3(1), dim3(kScanThreads), 0, st, in, out, count, total_out));
    DSVT_LAUNCHED(ctx);
    return DSVT_OK;
  }
  const int64_t nblocks = dsvt_ceil_div(count, kScanTile);
  DSVT_CUDA_TRY(ctx, launch_pdl(scan_local_kernel, dim3((unsigned)nblocks), dim3(kScanThreads), 0, st, in, out, count,
                                ctx->scan_tmp));
  DSVT_LAUNCHED(ctx);
  DSVT_CUDA_TRY(ctx, launch_pdl(scan_loop_kernel, dim3(1), dim3(kScanThreads), 0, st, (const int32_t*)ctx->scan_tmp,
                                ctx->scan_tmp, nblocks, (int32_t*)nullptr));
  DSVT_LAUNCHED(ctx);
  DSVT_CUDA_TRY(ctx, launch_pdl(scan_add_kernel, dim3((unsigned)nblocks), dim3(kScanThreads), 0, st, out, count,
                                (const int32_t*)ctx->scan_tmp, nblocks, total_out));
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}

// Sorts ctx->keys[0] / ctx->vals[0] (n pairs) by the low key_bits bits; *final_buf = index of the
// buffer pair that holds the result.
int dsvt_launch_sort_pairs(dsvt_ctx* ctx, int32_t n, int key_bits, int* final_buf) {
  const int passes = key_bits <= 0 ? 1 : (key_bits + kRadixBits - 1) / kRadixBits;
  const int32_t ntiles = (int32_t)dsvt_ceil_div(n, kSortTile);
  int cur = 0;
  for (int p = 0; p < passes; ++p) {
    const int shift = p * kRadixBits;
    radix_hist_kernel<<<ntiles, kSortThreads, 0, ctx->stream>>>(ctx->keys[cur], n, shift, ctx->hist, ntiles);
    DSVT_LAUNCHED(ctx);
    int rc = dsvt_launch_scan_i32(ctx, ctx->hist, ctx->hist, (int64_t)kRadix * ntiles, nullptr);
    if (rc != DSVT_OK) return rc;
    radix_scatter_kernel<<<ntiles, kSortThreads, 0, ctx->stream>>>(ctx->keys[cur], ctx->vals[cur], ctx->keys[cur ^ 1],
                                                                    ctx->vals[cur ^ 1], n, shift, ctx->hist, ntiles);
    DSVT_LAUNCHED(ctx);
    cur ^= 1;
  }
  *final_buf = cur;
  return DSVT_OK;
}

int dsvt_launch_rowoff_from_table(dsvt_ctx* ctx, const int32_t* table, int32_t cap_sets, const int32_t* num_sets,
                                  int32_t set_size, int32_t* rowoff) {
  const int warps_per_block = 8;
  if (cap_sets > 0) {
    const unsigned blocks = (unsigned)dsvt_ceil_div(cap_sets, warps_per_block);
    table_unique_count_kernel<<<blocks, warps_per_block * 32, 0, ctx->stream>>>(table, cap_sets, num_sets, set_size,
                                                                                rowoff);
    DSVT_LAUNCHED(ctx);
  }
  return dsvt_launch_scan_i32(ctx, rowoff, rowoff, cap_sets, nullptr);
}

// Tile plans behind the row offsets of one or two buffers: set_rowoff + cap_sets + 1 (see include/dsvt.h).
static int launch_tile_plans(dsvt_ctx* ctx, const int32_t* num_sets, int32_t cap_sets, int32_t* set_rowoff,
                             int32_t* set_rowoff1, PlanWindows pw) {
  const int32_t smax = cap_sets < kPlanMaxSets ? cap_sets : kPlanMaxSets;
  const size_t smem = plan_smem_bytes(smax);
  if (smem > 48 * 1024 && !(ctx->attr_flags & 2u)) {  // (once per context: the attribute belongs to its device)
    DSVT_CUDA_TRY(ctx, cudaFuncSetAttribute(tile_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)plan_smem_bytes(kPlanMaxSets)));
    ctx->attr_flags |= 2u;
  }
  tile_plan_kernel<<<set_rowoff1 ? 2 : 1, kScanThreads, smem, ctx->stream>>>(set_rowoff, set_rowoff1, num_sets,
                                                                            cap_sets, smax, 128, pw);
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}

int dsvt_launch_tile_plan(dsvt_ctx* ctx, const int32_t* num_sets, int32_t cap_sets, int32_t* set_rowoff) {
  return launch_tile_plans(ctx, num_sets, cap_sets, set_rowoff, nullptr, PlanWindows{nullptr, nullptr, 0});
}

static int key_bits_for(uint64_t max_key) {
  int b = 0;
  while (b < 32 && (max_key >> b) != 0) ++b;
  return b;
}

namespace {

struct PartOut {  // device outputs of one sort axis
  int32_t axis;
  int32_t* set_table;
  int32_t* num_sets;
  int32_t* set_rowoff;
  int32_t* perm;
};

struct PartCall {
  const int32_t* coords;
  const int32_t* n_dev;  // optional device count: the call takes min(n, *n_dev) voxels
  int32_t n, set_size, cap_sets, nw;
  PartGeom g;
  uint64_t V;
  int32_t *win_start, *win_count, *win_setoff;  // optional outputs
};

int validate(dsvt_ctx* ctx, const int32_t* coords, int32_t n, int32_t batch, const int32_t grid[3],
             const int32_t window[3], const int32_t shift[3], int32_t set_size, int32_t cap_sets, PartCall* pc) {
  if (!ctx || !grid || !window || n < 0 || batch < 1 || set_size < 1 || cap_sets < 0) return DSVT_ERR_INVALID_ARG;
  for (int a = 0; a < 3; ++a) {
    if (grid[a] < 1 || window[a] < 1) return DSVT_ERR_INVALID_ARG;
    if (shift && (shift[a] < 0 || shift[a] >= window[a])) return DSVT_ERR_INVALID_ARG;
    if ((int64_t)grid[a] + window[a] >= (1ll << 31)) return DSVT_ERR_UNSUPPORTED;
  }
  if (n > 0 && !coords) return DSVT_ERR_INVALID_ARG;
  if (((uintptr_t)coords & 15) != 0) return DSVT_ERR_INVALID_ARG;
  PartGeom& g = pc->g;
  g.batch = batch; g.gx = grid[0]; g.gy = grid[1]; g.gz = grid[2];
  g.L = window[0]; g.W = window[1]; g.H = window[2];
  g.sx = shift ? shift[0] : 0; g.sy = shift ? shift[1] : 0; g.sz = shift ? shift[2] : 0;
  g.nWx = (int32_t)dsvt_ceil_div((int64_t)grid[0] + g.sx, window[0]);
  g.nWy = (int32_t)dsvt_ceil_div((int64_t)grid[1] + g.sy, window[1]);
  g.nWz = (int32_t)dsvt_ceil_div((int64_t)grid[2] + g.sz, window[2]);
  g.axis = 0;
  const uint64_t V = (uint64_t)window[0] * window[1] * window[2];
  const uint64_t num_windows = (uint64_t)batch * g.nWx * g.nWy * g.nWz;
  if (V >= (1ull << 31) || num_windows >= (1ull << 31) || num_windows * V > 0xFFFFFFFFull) return DSVT_ERR_UNSUPPORTED;
  g.V = (uint32_t)V;
  if (n > ctx->max_voxels || (int64_t)num_windows > ctx->max_windows) return DSVT_ERR_CAPACITY;
  pc->coords = coords; pc->n_dev = nullptr; pc->n = n; pc->set_size = set_size; pc->cap_sets = cap_sets;
  pc->nw = (int32_t)num_windows;
  pc->V = V;
  return DSVT_OK;
}

// upper bound of the number of sets: floor(n / tau) + (non-empty windows), at most min(cap_sets, n)
int64_t sets_bound(const PartCall& pc) {
  int64_t b = (int64_t)pc.n / pc.set_size + (int64_t)(pc.nw < pc.n ? pc.nw : pc.n);
  if (b > pc.n) b = pc.n;
  if (b > pc.cap_sets) b = pc.cap_sets;
  return b;
}

int copy_window_arrays(dsvt_ctx* ctx, const PartCall& pc, const int32_t* counts) {
  cudaStream_t st = ctx->stream;
  const size_t nw = (size_t)pc.nw;
  if (pc.win_count)
    DSVT_CUDA_TRY(ctx, cudaMemcpyAsync(pc.win_count, counts, sizeof(int32_t) * nw, cudaMemcpyDeviceToDevice, st));
  if (pc.win_start)
    DSVT_CUDA_TRY(ctx, cudaMemcpyAsync(pc.win_start, ctx->win_start, sizeof(int32_t) * (nw + 1), cudaMemcpyDeviceToDevice, st));
  if (pc.win_setoff)
    DSVT_CUDA_TRY(ctx, cudaMemcpyAsync(pc.win_setoff, ctx->win_setoff, sizeof(int32_t) * (nw + 1), cudaMemcpyDeviceToDevice, st));
  return DSVT_OK;
}

// Sorting route: one axis per call; works for any key space below 2^32.
int partition_sorted(dsvt_ctx* ctx, const PartCall& pc, const PartOut& o) {
  cudaStream_t st = ctx->stream;
  const int32_t n = pc.n, nw = pc.nw, cap_sets = pc.cap_sets;
  PartGeom g = pc.g;
  g.axis = o.axis;
  DSVT_CUDA_TRY(ctx, cudaMemsetAsync(ctx->win_count, 0, sizeof(int32_t) * (size_t)(nw + 1), st));
  int fin = 0;
  if (n > 0) {
    window_key_kernel<<<(unsigned)dsvt_ceil_div(n, 256), 256, 0, st>>>((const int4*)pc.coords, n, g, ctx->keys[0],
                                                                       ctx->vals[0], ctx->win_count, ctx->status);
    DSVT_LAUNCHED(ctx);
    int rc = dsvt_launch_sort_pairs(ctx, n, key_bits_for((uint64_t)nw * pc.V - 1), &fin);
    if (rc != DSVT_OK) return rc;
  }
  window_scan_kernel<<<1, kScanThreads, 0, st>>>(ctx->win_count, nw, pc.set_size, ctx->win_start, ctx->win_setoff,
                                                 cap_sets, o.num_sets, ctx->status);
  DSVT_LAUNCHED(ctx);
  if (n > 0) {
    const int64_t s_bound = sets_bound(pc);
    if (s_bound > 0) {
      FillAxis f{ctx->vals[fin], o.num_sets, o.set_table, o.set_rowoff};
      table_fill_kernel<<<(unsigned)dsvt_ceil_div(s_bound, 8), 256, 0, st>>>(f, f, ctx->win_count, ctx->win_start,
                                                                             ctx->win_setoff, nw, pc.set_size);
      DSVT_LAUNCHED(ctx);
    }
    if (o.set_rowoff && s_bound > 0) {
      int rc = launch_tile_plans(ctx, o.num_sets, cap_sets, o.set_rowoff, nullptr,
                                 PlanWindows{ctx->win_setoff, ctx->win_count, nw});
      if (rc != DSVT_OK) return rc;
    }
    if (o.perm)
      DSVT_CUDA_TRY(ctx, cudaMemcpyAsync(o.perm, ctx->vals[fin], sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToDevice, st));
  }
  if (o.set_rowoff && (n == 0 || cap_sets == 0))  // no sets: row offset 0, empty tile plan
    DSVT_CUDA_TRY(ctx, cudaMemsetAsync(o.set_rowoff, 0, sizeof(int32_t) * (size_t)(2 * (size_t)cap_sets + 3), st));
  return copy_window_arrays(ctx, pc, ctx->win_count);
}

// Words of bitmap per window, or 0 if the bitmap route cannot take this call.
int32_t bitmap_words_per_window(const dsvt_ctx* ctx, const PartCall& pc) {
  if (ctx->bm_words == 0 || pc.n == 0 || pc.cap_sets == 0) return 0;
  const uint64_t wpw = (pc.V + 31) / 32;
  if ((uint64_t)pc.nw * wpw > ctx->bm_words || (uint64_t)pc.nw * wpw * 32 > 0xFFFFFFFFull) return 0;
  return (int32_t)wpw;
}

// Bitmap route: one or both axes in three launches and a memset.
int partition_bitmap(dsvt_ctx* ctx, const PartCall& pc, int32_t wpw, int naxes, const PartOut* o) {
  cudaStream_t st = ctx->stream;
  const int32_t n = pc.n, nw = pc.nw;
  const size_t words = (size_t)nw * wpw;
  // cleared region: [win_count nw + 1 | dup_count nw + 1 | bitmap of axis slot 0 | bitmap of axis slot 1]
  int32_t* counts = ctx->bm_zero;
  int32_t* dup_count = counts + (nw + 1);
  uint32_t* bitmap0 = reinterpret_cast<uint32_t*>(dup_count + (nw + 1));
  DSVT_CUDA_TRY(ctx, cudaMemsetAsync(counts, 0, sizeof(int32_t) * (2 * (size_t)(nw + 1) + (size_t)naxes * words), st));
  BmJob job;
  job.naxes = naxes;
  for (int a = 0; a < 2; ++a) {
    const int b = a < naxes ? a : 0;
    job.ax[a].keys = ctx->keys[b];
    job.ax[a].bitmap = bitmap0 + (size_t)b * words;
    job.ax[a].wordrank = ctx->bm_wordrank + (size_t)b * words;
    job.ax[a].sorted = ctx->vals[b];
    job.ax[a].axis = o[b].axis;
  }
  const unsigned vox_blocks = (unsigned)dsvt_ceil_div(n, 256);
  bm_mark_kernel<<<vox_blocks, 256, 0, st>>>((const int4*)pc.coords, n, pc.n_dev, pc.g, (uint32_t)wpw * 32u, job, counts,
                                             dup_count, ctx->bm_dup, ctx->status);
  DSVT_LAUNCHED(ctx);
  int64_t rank_blocks = dsvt_ceil_div((int64_t)naxes * nw, kScanThreads / 32);
  if (rank_blocks > 2 * (int64_t)ctx->sm_count) rank_blocks = 2 * (int64_t)ctx->sm_count;
  int32_t* r0 = o[0].set_rowoff;
  int32_t* r1 = naxes > 1 ? o[1].set_rowoff : nullptr;
  DSVT_CUDA_TRY(ctx, launch_pdl(bm_scan_kernel, dim3((unsigned)(1 + rank_blocks)), dim3(kScanThreads), 0, st,
                                (const int32_t*)counts, nw, pc.set_size, ctx->win_start, ctx->win_setoff, pc.cap_sets,
                                o[0].num_sets, naxes > 1 ? o[1].num_sets : (int32_t*)nullptr, job, wpw, r0, r1,
                                ctx->status));
  DSVT_LAUNCHED(ctx);
  // plan capacity: no more sets than floor(n / tau) + non-empty windows
  const int64_t s_bound = sets_bound(pc);
  const int32_t smax = (int32_t)(s_bound < kPlanMaxSets ? s_bound : kPlanMaxSets);
  const size_t smem = (r0 || r1) ? plan_smem_bytes(smax) : 0;
  if (smem > 48 * 1024 && !(ctx->attr_flags & 1u)) {  // (once per context: the attribute belongs to its device)
    DSVT_CUDA_TRY(ctx, cudaFuncSetAttribute(bm_place_fill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)plan_smem_bytes(kPlanMaxSets)));
    ctx->attr_flags |= 1u;
  }
  FillOut fo;
  for (int a = 0; a < 2; ++a) {
    const bool on = a < naxes;
    fo.table[a] = on ? o[a].set_table : nullptr;
    fo.perm[a] = on ? o[a].perm : nullptr;
    fo.rowoff[a] = on ? o[a].set_rowoff : nullptr;
  }
  const unsigned fill_blocks = (unsigned)dsvt_ceil_div(n, kScanThreads);
  DSVT_CUDA_TRY(ctx, launch_pdl(bm_place_fill_kernel, dim3(fill_blocks + 1), dim3(kScanThreads), smem, st, n, pc.n_dev, job, wpw,
                                (const int32_t*)ctx->bm_dup, (const int32_t*)counts, (const int32_t*)ctx->win_start,
                                (const int32_t*)ctx->win_setoff, pc.set_size, pc.cap_sets,
                                (const int32_t*)o[0].num_sets, fo, smax, nw));
  DSVT_LAUNCHED(ctx);
  return copy_window_arrays(ctx, pc, counts);
}

}  // namespace

extern "C" int dsvt_partition(dsvt_ctx* ctx, const int32_t* coords, int32_t n, int32_t batch, const int32_t grid[3],
                              const int32_t window[3], int32_t set_size, int32_t axis, int32_t* set_table,
                              int32_t cap_sets, int32_t* num_sets, int32_t* set_rowoff, int32_t* perm,
                              int32_t* win_start, int32_t* win_count, int32_t* win_setoff) {
  if (!num_sets || (axis != 0 && axis != 1)) return DSVT_ERR_INVALID_ARG;
  PartCall pc;
  int rc = validate(ctx, coords, n, batch, grid, window, nullptr, set_size, cap_sets, &pc);
  if (rc != DSVT_OK) return rc;
  if (n > 0 && !set_table) return DSVT_ERR_INVALID_ARG;
  pc.win_start = win_start; pc.win_count = win_count; pc.win_setoff = win_setoff;
  const PartOut o{axis, set_table, num_sets, set_rowoff, perm};
  const int32_t wpw = bitmap_words_per_window(ctx, pc);
  if (wpw > 0) return partition_bitmap(ctx, pc, wpw, 1, &o);
  return partition_sorted(ctx, pc, o);
}

extern "C" int dsvt_partition_rotated(dsvt_ctx* ctx, const int32_t* coords, int32_t n, int32_t batch,
                                      const int32_t grid[3], const int32_t window[3], int32_t set_size,
                                      int32_t* const set_table[2], int32_t cap_sets, int32_t* const num_sets[2],
                                      int32_t* const set_rowoff[2], int32_t* const perm[2], int32_t* win_start,
                                      int32_t* win_count, int32_t* win_setoff) {
  return dsvt_partition_shifted(ctx, coords, n, batch, grid, window, nullptr, set_size, set_table, cap_sets, num_sets,
                                set_rowoff, perm, win_start, win_count, win_setoff);
}

extern "C" int dsvt_partition_shifted(dsvt_ctx* ctx, const int32_t* coords, int32_t n, int32_t batch,
                                      const int32_t grid[3], const int32_t window[3], const int32_t shift[3],
                                      int32_t set_size, int32_t* const set_table[2], int32_t cap_sets,
                                      int32_t* const num_sets[2], int32_t* const set_rowoff[2],
                                      int32_t* const perm[2], int32_t* win_start, int32_t* win_count,
                                      int32_t* win_setoff) {
  return dsvt_partition_counted(ctx, coords, n, nullptr, batch, grid, window, shift, set_size, set_table, cap_sets,
                                num_sets, set_rowoff, perm, win_start, win_count, win_setoff);
}

extern "C" int dsvt_partition_counted(dsvt_ctx* ctx, const int32_t* coords, int32_t n, const int32_t* n_dev,
                                      int32_t batch, const int32_t grid[3], const int32_t window[3],
                                      const int32_t shift[3], int32_t set_size, int32_t* const set_table[2],
                                      int32_t cap_sets, int32_t* const num_sets[2], int32_t* const set_rowoff[2],
                                      int32_t* const perm[2], int32_t* win_start, int32_t* win_count,
                                      int32_t* win_setoff) {
  if (!set_table || !num_sets || !num_sets[0] || !num_sets[1]) return DSVT_ERR_INVALID_ARG;
  PartCall pc;
  int rc = validate(ctx, coords, n, batch, grid, window, shift, set_size, cap_sets, &pc);
  if (rc != DSVT_OK) return rc;
  pc.n_dev = n_dev;
  if (n > 0 && (!set_table[0] || !set_table[1])) return DSVT_ERR_INVALID_ARG;
  pc.win_start = win_start; pc.win_count = win_count; pc.win_setoff = win_setoff;
  PartOut o[2];
  for (int a = 0; a < 2; ++a)
    o[a] = PartOut{a, set_table[a], num_sets[a], set_rowoff ? set_rowoff[a] : nullptr, perm ? perm[a] : nullptr};
  const int32_t wpw = bitmap_words_per_window(ctx, pc);
  if (wpw > 0) return partition_bitmap(ctx, pc, wpw, 2, o);
  if (n_dev && n > 0 && cap_sets > 0) return DSVT_ERR_UNSUPPORTED;  // (the sorting route wants the count on the host)
  rc = partition_sorted(ctx, pc, o[0]);
  if (rc != DSVT_OK) return rc;
  return partition_sorted(ctx, pc, o[1]);
}
