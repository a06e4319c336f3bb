// Fused DSVT layers on the 5th-generation tensor cores (tcgen05 + TMEM), bfloat16 operands, fp32
// accumulation: gather (Eq. 4) -> QKV projection -> per-set multi-head attention (Eq. 5) -> output
// projection -> residual + LayerNorm -> MLP with GELU -> residual + LayerNorm -> scatter (App. B.1.1).
//
// One launch runs a chain of layers (one layer, the two layers of a block, or every block of a stage): layer 0
// reads x and writes y, the later layers run in place on y.  Whole sets are packed into tiles of at most 128
// distinct rows (the UMMA M) by the partition's tile plan.  The persistent CTAs (one per SM) draw tiles from a
// global counter, all tiles of layer 0 first, then layer 1, ...; a tile of layer l may be gathered as soon as
// each of its rows carries layer l - 1's completion stamp (one int per voxel, written after the row's store), so
// no CTA ever waits for a whole layer to end, and a launch pays its start-up and its tail once per chain rather
// than once per layer.  Tiles are taken in counter order and a tile only ever waits for tiles with a smaller
// number, so the tile with the smallest unfinished number can always run: no CTA has to be resident for another
// to make progress.
//
// Roles (640 threads): warps 0-15 compute (gather, TMEM epilogues, attention); warp 16 is the scheduler
// and TMA producer: it draws tiles, publishes them through a two-entry ring, two ahead, and streams the layer's
// weight matrices through a three-stage shared-memory ring with plain (single-CTA) TMA loads; warp 17
// allocates TMEM and issues the tcgen05.mma instructions; warp 18 builds the next tile's row list
// while the current tile is computed and waits for its rows' stamps; warp 19 stamps a finished tile's rows.
// The compute warps gather the next tile's rows as soon as the current tile's MMAs have stopped reading the A
// operand (if its rows are ready by then), so that its first projections overlap the current tile's tail.
//
// The projections of a layer are chunks of at most 192 output columns (K, V, Q, O, MLP-1 in pieces of
// 128 or 64 hidden columns, MLP-2), accumulated in three TMEM regions (map at compute_role) so the
// tensor pipe works on one chunk while the compute warps drain another.  The fp32 residual stream never
// leaves the chip inside a layer: x is staged in shared memory for the first residual, and
// x1 + b_2 = LN1(x + attention) + b_2 is parked in TMEM, where MLP-2 accumulates on top of it.
//
// Every operand tile in shared memory uses the K-major 128-byte-swizzled layout that tcgen05.mma and
// TMA share: 64 bf16 columns per 128-byte row, 8-row groups of 1024 bytes, 16-byte chunk index XORed
// with (row & 7).  Q, K, V and the attention output live in that same layout, so the attention phase
// (mma.sync m16n8k16 with ldmatrix) reads it without bank conflicts and writes its result straight
// into the A operand of the output projection.
//
// Every wait (on an mbarrier, on a row stamp) is bounded; a wait that gives up raises DSVT_STATUS_TIMEOUT and
// all roles leave their loops.
#include <cuda.h>
#include <limits.h>

#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

#include "dsvt_common.cuh"
#include "tc_ptx.cuh"

namespace {
using namespace dsvt_tc;

constexpr int kComputeWarps = 16;
constexpr int kComputeThreads = 32 * kComputeWarps;
constexpr int kTmaWarp = kComputeWarps, kMmaWarp = kComputeWarps + 1;
constexpr int kLoadWarp0 = kComputeWarps + 2, kLoadWarps = 1;  // row-list warp, one tile ahead
constexpr int kLoadThreads = 32 * kLoadWarps;
constexpr int kStampWarp = kLoadWarp0 + kLoadWarps;  // writes the completion stamps of a finished tile's rows
constexpr int kThreads = kComputeThreads + 64 + kLoadThreads + 32;
constexpr int kStages = 3;             // weight ring depth
constexpr int kStampPolls = 1 << 18;  // polls of a row's stamp, about a microsecond each
constexpr int kMaxLayers = DSVT_MAX_CHAIN_LAYERS;  // layers one launch can chain

struct TcGeom {
  int hidden, heads, tau;
  int nkb_h;    // hidden / 64: K blocks of the MLP-2 contraction
  int NF;       // MLP-1 chunk width (128 or 64)
  int n_f1;     // hidden / NF
  int mode;     // 0: attention only, 1: attention + residual + LN1, 2: full layer
  uint32_t off_a, off_kv, off_stage, off_par;  // byte offsets from the 1024-aligned base
  // relative position bias (rb_len == 0: none): entries per head, strides of the x and y offsets in the table,
  // index of the zero offset, extent of the table
  int rb_len, rb_sx, rb_sy, rb_centre, rb_ext[3];
};

// One layer of a launch's chain: weight tensor maps, per-layer vectors, and the set table the layer runs on.
struct alignas(64) TcLayer {
  CUtensorMap qkv, o, w1, w2;
  const float *b_qkv, *b_o, *b_1, *b_2, *ln1_g, *ln1_b, *ln2_g, *ln2_b, *rpb;
  const float* pe;  // positional term added to the input of the query and key maps, [n][C], or NULL
  const int32_t *table, *num_sets, *rowoff;
  int32_t cap_sets;
  float eps;
};

struct TcArgs {
  const float* x;        // input of layer 0
  float* y;              // output of every layer; input of the layers after the first
  const int4* coords;    // (b, x, y, z) per voxel: read only with a position bias
  int32_t n, n_layers;
  int32_t* counter;      // [0] next tile of the launch, [1] CTAs that have left; both zero between launches
  int32_t* row_stamp;    // [n] completion stamps (n_layers > 1)
  int32_t stamp_base;    // layer l's stamp is stamp_base + l + 1
  int32_t* status;
  TcGeom g;
  TcLayer layer[kMaxLayers];
};

struct Misc {  // small shared state beside the big regions
  // weight ring; accumulator regions 0 / 1 / 2 (see the TMEM map at compute_role); operand hand-offs
  unsigned long long full[kStages], empty[kStages], acc_full[3], acc_free[3];
  unsigned long long a_ready;   // compute warps -> MMA: attention output / x1 / MLP hidden is in place
  unsigned long long x_ready;   // compute warps -> MMA: the gathered rows of a tile are in the A operand
  unsigned long long rl_ready[2];   // loader warp -> compute: row-list buffer b describes its next tile
  unsigned long long dep_ready[2];  // loader warp -> compute: the rows listed in buffer b carry the previous layer's stamp
  unsigned long long rl_free[2];    // compute + stamp warp -> loader warp: row-list buffer b is no longer read
  unsigned long long stored[2];     // compute -> stamp warp: the tile listed in buffer b has been stored
  unsigned long long drain;         // MMA issuer: every MMA issued before an abort has completed
  unsigned long long sched_full[2], sched_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  int exit_at;   // tile iteration at which the compute warps left their loop (-1: still running; read by the stamp warp)
  int tile[2][6];  // ring of tiles: first set, number of sets (< 0: no more tiles), first row, rows, layer
  // the scheduler's view of the chain: tiles before the end of each layer, sets per layer, plan or not
  int tile_end[kMaxLayers], lay_S[kMaxLayers];
  unsigned char lay_plan[kMaxLayers];
  // launch constants, written once before the roles start: the phase functions read them from here
  // instead of taking them as arguments, so that nothing has to stay in registers across their calls
  const float* x;   // input rows of the tile the compute warps are working on
  const float* pe;  // the layer's positional term (kernels with one)
  float* y;
  int32_t* status;
  unsigned char* sm;   // 1024-aligned base of the dynamic shared memory (generic address)
  uint32_t sbase;      // the same as a shared-space address
  uint32_t off_a, off_kv, off_par;
  int n, tau, heads, mode, NF, n_f1, ln1, ln2;
  float eps;
  // the tile the compute warps are working on, and which row-list buffer describes it
  int s_lo, nsets, base, rows, buf, layer;
  int next_rows[2];        // rows of the tile listed in buffer b (< 0: there is no such tile), valid after rl_ready[b]
  const float* next_x[2];  // where that tile's input rows are read from
  int st_rows[2], st_stamp[2];  // for the stamp warp: rows of the stored tile in buffer b, the stamp they get (0: none)
  // row lists, double buffered: the loader warp fills buffer (k + 1) & 1 while the compute warps work on tile k;
  // the compute warps gather tile k + 1 as soon as tile k's MMAs no longer read the A operand
  int rowvox[2][kTM];              // tile row -> voxel (-1: none)
  unsigned char row_lo[2][kTM], row_n[2][kTM];  // per tile row: first row and row count of its set
  // relative position bias.  The table index is linear in the coordinate offset, so one integer per row,
  // x * rb_sx + y * rb_sy + z, serves every (query, key) pair: index = lin[query] - lin[key] + rb_centre.  Offsets
  // inside a covered set are at most (table length - 1) / 2 < 2^15 in magnitude (tables of up to 65,535 entries
  // per head), so the low 16 bits are kept and differences are taken modulo 2^16.
  // Written by the gather of a tile (after the previous tile's attention), read by the tile's attention.
  const float* rpb;
  const int4* coords;
  int rb_len, rb_sx, rb_sy, rb_centre, rb_ext[3];
  short rowlin[kTM];
};
__shared__ Misc s_mi;

__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kComputeThreads) : "memory"); }

// gelu(t) = t Phi(t) with Phi(t) = 1 - h for t >= 0 and h for t < 0, h = erfc(|t| / sqrt 2) / 2; hence
// gelu(t) = max(t, 0) - |t| h.  h is evaluated as 2^p(|t|), p a degree-5 polynomial: a weighted least-squares
// fit of log2 erfc(|t| / sqrt 2) on |t| <= 8.4 (beyond that h < 1e-17), with the factor 1/2 folded into its
// constant term.  The polynomial runs on m = -min(|t|, 8.4) (odd coefficients negated), so that the last step
// is one fused multiply-add max(t, 0) + m h.  Two values at a time: the polynomial, the bias add and the last
// step are packed fp32x2 operations.  Absolute error of gelu below 2e-6 for all t, far under the bfloat16
// rounding applied to the result.
__device__ __forceinline__ float2 gelu_fast2(float2 t) {
  const float2 m = make_float2(fmaxf(-fabsf(t.x), -8.4f), fmaxf(-fabsf(t.y), -8.4f));
  float2 q = __ffma2_rn(make_float2(5.189499352e-04f, 5.189499352e-04f), m, make_float2(7.387642749e-03f, 7.387642749e-03f));
  q = __ffma2_rn(q, m, make_float2(5.253871530e-02f, 5.253871530e-02f));
  q = __ffma2_rn(q, m, make_float2(-4.592762589e-01f, -4.592762589e-01f));
  q = __ffma2_rn(q, m, make_float2(1.151083231e+00f, 1.151083231e+00f));
  q = __ffma2_rn(q, m, make_float2(-1.0f - 8.382420447e-07f, -1.0f - 8.382420447e-07f));
  const float2 h = make_float2(ex2_approx(q.x), ex2_approx(q.y));  // erfc(|t| / sqrt 2) / 2
  return __ffma2_rn(m, h, make_float2(fmaxf(t.x, 0.f), fmaxf(t.y, 0.f)));
}

// Relative position bias of (query, key) from their rows' linear coordinates; `tab` is the head's table, `root`
// the square root of the head dimension (the scores are still unscaled dot products when the bias is added).
__device__ __forceinline__ float rpb_term(const float* __restrict__ tab, int lin_q, int lin_k, float root) {
  const int idx = (int)(short)(lin_q - lin_k) + s_mi.rb_centre;
  return __ldg(tab + min((unsigned)idx, (unsigned)(s_mi.rb_len - 1))) * root;  // (a negative index clamps too)
}

// ---------------------------------------------------------------------------------------------
// Attention of one tile with mma.sync, blocked by 16 consecutive tile rows rather than by set: one warp per (row
// block, head).  The keys of a block are the rows of every set that the block touches; a score is
// kept only where query and key belong to the same set (row_lo / row_n give each row's set range).
// The arithmetic per query row is exactly the per-set softmax attention, but sparse regions with
// many tiny sets cost one item per 16 rows instead of one per set, and the running softmax over passes of four key
// blocks keeps the registers low for sets of any size (a version with one item per set and all of a set's scores in
// registers spilled for set sizes near 96 and was a quarter slower there).
// NTB = key blocks of 8 a row block can need: ceil((2 tau + 14) / 8), at most the 16 of a whole tile.
// ---------------------------------------------------------------------------------------------
template <int C, int D, int NTB, bool RPB>
__device__ __noinline__ void attend_blocked() {
  constexpr int DC = D / 8;  // 16-byte chunks per head
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t a_base = s_mi.sbase + s_mi.off_a, k_base = s_mi.sbase + s_mi.off_kv;
  const uint32_t v_base = k_base + (C / 64) * (kTM * 128);
  const unsigned char* row_lo = s_mi.row_lo[s_mi.buf];
  const unsigned char* row_n = s_mi.row_n[s_mi.buf];
  const int rows = s_mi.rows, heads = s_mi.heads;
  constexpr int PW = 4;      // key blocks of 8 per pass (running softmax across passes keeps registers low)
  const int t4 = lane & 3;
  const float sc = 1.4426950408889634f * rsqrtf((float)D);  // log2(e) / sqrt(d)
  const int nblk = (rows + 15) >> 4;
  for (int item = warp; item < nblk * heads; item += kComputeWarps) {
    const int blk = item / heads, h = item - blk * heads;
    const int c0 = h * DC;
    const int q0 = 16 * blk;
    const int k_lo = row_lo[q0];
    const int r_last = min(q0 + 15, rows - 1);
    const int ntu = min((row_lo[r_last] + row_n[r_last] - k_lo + 7) >> 3, NTB);
    const int ra = q0 + (lane >> 2), rb = ra + 8;
    // each thread's two query rows: first key and number of keys of their sets, relative to k_lo
    // (rows past the tile get zero keys)
    const unsigned loA = ra < rows ? (unsigned)(row_lo[ra] - k_lo) : 0u;
    const unsigned nA = ra < rows ? (unsigned)row_n[ra] : 0u;
    const unsigned loB = rb < rows ? (unsigned)(row_lo[rb] - k_lo) : 0u;
    const unsigned nB = rb < rows ? (unsigned)row_n[rb] : 0u;
    const float root = sqrtf((float)D);
    const float* tab = RPB ? s_mi.rpb + (size_t)h * s_mi.rb_len : nullptr;
    const int linA = RPB ? s_mi.rowlin[min(ra, kTM - 1)] : 0, linB = RPB ? s_mi.rowlin[min(rb, kTM - 1)] : 0;
    uint32_t qa[4], qb[4];
    {
      const int row = q0 + (lane & 15);  // <= 127
      ldsm_x4(a_base + swz(row, c0 + (lane >> 4)), qa);
      if (D > 16) ldsm_x4(a_base + swz(row, c0 + 2 + ((D == 32) ? (lane >> 4) : 0)), qb);
    }
    // Row addresses advance by one 1024-byte group per key block of 8 (the swizzle depends on row & 7 only).
    // Reads may run up to two groups past row 127: they land in the neighbouring operand block or, for the last
    // 64 value columns, in the weight ring, and meet zero probabilities.  Those bytes are this tile's own K / V
    // values or this layer's weights: a non-finite value among them (0 x Inf) could only come from a non-finite
    // weight or feature, and every output row of a layer depends on every weight of the layer, so such a layer has
    // no finite output row to spoil.
    uint32_t k_addr = k_base + swz(k_lo + (lane & 7), c0 + min(lane >> 3, DC - 1));
    uint32_t v_addr[DC];
#pragma unroll
    for (int dn = 0; dn < DC; ++dn) v_addr[dn] = v_base + swz(k_lo + (lane & 15), c0 + dn);
    float o[DC][4];
#pragma unroll
    for (int dn = 0; dn < DC; ++dn) o[dn][0] = o[dn][1] = o[dn][2] = o[dn][3] = 0.f;
    float mA = -INFINITY, mB = -INFINITY, l0 = 0.f, l1 = 0.f;  // running row maxima and sums
    for (int j0 = 0; j0 < ntu; j0 += PW) {
      float s[PW][4];
      float mx0 = mA, mx1 = mB;
#pragma unroll
      for (int jj = 0; jj < PW; ++jj) {
        if (j0 + jj < ntu) {
          s[jj][0] = s[jj][1] = s[jj][2] = s[jj][3] = 0.f;
          uint32_t kf[4];
          ldsm_x4(k_addr + 1024u * jj, kf);
          mma_16816(s[jj], qa, kf[0], kf[1]);
          if (D == 24) mma_1688(s[jj], qb[0], qb[1], kf[2]);
          if (D == 32) mma_16816(s[jj], qb, kf[2], kf[3]);
          const unsigned key = (unsigned)(8 * (j0 + jj) + 2 * t4);
          if (RPB) {
            const int kr = k_lo + (int)key;  // (rows past the tile are masked below: any entry will do)
            const int lk0 = s_mi.rowlin[min(kr, kTM - 1)], lk1 = s_mi.rowlin[min(kr + 1, kTM - 1)];
            s[jj][0] += rpb_term(tab, linA, lk0, root);
            s[jj][1] += rpb_term(tab, linA, lk1, root);
            s[jj][2] += rpb_term(tab, linB, lk0, root);
            s[jj][3] += rpb_term(tab, linB, lk1, root);
          }
          if (key - loA >= nA) s[jj][0] = -INFINITY;  // unsigned: also true for key < lo
          if (key + 1u - loA >= nA) s[jj][1] = -INFINITY;
          if (key - loB >= nB) s[jj][2] = -INFINITY;
          if (key + 1u - loB >= nB) s[jj][3] = -INFINITY;
          mx0 = fmaxf(mx0, fmaxf(s[jj][0], s[jj][1]));
          mx1 = fmaxf(mx1, fmaxf(s[jj][2], s[jj][3]));
        }
      }
      k_addr += 1024u * PW;
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      // rows without any key so far (rows past the tile) keep finite arithmetic
      const float off0 = (mx0 == -INFINITY) ? 0.f : -mx0 * sc, off1 = (mx1 == -INFINITY) ? 0.f : -mx1 * sc;
      if (j0 > 0) {  // rescale what the earlier passes accumulated to the new maxima
        const float al0 = (mA == -INFINITY) ? 0.f : ex2_approx(fmaf(mA, sc, off0));
        const float al1 = (mB == -INFINITY) ? 0.f : ex2_approx(fmaf(mB, sc, off1));
        l0 *= al0;
        l1 *= al1;
#pragma unroll
        for (int dn = 0; dn < DC; ++dn) { o[dn][0] *= al0; o[dn][1] *= al0; o[dn][2] *= al1; o[dn][3] *= al1; }
      }
      mA = mx0;
      mB = mx1;
#pragma unroll
      for (int kk = 0; kk < PW / 2; ++kk) {
        if (j0 + 2 * kk < ntu) {
          const bool two = j0 + 2 * kk + 1 < ntu;
          float e[8];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            e[u] = ex2_approx(fmaf(s[2 * kk][u], sc, u < 2 ? off0 : off1));
            e[4 + u] = two ? ex2_approx(fmaf(s[2 * kk + 1][u], sc, u < 2 ? off0 : off1)) : 0.f;
          }
          l0 += (e[0] + e[1]) + (e[4] + e[5]);
          l1 += (e[2] + e[3]) + (e[6] + e[7]);
          uint32_t pa[4];
          pa[0] = pack_bf16(e[0], e[1]);
          pa[1] = pack_bf16(e[2], e[3]);
          pa[2] = pack_bf16(e[4], e[5]);
          pa[3] = pack_bf16(e[6], e[7]);
#pragma unroll
          for (int dn = 0; dn < DC; ++dn) {
            uint32_t vf[2];
            ldsm_x2_trans(v_addr[dn] + 2048u * kk, vf);
            mma_16816(o[dn], pa, vf[0], vf[1]);
          }
        }
      }
#pragma unroll
      for (int dn = 0; dn < DC; ++dn) v_addr[dn] += 1024u * PW;
    }
    // the per-thread partial sums of a row live in the four threads of its quad
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float i0 = __fdividef(1.0f, l0), i1 = __fdividef(1.0f, l1);
    // the query rows of this block and head are dead now: their slots take the attention output
    if (ra < rows) {
#pragma unroll
      for (int dn = 0; dn < DC; ++dn)
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(a_base + swz(ra, c0 + dn) + 4 * t4),
                     "r"(pack_bf16(o[dn][0] * i0, o[dn][1] * i0)) : "memory");
    }
    if (rb < rows) {
#pragma unroll
      for (int dn = 0; dn < DC; ++dn)
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(a_base + swz(rb, c0 + dn) + 4 * t4),
                     "r"(pack_bf16(o[dn][2] * i1, o[dn][3] * i1)) : "memory");
    }
  }
}

// fp32 row staging in the K/V region: row r, 16-byte chunk c4 of C/4, rotated by the row so that both
// the warp-per-row pattern (global side) and the thread-per-row pattern (TMEM side) are conflict-free.
template <int C>
__device__ __forceinline__ uint32_t stage_off(int r, int c4) {
  constexpr int NCH = C / 4;
  int idx = c4 + (r % NCH);
  if (idx >= NCH) idx -= NCH;
  return (uint32_t)(r * (C * 4) + (idx << 4));
}

// ---------------------------------------------------------------------------------------------
// Roles
// ---------------------------------------------------------------------------------------------
struct RoleCtx {
  uint32_t sbase;     // 1024-aligned shared-memory base as a shared-space address
  uint32_t tmem;      // TMEM base address of the CTA's allocation
  // copies of the kernel parameters the two single-thread roles use (registers instead of parameter-space loads)
  int mode, n_f1, NF, nkb_h, tau, n_layers;
  int pe;  // the value projection comes first and the A operand is rewritten (x + pe) before the key and query ones
  uint32_t off_a, off_kv, off_stage;
};

__device__ __forceinline__ int ld_acquire_gpu(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_gpu(int32_t* p, int v) {
  asm volatile("st.relaxed.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// The scheduler and the MMA issuer are separate (not inlined) functions so that their polling loops get
// their own, spill-free register allocation; the compute role is inlined into the kernel, where the
// kernel parameters are constant-bank operands.

// ================= scheduler + TMA producer (one thread) ===============================================
// Tiles are numbered over the whole chain, layer after layer; a tile's number comes from the launch's counter.
// Inside a layer, tile t is entry t of the layer's plan (whole sets, at most 128 distinct rows); a layer without
// a plan is cut by row ranges instead: tile t holds the sets whose first row lies in [t R, (t + 1) R),
// R = 128 - tau + 1, found by binary search in the row offsets (slower to schedule, same results).
template <int C>
__device__ __noinline__ void producer_role(const TcArgs& a, const RoleCtx rc) {
  constexpr int NKB = C / 64;        // K blocks of a C-deep contraction
  constexpr uint32_t STAGE_BYTES = C * 128;
  Misc* mi = &s_mi;
  const uint32_t st_base = rc.sbase + rc.off_stage;
  volatile int* abort_flag = &mi->abort_flag;
  int32_t* status = a.status;
  const bool mlp = rc.mode == 2;
  const int n_chunks = 4 + (mlp ? rc.n_f1 + 1 : 0);
  const int L = rc.n_layers;
  const int Rv = kTM - rc.tau + 1;
  // the chain's tile counts
  int total = 0;
  for (int l = 0; l < L; ++l) {
    const TcLayer& ly = a.layer[l];
    const int S = min(__ldg(ly.num_sets), ly.cap_sets);
    int T = __ldg(ly.rowoff + ly.cap_sets + 1);
    mi->lay_S[l] = S;
    mi->lay_plan[l] = T < 0 ? 0 : (T & DSVT_PLAN_PACKED) ? 2 : 1;  // none / in table order / over a reordering
    if (T < 0) T = S > 0 ? (__ldg(ly.rowoff + S) + Rv - 1) / Rv : 0;
    else T = min(T & ~DSVT_PLAN_PACKED, S);
    total += max(T, 0);
    mi->tile_end[l] = total;
  }
  // next tile: layer, first set s0, ns sets (< 0: none left), first row, rows
  auto next_tile = [&](int& lay, int& s0, int& ns, int& base, int& rows) {
    for (;;) {
      lay = 0; s0 = 0; ns = -1; base = 0; rows = 0;
      if (*abort_flag) return;
      const int g = atomicAdd(a.counter, 1);
      if (g < 0 || g >= total) return;
      int l = 0;
      while (l + 1 < L && g >= mi->tile_end[l]) ++l;
      const int t = g - (l ? mi->tile_end[l - 1] : 0);
      const TcLayer& ly = a.layer[l];
      const int S = mi->lay_S[l];
      int f, e;
      if (mi->lay_plan[l]) {
        const int32_t* plan = ly.rowoff + ly.cap_sets + 1;
        f = __ldg(plan + 1 + t);
        e = __ldg(plan + 2 + t);
        if (f < 0 || e <= f || e > S) { atomicOr(status, DSVT_STATUS_BAD_INDEX); continue; }
      } else {
        const int r0 = t * Rv, r1 = r0 + Rv;
        int lo = 0, hi = S;
        while (lo < hi) { const int m = (lo + hi) >> 1; if (__ldg(ly.rowoff + m) < r0) lo = m + 1; else hi = m; }
        f = lo;
        hi = S;
        while (lo < hi) { const int m = (lo + hi) >> 1; if (__ldg(ly.rowoff + m) < r1) lo = m + 1; else hi = m; }
        e = lo;
        if (e <= f) continue;  // no set starts in this row range
      }
      // rows before a position: of the table's own order, or of the packed plan's
      const int32_t* ro = mi->lay_plan[l] == 2 ? ly.rowoff + 3 * (size_t)ly.cap_sets + 3 : ly.rowoff;
      base = __ldg(ro + f);
      rows = __ldg(ro + e) - base;
      if (rows <= 0 || rows > kTM || e - f > kTM) { atomicOr(status, DSVT_STATUS_BAD_INDEX); continue; }
      lay = l; s0 = f; ns = e - f;
      return;
    }
  };
  int stage = 0, slot = 0;
  uint32_t phase = 0, sphase = 0;
  int issued[kStages];  // loads issued into each stage so far
#pragma unroll
  for (int i = 0; i < kStages; ++i) issued[i] = 0;
  int lay, s, ns, base, rows;
  int wl[2] = {0, 0}, wcount = 0, wread = 0;  // layers of the published tiles whose weights are still to be streamed
  bool all_out = false;    // the end marker has been published
  // Tiles are published two ahead of the weights (the ring has two entries), so that the loader
  // warp can prepare tile k + 1 while tile k is being computed.
  auto publish = [&]() -> bool {
    next_tile(lay, s, ns, base, rows);
    if (!mbar_wait(&mi->sched_empty[slot], sphase ^ 1u, abort_flag)) return false;
    mi->tile[slot][0] = s; mi->tile[slot][1] = ns; mi->tile[slot][2] = base; mi->tile[slot][3] = rows;
    mi->tile[slot][4] = lay;
    mbar_arrive(&mi->sched_full[slot]);
    if (++slot == 2) { slot = 0; sphase ^= 1u; }
    if (ns < 0) { all_out = true; return true; }
    wl[(wread + wcount) & 1] = lay;
    ++wcount;
    return true;
  };
  if (!publish()) goto producer_done;
  if (!all_out && !publish()) goto producer_done;
  while (wcount > 0) {
    // the layer's weights for one tile, chunk by chunk, K block by K block
    const TcLayer& ly = a.layer[wl[wread & 1]];
    for (int c = 0; c < n_chunks; ++c) {
      const CUtensorMap* map;
      int row0, nkb;
      uint32_t bytes = STAGE_BYTES;
      if (c < 3) {  // K, V, Q; with a positional term V, K, Q
        map = &ly.qkv; nkb = NKB;
        row0 = (rc.pe ? (c == 0 ? 2 : c == 1 ? 1 : 0) : (c == 0 ? 1 : c == 1 ? 2 : 0)) * C;
      }
      else if (c == 3) { map = &ly.o; row0 = 0; nkb = NKB; }
      else if (c < 4 + rc.n_f1) { map = &ly.w1; row0 = (c - 4) * rc.NF; nkb = NKB; bytes = (uint32_t)rc.NF * 128u; }
      else { map = &ly.w2; row0 = 0; nkb = rc.nkb_h; }
      for (int kb = 0; kb < nkb; ++kb) {
        if (!mbar_wait(&mi->empty[stage], phase ^ 1u, abort_flag)) goto producer_done;
        mbar_expect_tx(&mi->full[stage], bytes);
        tma_load_2d(st_base + stage * STAGE_BYTES, map, kb * 64, row0, &mi->full[stage]);
        ++issued[stage];
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
    }
    ++wread;
    --wcount;
    if (!all_out && !publish()) goto producer_done;
  }
producer_done:
  if (*abort_flag) {
    // leaving early: no load may still be writing into this CTA's shared memory when it retires
#pragma unroll
    for (int i = 0; i < kStages; ++i)
      if (issued[i] > 0) {
        const uint32_t par = (uint32_t)(issued[i] - 1) & 1u;
        for (int it = 0; it < kMaxPolls && !mbar_try(&mi->full[i], par); ++it) {}
      }
  }
}

// ================= MMA issuer (one thread) =============================================================
template <int C>
__device__ __noinline__ void mma_role(const RoleCtx rc) {
  constexpr int NKB = C / 64;        // K blocks of a C-deep contraction
  constexpr uint32_t COL_B = C;      // second accumulator buffer
  constexpr uint32_t STAGE_BYTES = C * 128;
  const uint32_t sbase = rc.sbase, tmem = rc.tmem;
  Misc* mi = &s_mi;
  const uint32_t a_base = sbase + rc.off_a, kv_base = sbase + rc.off_kv, st_base = sbase + rc.off_stage;
  volatile int* abort_flag = &mi->abort_flag;
  const bool mlp = rc.mode == 2;
  const int n_chunks = 4 + (mlp ? rc.n_f1 + 1 : 0);
  int stage = 0, slot = 0;
  uint32_t phase = 0, a_phase = 0, x_phase = 0, sphase = 0;
  uint32_t uses[3] = {0u, 0u, 0u};  // how often each accumulator region has been used
  for (;;) {
    if (!mbar_wait(&mi->sched_full[slot], sphase, abort_flag)) break;
    const int ns = mi->tile[slot][1];
    mbar_arrive(&mi->sched_empty[slot]);
    if (++slot == 2) { slot = 0; sphase ^= 1u; }
    if (ns < 0) break;
    for (int c = 0; c < n_chunks; ++c) {
      // a fresh A operand: X (chunks 0-2), attention output (3), x1 (4..), MLP hidden (last)
      if (c == 0 || (c == 1 && rc.pe)) {  // (with a positional term the operand is rewritten after the V chunk)
        if (!mbar_wait(&mi->x_ready, x_phase, abort_flag)) goto mma_done;
        x_phase ^= 1u;
      } else if (c == 3 || c == 4 || c == 4 + rc.n_f1) {
        if (!mbar_wait(&mi->a_ready, a_phase, abort_flag)) goto mma_done;
        a_phase ^= 1u;
      }
      // accumulator placement: K -> region 0, V -> 1, Q -> 0, O -> 0, MLP-1 piece i -> i & 1, MLP-2 -> 2
      // (on top of the parked x1 + b_2)
      uint32_t bar, col, n;
      const int c_v = rc.pe ? 0 : 1;  // the V chunk
      if (c < 4) { bar = (c == c_v) ? 1u : 0u; col = (c == c_v) ? COL_B : 0u; n = C; }
      else if (c < 4 + rc.n_f1) { bar = (uint32_t)(c - 4) & 1u; col = bar * COL_B; n = (uint32_t)rc.NF; }
      else { bar = 2u; col = kTmemCols - C; n = C; }
      if (c == c_v) {
        // region 1 may overlap region 2: the previous tile's MLP-2 result must have been read
        if (!mbar_wait(&mi->acc_free[2], (uses[2] & 1u) ^ 1u, abort_flag)) goto mma_done;
      }
      if (bar != 2u && !mbar_wait(&mi->acc_free[bar], (uses[bar] & 1u) ^ 1u, abort_flag)) goto mma_done;
      ++uses[bar];
      tc_fence_after();
      const bool last = mlp && c == 4 + rc.n_f1;
      const uint32_t abase = last ? kv_base : a_base;
      const int nkb = last ? rc.nkb_h : NKB;
      const uint32_t idesc = umma_idesc((int)n);
      const uint32_t d_tmem = tmem + col;
      for (int kb = 0; kb < nkb; ++kb) {
        if (!mbar_wait(&mi->full[stage], phase, abort_flag)) goto mma_done;
        tc_fence_after();
        const uint32_t sa = abase + kb * (kTM * 128), sb = st_base + stage * STAGE_BYTES;
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
          umma_bf16(d_tmem, umma_desc(sa + k4 * 32), umma_desc(sb + k4 * 32), idesc, (last || (kb | k4) != 0) ? 1u : 0u);
        umma_commit(&mi->empty[stage]);  // frees the weight stage once these MMAs have read it
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
      umma_commit(&mi->acc_full[bar]);
    }
  }
mma_done:
  if (*abort_flag) {
    // leaving early: the MMAs already issued must have completed before the TMEM columns are returned
    umma_commit(&mi->drain);
    for (int it = 0; it < kMaxPolls && !mbar_try(&mi->drain, 0u); ++it) {}
  }
}

// ================= loader warp: row list, one tile ahead of the compute warps =============================
__device__ __forceinline__ void loader_sync() { asm volatile("bar.sync 6, %0;" ::"n"(kLoadThreads) : "memory"); }

// Distinct slots of each set -> tile rows (Eq. 4) and per-row set ranges: one thread per
// set (a tile of a sparse region holds dozens of tiny sets), walking the set's table row.
// `order` (or NULL: the identity) maps the positions [s_lo, s_lo + nsets) of the tile to sets, `rowoff` holds the
// rows before each position.
template <bool RPB>
__device__ __forceinline__ void loader_row_list(const int32_t* __restrict__ table, const int32_t* __restrict__ rowoff,
                                                const int32_t* __restrict__ order, int cap_sets, int b, int lt,
                                                int s_lo, int nsets, int base) {
  const int n = s_mi.n, tau = s_mi.tau;
  for (int si = lt; si < nsets; si += kLoadThreads) {
    const int p = s_lo + si;
    const int s = order ? __ldg(order + p) : p;
    if ((unsigned)s >= (unsigned)cap_sets) {  // (only a plan that this library did not write can do that)
      atomicOr(s_mi.status, DSVT_STATUS_BAD_INDEX);
      continue;
    }
    const int32_t* trow = table + (size_t)s * tau;
    const int lb = __ldg(rowoff + p) - base, cap = __ldg(rowoff + p + 1) - __ldg(rowoff + p);
    const bool inside = lb >= 0 && lb < kTM;
    const int cnt_max = inside ? min(cap, kTM - lb) : 0;  // tile rows this set may fill
    int pos = 0, prev = 0;
    bool bad = false;
    constexpr bool rpb = RPB;
    int lo3[3] = {INT_MAX, INT_MAX, INT_MAX}, hi3[3] = {INT_MIN, INT_MIN, INT_MIN};
    for (int k0 = 0; k0 < tau; k0 += 8) {
      int v4[8];  // eight independent loads per round trip to L2 (the loader warp runs a whole tile ahead)
#pragma unroll
      for (int u = 0; u < 8; ++u) v4[u] = k0 + u < tau ? __ldg(trow + k0 + u) : 0;
      if (rpb) {  // a set spread wider than the bias table's extent is reported
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          if (k0 + u < tau && v4[u] >= 0 && v4[u] < n) {
            const int4 c = __ldg(s_mi.coords + v4[u]);
            lo3[0] = min(lo3[0], c.y); hi3[0] = max(hi3[0], c.y);
            lo3[1] = min(lo3[1], c.z); hi3[1] = max(hi3[1], c.z);
            lo3[2] = min(lo3[2], c.w); hi3[2] = max(hi3[2], c.w);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (k0 + u < tau) {
          int v = v4[u];
          const bool uniq = (k0 + u == 0) || (v != prev);
          prev = v;
          if (uniq) {
            if (pos < cnt_max) {
              if (v < 0 || v >= n) { bad = true; v = -1; }
              s_mi.rowvox[b][lb + pos] = v;
              s_mi.row_lo[b][lb + pos] = (unsigned char)lb;
              s_mi.row_n[b][lb + pos] = (unsigned char)cnt_max;
            }
            ++pos;
          }
        }
      }
    }
    if (rpb)
      for (int q = 0; q < 3; ++q) bad |= hi3[q] >= lo3[q] && hi3[q] - lo3[q] > s_mi.rb_ext[q] - 1;
    if (bad || pos != cap) atomicOr(s_mi.status, DSVT_STATUS_BAD_INDEX);
  }
}

template <int C, bool RPB>
__device__ __noinline__ void loader_role(const TcArgs& a) {
  const int lt = threadIdx.x - 32 * kLoadWarp0, lane = lt & 31;
  volatile int* abort_flag = &s_mi.abort_flag;
  int slot = 0;
  uint32_t sphase = 0;
  bool ok = true;
  for (int k = 0;; ++k) {
    ok = mbar_wait(&s_mi.sched_full[slot], sphase, abort_flag) && ok;
    // every exit from this loop is taken by all loader threads together
    if (bar_or(6, kLoadThreads, !ok || *abort_flag != 0)) break;
    const int s_lo = s_mi.tile[slot][0], nsets = s_mi.tile[slot][1], base = s_mi.tile[slot][2], rows = s_mi.tile[slot][3];
    const int lay = s_mi.tile[slot][4];
    __syncwarp();
    if (lane == 0) mbar_arrive(&s_mi.sched_empty[slot]);
    if (++slot == 2) { slot = 0; sphase ^= 1u; }
    const int b = k & 1;
    // buffer b was last used by tile k - 2: the compute warps and the stamp warp release it when they are done with it
    if (k >= 2) ok = mbar_wait(&s_mi.rl_free[b], (uint32_t)((k >> 1) - 1) & 1u, abort_flag) && ok;
    if (nsets >= 0) {
      for (int i = lt; i < kTM; i += kLoadThreads) {
        s_mi.rowvox[b][i] = -1;
        s_mi.row_lo[b][i] = (unsigned char)i;
        s_mi.row_n[b][i] = 1;
      }
      loader_sync();
      const TcLayer& ly = a.layer[lay];
      const bool packed = s_mi.lay_plan[lay] == 2;
      loader_row_list<RPB>(ly.table, packed ? ly.rowoff + 3 * (size_t)ly.cap_sets + 3 : ly.rowoff,
                           packed ? ly.rowoff + 2 * (size_t)ly.cap_sets + 3 : nullptr, ly.cap_sets, b, lt, s_lo, nsets, base);
      if (lt == 0) s_mi.next_x[b] = lay == 0 ? a.x : a.y;
    }
    if (lt == 0) s_mi.next_rows[b] = nsets < 0 ? -1 : rows;
    mbar_arrive(&s_mi.rl_ready[b]);
    if (nsets < 0) break;
    // a tile of a later layer reads rows the previous layer wrote, possibly on other SMs: each row must carry that
    // layer's stamp (written after the row's store) before the tile is gathered
    if (lay > 0) {
      loader_sync();  // the row list is complete
      const int want = a.stamp_base + lay;
      for (int r = lt; r < rows && ok; r += kLoadThreads) {
        const int v = s_mi.rowvox[b][r];
        if (v < 0) continue;
        int it = 0;
        while (ld_acquire_gpu(a.row_stamp + v) != want) {
          if (++it >= kStampPolls || *abort_flag) { *abort_flag = 1; ok = false; break; }
          __nanosleep(256);
        }
      }
    }
    mbar_arrive(&s_mi.dep_ready[b]);
  }
}

// ================= stamp warp: completion stamps of a stored tile's rows ==================================
__device__ __noinline__ void stamp_role(int32_t* __restrict__ row_stamp) {
  const int lane = threadIdx.x & 31;
  volatile int* abort_flag = &s_mi.abort_flag;
  for (int k = 0;; ++k) {
    const int b = k & 1;
    // (a failed wait has raised the abort flag: the compute warps leave their loop, and so does this warp)
    if (!mbar_wait(&s_mi.stored[b], (uint32_t)(k >> 1) & 1u, abort_flag)) break;
    if (s_mi.exit_at == k) break;
    const int rows = s_mi.st_rows[b], stamp = s_mi.st_stamp[b];
    if (stamp != 0) {
      __threadfence();  // the rows' stores (ordered before this warp by the barrier) are visible before the stamps
      for (int r = lane; r < rows; r += 32) {
        const int v = s_mi.rowvox[b][r];
        if (v >= 0) st_relaxed_gpu(row_stamp + v, stamp);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&s_mi.rl_free[b]);
  }
}

// ================= compute warps ========================================================================
// Each phase of a tile is a separate (not inlined) function that takes at most a few scalars and reads the
// rest from s_mi, so that each gets a register allocation of its own and the tile loop keeps almost nothing
// alive across the calls.

// Gather (Eq. 4): the fp32 rows listed in buffer b -> bf16 A operand, four rows in flight per warp; all 128 rows
// are written (rows past the tile as zeros).  ADD_PE: the current tile's rows once more, with the positional
// term added (the operand of the key and query projections).
template <int C, bool RPB, bool ADD_PE>
__device__ __noinline__ void phase_gather(int b, int rows) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* x = ADD_PE ? s_mi.x : s_mi.next_x[b];
  unsigned char* a_tile = s_mi.sm + s_mi.off_a;
  const int* rowvox = s_mi.rowvox[b];
  for (int r0 = warp; r0 < kTM; r0 += 4 * kComputeWarps) {
    float4 f[4][2];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int r = r0 + kComputeWarps * u;
      const int v = r < rows ? rowvox[r] : -1;
      f[u][0] = f[u][1] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (v >= 0 && lane < (C >> 3)) {
        const float4* src = reinterpret_cast<const float4*>(x + (size_t)v * C) + 2 * lane;
        f[u][0] = __ldcg(src);  // (L2: the rows of a later layer were written during this launch, by any SM)
        f[u][1] = __ldcg(src + 1);
        if (ADD_PE) {
          const float4* pp = reinterpret_cast<const float4*>(s_mi.pe + (size_t)v * C) + 2 * lane;
          const float4 p0 = __ldg(pp), p1 = __ldg(pp + 1);
          f[u][0].x += p0.x; f[u][0].y += p0.y; f[u][0].z += p0.z; f[u][0].w += p0.w;
          f[u][1].x += p1.x; f[u][1].y += p1.y; f[u][1].z += p1.z; f[u][1].w += p1.w;
        }
      }
      if (RPB && !ADD_PE && lane == 31) {  // (lane 31 carries no feature columns: C / 8 <= 24)
        int lin = 0;
        if (v >= 0) {
          const int4 c = __ldg(s_mi.coords + v);
          lin = c.y * s_mi.rb_sx + c.z * s_mi.rb_sy + c.w;
        }
        s_mi.rowlin[r] = (short)lin;
      }
    }
    if (lane < (C >> 3)) {
#pragma unroll
      for (int u = 0; u < 4; ++u)
        *reinterpret_cast<uint4*>(a_tile + swz(r0 + kComputeWarps * u, lane)) =
            make_uint4(pack_bf16(f[u][0].x, f[u][0].y), pack_bf16(f[u][0].z, f[u][0].w),
                       pack_bf16(f[u][1].x, f[u][1].y), pack_bf16(f[u][1].z, f[u][1].w));
    }
  }
}

// Epilogue of a projection chunk: QC accumulator columns per thread + bias -> bf16 into an operand tile.
// Four threads per tile row: warp w owns TMEM lanes 32 (w % 4) .. + 31 and column quarter w / 4.
//   tcol      first TMEM column of the chunk's accumulator
//   bar       accumulator barrier pair to release
//   bias_off  float offset of the chunk's bias in the parameter block
//   dst_off   byte offset of the destination operand tile from the shared-memory base
//   c8_0      16-byte chunk index of the chunk's first column in the destination rows
//   need      number of leading tile rows whose results are needed (warps wholly past it only release)
// GELU = true applies gelu first (MLP-1); BIAS = false skips the bias (the key projection: a key bias adds
// the same amount q . b_k to every score of a query, which the softmax cancels).
template <int QC, bool GELU, bool BIAS>
__device__ __noinline__ void phase_epi_bf16(uint32_t tcol, int bar, int bias_off, uint32_t dst_off, int c8_0, int need) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = 32 * (warp & 3) + lane, hq = warp >> 2;
  if (32 * (warp & 3) >= need) {
    tc_fence_before();
    mbar_arrive(&s_mi.acc_free[bar]);
    return;
  }
  const uint32_t taddr = s_mi.tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + tcol + hq * QC;
  const float* bias = reinterpret_cast<const float*>(s_mi.sm + s_mi.off_par) + bias_off + hq * QC;
  unsigned char* dst = s_mi.sm + dst_off;
  const int c8 = c8_0 + ((hq * QC) >> 3);
  float rr[QC];
  tmem_ld_row(taddr, rr);
  tmem_wait_ld();
  tc_fence_before();
  mbar_arrive(&s_mi.acc_free[bar]);  // the accumulator is in registers now
#pragma unroll
  for (int q = 0; q < QC / 8; ++q) {
    float2 v[4] = {make_float2(rr[8 * q], rr[8 * q + 1]), make_float2(rr[8 * q + 2], rr[8 * q + 3]),
                   make_float2(rr[8 * q + 4], rr[8 * q + 5]), make_float2(rr[8 * q + 6], rr[8 * q + 7])};
    if (BIAS) {
      const float4 b0 = *reinterpret_cast<const float4*>(bias + 8 * q), b1 = *reinterpret_cast<const float4*>(bias + 8 * q + 4);
      v[0] = __fadd2_rn(v[0], make_float2(b0.x, b0.y));
      v[1] = __fadd2_rn(v[1], make_float2(b0.z, b0.w));
      v[2] = __fadd2_rn(v[2], make_float2(b1.x, b1.y));
      v[3] = __fadd2_rn(v[3], make_float2(b1.z, b1.w));
    }
    if (GELU) {
#pragma unroll
      for (int e = 0; e < 4; ++e) v[e] = gelu_fast2(v[e]);
    }
    *reinterpret_cast<uint4*>(dst + swz(row, c8 + q)) =
        make_uint4(pack_bf16(v[0].x, v[0].y), pack_bf16(v[1].x, v[1].y), pack_bf16(v[2].x, v[2].y), pack_bf16(v[3].x, v[3].y));
  }
}

// x rows (fp32) for the first residual: asynchronous 16-byte copies global -> shared staging.
template <int C>
__device__ __noinline__ void phase_stage_x() {
  constexpr int C4 = C / 4;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* __restrict__ x = s_mi.x;
  unsigned char* stage = s_mi.sm + s_mi.off_kv;
  const uint32_t stage_saddr = s_mi.sbase + s_mi.off_kv;
  const int rows = s_mi.rows;
  const int* rowvox = s_mi.rowvox[s_mi.buf];
  for (int r = warp; r < rows; r += kComputeWarps) {
    const int v = rowvox[r];
    for (int c4 = lane; c4 < C4; c4 += 32) {
      const uint32_t off = stage_off<C>(r, c4);
      if (v >= 0)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_saddr + off),
                     "l"(reinterpret_cast<const float4*>(x + (size_t)v * C) + c4) : "memory");
      else
        *reinterpret_cast<float4*>(stage + off) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
}

// fp32 rows staged in shared memory -> coalesced global rows.
template <int C>
__device__ __noinline__ void phase_store_rows() {
  constexpr int C4 = C / 4;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* __restrict__ y = s_mi.y;
  const unsigned char* stage = s_mi.sm + s_mi.off_kv;
  const int rows = s_mi.rows;
  const int* rowvox = s_mi.rowvox[s_mi.buf];
  for (int r = warp; r < rows; r += kComputeWarps) {
    const int v = rowvox[r];
    if (v < 0) continue;
    for (int c4 = lane; c4 < C4; c4 += 32)
      reinterpret_cast<float4*>(y + (size_t)v * C)[c4] = *reinterpret_cast<const float4*>(stage + stage_off<C>(r, c4));
  }
}

// Per-layer vectors staged in shared memory (float offsets into the parameter block).
template <int C>
struct ParOff {
  static constexpr int b_q = 0, b_v = C, b_o = 2 * C, b_2 = 3 * C, ln1_g = 4 * C, ln1_b = 5 * C, ln2_g = 6 * C,
                       ln2_b = 7 * C, b_1 = 8 * C;  // b_1 has `hidden` entries and comes last; no key bias
  static constexpr int vectors = 8;
};

// LayerNorm over the row that four threads share: t holds this thread's QC values, sum their sum.  Each
// thread reduces its own quarter to (mean, sum of squared deviations), the four pairs are exchanged once
// through 8-byte slots that the caller picks (slot(quarter)) and combined exactly (pairwise update of
// Chan et al.).  The four threads of a row sit in warps q, q + 4, q + 8, q + 12 and meet at a barrier of
// their own.  Leaves t normalised; a caller whose slots are overwritten by the results calls quarter_sync()
// before it stores them.
__device__ __forceinline__ void quarter_sync() {
  asm volatile("bar.sync %0, 128;" ::"r"(2 + ((threadIdx.x >> 5) & 3)) : "memory");
}
template <int C, int QC, class Slot>
__device__ __forceinline__ void layer_norm_rows(float (&t)[QC], float sum, const float* gain, const float* shift, float eps,
                                                int hq, Slot slot) {
  const float mq = sum * (1.0f / (float)QC);
  float m2 = 0.f;
#pragma unroll
  for (int i = 0; i < QC; ++i) { const float d = t[i] - mq; m2 = fmaf(d, d, m2); }
  *slot(hq) = make_float2(mq, m2);
  quarter_sync();
  const float2 s0 = *slot(0), s1 = *slot(1), s2 = *slot(2), s3 = *slot(3);
  const float mean = 0.25f * ((s0.x + s1.x) + (s2.x + s3.x));
  const float d0 = s0.x - mean, d1 = s1.x - mean, d2 = s2.x - mean, d3 = s3.x - mean;
  const float ssq = ((s0.y + s1.y) + (s2.y + s3.y)) + (float)QC * ((d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3));
  const float inv = rsqrtf(ssq * (1.0f / (float)C) + eps);
#pragma unroll
  for (int i4 = 0; i4 < QC / 4; ++i4) {
    const float4 g4 = *reinterpret_cast<const float4*>(gain + hq * QC + 4 * i4);
    const float4 b4 = *reinterpret_cast<const float4*>(shift + hq * QC + 4 * i4);
    t[4 * i4] = (t[4 * i4] - mean) * inv * g4.x + b4.x;
    t[4 * i4 + 1] = (t[4 * i4 + 1] - mean) * inv * g4.y + b4.y;
    t[4 * i4 + 2] = (t[4 * i4 + 2] - mean) * inv * g4.z + b4.z;
    t[4 * i4 + 3] = (t[4 * i4 + 3] - mean) * inv * g4.w + b4.w;
  }
}

// Output-projection epilogue: t = Z + b_o (+ staged x); LayerNorm 1; then either the fp32 rows go to the
// staging area (mode 0 / 1: final result of the call) or x1 goes to the A operand (bf16) and x1 + b_2 to
// TMEM region 2 (fp32), where the MLP-2 MMAs accumulate on top of it.  The accumulator is region 0.
template <int C, int QC>
__device__ __noinline__ void phase_epi_o() {
  constexpr uint32_t COL_PARK = kTmemCols - C;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = 32 * (warp & 3) + lane, hq = warp >> 2;
  const uint32_t taddr = s_mi.tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + hq * QC;
  const float* par = reinterpret_cast<const float*>(s_mi.sm + s_mi.off_par);
  unsigned char* stage = s_mi.sm + s_mi.off_kv;
  const int mode = s_mi.mode;
  const bool add_x = mode != 0 && row < s_mi.rows;
  float t[QC];
  float sum = 0.f;
  tmem_ld_row(taddr, t);
  tmem_wait_ld();
  tc_fence_before();
  mbar_arrive(&s_mi.acc_free[0]);
#pragma unroll
  for (int q = 0; q < QC / 4; ++q) {
    float4 x4 = make_float4(0.f, 0.f, 0.f, 0.f);
    if (add_x) x4 = *reinterpret_cast<const float4*>(stage + stage_off<C>(row, hq * (QC / 4) + q));
    const float4 b4 = *reinterpret_cast<const float4*>(par + ParOff<C>::b_o + hq * QC + 4 * q);
    t[4 * q] += x4.x + b4.x;
    t[4 * q + 1] += x4.y + b4.y;
    t[4 * q + 2] += x4.z + b4.z;
    t[4 * q + 3] += x4.w + b4.w;
    sum += (t[4 * q] + t[4 * q + 1]) + (t[4 * q + 2] + t[4 * q + 3]);
  }
  if (mode != 0 && s_mi.ln1) {
    // exchange slots: the first eight bytes of each thread's own (already consumed) x staging chunk
    auto slot = [&](int quarter) { return reinterpret_cast<float2*>(stage + stage_off<C>(row, quarter * (QC / 4))); };
    layer_norm_rows<C, QC>(t, sum, par + ParOff<C>::ln1_g, par + ParOff<C>::ln1_b, s_mi.eps, hq, slot);
  }
  if (mode != 2) {
    compute_sync();  // the x staging (and the exchange slots in it) is dead once every thread has its t
#pragma unroll
    for (int i4 = 0; i4 < QC / 4; ++i4)
      *reinterpret_cast<float4*>(stage + stage_off<C>(row, hq * (QC / 4) + i4)) =
          make_float4(t[4 * i4], t[4 * i4 + 1], t[4 * i4 + 2], t[4 * i4 + 3]);
    return;
  }
  unsigned char* a_tile = s_mi.sm + s_mi.off_a;
#pragma unroll
  for (int q = 0; q < QC / 8; ++q)
    *reinterpret_cast<uint4*>(a_tile + swz(row, ((hq * QC) >> 3) + q)) =
        make_uint4(pack_bf16(t[8 * q], t[8 * q + 1]), pack_bf16(t[8 * q + 2], t[8 * q + 3]),
                   pack_bf16(t[8 * q + 4], t[8 * q + 5]), pack_bf16(t[8 * q + 6], t[8 * q + 7]));
#pragma unroll
  for (int q = 0; q < QC / 4; ++q) {
    const float4 b4 = *reinterpret_cast<const float4*>(par + ParOff<C>::b_2 + hq * QC + 4 * q);
    t[4 * q] += b4.x;
    t[4 * q + 1] += b4.y;
    t[4 * q + 2] += b4.z;
    t[4 * q + 3] += b4.w;
  }
  tmem_st_row(taddr + COL_PARK, t);
  tmem_wait_st();
  tc_fence_before();
}

// MLP-2 epilogue: region 2 holds x1 + b_2 + M; LayerNorm 2; fp32 rows to the staging area (the MLP-2 MMAs
// have read H: its region takes the output rows).  The exchange slots are the first eight bytes of each
// thread's own output chunk, which is therefore stored last, after one more meeting of the row's threads.
template <int C, int QC>
__device__ __noinline__ void phase_epi_f2() {
  constexpr uint32_t COL_PARK = kTmemCols - C;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = 32 * (warp & 3) + lane, hq = warp >> 2;
  const uint32_t taddr = s_mi.tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + COL_PARK + hq * QC;
  const float* par = reinterpret_cast<const float*>(s_mi.sm + s_mi.off_par);
  unsigned char* stage = s_mi.sm + s_mi.off_kv;
  float t[QC];
  tmem_ld_row(taddr, t);
  tmem_wait_ld();
  tc_fence_before();
  mbar_arrive(&s_mi.acc_free[2]);
  const bool ln = s_mi.ln2 != 0;
  if (ln) {
    float sum = 0.f;
#pragma unroll
    for (int q = 0; q < QC / 4; ++q) sum += (t[4 * q] + t[4 * q + 1]) + (t[4 * q + 2] + t[4 * q + 3]);
    auto slot = [&](int quarter) { return reinterpret_cast<float2*>(stage + stage_off<C>(row, quarter * (QC / 4))); };
    layer_norm_rows<C, QC>(t, sum, par + ParOff<C>::ln2_g, par + ParOff<C>::ln2_b, s_mi.eps, hq, slot);
  }
#pragma unroll
  for (int i4 = 1; i4 < QC / 4; ++i4)
    *reinterpret_cast<float4*>(stage + stage_off<C>(row, hq * (QC / 4) + i4)) =
        make_float4(t[4 * i4], t[4 * i4 + 1], t[4 * i4 + 2], t[4 * i4 + 3]);
  if (ln) quarter_sync();  // the row's other threads have read this thread's slot
  *reinterpret_cast<float4*>(stage + stage_off<C>(row, hq * (QC / 4))) = make_float4(t[0], t[1], t[2], t[3]);
}

// The layer's biases and LayerNorm vectors into the parameter block (absent vectors as zeros), and its scalars.
// Order of ParOff: b_q, b_v, b_o, b_2, ln1_g, ln1_b, ln2_g, ln2_b, then b_1 (the key bias is not needed).
template <int C>
__device__ __forceinline__ void load_layer_params(const TcLayer& ly, int hidden) {
  float* par = reinterpret_cast<float*>(s_mi.sm + s_mi.off_par);
  const uint32_t par_saddr = s_mi.sbase + s_mi.off_par;
  const int n_par = ParOff<C>::vectors * C + hidden;
  // asynchronous 4-byte copies, all in flight at once: the first reader is the V epilogue, which waits for them
  // (wait_layer_params) after the K epilogue
  for (int i = threadIdx.x; i < n_par; i += kComputeThreads) {
    const int which = i / C;
    const float* v = which == 0 ? ly.b_qkv : which == 1 ? (ly.b_qkv ? ly.b_qkv + 2 * C : nullptr) : which == 2 ? ly.b_o
                   : which == 3 ? ly.b_2 : which == 4 ? ly.ln1_g : which == 5 ? ly.ln1_b : which == 6 ? ly.ln2_g
                   : which == 7 ? ly.ln2_b : (ly.b_1 ? ly.b_1 - ParOff<C>::b_1 + which * C : nullptr);
    if (v) asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(par_saddr + 4u * (uint32_t)i), "l"(v + i % C) : "memory");
    else par[i] = 0.f;
  }
  if (threadIdx.x == 0) {
    s_mi.ln1 = ly.ln1_g != nullptr;
    s_mi.ln2 = ly.ln2_g != nullptr;
    s_mi.eps = ly.eps;
    s_mi.rpb = ly.rpb;
    s_mi.pe = ly.pe;
  }
}

__device__ __forceinline__ void wait_layer_params() {
  asm volatile("cp.async.wait_all;" ::: "memory");
  compute_sync();
}

// Barrier over the compute threads that also ANDs a predicate.
__device__ __forceinline__ bool compute_all(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %2, 0;\n\t"
      "bar.red.and.pred p, 1, %1, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "n"(kComputeThreads), "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

// TMEM map (512 columns): region 0 = [0, C): K, Q, O and the even MLP-1 pieces; region 1 = [C, 2C): V and
// the odd MLP-1 pieces; region 2 = [512 - C, 512): x1 + b_2 parked by the output-projection epilogue, then
// the MLP-2 accumulator.  Each region has its own full / free barrier pair.  For C = 192 regions 1 and 2
// overlap, which is why the MMA issuer waits for region 2 before it starts the next tile's V.
template <int C, int D, int NT, int VAR>
__device__ __forceinline__ void compute_role(const TcArgs& a) {
  constexpr bool RPB = VAR == 1, PE = VAR == 2;
  constexpr int NKB = C / 64;        // K blocks of a C-deep contraction
  constexpr int QC = C / 4;          // epilogue columns per thread for a C-wide chunk (four threads per row)
  constexpr uint32_t COL_B = C;      // accumulator region 1
  volatile int* abort_flag = &s_mi.abort_flag;
  uint32_t uses[3] = {0u, 0u, 0u};
  int slot = 0;
  uint32_t sphase = 0;
  bool ok = true;
  bool gathered = false;  // the tile about to start was gathered under the previous tile's tail
  int cur_layer = -1;     // layer whose vectors are in the parameter block
  auto acc_wait = [&](uint32_t bar) {
    ok = mbar_wait(&s_mi.acc_full[bar], uses[bar] & 1u, abort_flag) && ok;
    ++uses[bar];
    tc_fence_after();
  };
  // The next tile's rows are gathered as soon as the current tile's MMAs have stopped reading the A operand
  // (the caller has just waited for the accumulator of the last such chunk), so that its first projections
  // run on the tensor pipe while the compute warps finish the current tile; unless its rows are not all stamped
  // yet: then the gather waits until this tile is done (the row that is missing may be one of this tile's own).
  auto gather_next = [&](int k) {
    const int b = (k + 1) & 1;
    const uint32_t par = (uint32_t)((k + 1) >> 1) & 1u;
    ok = mbar_wait(&s_mi.rl_ready[b], par, abort_flag) && ok;
    const int nr = s_mi.next_rows[b];
    if (compute_all(ok && nr >= 0 && mbar_try(&s_mi.dep_ready[b], par))) {
      phase_gather<C, RPB, false>(b, nr);
      fence_proxy_async();
      mbar_arrive(&s_mi.x_ready);
      gathered = true;
    }
  };
  int k = 0;
  for (;; ++k) {
    ok = mbar_wait(&s_mi.sched_full[slot], sphase, abort_flag) && ok;
    // also orders the previous tile's last shared-memory reads before this tile's writes; every exit from
    // this loop is taken by all compute threads together
    if (bar_or(1, kComputeThreads, !ok || *abort_flag != 0)) break;
    const int nsets = s_mi.tile[slot][1], rows = s_mi.tile[slot][3], layer = s_mi.tile[slot][4];
    if (threadIdx.x == 0) {
      s_mi.s_lo = s_mi.tile[slot][0];
      s_mi.nsets = nsets;
      s_mi.base = s_mi.tile[slot][2];
      s_mi.rows = rows;
      s_mi.buf = k & 1;
      s_mi.layer = layer;
      s_mi.x = layer == 0 ? a.x : a.y;
      if (k >= 1) mbar_arrive(&s_mi.rl_free[(k - 1) & 1]);  // the previous tile's row list is dead
    }
    mbar_arrive(&s_mi.sched_empty[slot]);
    if (++slot == 2) { slot = 0; sphase ^= 1u; }
    if (nsets < 0) break;
    const bool new_params = layer != cur_layer;
    if (new_params) {  // (the previous tile's last use of the block lies before the barrier above)
      load_layer_params<C>(a.layer[layer], a.g.hidden);
      cur_layer = layer;
    }
    if (!gathered) {  // a CTA's first tile, or a tile whose rows were not ready in time
      const uint32_t par = (uint32_t)(k >> 1) & 1u;
      ok = mbar_wait(&s_mi.rl_ready[k & 1], par, abort_flag) && ok;
      ok = mbar_wait(&s_mi.dep_ready[k & 1], par, abort_flag) && ok;
      if (compute_all(ok)) {
        phase_gather<C, RPB, false>(k & 1, rows);
        fence_proxy_async();
      }
      mbar_arrive(&s_mi.x_ready);  // X is in place
    }
    gathered = false;
    compute_sync();  // the tile's fields are visible to the phase functions

    // ---- chunks 0..2: K, V, Q epilogues: (+ bias,) to bf16, into the operand layout ----
    // (the attention pads its key blocks up to 15 rows past the tile: those K / V rows must be real bf16)
    if (PE) {
      // the values come from the bare rows; the operand is then rewritten with the positional term added, for
      // the keys and the queries (the V chunk's accumulator being complete, nothing reads the operand any more)
      acc_wait(1u);
      if (new_params) wait_layer_params();
      phase_epi_bf16<QC, false, true>(COL_B, 1, ParOff<C>::b_v, s_mi.off_kv + NKB * kTM * 128, 0, rows + 16);
      phase_gather<C, false, true>(k & 1, rows);
      fence_proxy_async();
      mbar_arrive(&s_mi.x_ready);
      acc_wait(0u);
      phase_epi_bf16<QC, false, false>(0u, 0, 0, s_mi.off_kv, 0, rows + 16);
    } else {
      acc_wait(0u);
      phase_epi_bf16<QC, false, false>(0u, 0, 0, s_mi.off_kv, 0, rows + 16);
      acc_wait(1u);
      if (new_params) wait_layer_params();  // (the key epilogue adds no bias: it needs none of the vectors)
      phase_epi_bf16<QC, false, true>(COL_B, 1, ParOff<C>::b_v, s_mi.off_kv + NKB * kTM * 128, 0, rows + 16);
    }
    acc_wait(0u);
    phase_epi_bf16<QC, false, true>(0u, 0, ParOff<C>::b_q, s_mi.off_a, 0, rows);
    compute_sync();
    // ---- attention inside each set ----
    attend_blocked<C, D, NT, RPB>();
    fence_proxy_async();
    mbar_arrive(&s_mi.a_ready);  // attention output is the A operand of the output projection
    compute_sync();              // every warp is done with K and V: their region becomes fp32 staging
    const int mode = s_mi.mode;
    if (mode != 0) {
      phase_stage_x<C>();
      compute_sync();
    }
    // ---- chunk 3: output projection epilogue: Z + b_o (+ x, LayerNorm) ----
    acc_wait(0u);
    phase_epi_o<C, QC>();
    if (mode != 2) {  // final result of this layer
      gather_next(k);  // the output projection was the last chunk to read the A operand
    } else {
      fence_proxy_async();
      mbar_arrive(&s_mi.a_ready);  // x1 (bf16) is the A operand of MLP-1
      // ---- MLP-1 pieces: H = gelu(x1 W_1^T + b_1) as the A operand of MLP-2 ----
      const int n_f1 = s_mi.n_f1, NF = s_mi.NF;
      for (int c = 0; c < n_f1; ++c) {
        const int bar = c & 1;
        acc_wait((uint32_t)bar);
        if (NF == 128)
          phase_epi_bf16<32, true, true>(bar * COL_B, bar, ParOff<C>::b_1 + c * NF, s_mi.off_kv, (c * NF) >> 3, rows);
        else
          phase_epi_bf16<16, true, true>(bar * COL_B, bar, ParOff<C>::b_1 + c * NF, s_mi.off_kv, (c * NF) >> 3, rows);
      }
      fence_proxy_async();
      mbar_arrive(&s_mi.a_ready);  // H is in place
      gather_next(k);  // the last MLP-1 piece has been drained: nothing reads the A operand any more
      // ---- MLP-2 epilogue: y = LN2(x1 + M) ----
      acc_wait(2u);
      phase_epi_f2<C, QC>();
    }
    compute_sync();
    phase_store_rows<C>();
    if (threadIdx.x == 0) {
      s_mi.st_rows[k & 1] = rows;
      s_mi.st_stamp[k & 1] = a.n_layers > 1 ? a.stamp_base + layer + 1 : 0;
    }
    mbar_arrive(&s_mi.stored[k & 1]);  // the stamp warp takes it from here
  }
  // tell the stamp warp to leave at iteration k, once it is done with tile k - 2 (which signalled on the same barrier)
  if (k >= 2) mbar_wait(&s_mi.rl_free[k & 1], (uint32_t)((k >> 1) - 1) & 1u, abort_flag);
  if (threadIdx.x == 0) s_mi.exit_at = k;
  mbar_arrive(&s_mi.stored[k & 1]);
  if (!ok || *abort_flag) {
    if (threadIdx.x == 0) atomicOr(s_mi.status, DSVT_STATUS_TIMEOUT);
  }
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
// VAR: 0 plain, 1 relative position bias on the logits, 2 additive positional term on the query / key inputs
template <int C, int D, int NT, int VAR>
__global__ void __launch_bounds__(kThreads, 1) layer_tc_kernel(const __grid_constant__ TcArgs a) {
  constexpr bool RPB = VAR == 1;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* sm = smem_raw + pad;
  Misc* mi = &s_mi;
  const int tid = threadIdx.x, warp = tid >> 5;
  const TcGeom& g = a.g;
  if (tid == 0) {  // launch constants for the phase functions
    mi->abort_flag = 0;
    mi->exit_at = -1;
    mi->x = a.x; mi->y = a.y; mi->status = a.status;
    mi->sm = sm; mi->sbase = raw + pad;
    mi->off_a = g.off_a; mi->off_kv = g.off_kv; mi->off_par = g.off_par;
    mi->n = a.n; mi->tau = g.tau; mi->heads = g.heads; mi->mode = g.mode; mi->NF = g.NF; mi->n_f1 = g.n_f1;
    mi->ln1 = mi->ln2 = 0;
    mi->eps = 0.f;
    mi->rpb = nullptr; mi->pe = nullptr; mi->coords = a.coords;
    mi->rb_len = g.rb_len; mi->rb_sx = g.rb_sx; mi->rb_sy = g.rb_sy; mi->rb_centre = g.rb_centre;
    mi->rb_ext[0] = g.rb_ext[0]; mi->rb_ext[1] = g.rb_ext[1]; mi->rb_ext[2] = g.rb_ext[2];
    mi->s_lo = mi->nsets = mi->base = mi->rows = mi->buf = mi->layer = 0;
    mi->next_rows[0] = mi->next_rows[1] = -1;
    mi->next_x[0] = mi->next_x[1] = a.x;
    mi->st_rows[0] = mi->st_rows[1] = mi->st_stamp[0] = mi->st_stamp[1] = 0;
  }
  if (tid == 32 * kLoadWarp0) {  // barriers
    for (int i = 0; i < kStages; ++i) { mbar_init(&mi->full[i], 1); mbar_init(&mi->empty[i], 1); }
    for (int i = 0; i < 3; ++i) {
      mbar_init(&mi->acc_full[i], 1);
      mbar_init(&mi->acc_free[i], kComputeThreads);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&mi->sched_full[i], 1);
      mbar_init(&mi->sched_empty[i], kComputeThreads + 1 + kLoadWarps);  // compute threads, MMA issuer, loader warp
      mbar_init(&mi->rl_free[i], 2);  // the compute warps' first thread and the stamp warp
      mbar_init(&mi->rl_ready[i], kLoadThreads);
      mbar_init(&mi->dep_ready[i], kLoadThreads);
      mbar_init(&mi->stored[i], kComputeThreads);
    }
    mbar_init(&mi->a_ready, kComputeThreads);
    mbar_init(&mi->x_ready, kComputeThreads);
    mbar_init(&mi->drain, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&mi->tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // rows of K / V past the end of a tile are read (and masked) by the attention: never let them hold
  // uninitialised bit patterns
  // (the weight ring behind it as well: key blocks that run past row 127 read a little of it)
  for (uint32_t i = tid; i < ((uint32_t)kTM * 2 * C * 2 + kStages * (uint32_t)C * 128u) / 16; i += kThreads)
    reinterpret_cast<uint4*>(sm + g.off_kv)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async();  // the TMA writes that follow must not be overtaken by these generic stores
  // everything above touched only this CTA's own state; from here on the kernel reads what earlier kernels in the
  // stream wrote (tables, features, the launch counters): wait for them if this launch was allowed to start early
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  RoleCtx rc;
  rc.sbase = raw + pad;
  rc.tmem = mi->tmem_base;
  rc.mode = g.mode; rc.n_f1 = g.n_f1; rc.NF = g.NF; rc.nkb_h = g.nkb_h; rc.tau = g.tau; rc.n_layers = a.n_layers;
  rc.off_a = g.off_a; rc.off_kv = g.off_kv; rc.off_stage = g.off_stage;
  rc.pe = VAR == 2;

  if (warp == kTmaWarp) {
    if ((tid & 31) == 0) producer_role<C>(a, rc);
    __syncwarp();
  } else if (warp == kMmaWarp) {
    if ((tid & 31) == 0) mma_role<C>(rc);
    __syncwarp();
  } else if (warp == kStampWarp) {
    stamp_role(a.row_stamp);
  } else if (warp >= kLoadWarp0) {
    loader_role<C, RPB>(a);
  } else {
    compute_role<C, D, NT, VAR>(a);
  }
  // ---- teardown: everyone meets here, then the allocating warp returns the TMEM columns ----
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(rc.tmem), "r"(kTmemCols) : "memory");
  }
  // the last CTA to leave puts the launch's counters back to zero for the next launch on this context
  if (tid == 0) {
    const int left = atomicAdd(a.counter + 1, 1);
    if (left == (int)gridDim.x - 1) {
      a.counter[0] = 0;
      a.counter[1] = 0;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

// bf16 matrix [rows][cols] row-major; box = 64 columns x box_rows rows, 128-byte swizzle.
bool make_weight_map(CUtensorMap* m, const void* w, int rows, int cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(w), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Tensor maps are encoded once per (matrix, shape, box) and context and kept: a backbone calls the same layers
// frame after frame.
struct dsvt_map_cache {
  struct Entry {
    const void* w;
    int rows, cols, box_rows;
    CUtensorMap map;
  };
  std::vector<Entry> entries;
  unsigned attr_done = 0;  // kernel instantiations whose shared-memory attribute is set on this context's device
};

void dsvt_map_cache_destroy(dsvt_map_cache* c) { delete c; }

namespace {

bool cached_weight_map(dsvt_ctx* ctx, CUtensorMap* out, const void* w, int rows, int cols, int box_rows) {
  if (!ctx->maps) ctx->maps = new (std::nothrow) dsvt_map_cache();
  if (!ctx->maps) return false;
  auto& v = ctx->maps->entries;
  for (const auto& e : v)
    if (e.w == w && e.rows == rows && e.cols == cols && e.box_rows == box_rows) { *out = e.map; return true; }
  dsvt_map_cache::Entry e;
  e.w = w; e.rows = rows; e.cols = cols; e.box_rows = box_rows;
  if (!make_weight_map(&e.map, w, rows, cols, box_rows)) return false;
  if (v.size() >= 256) v.erase(v.begin(), v.begin() + 128);  // (a caller that keeps changing its weights)
  v.push_back(e);
  *out = e.map;
  return true;
}

template <int C, int D, int NT, int VAR>
int launch_tc_one(dsvt_ctx* ctx, const TcArgs& a, int grid, size_t smem, int inst) {
  if (!(ctx->maps->attr_done & (1u << inst))) {  // once per instantiation and context (the attribute is per device)
    cudaError_t e = cudaFuncSetAttribute(layer_tc_kernel<C, D, NT, VAR>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return DSVT_ERR_CUDA; }
    ctx->maps->attr_done |= 1u << inst;
  }
  // launched so that it may be set up under the tail of the kernel before it in the stream (the partition, an
  // earlier chain): the kernel waits for that kernel's completion before it reads anything but its parameters
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = ctx->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  cudaError_t le = cudaLaunchKernelEx(&cfg, layer_tc_kernel<C, D, NT, VAR>, a);
  if (le != cudaSuccess) { ctx->last_cuda_error = (int)le; cudaGetLastError(); return DSVT_ERR_CUDA; }
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}

// The position bias and the positional term are compile-time variants: a layer without them runs a kernel that
// holds none of their code.
template <int C, int D, int NT>
int launch_tc(dsvt_ctx* ctx, const TcArgs& a, int grid, size_t smem, int inst) {
  if (a.g.rb_len != 0) return launch_tc_one<C, D, NT, 1>(ctx, a, grid, smem, 2 * inst + 1);
  if (a.layer[0].pe) {
    // (the variant with a positional term is built for the paper's shape only: C = 192, set size up to 48)
    if constexpr (C == 192 && NT <= 14) return launch_tc_one<C, D, NT, 2>(ctx, a, grid, smem, 24 + inst);
    return DSVT_ERR_UNSUPPORTED;
  }
  return launch_tc_one<C, D, NT, 0>(ctx, a, grid, smem, 2 * inst);
}

template <int C, int D>
int launch_tc_nt(dsvt_ctx* ctx, const TcArgs& a, int grid, size_t smem, int inst) {
  // NT = key blocks of 8 a 16-row block can need: the rows of every set it touches, ceil((2 tau + 14) / 8), at most
  // the 16 blocks of a whole tile
  if (a.g.tau <= 36) return launch_tc<C, D, 11>(ctx, a, grid, smem, 3 * inst);
  if (a.g.tau <= 48) return launch_tc<C, D, 14>(ctx, a, grid, smem, 3 * inst + 1);
  return launch_tc<C, D, 16>(ctx, a, grid, smem, 3 * inst + 2);
}

int tc_hidden(const dsvt_fused_args& a) { return a.attention_only ? 0 : a.p.hidden; }

}  // namespace

// Shapes the tensor-core kernel covers; everything else goes to the FMA kernel.
bool dsvt_layer_tc_supported(const dsvt_fused_args& a) {
  const dsvt_layer_params& p = a.p;
  if (p.precision != DSVT_BF16_FP32ACC) return false;
  if (p.pe && (p.rpb || p.C != 192 || p.set_size > 48)) return false;  // (see launch_tc)
  if (p.rpb) {
    // row coordinates are kept as linear indices modulo 2^16 and differences are taken modulo 2^16: exact while every
    // offset inside a covered set, at most (len - 1) / 2 in magnitude, is below 2^15
    const int64_t len = (int64_t)(2 * p.rpb_extent[0] - 1) * (2 * p.rpb_extent[1] - 1) * (2 * p.rpb_extent[2] - 1);
    if (len > 65535) return false;
  }
  const int d = p.C / p.heads;
  const bool shape = (p.C == 192 && d == 24) || (p.C == 128 && (d == 16 || d == 32)) || (p.C == 64 && d == 16);
  if (!shape || p.set_size > 96) return false;
  const int hidden = tc_hidden(a);
  if (hidden != 0 && hidden != p.C && hidden != 2 * p.C) return false;
  return encode_fn() != nullptr;
}

// Two layers can share a launch if they have the same shape (one kernel instantiation, one geometry).
bool dsvt_layer_tc_chainable(const dsvt_fused_args& a, const dsvt_fused_args& b) {
  const dsvt_layer_params &p = a.p, &q = b.p;
  if (a.attention_only || b.attention_only || a.n != b.n || a.y != b.y) return false;
  if (p.C != q.C || p.heads != q.heads || tc_hidden(a) != tc_hidden(b) || p.set_size != q.set_size) return false;
  if ((p.rpb != nullptr) != (q.rpb != nullptr) || (p.pe != nullptr) != (q.pe != nullptr)) return false;
  if (p.rpb && (p.coords != q.coords || p.rpb_extent[0] != q.rpb_extent[0] || p.rpb_extent[1] != q.rpb_extent[1] ||
                p.rpb_extent[2] != q.rpb_extent[2]))
    return false;
  return true;
}

// One launch for layers[0 .. n_layers): layers[0] reads its x and writes y, every later layer runs in place on y
// (its x must be that y).  All layers pass dsvt_layer_tc_supported and are chainable with layers[0].
int dsvt_launch_layers_tc(dsvt_ctx* ctx, const dsvt_fused_args* layers, int n_layers) {
  if (n_layers < 1 || n_layers > kMaxLayers) return DSVT_ERR_INVALID_ARG;
  if (!ctx->maps) ctx->maps = new (std::nothrow) dsvt_map_cache();
  if (!ctx->maps) return DSVT_ERR_CUDA;
  const dsvt_fused_args& a0 = layers[0];
  const dsvt_layer_params& p = a0.p;
  const int C = p.C;
  TcArgs ta = {};
  TcGeom& g = ta.g;
  g.hidden = tc_hidden(a0);
  g.heads = p.heads;
  g.tau = p.set_size;
  g.mode = a0.attention_only ? 0 : (g.hidden > 0 ? 2 : 1);
  g.nkb_h = g.hidden / 64;
  g.NF = (g.hidden % 128 == 0 && C >= 128) ? 128 : 64;
  g.n_f1 = g.hidden / g.NF;
  g.rb_len = g.rb_sx = g.rb_sy = g.rb_centre = 0;
  g.rb_ext[0] = g.rb_ext[1] = g.rb_ext[2] = 0;
  if (p.rpb) {
    const int L = p.rpb_extent[0], W = p.rpb_extent[1], H = p.rpb_extent[2];
    g.rb_sy = 2 * H - 1;
    g.rb_sx = (2 * W - 1) * g.rb_sy;
    g.rb_len = (2 * L - 1) * g.rb_sx;
    g.rb_centre = (L - 1) * g.rb_sx + (W - 1) * g.rb_sy + (H - 1);
    g.rb_ext[0] = L; g.rb_ext[1] = W; g.rb_ext[2] = H;
  }
  const uint32_t a_bytes = kTM * C * 2;
  g.off_a = 0;
  g.off_kv = a_bytes;
  g.off_stage = g.off_kv + (uint32_t)kTM * 2 * C * 2;  // K + V (bf16) = fp32 staging = MLP hidden (<= 2C) bytes
  g.off_par = g.off_stage + kStages * (uint32_t)C * 128u;
  const size_t smem = (size_t)g.off_par + (size_t)(8 * C + g.hidden) * sizeof(float) + 1024;
  if (smem + sizeof(Misc) + 16 > 227 * 1024) return DSVT_ERR_UNSUPPORTED;  // s_mi is static shared memory
  int64_t grid = 1;
  for (int l = 0; l < n_layers; ++l) {
    const dsvt_fused_args& a = layers[l];
    const dsvt_layer_params& q = a.p;
    TcLayer& ly = ta.layer[l];
    bool okm = cached_weight_map(ctx, &ly.qkv, q.W_qkv, 3 * C, C, C) && cached_weight_map(ctx, &ly.o, q.W_o, C, C, C);
    if (g.hidden > 0)
      okm = okm && cached_weight_map(ctx, &ly.w1, q.W_1, g.hidden, C, g.NF) &&
            cached_weight_map(ctx, &ly.w2, q.W_2, C, g.hidden, C);
    else {
      ly.w1 = ly.o;
      ly.w2 = ly.o;
    }
    if (!okm) return DSVT_ERR_CUDA;
    ly.b_qkv = q.b_qkv; ly.b_o = q.b_o; ly.rpb = q.rpb; ly.pe = q.pe;
    const bool full = !a.attention_only;
    ly.b_1 = full ? q.b_1 : nullptr; ly.b_2 = full ? q.b_2 : nullptr;
    ly.ln1_g = full ? q.ln1_g : nullptr; ly.ln1_b = full ? q.ln1_b : nullptr;
    ly.ln2_g = full ? q.ln2_g : nullptr; ly.ln2_b = full ? q.ln2_b : nullptr;
    ly.table = a.table; ly.num_sets = a.num_sets; ly.rowoff = a.rowoff; ly.cap_sets = a.cap_sets;
    ly.eps = q.ln_eps;
    const int64_t cap = a.cap_sets < a.n ? a.cap_sets : a.n;
    if (cap > grid) grid = cap;
  }
  ta.x = a0.x; ta.y = a0.y; ta.n = a0.n; ta.n_layers = n_layers;
  ta.coords = reinterpret_cast<const int4*>(p.coords);
  ta.counter = ctx->tc_counter;
  ta.row_stamp = ctx->row_stamp;
  ctx->stamp_serial = (ctx->stamp_serial + 1) & 0x3ffffff;  // (stamps of launches 2^26 apart never meet)
  if (ctx->stamp_serial == 0) ctx->stamp_serial = 1;
  ta.stamp_base = (int32_t)(ctx->stamp_serial * 32u);
  ta.status = ctx->status;
  // one CTA per SM, but no more CTAs than there can be sets
  if (grid > ctx->sm_count) grid = ctx->sm_count;
  if (ctx->layer_ctas > 0 && grid > ctx->layer_ctas) grid = ctx->layer_ctas;
  if (grid < 1) grid = 1;
  const int d = C / p.heads;
  if (C == 192) return launch_tc_nt<192, 24>(ctx, ta, (int)grid, smem, 0);
  if (C == 128 && d == 16) return launch_tc_nt<128, 16>(ctx, ta, (int)grid, smem, 1);
  if (C == 128) return launch_tc_nt<128, 32>(ctx, ta, (int)grid, smem, 2);
  return launch_tc_nt<64, 16>(ctx, ta, (int)grid, smem, 3);
}

int dsvt_launch_layer_tc(dsvt_ctx* ctx, const dsvt_fused_args& a) { return dsvt_launch_layers_tc(ctx, &a, 1); }

// Tensor map of a row-major bf16 matrix [rows][cols] for boxes of 64 columns x box_rows rows with the 128-byte
// swizzle (the layout every operand tile here uses), from the context's cache; false if the driver entry point is
// missing or refuses.
bool dsvt_cached_weight_map(dsvt_ctx* ctx, void* tensor_map, const void* w, int rows, int cols, int box_rows) {
  return cached_weight_map(ctx, reinterpret_cast<CUtensorMap*>(tensor_map), w, rows, cols, box_rows);
}
