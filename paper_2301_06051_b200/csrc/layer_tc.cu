// Fused DSVT layer on the 5th-generation tensor cores (tcgen05 + TMEM), bfloat16 operands, fp32
// accumulation: gather (Eq. 4) -> QKV projection -> per-set multi-head attention (Eq. 5) -> output
// projection -> residual + LayerNorm -> MLP with GELU -> residual + LayerNorm -> scatter (App. B.1.1).
//
// One persistent CTA per SM.  Whole sets are packed greedily into tiles of at most 128 distinct rows (the
// UMMA M); the tile plan comes from the partition (tile t goes to CTA t mod gridDim.x), or, without a
// plan, each CTA cuts its own contiguous row segment into tiles.
//
// Roles (640 threads): warps 0-15 compute (gather, TMEM epilogues, attention); warp 16 is the scheduler
// and TMA producer: it publishes tiles through a two-entry ring, two ahead, and streams the layer's
// weight matrices through a three-stage shared-memory ring with plain (single-CTA) TMA loads; warp 17
// allocates TMEM and issues the tcgen05.mma instructions; warps 18-19 build the next tile's row list
// while the current tile is computed.  The compute warps gather the next tile's rows as soon as the
// current tile's MMAs have stopped reading the A operand, so that its first projections overlap the
// current tile's tail.
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
// Every wait on an mbarrier is bounded; a wait that gives up raises DSVT_STATUS_TIMEOUT and all roles
// leave their loops.
#include <cuda.h>
#include <limits.h>

#include <type_traits>

#include "dsvt_common.cuh"

namespace {

constexpr int kTM = 128;               // tile rows = UMMA M
constexpr int kComputeWarps = 16;
constexpr int kComputeThreads = 32 * kComputeWarps;
constexpr int kTmaWarp = kComputeWarps, kMmaWarp = kComputeWarps + 1;
constexpr int kLoadWarp0 = kComputeWarps + 2, kLoadWarps = 2;  // row-list + gather warps, one tile ahead
constexpr int kLoadThreads = 32 * kLoadWarps;
constexpr int kThreads = kComputeThreads + 64 + kLoadThreads;
constexpr int kStages = 3;             // weight ring depth
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxPolls = 1 << 20;

struct TcGeom {
  int hidden, heads, tau;
  int nkb_h;    // hidden / 64: K blocks of the MLP-2 contraction
  int NF;       // MLP-1 chunk width (128 or 64)
  int n_f1;     // hidden / NF
  int mode;     // 0: attention only, 1: attention + residual + LN1, 2: full layer
  uint32_t off_a, off_kv, off_stage, off_par;  // byte offsets from the 1024-aligned base
  // relative position bias (rb_len == 0: none): entries per head, strides of the x and y offsets in the table,
  // index of the zero offset
  int rb_len, rb_sx, rb_sy, rb_centre;
};

struct Misc {  // small shared state beside the big regions
  // weight ring; accumulator regions 0 / 1 / 2 (see the TMEM map at compute_role); operand hand-offs
  unsigned long long full[kStages], empty[kStages], acc_full[3], acc_free[3];
  unsigned long long a_ready;   // compute warps -> MMA: attention output / x1 / MLP hidden is in place
  unsigned long long x_ready;   // compute warps -> MMA: the gathered rows of a tile are in the A operand
  unsigned long long rl_ready[2];  // loader warps -> compute: row-list buffer b describes its next tile
  unsigned long long rl_free[2];   // compute -> loader warps: row-list buffer b is no longer read
  unsigned long long sched_full[2], sched_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  int tile[2][4];  // ring of tiles: first set, number of sets (< 0: no more tiles), first row, rows
  // launch constants, written once before the roles start: the phase functions read them from here
  // instead of taking them as arguments, so that nothing has to stay in registers across their calls
  const float* x;
  float* y;
  const int32_t* table;
  const int32_t* rowoff;
  int32_t* status;
  unsigned char* sm;   // 1024-aligned base of the dynamic shared memory (generic address)
  uint32_t sbase;      // the same as a shared-space address
  uint32_t off_a, off_kv, off_par;
  int n, tau, heads, mode, NF, n_f1, ln1, ln2;
  float eps;
  // the tile the compute warps are working on, and which row-list buffer describes it
  int s_lo, nsets, base, rows, buf;
  int pre0;  // the CTA's first tile was listed and gathered during the kernel's set-up
  int next_rows[2];  // rows of the tile listed in buffer b (< 0: there is no such tile), valid after rl_ready[b]
  // row lists, double buffered: the loader warps fill buffer (k + 1) & 1 while the compute warps work on tile k;
  // the compute warps gather tile k + 1 as soon as tile k's MMAs no longer read the A operand
  int rowvox[2][kTM];              // tile row -> voxel (-1: none)
  unsigned char set_lo[2][kTM + 1];  // first tile row of each set of the tile
  unsigned char row_lo[2][kTM], row_n[2][kTM];  // per tile row: first row and row count of its set
  // relative position bias.  The table index is linear in the coordinate offset, so one integer per row,
  // x * rb_sx + y * rb_sy + z, serves every (query, key) pair: index = lin[query] - lin[key] + rb_centre.  Offsets
  // inside a set are below 2^15 in magnitude, so the low 16 bits are kept and differences are taken modulo 2^16.
  // Written by the gather of a tile (after the previous tile's attention), read by the tile's attention.
  const float* rpb;
  const int4* coords;
  int rb_len, rb_sx, rb_sy, rb_centre, rb_ext[3];
  short rowlin[kTM];
};
__shared__ Misc s_mi;

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned long long* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the abort flag) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < kMaxPolls; ++i) {
    if (mbar_try(bar, parity)) return true;
    if ((i & 255) == 255 && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kComputeThreads) : "memory"); }
// Barrier `id` over `nthreads` threads that also ORs a predicate: every participant gets the same answer, so a
// loop exit taken on it is taken by all of them together.
__device__ __forceinline__ bool bar_or(int id, int nthreads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %3, 0;\n\t"
      "bar.red.or.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(id), "r"(nthreads), "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 16 fp32 columns of this thread's TMEM lane into / from elements [OFF, OFF + 16) of a register array
// (compile-time offsets keep the array in registers).
template <int OFF, int N>
__device__ __forceinline__ void tmem_ld16_at(uint32_t taddr, float (&r)[N]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=f"(r[OFF + 0]), "=f"(r[OFF + 1]), "=f"(r[OFF + 2]), "=f"(r[OFF + 3]), "=f"(r[OFF + 4]), "=f"(r[OFF + 5]),
        "=f"(r[OFF + 6]), "=f"(r[OFF + 7]), "=f"(r[OFF + 8]), "=f"(r[OFF + 9]), "=f"(r[OFF + 10]), "=f"(r[OFF + 11]),
        "=f"(r[OFF + 12]), "=f"(r[OFF + 13]), "=f"(r[OFF + 14]), "=f"(r[OFF + 15])
      : "r"(taddr));
}
template <int OFF, int N>
__device__ __forceinline__ void tmem_st16_at(uint32_t taddr, const float (&v)[N]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "f"(v[OFF + 0]), "f"(v[OFF + 1]), "f"(v[OFF + 2]), "f"(v[OFF + 3]), "f"(v[OFF + 4]), "f"(v[OFF + 5]),
        "f"(v[OFF + 6]), "f"(v[OFF + 7]), "f"(v[OFF + 8]), "f"(v[OFF + 9]), "f"(v[OFF + 10]), "f"(v[OFF + 11]),
        "f"(v[OFF + 12]), "f"(v[OFF + 13]), "f"(v[OFF + 14]), "f"(v[OFF + 15])
      : "memory");
}
template <int N>
__device__ __forceinline__ void tmem_ld_row(uint32_t taddr, float (&r)[N]) {
  static_assert(N == 16 || N == 32 || N == 48, "column count per thread");
  tmem_ld16_at<0>(taddr, r);
  if constexpr (N > 16) tmem_ld16_at<16>(taddr + 16, r);
  if constexpr (N > 32) tmem_ld16_at<32>(taddr + 32, r);
}
template <int N>
__device__ __forceinline__ void tmem_st_row(uint32_t taddr, const float (&v)[N]) {
  tmem_st16_at<0>(taddr, v);
  if constexpr (N > 16) tmem_st16_at<16>(taddr + 16, v);
  if constexpr (N > 32) tmem_st16_at<32>(taddr + 32, v);
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2_trans(uint32_t addr, uint32_t (&r)[2]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_1688(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5}, {%6}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(b0));
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Byte offset of the 16-byte chunk (row, c8) inside an operand region in the swizzled K-major layout.
__device__ __forceinline__ uint32_t swz(int row, int c8) {
  return (uint32_t)((c8 >> 3) * (kTM * 128) + (row >> 3) * 1024 + (row & 7) * 128 + (((c8 & 7) ^ (row & 7)) << 4));
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTM >> 4) << 24);
}

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

struct TcMaps {
  CUtensorMap qkv, o, w1, w2;
};

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
    // Reads may run up to two groups past row 127: they land in the neighbouring operand block or the weight
    // ring, which hold finite bf16 values, and meet zero probabilities.
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
  unsigned char* sm;  // 1024-aligned shared-memory base (generic address) and its shared-space address
  uint32_t sbase;
  uint32_t tmem;      // TMEM base address of the CTA's allocation
  // read by the scheduler thread while the other threads set up shared memory (see prefetch_first_tile)
  int S;              // number of sets
  int n_plan;         // tiles in the plan (< 0: no plan)
  int pre_ok;         // the CTA's first plan tile below is valid
  int pre_s, pre_ns, pre_base, pre_rows;
  // copies of the kernel parameters the two single-thread roles use (registers instead of parameter-space loads)
  const int32_t* rowoff;
  int cap_sets, mode, n_f1, NF, nkb_h;
  uint32_t off_a, off_kv, off_stage;
};

// The scheduler thread's first global reads (set count, plan header, the CTA's first tile and its row range)
// are issued at kernel entry, so that their two round trips overlap the shared-memory set-up.
__device__ __forceinline__ void prefetch_first_tile(const dsvt_fused_args& a, RoleCtx& rc) {
  const int32_t* plan = a.rowoff + a.cap_sets + 1;
  const int n_plan = plan[0];
  const int S = min(*a.num_sets, a.cap_sets);
  // in bounds for every block index: the grid has at most cap_sets CTAs and the plan cap_sets + 2 entries
  const int f = plan[1 + blockIdx.x], l = plan[2 + blockIdx.x];
  rc.n_plan = n_plan;
  rc.S = S;
  rc.pre_ok = 0;
  rc.pre_s = rc.pre_ns = rc.pre_base = rc.pre_rows = 0;
  if (n_plan >= 0 && (int)blockIdx.x < n_plan && f >= 0 && l > f && l <= S && l - f <= kTM) {
    const int base = a.rowoff[f], rows = a.rowoff[l] - base;
    if (rows > 0 && rows <= kTM) {
      rc.pre_ok = 1;
      rc.pre_s = f; rc.pre_ns = l - f; rc.pre_base = base; rc.pre_rows = rows;
    }
  }
}


// The scheduler and the MMA issuer are separate (not inlined) functions so that their polling loops get
// their own, spill-free register allocation; the compute role is inlined into the kernel, where the
// kernel parameters are constant-bank operands.

// ================= scheduler + TMA producer (one thread) ===============================================
template <int C>
__device__ __noinline__ void producer_role(const dsvt_fused_args& a, const TcGeom& g, const TcMaps& maps,
                                           int32_t* __restrict__ status, const RoleCtx rc) {
  constexpr int NKB = C / 64;        // K blocks of a C-deep contraction
  constexpr uint32_t COL_B = C;      // second accumulator buffer
  constexpr uint32_t STAGE_BYTES = C * 128;
  const uint32_t sbase = rc.sbase, tmem = rc.tmem;
  Misc* mi = &s_mi;
  const uint32_t a_base = sbase + rc.off_a, kv_base = sbase + rc.off_kv, st_base = sbase + rc.off_stage;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  volatile int* abort_flag = &mi->abort_flag;
  const int S = rc.S;
  const bool mlp = rc.mode == 2;
  const int n_chunks = 4 + (mlp ? rc.n_f1 + 1 : 0);
  (void)NKB; (void)COL_B; (void)STAGE_BYTES; (void)a_base; (void)kv_base; (void)st_base; (void)lane; (void)warp;
  (void)tmem; (void)S; (void)n_chunks; (void)tid;
    if (lane == 0) {
      // Tiles come from the plan behind the row offsets (greedy packing of the whole frame, tile t goes to
      // CTA t mod G); without a plan each CTA packs its own segment, the sets whose first row lies in
      // [b R / G, (b + 1) R / G).
      const int32_t* plan = rc.rowoff + rc.cap_sets + 1;
      const int n_plan = rc.n_plan;
      int t_next = blockIdx.x;
      int s = 0, s_end = 0;
      if (n_plan < 0) {
        const int R = S > 0 ? rc.rowoff[S] : 0;
        const int row_lo = (int)(((long long)blockIdx.x * R) / gridDim.x);
        const int row_hi = (int)(((long long)(blockIdx.x + 1) * R) / gridDim.x);
        int lo = 0, hi = S;
        while (lo < hi) { const int m = (lo + hi) >> 1; if (rc.rowoff[m] < row_lo) lo = m + 1; else hi = m; }
        s = lo;
        hi = S;
        while (lo < hi) { const int m = (lo + hi) >> 1; if (rc.rowoff[m] < row_hi) lo = m + 1; else hi = m; }
        s_end = lo;
      }
      // next tile: first set s0, ns sets (< 0: none left), first row, rows
      auto next_tile = [&](int& s0, int& ns, int& base, int& rows) {
        ns = -1; base = 0; rows = 0;
        if (n_plan >= 0) {
          while (t_next < n_plan) {
            const int f = plan[1 + t_next], l = plan[2 + t_next];
            t_next += gridDim.x;
            if (f < 0 || l <= f || l > S) { atomicOr(status, DSVT_STATUS_BAD_INDEX); continue; }
            base = rc.rowoff[f];
            rows = rc.rowoff[l] - base;
            if (rows <= 0 || rows > kTM || l - f > kTM) { atomicOr(status, DSVT_STATUS_BAD_INDEX); continue; }
            s0 = f;
            ns = l - f;
            return;
          }
          return;
        }
        while (s0 < s_end) {
          base = rc.rowoff[s0];
          const int first = rc.rowoff[s0 + 1] - base;
          if (first <= 0 || first > kTM) {  // offsets that do not describe a set: skip it
            atomicOr(status, DSVT_STATUS_BAD_INDEX);
            ++s0;
            continue;
          }
          int l2 = s0 + 1, h2 = s_end;  // last e in (s0, s_end] with rowoff[e] - base <= 128
          while (l2 < h2) { const int m = (l2 + h2 + 1) >> 1; if (rc.rowoff[m] - base <= kTM) l2 = m; else h2 = m - 1; }
          ns = l2 - s0;
          rows = rc.rowoff[l2] - base;
          return;
        }
      };
      int stage = 0, slot = 0;
      uint32_t phase = 0, sphase = 0;
      int ns, base, rows;
      if (rc.pre_ok) {  // the first tile was looked up at kernel entry
        s = rc.pre_s; ns = rc.pre_ns; base = rc.pre_base; rows = rc.pre_rows;
        t_next += gridDim.x;
      } else {
        next_tile(s, ns, base, rows);
      }
      // Tiles are published two ahead of the weights (the ring has two entries), so that the loader
      // warps can prepare tile k + 1 while tile k is being computed.
      int ahead = 0;          // published tiles whose weights have not been streamed yet
      bool all_out = false;   // the end marker has been published
      auto publish = [&]() -> bool {
        if (!mbar_wait(&mi->sched_empty[slot], sphase ^ 1u, abort_flag)) return false;
        mi->tile[slot][0] = s; mi->tile[slot][1] = ns; mi->tile[slot][2] = base; mi->tile[slot][3] = rows;
        mbar_arrive(&mi->sched_full[slot]);
        if (++slot == 2) { slot = 0; sphase ^= 1u; }
        if (ns < 0) { all_out = true; return true; }
        ++ahead;
        s += ns;
        next_tile(s, ns, base, rows);
        return true;
      };
      if (!publish()) goto producer_done;
      if (!all_out && !publish()) goto producer_done;
      while (ahead > 0) {
        // the layer's weights for one tile, chunk by chunk, K block by K block
        for (int c = 0; c < n_chunks; ++c) {
          const CUtensorMap* map;
          int row0, nkb;
          uint32_t bytes = STAGE_BYTES;
          if (c < 3) { map = &maps.qkv; row0 = (c == 0 ? 1 : c == 1 ? 2 : 0) * C; nkb = NKB; }   // K, V, Q
          else if (c == 3) { map = &maps.o; row0 = 0; nkb = NKB; }
          else if (c < 4 + rc.n_f1) { map = &maps.w1; row0 = (c - 4) * rc.NF; nkb = NKB; bytes = (uint32_t)rc.NF * 128u; }
          else { map = &maps.w2; row0 = 0; nkb = rc.nkb_h; }
          for (int kb = 0; kb < nkb; ++kb) {
            if (!mbar_wait(&mi->empty[stage], phase ^ 1u, abort_flag)) goto producer_done;
            mbar_expect_tx(&mi->full[stage], bytes);
            tma_load_2d(st_base + stage * STAGE_BYTES, map, kb * 64, row0, &mi->full[stage]);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
        --ahead;
        if (!all_out && !publish()) goto producer_done;
      }
    producer_done:;
    }
}

// ================= MMA issuer (one thread) =============================================================
template <int C>
__device__ __noinline__ void mma_role(const dsvt_fused_args& a, const TcGeom& g, const RoleCtx rc) {
  constexpr int NKB = C / 64;        // K blocks of a C-deep contraction
  constexpr uint32_t COL_B = C;      // second accumulator buffer
  constexpr uint32_t STAGE_BYTES = C * 128;
  const uint32_t sbase = rc.sbase, tmem = rc.tmem;
  Misc* mi = &s_mi;
  const uint32_t a_base = sbase + rc.off_a, kv_base = sbase + rc.off_kv, st_base = sbase + rc.off_stage;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  volatile int* abort_flag = &mi->abort_flag;
  const bool mlp = rc.mode == 2;
  const int n_chunks = 4 + (mlp ? rc.n_f1 + 1 : 0);
  (void)NKB; (void)COL_B; (void)STAGE_BYTES; (void)a_base; (void)kv_base; (void)st_base; (void)lane; (void)warp;
  (void)tmem; (void)n_chunks; (void)tid;
    if (lane == 0) {
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
          if (c == 0) {
            if (!mbar_wait(&mi->x_ready, x_phase, abort_flag)) goto mma_done;
            x_phase ^= 1u;
          } else if (c == 3 || c == 4 || c == 4 + rc.n_f1) {
            if (!mbar_wait(&mi->a_ready, a_phase, abort_flag)) goto mma_done;
            a_phase ^= 1u;
          }
          // accumulator placement: K -> region 0, V -> 1, Q -> 0, O -> 0, MLP-1 piece i -> i & 1, MLP-2 -> 2
          // (on top of the parked x1 + b_2)
          uint32_t bar, col, n;
          if (c < 4) { bar = (c == 1) ? 1u : 0u; col = (c == 1) ? COL_B : 0u; n = C; }
          else if (c < 4 + rc.n_f1) { bar = (uint32_t)(c - 4) & 1u; col = bar * COL_B; n = (uint32_t)rc.NF; }
          else { bar = 2u; col = kTmemCols - C; n = C; }
          if (c == 1) {
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
    mma_done:;
    }
}

// ================= loader warps: row list + gather, one tile ahead of the compute warps ==================
__device__ __forceinline__ void loader_sync() { asm volatile("bar.sync 6, %0;" ::"n"(kLoadThreads) : "memory"); }

// Distinct slots of each set -> tile rows (Eq. 4), per-row set ranges, per-set first rows: one thread per
// set (a tile of a sparse region holds dozens of tiny sets), walking the set's table row.
template <bool RPB>
__device__ __forceinline__ void loader_row_list(int b, int lt, int s_lo, int nsets, int base) {
  const int32_t* __restrict__ table = s_mi.table;
  const int32_t* __restrict__ rowoff = s_mi.rowoff;
  const int n = s_mi.n, tau = s_mi.tau;
  for (int si = lt; si < nsets; si += kLoadThreads) {
    const int s = s_lo + si;
    const int32_t* trow = table + (size_t)s * tau;
    const int lb = __ldg(rowoff + s) - base, cap = __ldg(rowoff + s + 1) - __ldg(rowoff + s);
    const bool inside = lb >= 0 && lb < kTM;
    const int cnt_max = inside ? min(cap, kTM - lb) : 0;  // tile rows this set may fill
    int pos = 0, prev = 0;
    bool bad = false;
    constexpr bool rpb = RPB;
    int lo3[3] = {INT_MAX, INT_MAX, INT_MAX}, hi3[3] = {INT_MIN, INT_MIN, INT_MIN};
    for (int k0 = 0; k0 < tau; k0 += 8) {
      int v4[8];  // eight independent loads per round trip to L2 (the loader warps run a whole tile ahead)
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
    s_mi.set_lo[b][si] = (unsigned char)min(max(lb, 0), kTM);
    if (rpb)
      for (int q = 0; q < 3; ++q) bad |= hi3[q] >= lo3[q] && hi3[q] - lo3[q] > s_mi.rb_ext[q] - 1;
    if (bad || pos != cap) atomicOr(s_mi.status, DSVT_STATUS_BAD_INDEX);
  }
}

template <int C, bool RPB>
__device__ __noinline__ void loader_role() {
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
    __syncwarp();
    if (lane == 0) mbar_arrive(&s_mi.sched_empty[slot]);
    if (++slot == 2) { slot = 0; sphase ^= 1u; }
    const int b = k & 1;
    if (k == 0) {  // the compute warps list a CTA's first tile themselves (nothing can run ahead of it)
      mbar_arrive(&s_mi.rl_ready[b]);
      if (nsets < 0) break;
      continue;
    }
    // buffer b was last used by tile k - 2: the compute warps release it when they are done with that tile
    if (k >= 2) ok = mbar_wait(&s_mi.rl_free[b], (uint32_t)((k >> 1) - 1) & 1u, abort_flag) && ok;
    if (nsets >= 0) {
      for (int i = lt; i < kTM; i += kLoadThreads) {
        s_mi.rowvox[b][i] = -1;
        s_mi.row_lo[b][i] = (unsigned char)i;
        s_mi.row_n[b][i] = 1;
      }
      loader_sync();
      loader_row_list<RPB>(b, lt, s_lo, nsets, base);
      if (lt == 0) s_mi.set_lo[b][nsets] = (unsigned char)rows;
    }
    if (lt == 0) s_mi.next_rows[b] = nsets < 0 ? -1 : rows;
    mbar_arrive(&s_mi.rl_ready[b]);
    if (nsets < 0) break;
  }
}

// ================= compute warps ========================================================================
// Each phase of a tile is a separate (not inlined) function that takes at most a few scalars and reads the
// rest from s_mi, so that each gets a register allocation of its own and the tile loop keeps almost nothing
// alive across the calls.

// Row list of a CTA's first tile by the compute warps (one warp per set), into buffer 0.
template <bool RPB>
__device__ __noinline__ void phase_row_list() {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int32_t* __restrict__ table = s_mi.table;
  const int32_t* __restrict__ rowoff = s_mi.rowoff;
  const int n = s_mi.n, tau = s_mi.tau, s_lo = s_mi.s_lo, nsets = s_mi.nsets, base = s_mi.base;
  // (runs once per CTA: loops kept rolled, the kernel's text is better spent elsewhere)
#pragma unroll 1
  for (int si = warp; si < nsets; si += kComputeWarps) {
    const int s = s_lo + si;
    const int32_t* trow = table + (size_t)s * tau;
    const int lb = rowoff[s] - base, cap = rowoff[s + 1] - rowoff[s];
    const int cnt_max = (lb >= 0 && lb < kTM) ? min(cap, kTM - lb) : 0;
    int cnt = 0;
    int lo3[3] = {INT_MAX, INT_MAX, INT_MAX}, hi3[3] = {INT_MIN, INT_MIN, INT_MIN};
#pragma unroll 1
    for (int k0 = 0; k0 < tau; k0 += 32) {
      const int k = k0 + lane;
      int v = -1;
      bool uniq = false;
      if (k < tau) { v = trow[k]; uniq = (k == 0) || (v != trow[k - 1]); }
      if (RPB && v >= 0 && v < n) {
        const int4 c = __ldg(s_mi.coords + v);
        lo3[0] = min(lo3[0], c.y); hi3[0] = max(hi3[0], c.y);
        lo3[1] = min(lo3[1], c.z); hi3[1] = max(hi3[1], c.z);
        lo3[2] = min(lo3[2], c.w); hi3[2] = max(hi3[2], c.w);
      }
      const unsigned bal = __ballot_sync(0xffffffffu, uniq);
      const int pos = cnt + __popc(bal & ((1u << lane) - 1u));
      if (uniq && pos < cnt_max) {
        if (v < 0 || v >= n) { atomicOr(s_mi.status, DSVT_STATUS_BAD_INDEX); v = -1; }
        s_mi.rowvox[0][lb + pos] = v;
      }
      cnt += __popc(bal);
    }
#pragma unroll 1
    for (int i = lane; i < cnt_max; i += 32) {
      s_mi.row_lo[0][lb + i] = (unsigned char)lb;
      s_mi.row_n[0][lb + i] = (unsigned char)cnt_max;
    }
    bool wide = false;
    if (RPB) {  // a set spread wider than the bias table's extent is reported
#pragma unroll
      for (int q = 0; q < 3; ++q) {
        const int l = __reduce_min_sync(0xffffffffu, lo3[q]), hmax = __reduce_max_sync(0xffffffffu, hi3[q]);
        wide |= hmax >= l && hmax - l > s_mi.rb_ext[q] - 1;
      }
    }
    if (lane == 0) {
      s_mi.set_lo[0][si] = (unsigned char)min(max(lb, 0), kTM);
      if (cnt != cap || wide) atomicOr(s_mi.status, DSVT_STATUS_BAD_INDEX);
    }
  }
  if (tid == 0) s_mi.set_lo[0][nsets] = (unsigned char)s_mi.rows;
}

// Gather (Eq. 4): the fp32 rows listed in buffer b -> bf16 A operand, four rows in flight per warp; all 128 rows
// are written (rows past the tile as zeros).
template <int C, bool RPB>
__device__ __noinline__ void phase_gather(int b, int rows) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* __restrict__ x = s_mi.x;
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
        f[u][0] = __ldg(src);
        f[u][1] = __ldg(src + 1);
      }
      if (RPB && lane == 31) {  // (lane 31 carries no feature columns: C / 8 <= 24)
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

// TMEM map (512 columns): region 0 = [0, C): K, Q, O and the even MLP-1 pieces; region 1 = [C, 2C): V and
// the odd MLP-1 pieces; region 2 = [512 - C, 512): x1 + b_2 parked by the output-projection epilogue, then
// the MLP-2 accumulator.  Each region has its own full / free barrier pair.  For C = 192 regions 1 and 2
// overlap, which is why the MMA issuer waits for region 2 before it starts the next tile's V.
template <int C, int D, int NT, bool RPB>
__device__ __forceinline__ void compute_role() {
  constexpr int NKB = C / 64;        // K blocks of a C-deep contraction
  constexpr int QC = C / 4;          // epilogue columns per thread for a C-wide chunk (four threads per row)
  constexpr uint32_t COL_B = C;      // accumulator region 1
  volatile int* abort_flag = &s_mi.abort_flag;
  uint32_t uses[3] = {0u, 0u, 0u};
  int slot = 0;
  uint32_t sphase = 0;
  bool ok = true;
  auto acc_wait = [&](uint32_t bar) {
    ok = mbar_wait(&s_mi.acc_full[bar], uses[bar] & 1u, abort_flag) && ok;
    ++uses[bar];
    tc_fence_after();
  };
  // The next tile's rows are gathered as soon as the current tile's MMAs have stopped reading the A operand
  // (the caller has just waited for the accumulator of the last such chunk), so that its first projections
  // run on the tensor pipe while the compute warps finish the current tile.
  auto gather_next = [&](int k) {
    const int b = (k + 1) & 1;
    ok = mbar_wait(&s_mi.rl_ready[b], (uint32_t)((k + 1) >> 1) & 1u, abort_flag) && ok;
    const int nr = s_mi.next_rows[b];
    if (ok && nr >= 0) {
      phase_gather<C, RPB>(b, nr);
      fence_proxy_async();
      mbar_arrive(&s_mi.x_ready);
    }
  };
  for (int k = 0;; ++k) {
    ok = mbar_wait(&s_mi.sched_full[slot], sphase, abort_flag) && ok;
    // also orders the previous tile's last shared-memory reads before this tile's writes; every exit from
    // this loop is taken by all compute threads together
    if (bar_or(1, kComputeThreads, !ok || *abort_flag != 0)) break;
    const int nsets = s_mi.tile[slot][1], rows = s_mi.tile[slot][3];
    if (threadIdx.x == 0) {
      s_mi.s_lo = s_mi.tile[slot][0];
      s_mi.nsets = nsets;
      s_mi.base = s_mi.tile[slot][2];
      s_mi.rows = rows;
      s_mi.buf = k & 1;
      if (k >= 1) mbar_arrive(&s_mi.rl_free[(k - 1) & 1]);  // the previous tile's row list is dead
    }
    mbar_arrive(&s_mi.sched_empty[slot]);
    if (++slot == 2) { slot = 0; sphase ^= 1u; }
    if (nsets < 0) break;
    const bool listed = k != 0 || s_mi.pre0 != 0;  // (pre0 is not written after the kernel's set-up)
    if (!listed && threadIdx.x < kTM) {
      s_mi.rowvox[0][threadIdx.x] = -1;
      s_mi.row_lo[0][threadIdx.x] = (unsigned char)threadIdx.x;
      s_mi.row_n[0][threadIdx.x] = 1;
    }
    compute_sync();  // the tile's fields are visible to the phase functions
    if (k == 0) {  // nothing runs ahead of a CTA's first tile: the compute warps list and gather it themselves,
                   // as a rule already during the kernel's set-up
      if (!listed) {
        phase_row_list<RPB>();
        compute_sync();
        phase_gather<C, RPB>(0, rows);
        fence_proxy_async();
      }
      mbar_arrive(&s_mi.x_ready);  // X is in place
    }

    // ---- chunks 0..2: K, V, Q epilogues: (+ bias,) to bf16, into the operand layout ----
    // (the attention pads its key blocks up to 15 rows past the tile: those K / V rows must be real bf16)
    acc_wait(0u);
    phase_epi_bf16<QC, false, false>(0u, 0, 0, s_mi.off_kv, 0, rows + 16);
    acc_wait(1u);
    phase_epi_bf16<QC, false, true>(COL_B, 1, ParOff<C>::b_v, s_mi.off_kv + NKB * kTM * 128, 0, rows + 16);
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
    if (mode != 2) {  // final result of this call
      gather_next(k);  // the output projection was the last chunk to read the A operand
      compute_sync();
      phase_store_rows<C>();
      continue;
    }
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
    compute_sync();
    phase_store_rows<C>();
  }
  if (!ok || *abort_flag) {
    if (threadIdx.x == 0) atomicOr(s_mi.status, DSVT_STATUS_TIMEOUT);
  }
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int C, int D, int NT, bool RPB>
__global__ void __launch_bounds__(kThreads, 1)
layer_tc_kernel(const __grid_constant__ dsvt_fused_args a, const __grid_constant__ TcGeom g,
                const __grid_constant__ TcMaps maps, int32_t* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* sm = smem_raw + pad;
  Misc* mi = &s_mi;
  const int tid = threadIdx.x, warp = tid >> 5;
  RoleCtx rc;
  rc.S = rc.n_plan = rc.pre_ok = rc.pre_s = rc.pre_ns = rc.pre_base = rc.pre_rows = 0;
  if (tid == 32 * kTmaWarp) prefetch_first_tile(a, rc);
  // (the scheduler warp takes no part in the set-up loops: its first thread is busy with the plan look-ups)
  const bool setup = warp != kTmaWarp;
  const int stid = warp > kTmaWarp ? tid - 32 : tid;  // dense index of the threads that take part
  constexpr int kSetupThreads = kThreads - 32;
  // biases and LayerNorm vectors (absent vectors read as zeros): the loads are issued first, the values go to
  // shared memory at the end of the set-up.  Order of ParOff: b_q, b_v, b_o, b_2, ln1_g, ln1_b, ln2_g, ln2_b,
  // then b_1 (the key bias is not needed).
  constexpr int kParSlots = (ParOff<C>::vectors * C + 2 * C + kSetupThreads - 1) / kSetupThreads;
  const int n_par = ParOff<C>::vectors * C + g.hidden;
  float pv[kParSlots];
#pragma unroll
  for (int j = 0; j < kParSlots; ++j) {
    const int i = stid + j * kSetupThreads;
    pv[j] = 0.f;
    if (setup && i < n_par) {
      const dsvt_layer_params& p = a.p;
      const int which = i / C;
      const float* v = which == 0 ? p.b_qkv : which == 1 ? (p.b_qkv ? p.b_qkv + 2 * C : nullptr) : which == 2 ? p.b_o
                     : which == 3 ? p.b_2 : which == 4 ? p.ln1_g : which == 5 ? p.ln1_b : which == 6 ? p.ln2_g
                     : which == 7 ? p.ln2_b : (p.b_1 ? p.b_1 - ParOff<C>::b_1 + which * C : nullptr);
      if (v) pv[j] = __ldg(v + i % C);
    }
  }
  if (tid == 0) {  // launch constants for the phase functions
    mi->abort_flag = 0;
    mi->x = a.x; mi->y = a.y; mi->table = a.table; mi->rowoff = a.rowoff; mi->status = status;
    mi->sm = sm; mi->sbase = raw + pad;
    mi->off_a = g.off_a; mi->off_kv = g.off_kv; mi->off_par = g.off_par;
    mi->n = a.n; mi->tau = g.tau; mi->heads = g.heads; mi->mode = g.mode; mi->NF = g.NF; mi->n_f1 = g.n_f1;
    mi->ln1 = a.p.ln1_g != nullptr; mi->ln2 = a.p.ln2_g != nullptr;
    mi->eps = a.p.ln_eps;
    mi->rpb = a.p.rpb; mi->coords = reinterpret_cast<const int4*>(a.p.coords);
    mi->rb_len = g.rb_len; mi->rb_sx = g.rb_sx; mi->rb_sy = g.rb_sy; mi->rb_centre = g.rb_centre;
    mi->rb_ext[0] = a.p.rpb_extent[0]; mi->rb_ext[1] = a.p.rpb_extent[1]; mi->rb_ext[2] = a.p.rpb_extent[2];
    mi->s_lo = mi->nsets = mi->base = mi->rows = mi->buf = mi->pre0 = 0;
    mi->next_rows[0] = mi->next_rows[1] = -1;
  }
  if (tid == 32 * kLoadWarp0) {  // barriers
    for (int i = 0; i < kStages; ++i) { mbar_init(&mi->full[i], 1); mbar_init(&mi->empty[i], 1); }
    for (int i = 0; i < 3; ++i) {
      mbar_init(&mi->acc_full[i], 1);
      mbar_init(&mi->acc_free[i], kComputeThreads);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&mi->sched_full[i], 1);
      mbar_init(&mi->sched_empty[i], kComputeThreads + 1 + kLoadWarps);  // compute threads, MMA issuer, loader warps
      mbar_init(&mi->rl_free[i], 1);
      mbar_init(&mi->rl_ready[i], kLoadThreads);
    }
    mbar_init(&mi->a_ready, kComputeThreads);
    mbar_init(&mi->x_ready, kComputeThreads);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&mi->tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // The compute warps look up the CTA's first tile themselves (the same plan entries the scheduler reads) and
  // list and gather it right here, under the rest of the set-up; the A operand is not touched by the loops below.
  if (warp < kComputeWarps) {
    const int32_t* plan = a.rowoff + a.cap_sets + 1;
    const int n_plan = plan[0];
    const int S = min(*a.num_sets, a.cap_sets);
    const int f = plan[1 + blockIdx.x], l = plan[2 + blockIdx.x];  // in bounds: see prefetch_first_tile
    bool pre = n_plan >= 0 && (int)blockIdx.x < n_plan && f >= 0 && l > f && l <= S && l - f <= kTM;
    int base = 0, rows = 0;
    if (pre) {
      base = a.rowoff[f];
      rows = a.rowoff[l] - base;
      pre = rows > 0 && rows <= kTM;
    }
    compute_sync();  // thread 0's constants are in place
    if (pre) {
      if (tid == 0) { mi->s_lo = f; mi->nsets = l - f; mi->base = base; mi->rows = rows; mi->buf = 0; mi->pre0 = 1; }
      if (tid < kTM) {
        mi->rowvox[0][tid] = -1;
        mi->row_lo[0][tid] = (unsigned char)tid;
        mi->row_n[0][tid] = 1;
      }
      compute_sync();
      phase_row_list<RPB>();
      compute_sync();
      phase_gather<C, RPB>(0, rows);
      fence_proxy_async();
    }
  }
  // rows of K / V past the end of a tile are read (and masked) by the attention: never let them hold
  // uninitialised bit patterns
  // (the weight ring behind it as well: key blocks that run past row 127 read a little of it)
  if (setup)
    for (uint32_t i = stid; i < ((uint32_t)kTM * 2 * C * 2 + kStages * (uint32_t)C * 128u) / 16; i += kSetupThreads)
      reinterpret_cast<uint4*>(sm + g.off_kv)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async();  // the TMA writes that follow must not be overtaken by these generic stores
  {
    float* par = reinterpret_cast<float*>(sm + g.off_par);
#pragma unroll
    for (int j = 0; j < kParSlots; ++j) {
      const int i = stid + j * kSetupThreads;
      if (setup && i < n_par) par[i] = pv[j];
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  rc.sm = sm;
  rc.sbase = raw + pad;
  rc.tmem = mi->tmem_base;
  rc.rowoff = a.rowoff; rc.cap_sets = a.cap_sets;
  rc.mode = g.mode; rc.n_f1 = g.n_f1; rc.NF = g.NF; rc.nkb_h = g.nkb_h;
  rc.off_a = g.off_a; rc.off_kv = g.off_kv; rc.off_stage = g.off_stage;

  if (warp == kTmaWarp) {
    if ((tid & 31) == 0) producer_role<C>(a, g, maps, status, rc);
    __syncwarp();
  } else if (warp == kMmaWarp) {
    if ((tid & 31) == 0) mma_role<C>(a, g, rc);
    __syncwarp();
  } else if (warp >= kLoadWarp0) {
    loader_role<C, RPB>();
  } else {
    compute_role<C, D, NT, RPB>();
  }
  // ---- teardown: everyone meets here, then the allocating warp returns the TMEM columns ----
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(rc.tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
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

template <int C, int D, int NT, bool RPB>
int launch_tc_one(dsvt_ctx* ctx, const dsvt_fused_args& a, const TcGeom& g, const TcMaps& maps, int grid, size_t smem) {
  cudaError_t e = cudaFuncSetAttribute(layer_tc_kernel<C, D, NT, RPB>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return DSVT_ERR_CUDA; }
  layer_tc_kernel<C, D, NT, RPB><<<grid, kThreads, smem, ctx->stream>>>(a, g, maps, ctx->status);
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}

// The position bias is a compile-time variant: a layer without one runs a kernel that holds none of its code.
template <int C, int D, int NT>
int launch_tc(dsvt_ctx* ctx, const dsvt_fused_args& a, const TcGeom& g, const TcMaps& maps, int grid, size_t smem) {
  if (g.rb_len != 0) return launch_tc_one<C, D, NT, true>(ctx, a, g, maps, grid, smem);
  return launch_tc_one<C, D, NT, false>(ctx, a, g, maps, grid, smem);
}

template <int C, int D>
int launch_tc_nt(dsvt_ctx* ctx, const dsvt_fused_args& a, const TcGeom& g, const TcMaps& maps, int grid, size_t smem) {
  // NT = key blocks of 8 a 16-row block can need: the rows of every set it touches, ceil((2 tau + 14) / 8), at most
  // the 16 blocks of a whole tile
  if (g.tau <= 36) return launch_tc<C, D, 11>(ctx, a, g, maps, grid, smem);
  if (g.tau <= 48) return launch_tc<C, D, 14>(ctx, a, g, maps, grid, smem);
  return launch_tc<C, D, 16>(ctx, a, g, maps, grid, smem);
}

}  // namespace

// Tensor map of a row-major bf16 matrix [rows][cols] for boxes of 64 columns x box_rows rows with the 128-byte
// swizzle (the layout every operand tile here uses); false if the driver entry point is missing or refuses.
bool dsvt_make_weight_map(void* tensor_map, const void* w, int rows, int cols, int box_rows) {
  return make_weight_map(reinterpret_cast<CUtensorMap*>(tensor_map), w, rows, cols, box_rows);
}

// Shapes the tensor-core kernel covers; everything else goes to the FMA kernel.
bool dsvt_layer_tc_supported(const dsvt_fused_args& a) {
  const dsvt_layer_params& p = a.p;
  if (p.precision != DSVT_BF16_FP32ACC || p.pe) return false;
  if (p.rpb) {  // row coordinates are kept as 16-bit linear indices: every table offset must be below 2^15
    const int64_t len = (int64_t)(2 * p.rpb_extent[0] - 1) * (2 * p.rpb_extent[1] - 1) * (2 * p.rpb_extent[2] - 1);
    if (len > 32767) return false;
  }
  const int d = p.C / p.heads;
  const bool shape = (p.C == 192 && d == 24) || (p.C == 128 && (d == 16 || d == 32)) || (p.C == 64 && d == 16);
  if (!shape || p.set_size > 96) return false;
  const int hidden = a.attention_only ? 0 : p.hidden;
  if (hidden != 0 && hidden != p.C && hidden != 2 * p.C) return false;
  return encode_fn() != nullptr;
}

int dsvt_launch_layer_tc(dsvt_ctx* ctx, const dsvt_fused_args& a) {
  const dsvt_layer_params& p = a.p;
  const int C = p.C;
  TcGeom g;
  g.hidden = a.attention_only ? 0 : p.hidden;
  g.heads = p.heads;
  g.tau = p.set_size;
  g.mode = a.attention_only ? 0 : (g.hidden > 0 ? 2 : 1);
  g.nkb_h = g.hidden / 64;
  g.NF = (g.hidden % 128 == 0 && C >= 128) ? 128 : 64;
  g.n_f1 = g.hidden / g.NF;
  g.rb_len = g.rb_sx = g.rb_sy = g.rb_centre = 0;
  if (p.rpb) {
    const int L = p.rpb_extent[0], W = p.rpb_extent[1], H = p.rpb_extent[2];
    g.rb_sy = 2 * H - 1;
    g.rb_sx = (2 * W - 1) * g.rb_sy;
    g.rb_len = (2 * L - 1) * g.rb_sx;
    g.rb_centre = (L - 1) * g.rb_sx + (W - 1) * g.rb_sy + (H - 1);
  }
  const uint32_t a_bytes = kTM * C * 2;
  g.off_a = 0;
  g.off_kv = a_bytes;
  g.off_stage = g.off_kv + (uint32_t)kTM * 2 * C * 2;  // K + V (bf16) = fp32 staging = MLP hidden (<= 2C) bytes
  g.off_par = g.off_stage + kStages * (uint32_t)C * 128u;
  const size_t smem = (size_t)g.off_par + (size_t)(8 * C + g.hidden) * sizeof(float) + 1024;
  if (smem + sizeof(Misc) + 16 > 227 * 1024) return DSVT_ERR_UNSUPPORTED;  // s_mi is static shared memory
  TcMaps maps;
  bool okm = make_weight_map(&maps.qkv, p.W_qkv, 3 * C, C, C) && make_weight_map(&maps.o, p.W_o, C, C, C);
  if (g.hidden > 0)
    okm = okm && make_weight_map(&maps.w1, p.W_1, g.hidden, C, g.NF) && make_weight_map(&maps.w2, p.W_2, C, g.hidden, C);
  else {
    maps.w1 = maps.o;
    maps.w2 = maps.o;
  }
  if (!okm) return DSVT_ERR_CUDA;
  // one CTA per SM, but no more CTAs than there can be sets
  int64_t grid = a.cap_sets < a.n ? a.cap_sets : a.n;
  if (grid > ctx->sm_count) grid = ctx->sm_count;
  if (ctx->layer_ctas > 0 && grid > ctx->layer_ctas) grid = ctx->layer_ctas;
  if (grid < 1) grid = 1;
  const int d = C / p.heads;
  if (C == 192) return launch_tc_nt<192, 24>(ctx, a, g, maps, (int)grid, smem);
  if (C == 128 && d == 16) return launch_tc_nt<128, 16>(ctx, a, g, maps, (int)grid, smem);
  if (C == 128) return launch_tc_nt<128, 32>(ctx, a, g, maps, (int)grid, smem);
  return launch_tc_nt<64, 16>(ctx, a, g, maps, (int)grid, smem);
}
