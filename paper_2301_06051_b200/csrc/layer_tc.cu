// Fused DSVT layer on the 5th-generation tensor cores (tcgen05 + TMEM), bfloat16 operands, fp32
// accumulation: gather (Eq. 4) -> QKV projection -> per-set multi-head attention (Eq. 5) -> output
// projection -> residual + LayerNorm -> MLP with GELU -> residual + LayerNorm -> scatter (App. B.1.1).
//
// One persistent CTA per SM walks over tiles of up to 128 distinct voxel rows made of whole sets.
// Roles: warps 0-7 compute (gather, TMEM epilogues, attention), warp 8 streams the weight matrices
// through a shared-memory ring with TMA (no cluster multicast), warp 9 allocates TMEM and issues the
// tcgen05.mma instructions.  The four projections of a layer are seven "chunks" of N = C output
// columns (K, V, Q, O, MLP-1a, MLP-1b, MLP-2); chunk g accumulates in TMEM buffer g & 1, so the
// tensor pipe works on one chunk while the compute warps drain the previous one.
//
// Every operand tile in shared memory uses the K-major 128-byte-swizzled layout that tcgen05.mma and
// TMA share: 64 bf16 columns per 128-byte row, 8-row groups of 1024 bytes, 16-byte chunk index XORed
// with (row & 7).  Q, K, V and the attention output live in that same layout, so the attention phase
// (mma.sync m16n8k16 with ldmatrix) reads it without bank conflicts and writes its result straight
// into the A operand of the output projection.
//
// Every wait on an mbarrier is bounded; a wait that gives up raises DSVT_STATUS_TIMEOUT and all roles
// leave the tile loop together.
#include <cuda.h>

#include "dsvt_common.cuh"

namespace {

constexpr int kTM = 128;               // tile rows = UMMA M
constexpr int kComputeThreads = 256;   // warps 0-7
constexpr int kThreads = 320;          // + TMA warp + MMA warp
constexpr int kStages = 3;             // weight ring depth
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxPolls = 1 << 20;

struct TcGeom {
  int C, hidden, heads, tau, TMn;
  int nkb;      // C / 64: K blocks of a C-deep contraction
  int nkb_h;    // hidden / 64
  int n_f1;     // hidden / C: MLP-1 chunks
  uint32_t stage_bytes;  // C * 128
  uint32_t off_a, off_kv, off_stage, off_misc;  // byte offsets from the 1024-aligned base
};

struct Misc {  // small shared state behind the big regions
  unsigned long long full[kStages], empty[kStages], acc_full[2], acc_free[2], a_ready;
  uint32_t tmem_base;
  int abort_flag;
  int tile[4];  // s_lo, nsets, base row, rows
  int rowvox[kTM];
  int set_lo[kTM + 1];
  float red[2][2][kTM];  // [exchange][column half][row]
};

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
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

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
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

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

__device__ __forceinline__ float gelu_erf(float t) { return 0.5f * t * (1.0f + erff(t * 0.70710678118654752440f)); }

// Sets whose first distinct row lies in [t*TMn, (t+1)*TMn).  Same answer for every role.
__device__ __forceinline__ bool tile_range(const int32_t* __restrict__ rowoff, int S, int t, int TMn, int* out) {
  const int lo_row = t * TMn, hi_row = lo_row + TMn;
  int lo = 0, hi = S;
  while (lo < hi) { const int m = (lo + hi) >> 1; if (rowoff[m] < lo_row) lo = m + 1; else hi = m; }
  const int s_lo = lo;
  hi = S;
  while (lo < hi) { const int m = (lo + hi) >> 1; if (rowoff[m] < hi_row) lo = m + 1; else hi = m; }
  out[0] = s_lo;
  out[1] = lo - s_lo;
  out[2] = rowoff[s_lo];
  out[3] = rowoff[lo] - rowoff[s_lo];
  return out[1] > 0 && out[1] <= kTM && out[3] > 0 && out[3] <= kTM;
}

struct TcMaps {
  CUtensorMap qkv, o, w1, w2;
};

// ---------------------------------------------------------------------------------------------
// Attention of one tile with mma.sync: one warp per (set, head, 16-query block).
// D = head dim (16 / 24 / 32), NT = key blocks of 8 a set can have.
// ---------------------------------------------------------------------------------------------
template <int D, int NT>
__device__ __forceinline__ void attend_tile(uint32_t a_base, uint32_t k_base, uint32_t v_base, const int* set_lo,
                                            int nsets, int heads, int warp, int lane) {
  constexpr int DC = D / 8;  // 16-byte chunks per head
  const int g = lane >> 2, t4 = lane & 3;
  const float sc = 1.4426950408889634f * rsqrtf((float)D);  // log2(e) / sqrt(d)
  int item = 0;
  for (int si = 0; si < nsets; ++si) {
    const int r0 = set_lo[si], m = set_lo[si + 1] - r0;
    const int mtiles = (m + 15) >> 4, ntu = (m + 7) >> 3;
    for (int hm = 0; hm < heads * mtiles; ++hm, ++item) {
      if ((item & 7) != warp) continue;
      const int h = hm / mtiles, mt = hm - h * mtiles;
      const int c0 = h * DC;
      const int q0 = r0 + 16 * mt;
      // Q fragments (A operand, 16 x D)
      uint32_t qa[4], qb[4];
      {
        const int row = min(q0 + (lane & 15), kTM - 1);
        ldsm_x4(a_base + swz(row, c0 + (lane >> 4)), qa);
        if (D > 16) ldsm_x4(a_base + swz(row, c0 + 2 + ((D == 32) ? (lane >> 4) : 0)), qb);
      }
      float s[NT][4];
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
        if (j < ntu) {
          uint32_t kf[4];
          const int row = min(r0 + 8 * j + (lane & 7), kTM - 1);
          const int ch = min(lane >> 3, DC - 1);
          ldsm_x4(k_base + swz(row, c0 + ch), kf);
          mma_16816(s[j], qa, kf[0], kf[1]);
          if (D == 24) mma_1688(s[j], qb[0], qb[1], kf[2]);
          if (D == 32) mma_16816(s[j], qb, kf[2], kf[3]);
        }
      }
      // masked softmax over the set's m keys (rows g and g + 8 of the query block)
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const int key = 8 * j + 2 * t4;
        if (key >= m) s[j][0] = s[j][2] = -INFINITY;
        if (key + 1 >= m) s[j][1] = s[j][3] = -INFINITY;
        mx0 = fmaxf(mx0, fmaxf(s[j][0], s[j][1]));
        mx1 = fmaxf(mx1, fmaxf(s[j][2], s[j][3]));
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      float l0 = 0.f, l1 = 0.f;
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        s[j][0] = exp2f((s[j][0] - mx0) * sc);
        s[j][1] = exp2f((s[j][1] - mx0) * sc);
        s[j][2] = exp2f((s[j][2] - mx1) * sc);
        s[j][3] = exp2f((s[j][3] - mx1) * sc);
        l0 += s[j][0] + s[j][1];
        l1 += s[j][2] + s[j][3];
      }
      l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
      l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
      // O = P V
      float o[DC][4];
#pragma unroll
      for (int dn = 0; dn < DC; ++dn) o[dn][0] = o[dn][1] = o[dn][2] = o[dn][3] = 0.f;
#pragma unroll
      for (int kk = 0; kk < (NT + 1) / 2; ++kk) {
        if (2 * kk < ntu) {
          uint32_t pa[4];
          pa[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
          pa[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
          const bool two = (2 * kk + 1 < NT);
          pa[2] = two ? pack_bf16(s[(2 * kk + 1 < NT) ? 2 * kk + 1 : 0][0], s[(2 * kk + 1 < NT) ? 2 * kk + 1 : 0][1]) : 0u;
          pa[3] = two ? pack_bf16(s[(2 * kk + 1 < NT) ? 2 * kk + 1 : 0][2], s[(2 * kk + 1 < NT) ? 2 * kk + 1 : 0][3]) : 0u;
          const int row = min(r0 + 16 * kk + (lane & 15), kTM - 1);
#pragma unroll
          for (int dn = 0; dn < DC; ++dn) {
            uint32_t vf[2];
            ldsm_x2_trans(v_base + swz(row, c0 + dn), vf);
            mma_16816(o[dn], pa, vf[0], vf[1]);
          }
        }
      }
      const float i0 = 1.0f / l0, i1 = 1.0f / l1;
      const int qa_row = 16 * mt + g;
#pragma unroll
      for (int dn = 0; dn < DC; ++dn) {
        // the query rows of this block and head are dead now: their slots take the attention output
        if (qa_row < m)
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(a_base + swz(q0 + g, c0 + dn) + 4 * t4),
                       "r"(pack_bf16(o[dn][0] * i0, o[dn][1] * i0)) : "memory");
        if (qa_row + 8 < m)
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(a_base + swz(q0 + g + 8, c0 + dn) + 4 * t4),
                       "r"(pack_bf16(o[dn][2] * i1, o[dn][3] * i1)) : "memory");
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int D, int NT>
__global__ void __launch_bounds__(kThreads, 1)
layer_tc_kernel(dsvt_fused_args a, TcGeom g, const __grid_constant__ TcMaps maps, int32_t* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* sm = smem_raw + pad;
  const uint32_t sbase = raw + pad;
  Misc* mi = reinterpret_cast<Misc*>(sm + g.off_misc);
  const uint32_t a_base = sbase + g.off_a, kv_base = sbase + g.off_kv, st_base = sbase + g.off_stage;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int C = g.C;
  const dsvt_layer_params& p = a.p;
  volatile int* abort_flag = &mi->abort_flag;

  const int S = min(*a.num_sets, a.cap_sets);
  const int R = S > 0 ? a.rowoff[S] : 0;
  const int num_tiles = (R + g.TMn - 1) / g.TMn;
  const bool mlp = g.hidden > 0 && !a.attention_only;
  const int n_chunks = 4 + (mlp ? g.n_f1 + 1 : 0);

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(&mi->full[i], 1); mbar_init(&mi->empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&mi->acc_full[i], 1); mbar_init(&mi->acc_free[i], kComputeThreads); }
    mbar_init(&mi->a_ready, kComputeThreads);
    mi->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&mi->tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = mi->tmem_base;

  if (warp == 8) {
    // ================= TMA producer: the layer's weights, chunk by chunk, K block by K block ==========
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int t = blockIdx.x; t < num_tiles && !*abort_flag; t += gridDim.x) {
        int info[4];
        if (!tile_range(a.rowoff, S, t, g.TMn, info)) continue;
        for (int c = 0; c < n_chunks; ++c) {
          const CUtensorMap* map;
          int row0, nkb;
          if (c < 3) { map = &maps.qkv; row0 = (c == 0 ? 1 : c == 1 ? 2 : 0) * C; nkb = g.nkb; }   // K, V, Q
          else if (c == 3) { map = &maps.o; row0 = 0; nkb = g.nkb; }
          else if (c < 4 + g.n_f1) { map = &maps.w1; row0 = (c - 4) * C; nkb = g.nkb; }
          else { map = &maps.w2; row0 = 0; nkb = g.nkb_h; }
          for (int kb = 0; kb < nkb; ++kb) {
            if (!mbar_wait(&mi->empty[stage], phase ^ 1u, abort_flag)) goto producer_done;
            mbar_expect_tx(&mi->full[stage], g.stage_bytes);
            tma_load_2d(st_base + stage * g.stage_bytes, map, kb * 64, row0, &mi->full[stage]);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    producer_done:;
    }
    __syncwarp();
  } else if (warp == 9) {
    // ================= MMA issuer ====================================================================
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(C);
      int stage = 0;
      uint32_t phase = 0, a_phase = 0;
      uint32_t chunk_seq = 0;  // running chunk number: TMEM buffer = chunk_seq & 1
      for (int t = blockIdx.x; t < num_tiles && !*abort_flag; t += gridDim.x) {
        int info[4];
        if (!tile_range(a.rowoff, S, t, g.TMn, info)) continue;
        for (int c = 0; c < n_chunks; ++c, ++chunk_seq) {
          // a fresh A operand: X (chunks 0-2), attention output (3), x1 (4..), MLP hidden (last)
          if (c == 0 || c == 3 || c == 4 || c == 4 + g.n_f1) {
            if (!mbar_wait(&mi->a_ready, a_phase, abort_flag)) goto mma_done;
            a_phase ^= 1u;
          }
          const uint32_t buf = chunk_seq & 1u;
          if (!mbar_wait(&mi->acc_free[buf], ((chunk_seq >> 1) & 1u) ^ 1u, abort_flag)) goto mma_done;
          tc_fence_after();
          const bool last = mlp && c == 4 + g.n_f1;
          const uint32_t abase = last ? kv_base : a_base;
          const int nkb = last ? g.nkb_h : g.nkb;
          const uint32_t d_tmem = tmem + buf * 256u;
          for (int kb = 0; kb < nkb; ++kb) {
            if (!mbar_wait(&mi->full[stage], phase, abort_flag)) goto mma_done;
            tc_fence_after();
            const uint32_t sa = abase + kb * (kTM * 128), sb = st_base + stage * g.stage_bytes;
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4)
              umma_bf16(d_tmem, umma_desc(sa + k4 * 32), umma_desc(sb + k4 * 32), idesc, (kb | k4) != 0 ? 1u : 0u);
            umma_commit(&mi->empty[stage]);  // frees the weight stage once these MMAs have read it
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          umma_commit(&mi->acc_full[buf]);
        }
      }
    mma_done:;
    }
    __syncwarp();
  } else {
    // ================= compute warps =================================================================
    const int row = 32 * (warp & 3) + lane;  // TMEM lane owned in the epilogues
    const int hh = warp >> 2;                // column half owned in the epilogues
    const int half = C >> 1;
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    uint32_t chunk_seq = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      compute_sync();
      if (*abort_flag) break;
      if (tid == 0) {
        int info[4];
        const bool valid = tile_range(a.rowoff, S, t, g.TMn, info);
        mi->tile[0] = info[0]; mi->tile[1] = valid ? info[1] : 0; mi->tile[2] = info[2]; mi->tile[3] = info[3];
        if (!valid && info[1] > 0) atomicOr(status, DSVT_STATUS_BAD_INDEX);
      }
      if (tid < kTM) mi->rowvox[tid] = -1;
      compute_sync();
      const int s_lo = mi->tile[0], nsets = mi->tile[1], base = mi->tile[2], rows = mi->tile[3];
      if (nsets <= 0) continue;
      // ---- distinct slots of each set -> tile rows (Eq. 4) ----
      for (int si = warp; si < nsets; si += 8) {
        const int s = s_lo + si;
        const int32_t* trow = a.table + (size_t)s * g.tau;
        const int lb = a.rowoff[s] - base, cap = a.rowoff[s + 1] - a.rowoff[s];
        int cnt = 0;
        for (int k0 = 0; k0 < g.tau; k0 += 32) {
          const int k = k0 + lane;
          int v = -1;
          bool uniq = false;
          if (k < g.tau) { v = trow[k]; uniq = (k == 0) || (v != trow[k - 1]); }
          const unsigned bal = __ballot_sync(0xffffffffu, uniq);
          const int pos = cnt + __popc(bal & ((1u << lane) - 1u));
          if (uniq && pos < cap && lb + pos < kTM) {
            if (v < 0 || v >= a.n) { atomicOr(status, DSVT_STATUS_BAD_INDEX); v = -1; }
            mi->rowvox[lb + pos] = v;
          }
          cnt += __popc(bal);
        }
        if (lane == 0) {
          mi->set_lo[si] = lb;
          if (cnt != cap) atomicOr(status, DSVT_STATUS_BAD_INDEX);
        }
      }
      if (tid == 0) mi->set_lo[nsets] = rows;
      compute_sync();
      // ---- gather: fp32 rows -> bf16 A operand ----
      for (int r = warp; r < kTM; r += 8) {
        const int v = r < rows ? mi->rowvox[r] : -1;
        if (lane < (C >> 3)) {
          uint4 pk = make_uint4(0u, 0u, 0u, 0u);
          if (v >= 0) {
            const float4* src = reinterpret_cast<const float4*>(a.x + (size_t)v * C) + 2 * lane;
            const float4 f0 = __ldg(src), f1 = __ldg(src + 1);
            pk = make_uint4(pack_bf16(f0.x, f0.y), pack_bf16(f0.z, f0.w), pack_bf16(f1.x, f1.y), pack_bf16(f1.z, f1.w));
          }
          *reinterpret_cast<uint4*>(sm + g.off_a + swz(r, lane)) = pk;
        }
      }
      fence_proxy_async();
      mbar_arrive(&mi->a_ready);  // X is in place

      const int my_v = row < rows ? mi->rowvox[row] : -1;
      // ---- chunks 0..2: K, V, Q epilogues: + bias, to bf16, into the operand layout ----
      for (int c = 0; c < 3; ++c, ++chunk_seq) {
        const uint32_t buf = chunk_seq & 1u;
        ok = mbar_wait(&mi->acc_full[buf], (chunk_seq >> 1) & 1u, abort_flag) && ok;
        tc_fence_after();
        const float* bias = p.b_qkv ? p.b_qkv + (c == 0 ? 1 : c == 1 ? 2 : 0) * C : nullptr;
        unsigned char* dst = sm + (c == 2 ? g.off_a : g.off_kv + (uint32_t)c * (uint32_t)g.nkb * (kTM * 128));
        for (int j0 = 0; j0 < half; j0 += 32) {
          float v[32];
          tmem_ld32(tmem + lane_addr + buf * 256u + hh * half + j0, v);
          const int col = hh * half + j0;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float b[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) b[e] = v[8 * q + e] + (bias ? __ldg(bias + col + 8 * q + e) : 0.f);
            *reinterpret_cast<uint4*>(dst + swz(row, (col >> 3) + q)) =
                make_uint4(pack_bf16(b[0], b[1]), pack_bf16(b[2], b[3]), pack_bf16(b[4], b[5]), pack_bf16(b[6], b[7]));
          }
        }
        tc_fence_before();
        mbar_arrive(&mi->acc_free[buf]);
      }
      compute_sync();
      // ---- attention inside each set ----
      attend_tile<D, NT>(a_base, kv_base, kv_base + (uint32_t)g.nkb * (kTM * 128), mi->set_lo, nsets, g.heads, warp, lane);
      fence_proxy_async();
      mbar_arrive(&mi->a_ready);  // attention output is the A operand of the output projection

      // ---- chunk 3: output projection epilogue ----
      {
        const uint32_t buf = chunk_seq & 1u;
        ok = mbar_wait(&mi->acc_full[buf], (chunk_seq >> 1) & 1u, abort_flag) && ok;
        tc_fence_after();
        ++chunk_seq;
        const uint32_t tsrc = tmem + lane_addr + buf * 256u + hh * half;
        if (a.attention_only) {
          for (int j0 = 0; j0 < half; j0 += 32) {
            float v[32];
            tmem_ld32(tsrc + j0, v);
            const int col = hh * half + j0;
            if (my_v >= 0) {
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                float4 o4;
                o4.x = v[4 * q] + (p.b_o ? __ldg(p.b_o + col + 4 * q) : 0.f);
                o4.y = v[4 * q + 1] + (p.b_o ? __ldg(p.b_o + col + 4 * q + 1) : 0.f);
                o4.z = v[4 * q + 2] + (p.b_o ? __ldg(p.b_o + col + 4 * q + 2) : 0.f);
                o4.w = v[4 * q + 3] + (p.b_o ? __ldg(p.b_o + col + 4 * q + 3) : 0.f);
                *reinterpret_cast<float4*>(a.y + (size_t)my_v * C + col + 4 * q) = o4;
              }
            }
          }
          tc_fence_before();
          mbar_arrive(&mi->acc_free[buf]);
          continue;
        }
        // x1 = LN1(x + Z): pass 1 sums, pass 2 centred squares, pass 3 normalise (TMEM is re-read)
        float sum = 0.f;
        for (int j0 = 0; j0 < half; j0 += 32) {
          float v[32];
          tmem_ld32(tsrc + j0, v);
          const int col = hh * half + j0;
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float4 x4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (my_v >= 0) x4 = __ldg(reinterpret_cast<const float4*>(a.x + (size_t)my_v * C + col + 4 * q));
            sum += v[4 * q] + x4.x + v[4 * q + 1] + x4.y + v[4 * q + 2] + x4.z + v[4 * q + 3] + x4.w;
            if (p.b_o) sum += __ldg(p.b_o + col + 4 * q) + __ldg(p.b_o + col + 4 * q + 1) + __ldg(p.b_o + col + 4 * q + 2) +
                              __ldg(p.b_o + col + 4 * q + 3);
          }
        }
        mi->red[0][hh][row] = sum;
        compute_sync();
        const float mean = (mi->red[0][0][row] + mi->red[0][1][row]) / (float)C;
        float sq = 0.f;
        if (p.ln1_g) {
          for (int j0 = 0; j0 < half; j0 += 32) {
            float v[32];
            tmem_ld32(tsrc + j0, v);
            const int col = hh * half + j0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              float4 x4 = make_float4(0.f, 0.f, 0.f, 0.f);
              if (my_v >= 0) x4 = __ldg(reinterpret_cast<const float4*>(a.x + (size_t)my_v * C + col + 4 * q));
              const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float tt = v[4 * q + e] + xs[e] + (p.b_o ? __ldg(p.b_o + col + 4 * q + e) : 0.f) - mean;
                sq += tt * tt;
              }
            }
          }
        }
        mi->red[1][hh][row] = sq;
        compute_sync();
        const float inv = p.ln1_g ? rsqrtf((mi->red[1][0][row] + mi->red[1][1][row]) / (float)C + p.ln_eps) : 1.f;
        for (int j0 = 0; j0 < half; j0 += 32) {
          float v[32];
          tmem_ld32(tsrc + j0, v);
          const int col = hh * half + j0;
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float4 x4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (my_v >= 0) x4 = __ldg(reinterpret_cast<const float4*>(a.x + (size_t)my_v * C + col + 4 * q));
            const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int cc = col + 4 * q + e;
              float tt = v[4 * q + e] + xs[e] + (p.b_o ? __ldg(p.b_o + cc) : 0.f);
              if (p.ln1_g) tt = (tt - mean) * inv * __ldg(p.ln1_g + cc) + (p.ln1_b ? __ldg(p.ln1_b + cc) : 0.f);
              v[4 * q + e] = tt;
            }
            // fp32 x1 parks in the voxel's output row (also the final result when there is no MLP)
            if (my_v >= 0)
              *reinterpret_cast<float4*>(a.y + (size_t)my_v * C + col + 4 * q) =
                  make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          }
          if (mlp) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<uint4*>(sm + g.off_a + swz(row, (col >> 3) + q)) =
                  make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                             pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
          }
        }
        tc_fence_before();
        mbar_arrive(&mi->acc_free[buf]);
        if (!mlp) continue;
        fence_proxy_async();
        mbar_arrive(&mi->a_ready);  // x1 (bf16) is the A operand of MLP-1
      }
      // ---- MLP-1 chunks: H = gelu(x1 W_1^T + b_1) as the A operand of MLP-2 ----
      for (int c = 0; c < g.n_f1; ++c, ++chunk_seq) {
        const uint32_t buf = chunk_seq & 1u;
        ok = mbar_wait(&mi->acc_full[buf], (chunk_seq >> 1) & 1u, abort_flag) && ok;
        tc_fence_after();
        for (int j0 = 0; j0 < half; j0 += 32) {
          float v[32];
          tmem_ld32(tmem + lane_addr + buf * 256u + hh * half + j0, v);
          const int col = c * C + hh * half + j0;  // hidden column
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float b[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) b[e] = gelu_erf(v[8 * q + e] + (p.b_1 ? __ldg(p.b_1 + col + 8 * q + e) : 0.f));
            *reinterpret_cast<uint4*>(sm + g.off_kv + swz(row, (col >> 3) + q)) =
                make_uint4(pack_bf16(b[0], b[1]), pack_bf16(b[2], b[3]), pack_bf16(b[4], b[5]), pack_bf16(b[6], b[7]));
          }
        }
        tc_fence_before();
        mbar_arrive(&mi->acc_free[buf]);
      }
      fence_proxy_async();
      mbar_arrive(&mi->a_ready);  // H is in place
      // ---- MLP-2 epilogue: y = LN2(x1 + M) ----
      {
        const uint32_t buf = chunk_seq & 1u;
        ok = mbar_wait(&mi->acc_full[buf], (chunk_seq >> 1) & 1u, abort_flag) && ok;
        tc_fence_after();
        ++chunk_seq;
        const uint32_t tsrc = tmem + lane_addr + buf * 256u + hh * half;
        float sum = 0.f;
        for (int j0 = 0; j0 < half; j0 += 32) {
          float v[32];
          tmem_ld32(tsrc + j0, v);
          const int col = hh * half + j0;
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float4 x4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (my_v >= 0) x4 = *reinterpret_cast<const float4*>(a.y + (size_t)my_v * C + col + 4 * q);
            sum += v[4 * q] + x4.x + v[4 * q + 1] + x4.y + v[4 * q + 2] + x4.z + v[4 * q + 3] + x4.w;
            if (p.b_2) sum += __ldg(p.b_2 + col + 4 * q) + __ldg(p.b_2 + col + 4 * q + 1) + __ldg(p.b_2 + col + 4 * q + 2) +
                              __ldg(p.b_2 + col + 4 * q + 3);
          }
        }
        mi->red[0][hh][row] = sum;
        compute_sync();
        const float mean = (mi->red[0][0][row] + mi->red[0][1][row]) / (float)C;
        float sq = 0.f;
        if (p.ln2_g) {
          for (int j0 = 0; j0 < half; j0 += 32) {
            float v[32];
            tmem_ld32(tsrc + j0, v);
            const int col = hh * half + j0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              float4 x4 = make_float4(0.f, 0.f, 0.f, 0.f);
              if (my_v >= 0) x4 = *reinterpret_cast<const float4*>(a.y + (size_t)my_v * C + col + 4 * q);
              const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float tt = v[4 * q + e] + xs[e] + (p.b_2 ? __ldg(p.b_2 + col + 4 * q + e) : 0.f) - mean;
                sq += tt * tt;
              }
            }
          }
        }
        mi->red[1][hh][row] = sq;
        compute_sync();
        const float inv = p.ln2_g ? rsqrtf((mi->red[1][0][row] + mi->red[1][1][row]) / (float)C + p.ln_eps) : 1.f;
        for (int j0 = 0; j0 < half; j0 += 32) {
          float v[32];
          tmem_ld32(tsrc + j0, v);
          const int col = hh * half + j0;
          if (my_v >= 0) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              float* yp = a.y + (size_t)my_v * C + col + 4 * q;
              const float4 x4 = *reinterpret_cast<const float4*>(yp);
              const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
              float o4[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int cc = col + 4 * q + e;
                float tt = v[4 * q + e] + xs[e] + (p.b_2 ? __ldg(p.b_2 + cc) : 0.f);
                if (p.ln2_g) tt = (tt - mean) * inv * __ldg(p.ln2_g + cc) + (p.ln2_b ? __ldg(p.ln2_b + cc) : 0.f);
                o4[e] = tt;
              }
              *reinterpret_cast<float4*>(yp) = make_float4(o4[0], o4[1], o4[2], o4[3]);
            }
          }
        }
        tc_fence_before();
        mbar_arrive(&mi->acc_free[buf]);
      }
    }
    if (!ok || *abort_flag) {
      if (tid == 0) atomicOr(status, DSVT_STATUS_TIMEOUT);
    }
  }
  // ---- teardown: everyone meets here, then the allocating warp returns the TMEM columns ----
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
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

template <int D, int NT>
int launch_tc(dsvt_ctx* ctx, const dsvt_fused_args& a, const TcGeom& g, const TcMaps& maps, int grid, size_t smem) {
  cudaError_t e = cudaFuncSetAttribute(layer_tc_kernel<D, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return DSVT_ERR_CUDA; }
  layer_tc_kernel<D, NT><<<grid, kThreads, smem, ctx->stream>>>(a, g, maps, ctx->status);
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}

}  // namespace

// Shapes the tensor-core kernel covers; everything else goes to the FMA kernel.
bool dsvt_layer_tc_supported(const dsvt_fused_args& a) {
  const dsvt_layer_params& p = a.p;
  if (p.precision != DSVT_BF16_FP32ACC || p.pe) return false;
  if (p.C != 64 && p.C != 128 && p.C != 192) return false;
  const int d = p.C / p.heads;
  if (d != 16 && d != 24 && d != 32) return false;
  if (p.set_size > 96) return false;
  const int hidden = a.attention_only ? 0 : p.hidden;
  if (hidden != 0 && hidden != p.C && hidden != 2 * p.C) return false;
  return encode_fn() != nullptr;
}

int dsvt_launch_layer_tc(dsvt_ctx* ctx, const dsvt_fused_args& a) {
  const dsvt_layer_params& p = a.p;
  TcGeom g;
  g.C = p.C; g.hidden = a.attention_only ? 0 : p.hidden; g.heads = p.heads; g.tau = p.set_size;
  g.TMn = kTM - g.tau + 1;
  g.nkb = p.C / 64; g.nkb_h = g.hidden / 64; g.n_f1 = g.hidden / p.C;
  g.stage_bytes = (uint32_t)p.C * 128u;
  const uint32_t a_bytes = kTM * p.C * 2;
  const int kv_cols = 2 * p.C > g.hidden ? 2 * p.C : g.hidden;
  g.off_a = 0;
  g.off_kv = a_bytes;
  g.off_stage = g.off_kv + (uint32_t)kTM * kv_cols * 2;
  g.off_stage = (g.off_stage + 1023u) & ~1023u;
  g.off_misc = g.off_stage + kStages * g.stage_bytes;
  const size_t smem = (size_t)g.off_misc + sizeof(Misc) + 1024;
  if (smem > 227 * 1024) return DSVT_ERR_UNSUPPORTED;
  TcMaps maps;
  bool okm = make_weight_map(&maps.qkv, p.W_qkv, 3 * p.C, p.C, p.C) && make_weight_map(&maps.o, p.W_o, p.C, p.C, p.C);
  if (g.hidden > 0)
    okm = okm && make_weight_map(&maps.w1, p.W_1, g.hidden, p.C, p.C) && make_weight_map(&maps.w2, p.W_2, p.C, g.hidden, p.C);
  else {
    maps.w1 = maps.o;
    maps.w2 = maps.o;
  }
  if (!okm) return DSVT_ERR_CUDA;
  int64_t rmax = (int64_t)a.cap_sets * g.tau;
  if (rmax > a.n) rmax = a.n;
  int64_t grid = dsvt_ceil_div(rmax, g.TMn);
  if (grid < 1) grid = 1;
  if (grid > ctx->sm_count) grid = ctx->sm_count;
  const int d = p.C / p.heads;
  const int nt = (g.tau + 7) / 8;
#define DSVT_TC_CASE(DD, NN) return launch_tc<DD, NN>(ctx, a, g, maps, (int)grid, smem)
  if (d == 16) { if (nt <= 5) DSVT_TC_CASE(16, 5); if (nt <= 6) DSVT_TC_CASE(16, 6); DSVT_TC_CASE(16, 12); }
  if (d == 24) { if (nt <= 5) DSVT_TC_CASE(24, 5); if (nt <= 6) DSVT_TC_CASE(24, 6); DSVT_TC_CASE(24, 12); }
  if (nt <= 5) DSVT_TC_CASE(32, 5);
  if (nt <= 6) DSVT_TC_CASE(32, 6);
  DSVT_TC_CASE(32, 12);
#undef DSVT_TC_CASE
}
