// Attention-style 3D pooling (Eq. 6, Eq. 7): dense cell map -> region ranks -> fused
// pad / max-pool / cross-attention kernel.  The region bookkeeping is exact integer work; the
// attention runs on the fp32 FMA pipes with float or bfloat16 weights.
#include <cuda.h>

#include "dsvt_common.cuh"
#include "fma_tile.cuh"

namespace {
using namespace dsvt_fma;

struct PoolGeom {
  int32_t batch, gx, gy, gz, l, w, h, GX, GY, GZ, nslots;
};

__device__ __forceinline__ int4 clamp_coord(int4 c, const PoolGeom& g, int32_t* status) {
  const bool bad =
      c.x < 0 || c.x >= g.batch || c.y < 0 || c.y >= g.gx || c.z < 0 || c.z >= g.gy || c.w < 0 || c.w >= g.gz;
  if (bad) {
    atomicOr(status, DSVT_STATUS_BAD_COORD);
    c.x = min(max(c.x, 0), g.batch - 1);
    c.y = min(max(c.y, 0), g.gx - 1);
    c.z = min(max(c.z, 0), g.gy - 1);
    c.w = min(max(c.w, 0), g.gz - 1);
  }
  return c;
}

// Each voxel claims its cell of the dense (region, slot) map and marks its region as non-empty.
__global__ void pool_mark_kernel(const int4* __restrict__ coords, int32_t n_max, const int32_t* __restrict__ n_dev,
                                 PoolGeom g, int32_t* __restrict__ cell_map,
                                 int32_t* __restrict__ region_flag, uint32_t* __restrict__ vox_region,
                                 int32_t* __restrict__ slot_of, int32_t* __restrict__ status) {
  pdl_enter();  // (lets the scan's first kernel start under this one's tail)
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int n = n_dev ? min(max(*n_dev, 0), n_max) : n_max;  // (a count that lives on the device)
  if (i >= n) return;
  const int4 c = clamp_coord(coords[i], g, status);
  const int X = c.y / g.l, Y = c.z / g.w, Z = c.w / g.h;
  const int slot = ((c.y - X * g.l) * g.w + (c.z - Y * g.w)) * g.h + (c.w - Z * g.h);
  const uint32_t region = (uint32_t)(((c.x * g.GX + X) * g.GY + Y) * g.GZ + Z);
  const int old = atomicExch(&cell_map[(size_t)region * g.nslots + slot], i);
  if (old != -1) atomicOr(status, DSVT_STATUS_DUPLICATE_CELL);
  region_flag[region] = 1;
  vox_region[i] = region;
  if (slot_of) slot_of[i] = slot;
}

// region rank -> output row: coordinates, region id per output row, region_of per voxel.
__global__ void pool_finish_kernel(int32_t n_max, const int32_t* __restrict__ n_dev, PoolGeom g,
                                   const uint32_t* __restrict__ vox_region,
                                   const int32_t* __restrict__ region_rank, int32_t num_regions, int32_t cap_m,
                                   int32_t* __restrict__ out_coords, int32_t* __restrict__ region_key,
                                   int32_t* __restrict__ region_of, int32_t* __restrict__ num_out,
                                   int32_t* __restrict__ status) {
  pdl_enter();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0) {
    const int m = region_rank[num_regions];
    if (m > cap_m) atomicOr(status, DSVT_STATUS_TABLE_OVERFLOW);
    *num_out = min(m, cap_m);
  }
  const int n = n_dev ? min(max(*n_dev, 0), n_max) : n_max;
  if (i >= n) return;
  const uint32_t region = vox_region[i];
  const int r = region_rank[region];
  if (region_of) region_of[i] = r;
  if (r < cap_m) {  // every member of a region writes the same values
    region_key[r] = (int32_t)region;
    uint32_t t = region;
    const int Z = t % g.GZ; t /= g.GZ;
    const int Y = t % g.GY; t /= g.GY;
    const int X = t % g.GX; t /= g.GX;
    reinterpret_cast<int4*>(out_coords)[r] = make_int4((int)t, X, Y, Z);
  }
}

struct PoolArgs {
  const float* feats;
  const int32_t* cell_map;
  const int32_t* region_key;
  const int32_t* num_out;
  int32_t cap_m, n;
  const void *W_q, *W_k, *W_v, *W_o;
  const float *b_q, *b_k, *b_v, *b_o, *slot_pe;
  float* out_feats;
  int32_t C, heads, nslots, mask_empty;
  int32_t TM, TR, LDQ;
};

template <typename WT, int RM>
__global__ void __launch_bounds__(kThreads, 1) pool_attn_kernel(PoolArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int C = a.C, LDQ = a.LDQ, TM = a.TM, TR = a.TR, ns = a.nslots;
  float* Xs = reinterpret_cast<float*>(smem_raw);  // [TM][C]
  float* Bs = Xs + (size_t)TM * C;                  // [TM][LDQ]
  float* Wst = Bs + (size_t)TM * LDQ;               // [kKC][kNC]
  int* rowvox = reinterpret_cast<int*>(Wst + kKC * kNC);  // [TM]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int C4 = C >> 2, d = C / a.heads, d4 = d >> 2;
  const float scale = 1.0f / sqrtf((float)d);
  const int m = min(*a.num_out, a.cap_m);
  const int num_tiles = (m + TR - 1) / TR;
  const WT* Wq = reinterpret_cast<const WT*>(a.W_q);
  const WT* Wk = reinterpret_cast<const WT*>(a.W_k);
  const WT* Wv = reinterpret_cast<const WT*>(a.W_v);
  const WT* Wo = reinterpret_cast<const WT*>(a.W_o);

  for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
    __syncthreads();
    const int r_lo = t * TR, nr = min(TR, m - r_lo), rows = nr * ns;
    for (int r = tid; r < rows; r += kThreads) {
      const int ri = r / ns, s = r - ri * ns;
      rowvox[r] = a.cell_map[(size_t)a.region_key[r_lo + ri] * ns + s];
    }
    __syncthreads();
    const int rm_rows = (rows + 15) >> 4, rm_reg = (nr + 15) >> 4;
    // padded region rows (zero rows for empty slots)
    for (int r = warp; r < (rm_rows << 4); r += kWarps) {
      const int v = r < rows ? rowvox[r] : -1;
      for (int c4 = lane; c4 < C4; c4 += 32) {
        float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
        if (v >= 0) f = reinterpret_cast<const float4*>(a.feats + (size_t)v * C)[c4];
        reinterpret_cast<float4*>(Xs + (size_t)r * C)[c4] = f;
      }
    }
    __syncthreads();
    // Eq. 6: P = channel-wise max over the slots -> Bs[:, 2C:3C) rows [0, nr)
    for (int idx = tid; idx < (rm_reg << 4) * C; idx += kThreads) {
      const int ri = idx / C, c = idx - ri * C;
      float mx = 0.f;
      if (ri < nr) {
        mx = -INFINITY;
        for (int s = 0; s < ns; ++s)
          if (!a.mask_empty || rowvox[ri * ns + s] >= 0) mx = fmaxf(mx, Xs[(size_t)(ri * ns + s) * C + c]);
      }
      Bs[(size_t)ri * LDQ + 2 * C + c] = mx;
    }
    __syncthreads();
    if (a.slot_pe) {
      for (int idx = tid; idx < rows * C4; idx += kThreads) {
        const int r = idx / C4, c4 = idx - r * C4;
        const float4 e = reinterpret_cast<const float4*>(a.slot_pe + (size_t)(r % ns) * C)[c4];
        float4* px = reinterpret_cast<float4*>(Xs + (size_t)r * C) + c4;
        float4 f = *px;
        f.x += e.x; f.y += e.y; f.z += e.z; f.w += e.w;
        *px = f;
      }
      __syncthreads();
    }
    // Eq. 7: keys, values from the padded slots; query from P
    gemm_tile<WT, RM>(Xs, C, rm_rows, Wk, C, C, a.b_k, Bs, LDQ, false, Wst);
    gemm_tile<WT, RM>(Xs, C, rm_rows, Wv, C, C, a.b_v, Bs + C, LDQ, false, Wst);
    gemm_tile<WT, RM>(Bs + 2 * C, LDQ, rm_reg, Wq, C, C, a.b_q, Xs, C, false, Wst);
    // one warp per (region, head): lane s scores slot s
    for (int item = warp; item < nr * a.heads; item += kWarps) {
      const int ri = item / a.heads, h = item - ri * a.heads;
      const bool use = lane < ns && (!a.mask_empty || rowvox[ri * ns + lane] >= 0);
      float lg = -INFINITY;
      if (use) {
        const float4* q4 = reinterpret_cast<const float4*>(Xs + (size_t)ri * C + h * d);
        const float4* k4 = reinterpret_cast<const float4*>(Bs + (size_t)(ri * ns + lane) * LDQ + h * d);
        float s = 0.f;
        for (int c = 0; c < d4; ++c) {
          const float4 qv = q4[c], kv = k4[c];
          s = fmaf(qv.x, kv.x, s); s = fmaf(qv.y, kv.y, s); s = fmaf(qv.z, kv.z, s); s = fmaf(qv.w, kv.w, s);
        }
        lg = s * scale;
      }
      const float mx = warp_max(lg);
      const float e = use ? expf(lg - mx) : 0.f;
      const float inv = 1.0f / warp_sum(e);
      for (int c0 = 0; c0 < d; c0 += 32) {
        const int c = c0 + lane;
        float acc = 0.f;
        for (int s = 0; s < ns; ++s) {
          const float ps = __shfl_sync(0xffffffffu, e, s);
          if (c < d) acc = fmaf(ps, Bs[(size_t)(ri * ns + s) * LDQ + C + h * d + c], acc);
        }
        if (c < d) Xs[(size_t)(TR + ri) * C + h * d + c] = acc * inv;
      }
    }
    __syncthreads();
    gemm_tile<WT, RM>(Xs + (size_t)TR * C, C, rm_reg, Wo, C, C, a.b_o, Bs + 2 * C, LDQ, false, Wst);
    for (int r = warp; r < nr; r += kWarps)
      for (int c4 = lane; c4 < C4; c4 += 32)
        reinterpret_cast<float4*>(a.out_feats + (size_t)(r_lo + r) * C)[c4] =
            *reinterpret_cast<const float4*>(Bs + (size_t)r * LDQ + 2 * C + 4 * c4);
  }
}

// ---------------------------------------------------------------------------------------------------
// Tensor-core version of the fused kernel for bfloat16 weights (mma.sync.m16n8k16, fp32 accumulation).
// Tile = up to 128 padded slot rows = TR regions.  Shared memory: X (padded slots, bf16, the A operand
// of the key / value projections), K, V (bf16), P (Eq. 6 maxima, bf16, later the attention output), a
// two-stage ring of 64-column weight blocks.  All operand tiles use the 128-byte-swizzled K-major layout
// (64 bf16 per 128-byte row, 8-row groups of 1024 bytes, chunk index XOR row & 7), which ldmatrix reads
// without bank conflicts.  The fp32 queries and the fp32 output rows reuse X's space once X is dead.
// ---------------------------------------------------------------------------------------------------
namespace mma_pool {
constexpr int kT = 512, kW = kT / 32;
constexpr int kRows = 128;  // slot rows per tile
constexpr int kRegs = 64;   // regions per tile at most

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// byte offset of 16-byte chunk c8 of `row` in a tile whose 64-column blocks hold rows_pb rows each
__device__ __forceinline__ uint32_t swz(int row, int c8, int rows_pb) {
  return (uint32_t)((c8 >> 3) * (rows_pb * 128) + (row >> 3) * 1024 + (row & 7) * 128 + (((c8 & 7) ^ (row & 7)) << 4));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ float bf16_at(const unsigned char* tile, int row, int col, int rows_pb) {
  const unsigned short u = *reinterpret_cast<const unsigned short*>(tile + swz(row, col >> 3, rows_pb) + (col & 7) * 2);
  return __uint_as_float((uint32_t)u << 16);
}

constexpr int kStages = 4;  // weight ring: 64-column blocks, prefetched three ahead
constexpr int kMaxHeads = 8;

struct Layout {  // byte offsets into dynamic shared memory (1024-aligned base)
  uint32_t x, kv, p, w, probs, rowvox, bars, total;
};
__host__ __device__ inline Layout make_layout(int C) {
  Layout L;
  L.x = 0;                                   // padded slot rows (bf16 A operand); at the end the fp32 output rows
  L.kv = L.x + kRows * C * 2;                // keys, later values (bf16)
  L.p = L.kv + kRows * C * 2;                // Eq. 6 maxima -> queries (in place) -> attention output (bf16)
  L.w = L.p + kRegs * C * 2;
  L.probs = L.w + kStages * (uint32_t)C * 128;
  L.rowvox = L.probs + 2 * kRows * kMaxHeads * 4;  // (regions x padded slots) < 2 x 128 per head
  L.bars = L.rowvox + kRows * 4;             // kStages mbarriers + the error flag
  L.total = L.bars + kStages * 8 + 8;
  return L;
}

struct PoolMaps {
  CUtensorMap w[4];  // W_q, W_k, W_v, W_o: boxes of 64 input columns x C rows, 128-byte swizzle
};
constexpr int kMaxPolls = 1 << 20;

// The weight blocks of a CTA form one stream: tile after tile, W_q, W_k, W_v, W_o, each in C / 64 blocks of
// 64 input columns.  Block g lives in stage g mod 4 and is requested three steps before it is used, by one
// thread, as a TMA load that completes on the stage's mbarrier.  Every wait is bounded (error flag).
struct WeightStream {
  const PoolMaps* maps;
  unsigned long long* full;  // [kStages] in shared memory
  int* error;                // shared flag: a wait gave up
  int C, nkb;
  long long total;   // blocks this CTA will consume
  long long next;    // next block to consume
  uint32_t base, stage_bytes;

  __device__ __forceinline__ void request(long long g) {
    if (g < total && threadIdx.x == 0) {
      const int kb = (int)(g % nkb), st = (int)(g % kStages);
      const uint32_t bar = smem_u32(&full[st]);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(stage_bytes) : "memory");
      asm volatile(
          "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
          ::"r"(base + (uint32_t)st * stage_bytes), "l"((uint64_t)&maps->w[(g / nkb) & 3]), "r"(bar), "r"(kb * 64), "r"(0)
          : "memory");
    }
  }
  __device__ __forceinline__ void prologue() {
    for (int g = 0; g < kStages - 1; ++g) request(g);
  }
  // Makes the next block usable by every thread and returns its stage; requests the block three ahead.
  __device__ __forceinline__ uint32_t acquire() {
    const int st = (int)(next % kStages);
    const uint32_t bar = smem_u32(&full[st]), parity = (uint32_t)((next / kStages) & 1);
    bool ok = false;
    for (int i = 0; i < kMaxPolls && !ok; ++i) {
      uint32_t done;
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                   : "=r"(done) : "r"(bar), "r"(parity) : "memory");
      ok = done != 0;
      if (!ok && (i & 255) == 255 && *reinterpret_cast<volatile int*>(error)) break;
    }
    if (!ok) *reinterpret_cast<volatile int*>(error) = 1;
    __syncthreads();  // everyone is done with the block before it: its stage may be overwritten
    request(next + kStages - 1);
    ++next;
    return base + (uint32_t)st * stage_bytes;
  }
};

// epi(row, col, v0, v1) receives out(row, col) and out(row, col + 1), out = A W^T + bias, for row < 16 mt_count.
// A: swizzled bf16 tile with rows_pb rows per 64-column block; W: the stream's next C / 64 blocks.  Work
// item = (16-row tile, 32 output columns); all A reads are complete before the first epi call.
template <class Epi>
__device__ __forceinline__ void gemm(uint32_t a_base, int rows_pb, int mt_count, WeightStream& ws, const float* bias,
                                     Epi epi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int C = ws.C, ng = C >> 5, items = mt_count * ng;
  float acc[3][4][4];
#pragma unroll
  for (int ii = 0; ii < 3; ++ii) {
    const int item = warp + kW * ii;
    const int g = item < items ? item % ng : 0;
#pragma unroll
    for (int nb = 0; nb < 4; ++nb) {
      const int col = g * 32 + nb * 8 + 2 * (lane & 3);
      const float b0 = bias ? __ldg(bias + col) : 0.f, b1 = bias ? __ldg(bias + col + 1) : 0.f;
      acc[ii][nb][0] = b0; acc[ii][nb][1] = b1; acc[ii][nb][2] = b0; acc[ii][nb][3] = b1;
    }
  }
  for (int kb = 0; kb < ws.nkb; ++kb) {
    const uint32_t wb = ws.acquire();
#pragma unroll
    for (int ii = 0; ii < 3; ++ii) {
      const int item = warp + kW * ii;
      if (item < items) {
        const int mt = item / ng, g = item - mt * ng;
        uint32_t af[4][4];
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          ldsm_x4(a_base + swz(16 * mt + (lane & 15), kb * 8 + ks * 2 + (lane >> 4), rows_pb), af[ks]);
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
          const int n0 = g * 32 + nb * 8;
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t bf[4];
            ldsm_x4(wb + swz(n0 + (lane & 7), half * 4 + (lane >> 3), 0), bf);
            mma_16816(acc[ii][nb], af[2 * half], bf[0], bf[1]);
            mma_16816(acc[ii][nb], af[2 * half + 1], bf[2], bf[3]);
          }
        }
      }
    }
  }
  __syncthreads();  // every warp has read its A fragments: the epilogue may overwrite A in place
#pragma unroll
  for (int ii = 0; ii < 3; ++ii) {
    const int item = warp + kW * ii;
    if (item < items) {
      const int mt = item / ng, g = item - mt * ng;
#pragma unroll
      for (int nb = 0; nb < 4; ++nb) {
        const int row = 16 * mt + (lane >> 2), col = g * 32 + nb * 8 + 2 * (lane & 3);
        epi(row, col, acc[ii][nb][0], acc[ii][nb][1]);
        epi(row + 8, col, acc[ii][nb][2], acc[ii][nb][3]);
      }
    }
  }
}

__device__ __forceinline__ void unpack8(const uint4 u, float (&f)[8]) {
  f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xFFFF0000u);
  f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xFFFF0000u);
  f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xFFFF0000u);
  f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xFFFF0000u);
}

__global__ void __launch_bounds__(kT, 1) pool_attn_mma_kernel(const __grid_constant__ PoolArgs a,
                                                              const __grid_constant__ PoolMaps maps,
                                                              int32_t* __restrict__ status) {
  extern __shared__ unsigned char pool_smem_raw[];
  const uint32_t raw = smem_u32(pool_smem_raw);
  unsigned char* sm = pool_smem_raw + ((1024u - (raw & 1023u)) & 1023u);
  const uint32_t sb = smem_u32(sm);
  const int C = a.C, ns = a.nslots, TR = a.TR, heads = a.heads;
  const Layout L = make_layout(C);
  int* rowvox = reinterpret_cast<int*>(sm + L.rowvox);
  float* probs = reinterpret_cast<float*>(sm + L.probs);  // [region][head][padded slot]
  float* outf = reinterpret_cast<float*>(sm + L.x);       // fp32 output rows [kRegs][C], once X is dead
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int C4 = C >> 2, d = C / heads;
  const float scale = 1.0f / sqrtf((float)d);
  const int m = min(*a.num_out, a.cap_m);
  const int num_tiles = (m + TR - 1) / TR;
  int nsp = 1;
  while (nsp < ns) nsp <<= 1;
  const int hpg = 32 / nsp;  // heads per pass of a warp

  WeightStream ws;
  ws.maps = &maps;
  ws.full = reinterpret_cast<unsigned long long*>(sm + L.bars);
  ws.error = reinterpret_cast<int*>(sm + L.bars + kStages * 8);
  if (tid == 0) {
    for (int i = 0; i < kStages; ++i)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&ws.full[i])) : "memory");
    *ws.error = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  ws.C = C; ws.nkb = C >> 6;
  const long long my_tiles = blockIdx.x < num_tiles ? (num_tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;
  ws.total = my_tiles * 4 * ws.nkb;
  ws.next = 0;
  ws.base = sb + L.w;
  ws.stage_bytes = (uint32_t)C * 128;
  ws.prologue();

  for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
    __syncthreads();
    const int r_lo = t * TR, nr = min(TR, m - r_lo), rows = nr * ns;
    const int mt_rows = (rows + 15) >> 4, mt_reg = (nr + 15) >> 4;
    for (int r = tid; r < kRows; r += kT) {
      int v = -1;
      if (r < rows) {
        const int ri = r / ns;
        v = a.cell_map[(size_t)a.region_key[r_lo + ri] * ns + (r - ri * ns)];
      }
      rowvox[r] = v;
    }
    __syncthreads();
    // padded slot rows (+ slot term) -> X as bf16; Eq. 6 maxima -> P as bf16.  One warp per region, the loads
    // of four slots in flight together.
    for (int ri = warp; ri < (mt_reg << 4); ri += kW) {
      for (int c4 = lane; c4 < C4; c4 += 32) {
        float4 mx = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ri < nr) {
          mx = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
          for (int s0 = 0; s0 < ns; s0 += 4) {
            float4 f[4];
            int vv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              vv[u] = s0 + u < ns ? rowvox[ri * ns + s0 + u] : -1;
              f[u] = make_float4(0.f, 0.f, 0.f, 0.f);
              if (vv[u] >= 0) f[u] = __ldg(reinterpret_cast<const float4*>(a.feats + (size_t)vv[u] * C) + c4);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              if (s0 + u < ns) {
                const int s = s0 + u, r = ri * ns + s;
                if (!a.mask_empty || vv[u] >= 0) {
                  mx.x = fmaxf(mx.x, f[u].x); mx.y = fmaxf(mx.y, f[u].y); mx.z = fmaxf(mx.z, f[u].z); mx.w = fmaxf(mx.w, f[u].w);
                }
                if (a.slot_pe) {
                  const float4 e = __ldg(reinterpret_cast<const float4*>(a.slot_pe + (size_t)s * C) + c4);
                  f[u].x += e.x; f[u].y += e.y; f[u].z += e.z; f[u].w += e.w;
                }
                *reinterpret_cast<uint2*>(sm + L.x + swz(r, c4 >> 1, kRows) + (c4 & 1) * 8) =
                    make_uint2(pack_bf16(f[u].x, f[u].y), pack_bf16(f[u].z, f[u].w));
              }
            }
          }
        }
        *reinterpret_cast<uint2*>(sm + L.p + swz(ri, c4 >> 1, kRegs) + (c4 & 1) * 8) =
            make_uint2(pack_bf16(mx.x, mx.y), pack_bf16(mx.z, mx.w));
      }
    }
    // rows between the last slot row and the end of its 16-row tile: zeros
    for (int idx = tid; idx < ((mt_rows << 4) - rows) * (C >> 3); idx += kT) {
      const int r = rows + idx / (C >> 3), c8 = idx % (C >> 3);
      *reinterpret_cast<uint4*>(sm + L.x + swz(r, c8, kRows)) = make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();
    // Eq. 7.  Queries from P, in place (bf16); keys from the padded slots.
    gemm(sb + L.p, kRegs, mt_reg, ws, a.b_q, [&](int row, int col, float v0, float v1) {
      *reinterpret_cast<uint32_t*>(sm + L.p + swz(row, col >> 3, kRegs) + (col & 7) * 2) = pack_bf16(v0, v1);
    });
    gemm(sb + L.x, kRows, mt_rows, ws, a.b_k, [&](int row, int col, float v0, float v1) {
      *reinterpret_cast<uint32_t*>(sm + L.kv + swz(row, col >> 3, kRows) + (col & 7) * 2) = pack_bf16(v0, v1);
    });
    __syncthreads();
    // scores and softmax: one warp per region, lane = (head of the current group, slot)
    for (int ri = warp; ri < nr; ri += kW) {
      const int s = lane & (nsp - 1), hh = lane / nsp;
      for (int h0 = 0; h0 < heads; h0 += hpg) {
        const int h = h0 + hh;
        const bool use = h < heads && s < ns && (!a.mask_empty || rowvox[ri * ns + s] >= 0);
        float lg = -INFINITY;
        if (use) {
          float acc = 0.f;
          if ((d & 7) == 0) {
            for (int j = 0; j < (d >> 3); ++j) {
              float q[8], k[8];
              unpack8(*reinterpret_cast<const uint4*>(sm + L.p + swz(ri, ((h * d) >> 3) + j, kRegs)), q);
              unpack8(*reinterpret_cast<const uint4*>(sm + L.kv + swz(ri * ns + s, ((h * d) >> 3) + j, kRows)), k);
#pragma unroll
              for (int e = 0; e < 8; ++e) acc = fmaf(q[e], k[e], acc);
            }
          } else {
            for (int c = 0; c < d; ++c)
              acc = fmaf(bf16_at(sm + L.p, ri, h * d + c, kRegs), bf16_at(sm + L.kv, ri * ns + s, h * d + c, kRows), acc);
          }
          lg = acc * scale;
        }
        float mx = lg;
        for (int o = nsp >> 1; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float e = use ? expf(lg - mx) : 0.f;
        float sum = e;
        for (int o = nsp >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (h < heads) probs[(ri * heads + h) * nsp + s] = sum > 0.f ? e / sum : 0.f;
      }
    }
    // values into the keys' space
    gemm(sb + L.x, kRows, mt_rows, ws, a.b_v, [&](int row, int col, float v0, float v1) {
      *reinterpret_cast<uint32_t*>(sm + L.kv + swz(row, col >> 3, kRows) + (col & 7) * 2) = pack_bf16(v0, v1);
    });
    __syncthreads();
    // attention output (bf16) over the queries: one thread per (region, 8-channel chunk) (or per channel)
    if ((d & 7) == 0) {
      const int cpr = C >> 3;
      for (int idx = tid; idx < (mt_reg << 4) * cpr; idx += kT) {
        const int ri = idx / cpr, c8 = idx - ri * cpr;
        float o[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (ri < nr) {
          const int h = (c8 << 3) / d;
          const float* pr = probs + (ri * heads + h) * nsp;
          for (int s2 = 0; s2 < ns; ++s2) {
            float v[8];
            unpack8(*reinterpret_cast<const uint4*>(sm + L.kv + swz(ri * ns + s2, c8, kRows)), v);
            const float ps = pr[s2];
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = fmaf(ps, v[e], o[e]);
          }
        }
        *reinterpret_cast<uint4*>(sm + L.p + swz(ri, c8, kRegs)) =
            make_uint4(pack_bf16(o[0], o[1]), pack_bf16(o[2], o[3]), pack_bf16(o[4], o[5]), pack_bf16(o[6], o[7]));
      }
    } else {
      for (int idx = tid; idx < (mt_reg << 4) * C; idx += kT) {
        const int ri = idx / C, c = idx - ri * C;
        float o = 0.f;
        if (ri < nr) {
          const float* pr = probs + (ri * heads + c / d) * nsp;
          for (int s2 = 0; s2 < ns; ++s2) o = fmaf(pr[s2], bf16_at(sm + L.kv, ri * ns + s2, c, kRows), o);
        }
        *reinterpret_cast<__nv_bfloat16*>(sm + L.p + swz(ri, c >> 3, kRegs) + (c & 7) * 2) = __float2bfloat16_rn(o);
      }
    }
    __syncthreads();
    gemm(sb + L.p, kRegs, mt_reg, ws, a.b_o, [&](int row, int col, float v0, float v1) {
      *reinterpret_cast<float2*>(outf + (size_t)row * C + col) = make_float2(v0, v1);  // X is dead
    });
    __syncthreads();
    for (int r = warp; r < nr; r += kW)
      for (int c4 = lane; c4 < C4; c4 += 32)
        reinterpret_cast<float4*>(a.out_feats + (size_t)(r_lo + r) * C)[c4] = *reinterpret_cast<const float4*>(outf + (size_t)r * C + 4 * c4);
  }
  if (tid == 0 && *ws.error) atomicOr(status, DSVT_STATUS_TIMEOUT);
}
}  // namespace mma_pool

size_t pool_smem_bytes(int TM, int C, int LDQ) {
  return ((size_t)TM * C + (size_t)TM * LDQ + kKC * kNC) * 4 + (size_t)TM * 4 + 16;
}

template <typename WT, int RM>
int launch_pool_one(dsvt_ctx* ctx, const PoolArgs& a, int grid) {
  const size_t smem = pool_smem_bytes(a.TM, a.C, a.LDQ);
  cudaError_t e = cudaFuncSetAttribute(pool_attn_kernel<WT, RM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return DSVT_ERR_CUDA; }
  pool_attn_kernel<WT, RM><<<grid, kThreads, smem, ctx->stream>>>(a);
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}

template <typename WT>
int launch_pool_rm(dsvt_ctx* ctx, const PoolArgs& a, int grid) {
  switch (a.TM / 16) {
    case 2: return launch_pool_one<WT, 2>(ctx, a, grid);
    case 3: return launch_pool_one<WT, 3>(ctx, a, grid);
    case 4: return launch_pool_one<WT, 4>(ctx, a, grid);
    case 6: return launch_pool_one<WT, 6>(ctx, a, grid);
    case 8: return launch_pool_one<WT, 8>(ctx, a, grid);
  }
  return DSVT_ERR_UNSUPPORTED;
}

}  // namespace

extern "C" int dsvt_pool(dsvt_ctx* ctx, const int32_t* coords, const float* feats, int32_t n, int32_t C, int32_t batch,
                         const int32_t grid[3], const int32_t pool[3], const void* W_q, const void* W_k,
                         const void* W_v, const void* W_o, const float* b_q, const float* b_k, const float* b_v,
                         const float* b_o, const float* slot_pe, int32_t heads, int32_t mask_empty, int precision,
                         int32_t* out_coords, float* out_feats, int32_t cap_m, int32_t* num_out, int32_t* region_of,
                         int32_t* slot_of) {
  return dsvt_pool_counted(ctx, coords, feats, n, nullptr, C, batch, grid, pool, W_q, W_k, W_v, W_o, b_q, b_k, b_v, b_o,
                           slot_pe, heads, mask_empty, precision, out_coords, out_feats, cap_m, num_out, region_of,
                           slot_of);
}

extern "C" int dsvt_pool_counted(dsvt_ctx* ctx, const int32_t* coords, const float* feats, int32_t n,
                                 const int32_t* n_dev, int32_t C, int32_t batch, const int32_t grid[3],
                                 const int32_t pool[3], const void* W_q, const void* W_k, const void* W_v,
                                 const void* W_o, const float* b_q, const float* b_k, const float* b_v,
                                 const float* b_o, const float* slot_pe, int32_t heads, int32_t mask_empty,
                                 int precision, int32_t* out_coords, float* out_feats, int32_t cap_m,
                                 int32_t* num_out, int32_t* region_of, int32_t* slot_of) {
  if (!ctx || !grid || !pool || !num_out || n < 0 || batch < 1 || cap_m < 0 || C < 1 || heads < 1)
    return DSVT_ERR_INVALID_ARG;
  if (precision != DSVT_FP32 && precision != DSVT_BF16_FP32ACC) return DSVT_ERR_INVALID_ARG;
  for (int a = 0; a < 3; ++a)
    if (grid[a] < 1 || pool[a] < 1) return DSVT_ERR_INVALID_ARG;
  if (n > 0 && (!coords || !feats || !out_coords || !out_feats || !W_q || !W_k || !W_v || !W_o))
    return DSVT_ERR_INVALID_ARG;
  if (((uintptr_t)coords & 15) || ((uintptr_t)feats & 15) || ((uintptr_t)out_feats & 15) || ((uintptr_t)out_coords & 15))
    return DSVT_ERR_INVALID_ARG;
  if (C % heads != 0 || C % 8 != 0 || (C / heads) % 4 != 0) return DSVT_ERR_UNSUPPORTED;
  PoolGeom g;
  g.batch = batch; g.gx = grid[0]; g.gy = grid[1]; g.gz = grid[2];
  g.l = pool[0]; g.w = pool[1]; g.h = pool[2];
  g.GX = (int32_t)dsvt_ceil_div(grid[0], pool[0]);
  g.GY = (int32_t)dsvt_ceil_div(grid[1], pool[1]);
  g.GZ = (int32_t)dsvt_ceil_div(grid[2], pool[2]);
  const int64_t nslots = (int64_t)pool[0] * pool[1] * pool[2];
  if (nslots > 32) return DSVT_ERR_UNSUPPORTED;
  g.nslots = (int32_t)nslots;
  const int64_t num_regions = (int64_t)batch * g.GX * g.GY * g.GZ;
  if (num_regions >= (1ll << 31) / nslots) return DSVT_ERR_UNSUPPORTED;
  if (n > ctx->max_voxels || num_regions > ctx->max_windows || C > ctx->max_channels) return DSVT_ERR_CAPACITY;
  cudaStream_t st = ctx->stream;
  if (n == 0) {
    DSVT_CUDA_TRY(ctx, cudaMemsetAsync(num_out, 0, sizeof(int32_t), st));
    return DSVT_OK;
  }
  const size_t cells = (size_t)num_regions * (size_t)nslots;
  if (cells > ctx->cell_map_entries) {  // grow the dense cell map (the one allocation a call may make)
    DSVT_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    if (ctx->cell_map) DSVT_CUDA_TRY(ctx, cudaFree(ctx->cell_map));
    ctx->cell_map = nullptr;
    ctx->cell_map_entries = 0;
    DSVT_CUDA_TRY(ctx, cudaMalloc((void**)&ctx->cell_map, cells * sizeof(int32_t)));
    ctx->cell_map_entries = cells;
  }
  DSVT_CUDA_TRY(ctx, cudaMemsetAsync(ctx->cell_map, 0xFF, cells * sizeof(int32_t), st));
  DSVT_CUDA_TRY(ctx, cudaMemsetAsync(ctx->win_count, 0, sizeof(int32_t) * (size_t)(num_regions + 1), st));
  const unsigned vb = (unsigned)dsvt_ceil_div(n, 256);
  pool_mark_kernel<<<vb, 256, 0, st>>>((const int4*)coords, n, n_dev, g, ctx->cell_map, ctx->win_count, ctx->keys[0], slot_of,
                                       ctx->status);
  DSVT_LAUNCHED(ctx);
  int rc = dsvt_launch_scan_i32(ctx, ctx->win_count, ctx->win_start, num_regions, nullptr);
  if (rc != DSVT_OK) return rc;
  DSVT_CUDA_TRY(ctx, launch_pdl(pool_finish_kernel, dim3(vb), dim3(256), 0, st, n, n_dev, g, (const uint32_t*)ctx->keys[0],
                                (const int32_t*)ctx->win_start, (int32_t)num_regions, cap_m, out_coords, ctx->region_key,
                                region_of, num_out, ctx->status));
  DSVT_LAUNCHED(ctx);
  if (cap_m == 0) return DSVT_OK;

  PoolArgs a;
  a.feats = feats; a.cell_map = ctx->cell_map; a.region_key = ctx->region_key; a.num_out = num_out;
  a.cap_m = cap_m; a.n = n;
  a.W_q = W_q; a.W_k = W_k; a.W_v = W_v; a.W_o = W_o;
  a.b_q = b_q; a.b_k = b_k; a.b_v = b_v; a.b_o = b_o; a.slot_pe = slot_pe;
  a.out_feats = out_feats; a.C = C; a.heads = heads; a.nslots = (int32_t)nslots; a.mask_empty = mask_empty ? 1 : 0;
  // bfloat16 weights, a power-of-two number of slots: the projections on tcgen05
  if (precision == DSVT_BF16_FP32ACC && dsvt_pool_tc_supported(C, heads, (int)nslots)) {
    dsvt_pool_tc_call c;
    c.feats = feats; c.cell_map = ctx->cell_map; c.region_key = ctx->region_key; c.num_out = num_out;
    c.cap_m = cap_m; c.n = n;
    c.W[0] = W_q; c.W[1] = W_k; c.W[2] = W_v; c.W[3] = W_o;
    c.b_q = b_q; c.b_k = b_k; c.b_v = b_v; c.b_o = b_o; c.slot_pe = slot_pe;
    c.out_feats = out_feats; c.C = C; c.heads = heads; c.nslots = (int32_t)nslots; c.mask_empty = mask_empty ? 1 : 0;
    return dsvt_launch_pool_tc(ctx, c);
  }
  // bfloat16 weights, C in {64, 128, 192}, head dim <= 32: other slot counts: the mma.sync kernel
  if (precision == DSVT_BF16_FP32ACC && (C == 64 || C == 128 || C == 192) && heads <= mma_pool::kMaxHeads) {
    a.TM = mma_pool::kRows;
    a.LDQ = 0;
    a.TR = (int32_t)(mma_pool::kRows / nslots);
    if (a.TR > mma_pool::kRegs) a.TR = mma_pool::kRegs;
    const size_t smem = (size_t)mma_pool::make_layout(C).total + 1024;
    int64_t tiles = dsvt_ceil_div(n < cap_m ? n : cap_m, a.TR);
    int64_t gridn = tiles < ctx->sm_count ? tiles : ctx->sm_count;
    if (gridn < 1) gridn = 1;
    cudaError_t e = cudaFuncSetAttribute(mma_pool::pool_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return DSVT_ERR_CUDA; }
    mma_pool::PoolMaps maps;
    const void* wm[4] = {W_q, W_k, W_v, W_o};
    for (int i = 0; i < 4; ++i)
      if (!dsvt_cached_weight_map(ctx, &maps.w[i], wm[i], C, C, C)) return DSVT_ERR_CUDA;
    mma_pool::pool_attn_mma_kernel<<<(unsigned)gridn, mma_pool::kT, smem, st>>>(a, maps, ctx->status);
    DSVT_LAUNCHED(ctx);
    return DSVT_OK;
  }
  a.LDQ = 3 * C + (36 - (3 * C) % 32) % 32;
  static const int kTiles[] = {128, 96, 64, 48, 32};
  a.TM = 0;
  for (int tm : kTiles)
    if (tm >= nslots && tm >= 32 && pool_smem_bytes(tm, C, a.LDQ) <= 227 * 1024) { a.TM = tm; break; }
  if (a.TM == 0) return DSVT_ERR_UNSUPPORTED;
  a.TR = (int32_t)(a.TM / nslots);
  if (a.TR > a.TM / 2) a.TR = a.TM / 2;
  int64_t mmax = n < cap_m ? n : cap_m;
  int64_t gridn = dsvt_ceil_div(mmax, a.TR);
  const int64_t gmax = (int64_t)ctx->sm_count * 16;
  if (gridn > gmax) gridn = gmax;
  if (gridn < 1) gridn = 1;
  if (precision == DSVT_FP32) return launch_pool_rm<float>(ctx, a, (int)gridn);
  return launch_pool_rm<__nv_bfloat16>(ctx, a, (int)gridn);
}
