// Attention-style 3D pooling (Eq. 6, Eq. 7): dense cell map -> region ranks -> fused
// pad / max-pool / cross-attention kernel.  The region bookkeeping is exact integer work; the
// attention runs on the fp32 FMA pipes with float or bfloat16 weights.
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
__global__ void pool_mark_kernel(const int4* __restrict__ coords, int32_t n, PoolGeom g, int32_t* __restrict__ cell_map,
                                 int32_t* __restrict__ region_flag, uint32_t* __restrict__ vox_region,
                                 int32_t* __restrict__ slot_of, int32_t* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
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
__global__ void pool_finish_kernel(int32_t n, PoolGeom g, const uint32_t* __restrict__ vox_region,
                                   const int32_t* __restrict__ region_rank, int32_t num_regions, int32_t cap_m,
                                   int32_t* __restrict__ out_coords, int32_t* __restrict__ region_key,
                                   int32_t* __restrict__ region_of, int32_t* __restrict__ num_out,
                                   int32_t* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0) {
    const int m = region_rank[num_regions];
    if (m > cap_m) atomicOr(status, DSVT_STATUS_TABLE_OVERFLOW);
    *num_out = min(m, cap_m);
  }
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
  pool_mark_kernel<<<vb, 256, 0, st>>>((const int4*)coords, n, g, ctx->cell_map, ctx->win_count, ctx->keys[0], slot_of,
                                       ctx->status);
  DSVT_LAUNCHED(ctx);
  int rc = dsvt_launch_scan_i32(ctx, ctx->win_count, ctx->win_start, num_regions, nullptr);
  if (rc != DSVT_OK) return rc;
  pool_finish_kernel<<<vb, 256, 0, st>>>(n, g, ctx->keys[0], ctx->win_start, (int32_t)num_regions, cap_m, out_coords,
                                         ctx->region_key, region_of, num_out, ctx->status);
  DSVT_LAUNCHED(ctx);
  if (cap_m == 0) return DSVT_OK;

  PoolArgs a;
  a.feats = feats; a.cell_map = ctx->cell_map; a.region_key = ctx->region_key; a.num_out = num_out;
  a.cap_m = cap_m; a.n = n;
  a.W_q = W_q; a.W_k = W_k; a.W_v = W_v; a.W_o = W_o;
  a.b_q = b_q; a.b_k = b_k; a.b_v = b_v; a.b_o = b_o; a.slot_pe = slot_pe;
  a.out_feats = out_feats; a.C = C; a.heads = heads; a.nslots = (int32_t)nslots; a.mask_empty = mask_empty ? 1 : 0;
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
