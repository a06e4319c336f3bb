// Projection of the voxel features to a dense bird's-eye-view map (Sec. 3.1): channel c*Z + z of cell (b, y, x)
// holds feature c of the voxel at (b, x, y, z), zero where the grid is empty.
//
// The map is far larger than the features (168 MB against 25 MB for 32 000 pillars on a 468 x 468 grid), so the
// work is writing the map at HBM speed.  Both layouts are produced dense: a cell -> voxel map is filled first (n
// scattered 4-byte writes), then one kernel walks the output in its own order, looks every cell up and writes the
// voxel's values or zeros, so the map is written exactly once with coalesced stores and needs no memset; the
// feature rows are read from L2, where the last block left them.
#include "dsvt_common.cuh"

namespace {

struct BevGeom {
  int32_t B, X, Y, Z, C;
};

__global__ void bev_mark_kernel(const int4* __restrict__ coords, int32_t n, BevGeom g, int32_t* __restrict__ cell_map,
                                int32_t* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int4 c = coords[i];
  if (c.x < 0 || c.x >= g.B || c.y < 0 || c.y >= g.X || c.z < 0 || c.z >= g.Y || c.w < 0 || c.w >= g.Z) {
    atomicOr(status, DSVT_STATUS_BAD_COORD);
    return;
  }
  // line-major: ((b*Z + z)*Y + y)*X + x, the order the channels-first writer walks
  const size_t cell = (((size_t)c.x * g.Z + c.w) * g.Y + c.z) * g.X + c.y;
  if (atomicExch(&cell_map[cell], i) >= 0) atomicOr(status, DSVT_STATUS_DUPLICATE_CELL);
}

constexpr int kThreads = 256;
constexpr int kGroup = 8;  // channels per block of the channels-first writer
constexpr int kUnroll = 4;

// Channels-first: out[b][c*Z + z][y][x].  A block owns `lines_per_block` consecutive grid lines (line = (b*Z + z)*Y + y,
// X cells each) and kGroup channels.  A thread takes a cell, reads 32 bytes of the occupying voxel's row (or nothing)
// and writes one value into each of the kGroup channel planes; consecutive lanes are consecutive cells, so every plane
// receives one contiguous run of lines_per_block * X floats per block.  No shared memory, no atomics.
__global__ void __launch_bounds__(kThreads)
bev_planes_kernel(const float* __restrict__ feats, const int32_t* __restrict__ cell_map, BevGeom g, int32_t groups,
                  int32_t lines_per_block, int64_t lines, float* __restrict__ out) {
  const int cg = blockIdx.x % groups;
  const int64_t line0 = (int64_t)(blockIdx.x / groups) * lines_per_block;
  const int c0 = cg * kGroup;
  const bool upper = c0 + 4 < g.C;  // C % 4 == 0: a group holds 8 or 4 channels
  const int64_t nline = min((int64_t)lines_per_block, lines - line0);
  const int cells = (int)(nline * g.X);
  const int32_t* map = cell_map + line0 * g.X;
  const size_t plane = (size_t)g.Y * g.X * g.Z;  // from channel c*Z + z to (c+1)*Z + z
  for (int i0 = threadIdx.x; i0 < cells; i0 += kThreads * kUnroll) {
    int v[kUnroll];
    float4 lo[kUnroll], hi[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int i = i0 + u * kThreads;
      v[u] = i < cells ? __ldg(map + i) : -1;
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      lo[u] = hi[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (v[u] >= 0) {
        const float4* src = reinterpret_cast<const float4*>(feats + (size_t)v[u] * g.C + c0);
        lo[u] = __ldg(src);
        if (upper) hi[u] = __ldg(src + 1);
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int i = i0 + u * kThreads;
      if (i >= cells) continue;
      const int64_t line = line0 + i / g.X;
      const int x = i % g.X;
      const int y = (int)(line % g.Y);
      const int64_t bz = line / g.Y;
      const int z = (int)(bz % g.Z);
      const int64_t b = bz / g.Z;
      float* dst = out + (((size_t)b * g.C + c0) * g.Z + z) * ((size_t)g.Y * g.X) + (size_t)y * g.X + x;
      __stcs(dst, lo[u].x);
      __stcs(dst + plane, lo[u].y);
      __stcs(dst + 2 * plane, lo[u].z);
      __stcs(dst + 3 * plane, lo[u].w);
      if (upper) {
        __stcs(dst + 4 * plane, hi[u].x);
        __stcs(dst + 5 * plane, hi[u].y);
        __stcs(dst + 6 * plane, hi[u].z);
        __stcs(dst + 7 * plane, hi[u].w);
      }
    }
  }
}

// The same for X % 4 == 0: a thread takes four consecutive cells of a line and writes one float4 per channel plane,
// so a warp's store covers 512 contiguous bytes.
__global__ void __launch_bounds__(kThreads)
bev_planes4_kernel(const float* __restrict__ feats, const int32_t* __restrict__ cell_map, BevGeom g, int32_t groups,
                   int32_t lines_per_block, int64_t lines, float* __restrict__ out) {
  const int cg = blockIdx.x % groups;
  const int64_t line0 = (int64_t)(blockIdx.x / groups) * lines_per_block;
  const int c0 = cg * kGroup;
  const bool upper = c0 + 4 < g.C;
  const int64_t nline = min((int64_t)lines_per_block, lines - line0);
  const int quads = (int)(nline * g.X) >> 2;
  const int4* map = reinterpret_cast<const int4*>(cell_map + line0 * g.X);
  const size_t plane = (size_t)g.Y * g.X * g.Z;
  for (int q = threadIdx.x; q < quads; q += kThreads) {
    const int4 v4 = __ldg(map + q);
    const int v[4] = {v4.x, v4.y, v4.z, v4.w};
    float f[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
      if (v[u] >= 0) {
        const float4* src = reinterpret_cast<const float4*>(feats + (size_t)v[u] * g.C + c0);
        lo = __ldg(src);
        if (upper) hi = __ldg(src + 1);
      }
      f[u][0] = lo.x; f[u][1] = lo.y; f[u][2] = lo.z; f[u][3] = lo.w;
      f[u][4] = hi.x; f[u][5] = hi.y; f[u][6] = hi.z; f[u][7] = hi.w;
    }
    const int i = q << 2;
    const int64_t line = line0 + i / g.X;
    const int x = i % g.X;  // a multiple of 4: the four cells lie in one line
    const int y = (int)(line % g.Y);
    const int64_t bz = line / g.Y;
    const int z = (int)(bz % g.Z);
    const int64_t b = bz / g.Z;
    float* dst = out + (((size_t)b * g.C + c0) * g.Z + z) * ((size_t)g.Y * g.X) + (size_t)y * g.X + x;
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j < 4 || upper)
        __stcs(reinterpret_cast<float4*>(dst + (size_t)j * plane), make_float4(f[0][j], f[1][j], f[2][j], f[3][j]));
  }
}

// Channels-last with Z == 1: out[b][y][x][c] is the cell map's order with C floats per cell, so the map is one flat
// array of float4 written front to back; element e belongs to cell e / (C/4).
__global__ void __launch_bounds__(kThreads)
bev_cells_kernel(const float4* __restrict__ feats, const int32_t* __restrict__ cell_map, int32_t C4, int64_t total4,
                 float4* __restrict__ out) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t e0 = (int64_t)blockIdx.x * kThreads + threadIdx.x; e0 < total4; e0 += stride * kUnroll) {
    int v[kUnroll];
    int c4[kUnroll];
    float4 f[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t e = e0 + u * stride;
      v[u] = -1;
      c4[u] = 0;
      if (e < total4) {
        const int64_t cell = e / C4;
        c4[u] = (int)(e - cell * C4);
        v[u] = __ldg(cell_map + cell);
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      f[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (v[u] >= 0) f[u] = __ldg(feats + (size_t)v[u] * C4 + c4[u]);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t e = e0 + u * stride;
      if (e < total4) __stcs(out + e, f[u]);
    }
  }
}

// Channels-last, general Z: out[b][y][x][c*Z + z]; element e = column * (C*Z) + ch, column = (b*Y + y)*X + x.
__global__ void __launch_bounds__(kThreads)
bev_columns_kernel(const float* __restrict__ feats, const int32_t* __restrict__ cell_map, BevGeom g, int64_t total,
                   float* __restrict__ out) {
  const int CH = g.C * g.Z;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < total; e += stride) {
    const int64_t col = e / CH;
    const int ch = (int)(e - col * CH);
    const int c = ch / g.Z, z = ch - c * g.Z;
    const int x = (int)(col % g.X);
    const int64_t by = col / g.X;
    const int y = (int)(by % g.Y);
    const int64_t b = by / g.Y;
    const int v = __ldg(cell_map + ((b * g.Z + z) * g.Y + y) * g.X + x);
    __stcs(out + e, v >= 0 ? __ldg(feats + (size_t)v * g.C + c) : 0.f);
  }
}

}  // namespace

extern "C" int dsvt_bev_scatter(dsvt_ctx* ctx, const int32_t* coords, const float* feats, int32_t n, int32_t C,
                                int32_t batch, const int32_t grid[3], int32_t channels_last, float* out) {
  if (!ctx || !grid || n < 0 || C < 1 || batch < 1 || !out) return DSVT_ERR_INVALID_ARG;
  if (grid[0] < 1 || grid[1] < 1 || grid[2] < 1) return DSVT_ERR_INVALID_ARG;
  if (n > 0 && (!coords || !feats)) return DSVT_ERR_INVALID_ARG;
  if (((uintptr_t)feats & 15) || ((uintptr_t)out & 15) || ((uintptr_t)coords & 15)) return DSVT_ERR_INVALID_ARG;
  if (C % 4 != 0) return DSVT_ERR_UNSUPPORTED;
  if (n > ctx->max_voxels) return DSVT_ERR_CAPACITY;
  BevGeom g;
  g.B = batch; g.X = grid[0]; g.Y = grid[1]; g.Z = grid[2]; g.C = C;
  const int64_t cells = (int64_t)batch * g.X * g.Y * g.Z;
  if (cells >= (1ll << 31)) return DSVT_ERR_UNSUPPORTED;
  cudaStream_t st = ctx->stream;
  if ((size_t)cells > ctx->cell_map_entries) {  // grow the dense cell map (the one allocation a call may make)
    DSVT_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    if (ctx->cell_map) DSVT_CUDA_TRY(ctx, cudaFree(ctx->cell_map));
    ctx->cell_map = nullptr;
    ctx->cell_map_entries = 0;
    DSVT_CUDA_TRY(ctx, cudaMalloc((void**)&ctx->cell_map, (size_t)cells * sizeof(int32_t)));
    ctx->cell_map_entries = (size_t)cells;
  }
  DSVT_CUDA_TRY(ctx, cudaMemsetAsync(ctx->cell_map, 0xFF, (size_t)cells * sizeof(int32_t), st));
  if (n > 0) {
    bev_mark_kernel<<<(unsigned)dsvt_ceil_div(n, 256), 256, 0, st>>>((const int4*)coords, n, g, ctx->cell_map,
                                                                      ctx->status);
    DSVT_LAUNCHED(ctx);
  }
  const int64_t grid_cap = (int64_t)ctx->sm_count * 8 * 4;  // grid-stride kernels: a few waves of resident blocks
  if (channels_last) {
    const int64_t total = cells * C;
    if (g.Z == 1) {
      const int64_t total4 = total / 4;
      int64_t blocks = dsvt_ceil_div(total4, (int64_t)kThreads * kUnroll);
      if (blocks > grid_cap) blocks = grid_cap;
      bev_cells_kernel<<<(unsigned)blocks, kThreads, 0, st>>>((const float4*)feats, ctx->cell_map, C / 4, total4,
                                                             (float4*)out);
    } else {
      int64_t blocks = dsvt_ceil_div(total, kThreads);
      if (blocks > grid_cap) blocks = grid_cap;
      bev_columns_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(feats, ctx->cell_map, g, total, out);
    }
    DSVT_LAUNCHED(ctx);
    return DSVT_OK;
  }
  const int64_t lines = (int64_t)batch * g.Z * g.Y;
  const int32_t groups = (int32_t)dsvt_ceil_div(C, kGroup);
  // whole lines, at most kUnroll cells per thread and block
  const int32_t lines_per_block = g.X >= kThreads * kUnroll ? 1 : (kThreads * kUnroll) / g.X;
  const int64_t blocks = dsvt_ceil_div(lines, lines_per_block) * groups;
  if (blocks >= (1ll << 31)) return DSVT_ERR_UNSUPPORTED;
  if (g.X % 4 == 0)
    bev_planes4_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(feats, ctx->cell_map, g, groups, lines_per_block, lines, out);
  else
    bev_planes_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(feats, ctx->cell_map, g, groups, lines_per_block, lines, out);
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}
