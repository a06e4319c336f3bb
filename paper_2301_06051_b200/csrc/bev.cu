// Projection of the voxel features to a dense bird's-eye-view map (Sec. 3.1): channel c*Z + z of cell (b, y, x)
// holds feature c of the voxel at (b, x, y, z), zero where the grid is empty.
//
// The map is far larger than the features (168 MB against 25 MB for 32 000 pillars on a 468 x 468 grid), so the
// work is writing the map at HBM speed.  Channels-first output is produced dense: a dense cell -> voxel map is
// filled first (n scattered 4-byte writes), then every block owns 32 consecutive x cells of one (b, z, y) line,
// stages the feature rows of the occupied cells in shared memory and writes one 128-byte line segment per
// channel, zeros included, so the map is written exactly once with full-width stores and needs no memset.
// Channels-last output is one memset and one row copy per voxel.
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
  // line-major: ((b*Z + z)*Y + y)*X + x, the order the dense writer walks
  const size_t cell = (((size_t)c.x * g.Z + c.w) * g.Y + c.z) * g.X + c.y;
  if (atomicExch(&cell_map[cell], i) >= 0) atomicOr(status, DSVT_STATUS_DUPLICATE_CELL);
}

constexpr int kCells = 32;     // x cells per block
constexpr int kThreads = 256;  // 8 warps

// out[b][c*Z + z][y][x]; one block per (line, 32-cell segment), line = (b*Z + z)*Y + y.
__global__ void __launch_bounds__(kThreads)
bev_dense_kernel(const float* __restrict__ feats, const int32_t* __restrict__ cell_map, BevGeom g, int32_t segs,
                 float* __restrict__ out) {
  extern __shared__ __align__(16) float rows[];  // [kCells][C + 1]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seg = blockIdx.x % segs;
  const int64_t line = blockIdx.x / segs;
  const int y = (int)(line % g.Y);
  const int64_t bz = line / g.Y;
  const int z = (int)(bz % g.Z), b = (int)(bz / g.Z);
  const int x0 = seg * kCells;
  const int x = x0 + lane;
  const int v = x < g.X ? cell_map[line * g.X + x] : -1;
  const unsigned occupied = __ballot_sync(0xffffffffu, v >= 0);
  const int C = g.C, ld = C + 1;
  if (occupied) {
    // warp w stages the rows of cells w, w + 8, ...: 128-bit loads, scalar stores (odd row stride: no conflicts later)
    for (int cell = warp; cell < kCells; cell += kThreads / 32) {
      const int vc = __shfl_sync(0xffffffffu, v, cell);
      if (vc < 0) continue;
      const float4* src = reinterpret_cast<const float4*>(feats + (size_t)vc * C);
      for (int c4 = lane; c4 < (C >> 2); c4 += 32) {
        const float4 f = __ldg(src + c4);
        float* d = rows + cell * ld + 4 * c4;
        d[0] = f.x; d[1] = f.y; d[2] = f.z; d[3] = f.w;
      }
    }
    __syncthreads();
  }
  if (x >= g.X) return;
  const size_t plane = (size_t)g.Y * g.X;
  float* dst = out + (((size_t)b * C * g.Z + z) * g.Y + y) * (size_t)g.X + x;  // channel 0*Z + z
  const size_t cstride = plane * g.Z;                                           // from channel c*Z+z to (c+1)*Z+z
  const float* mine = rows + lane * ld;
  if (v >= 0) {
    for (int c = warp; c < C; c += kThreads / 32) __stcs(dst + (size_t)c * cstride, mine[c]);
  } else {
    for (int c = warp; c < C; c += kThreads / 32) __stcs(dst + (size_t)c * cstride, 0.f);
  }
}

// out[b][y][x][c*Z + z]: one warp per voxel (the map was cleared before).
__global__ void bev_rows_kernel(const int4* __restrict__ coords, const float* __restrict__ feats, int32_t n, BevGeom g,
                                const int32_t* __restrict__ cell_map, float* __restrict__ out) {
  const int i = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
  if (i >= n) return;
  const int4 c = coords[i];
  if (c.x < 0 || c.x >= g.B || c.y < 0 || c.y >= g.X || c.z < 0 || c.z >= g.Y || c.w < 0 || c.w >= g.Z) return;
  const size_t cell = (((size_t)c.x * g.Z + c.w) * g.Y + c.z) * g.X + c.y;
  if (cell_map[cell] != i) return;  // of two voxels in one cell, the one the cell map kept
  const int C = g.C;
  float* dst = out + (((size_t)c.x * g.Y + c.z) * g.X + c.y) * (size_t)C * g.Z + c.w;
  const float* src = feats + (size_t)i * C;
  if (g.Z == 1) {
    for (int c4 = lane; c4 < (C >> 2); c4 += 32)
      reinterpret_cast<float4*>(dst)[c4] = __ldg(reinterpret_cast<const float4*>(src) + c4);
  } else {
    for (int ch = lane; ch < C; ch += 32) dst[(size_t)ch * g.Z] = __ldg(src + ch);
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
  const size_t smem = (size_t)kCells * (C + 1) * sizeof(float);
  if (!channels_last && smem > 200 * 1024) return DSVT_ERR_UNSUPPORTED;
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
  if (channels_last) {
    DSVT_CUDA_TRY(ctx, cudaMemsetAsync(out, 0, (size_t)cells * C * sizeof(float), st));
    if (n > 0) {
      bev_rows_kernel<<<(unsigned)dsvt_ceil_div((int64_t)n * 32, 256), 256, 0, st>>>((const int4*)coords, feats, n, g,
                                                                                      ctx->cell_map, out);
      DSVT_LAUNCHED(ctx);
    }
    return DSVT_OK;
  }
  const int32_t segs = (int32_t)dsvt_ceil_div(g.X, kCells);
  const int64_t blocks = (int64_t)batch * g.Z * g.Y * segs;
  if (blocks >= (1ll << 31)) return DSVT_ERR_UNSUPPORTED;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(bev_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return DSVT_ERR_CUDA; }
  }
  bev_dense_kernel<<<(unsigned)blocks, kThreads, smem, st>>>(feats, ctx->cell_map, g, segs, out);
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}
