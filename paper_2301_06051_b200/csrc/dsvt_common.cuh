// Shared declarations of the CUDA library: context layout, error helpers, launch bookkeeping.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dsvt.h"

struct dsvt_map_cache;  // tensor maps of the weight matrices seen so far (layer_tc.cu)
void dsvt_map_cache_destroy(dsvt_map_cache* c);

struct dsvt_ctx {
  int device;
  cudaStream_t stream;
  int64_t max_voxels, max_windows;
  int32_t max_channels;
  int sm_count;
  int layer_ctas;  // cap on the tensor-core layer kernel's grid (0: sm_count)
  int last_cuda_error;
  unsigned attr_flags;  // kernels whose shared-memory attribute has been raised on this context's device
  int64_t launches;
  // one device allocation carved into the arrays below
  void* arena;
  size_t arena_bytes;
  int32_t* status;      // device status word
  uint32_t* keys[2];    // radix sort ping-pong keys        [max_voxels]
  int32_t* vals[2];     // radix sort ping-pong voxel ids   [max_voxels]
  int32_t* hist;        // per-tile digit histograms        [256 * sort tiles + 1]
  int32_t* scan_tmp;    // block sums of the generic scan
  int32_t* win_count;   // [max_windows + 1]  (pooling: region occupancy flags)
  int32_t* win_start;   // [max_windows + 1]  (pooling: region rank)
  int32_t* win_setoff;  // [max_windows + 1]
  int32_t* rowoff_a;    // [4 max_voxels + 4] row offsets + tile plan derived from a caller table
  int32_t* rowoff_b;    // [4 max_voxels + 4]
  int32_t* region_key;  // [max_voxels] pooling: dense region id of each output row
  // partition, bitmap route (bm_words == 0: route not available)
  size_t bm_words;       // bitmap capacity per sort axis, in 32-bit words
  int32_t* bm_zero;      // [2 (max_windows + 1) + 2 bm_words] window counts, duplicate counts, bitmaps
  int32_t* bm_wordrank;  // [2 bm_words] popcount prefix of each bitmap word inside its window
  int32_t* bm_dup;       // [max_voxels] -1, or the voxel's ticket among the duplicates of its window
  // tensor-core layer kernel: tile counter of a launch ([0] next tile, [1] CTAs that have left; zero between
  // launches), per-voxel completion stamps of a chain of layers, and the serial number the stamps are built from
  int32_t* tc_counter;   // [2]
  int32_t* row_stamp;    // [max_voxels]
  uint32_t stamp_serial;
  dsvt_map_cache* maps;
  // pooling: dense cell -> voxel map, grown on demand
  int32_t* cell_map;
  size_t cell_map_entries;
};

#define DSVT_CUDA_TRY(ctx, expr)          \
  do {                                    \
    cudaError_t e_ = (expr);              \
    if (e_ != cudaSuccess) {              \
      (ctx)->last_cuda_error = (int)e_;   \
      return DSVT_ERR_CUDA;               \
    }                                     \
  } while (0)

// Call after every kernel launch: counts it and turns a launch error into DSVT_ERR_CUDA.
#define DSVT_LAUNCHED(ctx)                \
  do {                                    \
    (ctx)->launches += 1;                 \
    cudaError_t e_ = cudaGetLastError();  \
    if (e_ != cudaSuccess) {              \
      (ctx)->last_cuda_error = (int)e_;   \
      return DSVT_ERR_CUDA;               \
    }                                     \
  } while (0)

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may start while its
// predecessor in the stream still runs; it lets its own successor start early and then waits for the predecessor
// (and everything before it) to have completed and flushed.  Both are no-ops in an ordinary launch.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

// A launch that may overlap its predecessor's tail (see pdl_enter).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

static inline int64_t dsvt_ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ---- launchers implemented in the .cu files (all enqueue on ctx->stream) ----
// Exclusive scan; out has count + 1 entries (out[count] = total).  in == out is allowed.
int dsvt_launch_scan_i32(dsvt_ctx* ctx, const int32_t* in, int32_t* out, int64_t count, int32_t* total_out);
int dsvt_launch_sort_pairs(dsvt_ctx* ctx, int32_t n, int key_bits, int* final_buf);
int dsvt_launch_rowoff_from_table(dsvt_ctx* ctx, const int32_t* table, int32_t cap_sets, const int32_t* num_sets,
                                  int32_t set_size, int32_t* rowoff);

int dsvt_launch_tile_plan(dsvt_ctx* ctx, const int32_t* num_sets, int32_t cap_sets, int32_t* set_rowoff);

struct dsvt_fused_args {
  const float* x;
  float* y;
  int32_t n;
  const int32_t* table;
  const int32_t* num_sets;
  const int32_t* rowoff;
  int32_t cap_sets;
  dsvt_layer_params p;
  int32_t attention_only;  // 1: y = attention output (no residual, LN, MLP)
};
int dsvt_launch_layer_fma(dsvt_ctx* ctx, const dsvt_fused_args& a);
// tcgen05 path: bfloat16 weights, C in {64, 128, 192}, head dim in {16, 24, 32}, set size <= 96.
bool dsvt_layer_tc_supported(const dsvt_fused_args& a);
int dsvt_launch_layer_tc(dsvt_ctx* ctx, const dsvt_fused_args& a);
// A chain of layers in one launch: layers[0] reads its x and writes y; layers[i > 0] run in place on that y.  Every
// layer passes dsvt_layer_tc_supported and dsvt_layer_tc_chainable(layers[0], layers[i]); at most
// DSVT_MAX_CHAIN_LAYERS layers; every voxel a later layer reads must be written by the layer before it.
bool dsvt_layer_tc_chainable(const dsvt_fused_args& a, const dsvt_fused_args& b);
int dsvt_launch_layers_tc(dsvt_ctx* ctx, const dsvt_fused_args* layers, int n_layers);
// CUtensorMap (128 bytes, 64-byte aligned) of a row-major bf16 matrix [rows][cols]: boxes of 64 columns x box_rows
// rows, 128-byte swizzle; encoded once per matrix and context.  Returns false if the driver cannot encode it.
bool dsvt_cached_weight_map(dsvt_ctx* ctx, void* tensor_map, const void* w, int rows, int cols, int box_rows);

// Attention-style pooling with the projections on tcgen05 (pool_tc.cu): bfloat16 weights, C / head dim as for the
// layer kernel, a power-of-two number of slots per region (at most 32).  The region bookkeeping (cell map, region
// keys, output count) has been done by the caller.
struct dsvt_pool_tc_call {
  const float* feats;
  const int32_t* cell_map;
  const int32_t* region_key;
  const int32_t* num_out;
  int32_t cap_m, n;
  const void* W[4];  // W_q, W_k, W_v, W_o
  const float *b_q, *b_k, *b_v, *b_o, *slot_pe;
  float* out_feats;
  int32_t C, heads, nslots, mask_empty;
};
bool dsvt_pool_tc_supported(int C, int heads, int nslots);
int dsvt_launch_pool_tc(dsvt_ctx* ctx, const dsvt_pool_tc_call& c);
