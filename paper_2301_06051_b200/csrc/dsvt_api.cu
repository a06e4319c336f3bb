// Context management and the attention / layer / block entry points of the C ABI.
#include <new>

#include "dsvt_common.cuh"

namespace {

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Carver {
  unsigned char* base;
  size_t off;
  template <typename T>
  T* take(size_t count) {
    off = align_up(off, 256);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

void carve(dsvt_ctx* c, unsigned char* base, size_t* total) {
  Carver k{base, 0};
  const size_t nv = (size_t)c->max_voxels, nw = (size_t)c->max_windows;
  const size_t sort_tiles = (nv + 2047) / 2048 + 1;
  const size_t hist = 256 * sort_tiles + 1;
  size_t longest_scan = hist;
  if (nw + 1 > longest_scan) longest_scan = nw + 1;
  if (nv + 1 > longest_scan) longest_scan = nv + 1;
  c->status = k.take<int32_t>(64);
  c->keys[0] = k.take<uint32_t>(nv);
  c->keys[1] = k.take<uint32_t>(nv);
  c->vals[0] = k.take<int32_t>(nv);
  c->vals[1] = k.take<int32_t>(nv);
  c->hist = k.take<int32_t>(hist);
  c->scan_tmp = k.take<int32_t>(longest_scan / 8192 + 2);
  c->win_count = k.take<int32_t>(nw + 1);
  c->win_start = k.take<int32_t>(nw + 1);
  c->win_setoff = k.take<int32_t>(nw + 1);
  c->rowoff_a = k.take<int32_t>(4 * nv + 4);
  c->rowoff_b = k.take<int32_t>(4 * nv + 4);
  c->region_key = k.take<int32_t>(nv);
  c->bm_words = (size_t)1 << 21;  // 64 Mi keys per sort axis
  c->bm_zero = k.take<int32_t>(2 * (nw + 1) + 2 * c->bm_words);
  c->bm_wordrank = k.take<int32_t>(2 * c->bm_words);
  c->bm_dup = k.take<int32_t>(nv);
  c->tc_counter = k.take<int32_t>(64);
  c->row_stamp = k.take<int32_t>(nv);
  *total = align_up(k.off, 256);
}

int check_layer_shape(const dsvt_ctx* ctx, const dsvt_layer_params& p, bool attention_only) {
  if (p.C < 1 || p.heads < 1 || p.set_size < 1 || p.hidden < 0) return DSVT_ERR_INVALID_ARG;
  if (p.precision != DSVT_FP32 && p.precision != DSVT_BF16_FP32ACC) return DSVT_ERR_INVALID_ARG;
  if (!p.W_qkv || !p.W_o) return DSVT_ERR_INVALID_ARG;
  if (p.C % p.heads != 0 || p.C % 8 != 0 || (p.C / p.heads) % 4 != 0 || p.set_size > 128) return DSVT_ERR_UNSUPPORTED;
  if (!attention_only && p.hidden > 0) {
    if (!p.W_1 || !p.W_2) return DSVT_ERR_INVALID_ARG;
    if (p.hidden % 8 != 0 || p.hidden > 2 * p.C) return DSVT_ERR_UNSUPPORTED;
  }
  if (p.C > ctx->max_channels) return DSVT_ERR_CAPACITY;
  const void* ptrs[] = {p.W_qkv, p.W_o, p.W_1, p.W_2, p.b_qkv, p.b_o, p.b_1, p.b_2, p.pe, p.coords};
  for (const void* q : ptrs)
    if (((uintptr_t)q & 15) != 0) return DSVT_ERR_INVALID_ARG;
  if (p.rpb) {
    if (!p.coords || ((uintptr_t)p.rpb & 3) != 0) return DSVT_ERR_INVALID_ARG;
    int64_t len = p.heads;
    for (int a = 0; a < 3; ++a) {
      if (p.rpb_extent[a] < 1 || p.rpb_extent[a] > (1 << 12)) return DSVT_ERR_INVALID_ARG;
      len *= 2 * p.rpb_extent[a] - 1;
      if (len >= (1ll << 30)) return DSVT_ERR_UNSUPPORTED;
    }
  }
  return DSVT_OK;
}

// Runs one fused layer; derives the row offsets from the table when the caller has none.
int run_layer(dsvt_ctx* ctx, const float* x, int32_t n, const int32_t* table, int32_t cap_sets,
              const int32_t* num_sets, const int32_t* rowoff, const dsvt_layer_params& p, float* y,
              bool attention_only, int32_t* rowoff_scratch) {
  if (n == 0 || cap_sets == 0) return DSVT_OK;
  dsvt_fused_args a;
  a.x = x; a.y = y; a.n = n; a.table = table; a.num_sets = num_sets; a.rowoff = rowoff; a.cap_sets = cap_sets;
  a.p = p;
  a.attention_only = attention_only ? 1 : 0;
  const bool tc = dsvt_layer_tc_supported(a);
  if (!rowoff) {
    int rc = dsvt_launch_rowoff_from_table(ctx, table, cap_sets, num_sets, p.set_size, rowoff_scratch);
    if (rc != DSVT_OK) return rc;
    if (tc) {
      rc = dsvt_launch_tile_plan(ctx, num_sets, cap_sets, rowoff_scratch);
      if (rc != DSVT_OK) return rc;
    }
    a.rowoff = rowoff_scratch;
  }
  if (tc) return dsvt_launch_layer_tc(ctx, a);
  return dsvt_launch_layer_fma(ctx, a);
}

int check_common(const dsvt_ctx* ctx, const float* x, const float* y, int32_t n, const int32_t* table,
                 int32_t cap_sets, const int32_t* num_sets) {
  if (!ctx || n < 0 || cap_sets < 0) return DSVT_ERR_INVALID_ARG;
  if (n > 0 && cap_sets > 0 && (!x || !y || !table || !num_sets)) return DSVT_ERR_INVALID_ARG;
  if (((uintptr_t)x & 15) || ((uintptr_t)y & 15)) return DSVT_ERR_INVALID_ARG;
  if (n > ctx->max_voxels || cap_sets > ctx->max_voxels) return DSVT_ERR_CAPACITY;
  return DSVT_OK;
}


// A chain of layers, layer i on tables[i]: layer 0 reads x and writes y, the later ones run in place on y.
// Consecutive layers of one shape that the tensor-core kernel covers share a launch; the rest run one by one.
int run_layers(dsvt_ctx* ctx, const float* x, int32_t n, int32_t num_layers, const dsvt_table_ref* tables,
               const dsvt_layer_params* params, float* y) {
  dsvt_fused_args chain[DSVT_MAX_CHAIN_LAYERS];
  int len = 0;
  auto flush = [&]() -> int {
    if (len == 0) return DSVT_OK;
    const int rc = dsvt_launch_layers_tc(ctx, chain, len);
    len = 0;
    return rc;
  };
  for (int i = 0; i < num_layers; ++i) {
    const dsvt_table_ref& t = tables[i];
    if (n == 0 || t.cap_sets == 0) continue;
    dsvt_fused_args a;
    a.x = i == 0 ? x : y; a.y = y; a.n = n;
    a.table = t.set_table; a.num_sets = t.num_sets; a.rowoff = t.set_rowoff; a.cap_sets = t.cap_sets;
    a.p = params[i];
    a.attention_only = 0;
    const bool tc = t.set_rowoff != nullptr && dsvt_layer_tc_supported(a);
    if (len > 0 && (!tc || len == DSVT_MAX_CHAIN_LAYERS || !dsvt_layer_tc_chainable(chain[0], a))) {
      const int rc = flush();
      if (rc != DSVT_OK) return rc;
    }
    if (tc) {
      chain[len++] = a;
      continue;
    }
    const int rc = run_layer(ctx, a.x, n, t.set_table, t.cap_sets, t.num_sets, t.set_rowoff, params[i], y, false,
                             (i & 1) ? ctx->rowoff_b : ctx->rowoff_a);
    if (rc != DSVT_OK) return rc;
  }
  return flush();
}

}  // namespace

extern "C" int dsvt_create(dsvt_ctx** out, int device, void* cuda_stream, int64_t max_voxels, int64_t max_windows,
                           int32_t max_channels) {
  if (!out || max_voxels < 1 || max_windows < 1 || max_channels < 1) return DSVT_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    cudaGetLastError();
    return DSVT_ERR_CUDA;
  }
  if (cudaSetDevice(device) != cudaSuccess) return DSVT_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return DSVT_ERR_CUDA;
  if (prop.major != 10) return DSVT_ERR_UNSUPPORTED;  // kernels are built for sm_100a only
  dsvt_ctx* c = new (std::nothrow) dsvt_ctx();
  if (!c) return DSVT_ERR_INVALID_ARG;
  c->device = device;
  c->stream = (cudaStream_t)cuda_stream;
  c->max_voxels = max_voxels;
  c->max_windows = max_windows;
  c->max_channels = max_channels;
  c->sm_count = prop.multiProcessorCount;
  c->layer_ctas = 0;
  c->last_cuda_error = 0;
  c->launches = 0;
  c->cell_map = nullptr;
  c->cell_map_entries = 0;
  c->maps = nullptr;
  c->stamp_serial = 0;
  size_t total = 0;
  carve(c, nullptr, &total);
  cudaError_t e = cudaMalloc(&c->arena, total);
  if (e != cudaSuccess) {
    delete c;
    return e == cudaErrorMemoryAllocation ? DSVT_ERR_CAPACITY : DSVT_ERR_CUDA;
  }
  c->arena_bytes = total;
  carve(c, (unsigned char*)c->arena, &total);
  if (cudaMemsetAsync(c->status, 0, 64 * sizeof(int32_t), c->stream) != cudaSuccess ||
      cudaMemsetAsync(c->tc_counter, 0, 64 * sizeof(int32_t), c->stream) != cudaSuccess ||
      cudaMemsetAsync(c->row_stamp, 0, (size_t)max_voxels * sizeof(int32_t), c->stream) != cudaSuccess) {
    cudaFree(c->arena);
    delete c;
    return DSVT_ERR_CUDA;
  }
  *out = c;
  return DSVT_OK;
}

extern "C" int dsvt_destroy(dsvt_ctx* ctx) {
  if (!ctx) return DSVT_OK;
  cudaSetDevice(ctx->device);
  cudaStreamSynchronize(ctx->stream);
  if (ctx->cell_map) cudaFree(ctx->cell_map);
  cudaFree(ctx->arena);
  if (ctx->maps) dsvt_map_cache_destroy(ctx->maps);
  delete ctx;
  return DSVT_OK;
}

extern "C" int dsvt_status_sync(dsvt_ctx* ctx, int32_t* bits) {
  if (!ctx) return DSVT_ERR_INVALID_ARG;
  int32_t h = 0;
  DSVT_CUDA_TRY(ctx, cudaMemcpyAsync(&h, ctx->status, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
  DSVT_CUDA_TRY(ctx, cudaMemsetAsync(ctx->status, 0, sizeof(int32_t), ctx->stream));
  DSVT_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
  if (bits) *bits = h;
  if (h & DSVT_STATUS_TIMEOUT) return DSVT_ERR_TIMEOUT;
  if (h != 0) return DSVT_ERR_BAD_INPUT;
  return DSVT_OK;
}

extern "C" int dsvt_last_cuda_error(const dsvt_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
extern "C" int64_t dsvt_launch_count(const dsvt_ctx* ctx) { return ctx ? ctx->launches : 0; }
extern "C" int dsvt_set_layer_ctas(dsvt_ctx* ctx, int32_t max_ctas) {
  if (!ctx || max_ctas < 0) return DSVT_ERR_INVALID_ARG;
  ctx->layer_ctas = max_ctas;
  return DSVT_OK;
}

extern "C" const char* dsvt_error_string(int code) {
  switch (code) {
    case DSVT_OK: return "ok";
    case DSVT_ERR_INVALID_ARG: return "invalid argument";
    case DSVT_ERR_CAPACITY: return "beyond the capacity reserved by dsvt_create";
    case DSVT_ERR_UNSUPPORTED: return "shape not supported by the kernels";
    case DSVT_ERR_CUDA: return "CUDA runtime error (see dsvt_last_cuda_error)";
    case DSVT_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case DSVT_ERR_BAD_INPUT: return "bad input detected on the device (see the status bits)";
  }
  return "unknown code";
}

extern "C" int dsvt_set_attention(dsvt_ctx* ctx, const float* feats, int32_t n, int32_t C, const int32_t* set_table,
                                  int32_t cap_sets, const int32_t* num_sets, const int32_t* set_rowoff,
                                  int32_t set_size, const void* W_qkv, const float* b_qkv, const void* W_o,
                                  const float* b_o, int32_t heads, const float* pe, int precision, float* out) {
  return dsvt_set_attention_rpb(ctx, feats, n, C, set_table, cap_sets, num_sets, set_rowoff, set_size, W_qkv, b_qkv,
                                W_o, b_o, heads, pe, nullptr, nullptr, nullptr, precision, out);
}

extern "C" int dsvt_set_attention_rpb(dsvt_ctx* ctx, const float* feats, int32_t n, int32_t C,
                                      const int32_t* set_table, int32_t cap_sets, const int32_t* num_sets,
                                      const int32_t* set_rowoff, int32_t set_size, const void* W_qkv,
                                      const float* b_qkv, const void* W_o, const float* b_o, int32_t heads,
                                      const float* pe, const float* rpb, const int32_t* coords,
                                      const int32_t rpb_extent[3], int precision, float* out) {
  int rc = check_common(ctx, feats, out, n, set_table, cap_sets, num_sets);
  if (rc != DSVT_OK) return rc;
  if (n > 0 && feats == out) return DSVT_ERR_INVALID_ARG;
  dsvt_layer_params p = {};
  p.C = C; p.heads = heads; p.hidden = 0; p.set_size = set_size; p.precision = precision; p.ln_eps = 0.f;
  p.W_qkv = W_qkv; p.W_o = W_o; p.b_qkv = b_qkv; p.b_o = b_o; p.pe = pe;
  if (rpb) {
    if (!rpb_extent) return DSVT_ERR_INVALID_ARG;
    p.rpb = rpb; p.coords = coords;
    for (int a = 0; a < 3; ++a) p.rpb_extent[a] = rpb_extent[a];
  }
  rc = check_layer_shape(ctx, p, true);
  if (rc != DSVT_OK) return rc;
  return run_layer(ctx, feats, n, set_table, cap_sets, num_sets, set_rowoff, p, out, true, ctx->rowoff_a);
}

extern "C" int dsvt_layer(dsvt_ctx* ctx, const float* x, int32_t n, const int32_t* set_table, int32_t cap_sets,
                          const int32_t* num_sets, const int32_t* set_rowoff, const dsvt_layer_params* params,
                          float* y) {
  if (!params) return DSVT_ERR_INVALID_ARG;
  int rc = check_common(ctx, x, y, n, set_table, cap_sets, num_sets);
  if (rc != DSVT_OK) return rc;
  rc = check_layer_shape(ctx, *params, false);
  if (rc != DSVT_OK) return rc;
  return run_layer(ctx, x, n, set_table, cap_sets, num_sets, set_rowoff, *params, y, false, ctx->rowoff_a);
}

extern "C" int dsvt_layers(dsvt_ctx* ctx, const float* x, int32_t n, int32_t num_layers, const dsvt_table_ref* tables,
                           const dsvt_layer_params* params, float* y) {
  if (!ctx || num_layers < 0 || (num_layers > 0 && (!tables || !params))) return DSVT_ERR_INVALID_ARG;
  for (int i = 0; i < num_layers; ++i) {
    int rc = check_common(ctx, x, y, n, tables[i].set_table, tables[i].cap_sets, tables[i].num_sets);
    if (rc != DSVT_OK) return rc;
    rc = check_layer_shape(ctx, params[i], false);
    if (rc != DSVT_OK) return rc;
    if (params[i].C != params[0].C) return DSVT_ERR_INVALID_ARG;
  }
  return run_layers(ctx, x, n, num_layers, tables, params, y);
}

extern "C" int dsvt_block(dsvt_ctx* ctx, const float* x, int32_t n, const int32_t* table_axis0, int32_t cap_sets0,
                          const int32_t* num_sets0, const int32_t* set_rowoff0, const int32_t* table_axis1,
                          int32_t cap_sets1, const int32_t* num_sets1, const int32_t* set_rowoff1,
                          const dsvt_layer_params layers[2], float* y) {
  if (!layers) return DSVT_ERR_INVALID_ARG;
  // X-axis layer writes y (every voxel is in one set, so every row of y is produced); the Y-axis
  // layer then runs in place on y.
  const dsvt_table_ref tables[2] = {{table_axis0, cap_sets0, num_sets0, set_rowoff0},
                                    {table_axis1, cap_sets1, num_sets1, set_rowoff1}};
  return dsvt_layers(ctx, x, n, 2, tables, layers, y);
}
