/*
 * dsvt.h -- C ABI of the DSVT dynamic sparse window attention library for NVIDIA B200 (sm_100a).
 *
 * The library implements the hot path of the DSVT 3D backbone (arXiv 2301.06051):
 * rotated set partitioning (Sec. 3.2, Eq. 1-3), batched set attention (Eq. 4-5), the DSVT
 * layer and block (Eq. 5, Appendix B.1.1), the attention-style 3D pooling (Eq. 6-7) and the
 * projection of the voxel features to a bird's-eye-view map (Sec. 3.1).
 *
 * Conventions that hold for every call unless a comment says otherwise:
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library reads / writes it
 *     only during the call's kernels and keeps no reference afterwards.
 *   - `grid`, `window`, `pool` (3 x int32) and the parameter structs are HOST pointers, read
 *     before the call returns.
 *   - Calls are asynchronous: kernels are enqueued on the CUDA stream given to dsvt_create and
 *     the call returns without synchronising.  Counts produced on the device (`num_sets`,
 *     `num_out`) stay on the device.
 *   - Return value: DSVT_OK or a negative DSVT_ERR_* code for errors the host can see (bad
 *     arguments, unsupported shapes, workspace too small, CUDA launch errors).  Errors only the
 *     device can see (a coordinate outside the grid, a table index outside [0, n), a table
 *     larger than its capacity, two voxels in one cell) never trap: the offending item is
 *     clamped or skipped, a bit is set in the context's device status word, and
 *     dsvt_status_sync reports it.
 *   - No call throws, aborts, or frees caller memory.
 *   - Matrices are row-major; a linear map is y = W x + b with W stored [out][in].
 *   - precision = DSVT_FP32: weights are float, arithmetic is fp32 throughout.
 *     precision = DSVT_BF16_FP32ACC: weights are bfloat16 (16-bit storage); products
 *     accumulate in fp32; residual stream, LayerNorm, softmax and GELU are fp32.
 *     Features (x, y, feats, out) and biases / LayerNorm parameters are always float.
 */
#ifndef DSVT_H_
#define DSVT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DSVT_OK 0
#define DSVT_ERR_INVALID_ARG (-1) /* NULL where data is required, negative size, axis not 0/1, ... */
#define DSVT_ERR_CAPACITY (-2)    /* n, window count or channel count beyond what dsvt_create reserved */
#define DSVT_ERR_UNSUPPORTED (-3) /* shape the kernels do not cover (see each call) */
#define DSVT_ERR_CUDA (-4)        /* a CUDA runtime call failed; dsvt_last_cuda_error gives the code */
#define DSVT_ERR_TIMEOUT (-5)     /* a bounded device-side wait expired (reported by dsvt_status_sync) */
#define DSVT_ERR_BAD_INPUT (-6)   /* device-detected bad data (reported by dsvt_status_sync) */

/* Flag on the tile count of a set_rowoff buffer's tile plan (see dsvt_partition). */
#define DSVT_PLAN_PACKED 0x40000000

#define DSVT_FP32 0
#define DSVT_BF16_FP32ACC 1

/* Bits of the device status word returned through dsvt_status_sync's `bits`. */
#define DSVT_STATUS_BAD_COORD 1      /* coordinate or batch index outside the grid (clamped) */
#define DSVT_STATUS_TABLE_OVERFLOW 2 /* more sets / outputs than the caller's capacity (excess dropped) */
#define DSVT_STATUS_BAD_INDEX 4      /* set table entry outside [0, n) (slot skipped) */
#define DSVT_STATUS_DUPLICATE_CELL 8 /* two voxels in the same cell (pooling keeps one of them) */
#define DSVT_STATUS_TIMEOUT 16       /* a bounded wait inside a kernel expired */

typedef struct dsvt_ctx dsvt_ctx; /* opaque: device workspace, stream, device status word */

/*
 * Creates a context on CUDA device `device` whose kernels run on `cuda_stream` (a cudaStream_t;
 * NULL = the legacy default stream).  Reserves all workspace up front for calls with at most
 * `max_voxels` voxels, `max_windows` windows (or pooling regions) per call and `max_channels`
 * feature channels; later calls allocate nothing, except dsvt_pool, which grows its dense cell
 * map once if a call's grid has more cells than any earlier call.
 * The context must be used by one host thread at a time.
 */
int dsvt_create(dsvt_ctx** out, int device, void* cuda_stream, int64_t max_voxels, int64_t max_windows,
                int32_t max_channels);
int dsvt_destroy(dsvt_ctx* ctx);

/* Synchronises the context's stream, copies the device status word to *bits (may be NULL), clears
 * it, and returns DSVT_OK, DSVT_ERR_TIMEOUT, DSVT_ERR_BAD_INPUT or DSVT_ERR_CUDA. */
int dsvt_status_sync(dsvt_ctx* ctx, int32_t* bits);
/* The cudaError_t of the most recent failed runtime call on this context (0 if none). */
int dsvt_last_cuda_error(const dsvt_ctx* ctx);
/* Static, NUL-terminated description of a DSVT_* return code. */
const char* dsvt_error_string(int code);
/* Number of kernels this context has launched since it was created. */
int64_t dsvt_launch_count(const dsvt_ctx* ctx);
/* Caps the number of persistent CTAs (one per SM) the tensor-core layer kernel is launched with on this
 * context: max_ctas >= 1, or 0 for "as many as the device has SMs" (the default).  A context that shares the
 * GPU with other contexts' launches (several frames in flight on several streams) runs its tiles on fewer
 * CTAs, each taking more tiles, so that a launch's set-up is spread over more work and launches of different
 * frames run side by side.  No counterpart in the paper (a launch parameter).  Returns DSVT_ERR_INVALID_ARG
 * for a NULL context or a negative value. */
int dsvt_set_layer_ctas(dsvt_ctx* ctx, int32_t max_ctas);

/*
 * Rotated set partition: Sec. 3.2 "Dynamic set partition" (window partition, Eq. 1 inner-window
 * id from a sorting strategy, Eq. 2 number of sets, Eq. 3 set index rule) for one sort axis.
 *
 *   coords      int32 [n][4] = (b, x, y, z), 16-byte aligned; 0 <= b < batch, 0 <= x < grid[0], ...
 *   grid        cells per axis (x, y, z); window = (L, W, H); windows start at cell 0 and do not
 *               cross frames.  Window id = ((b*nWx + x/L)*nWy + y/W)*nWz + z/H, nW* = ceil(grid/window).
 *   axis        0: X main order, voxels of a window ordered by (x, y, z) of their in-window
 *               offsets; 1: Y main order, ordered by (y, x, z).  Voxels occupy distinct cells (the
 *               output of voxelisation).  Two voxels in one cell are an input error: every voxel
 *               still lands in exactly one set of its window, but the later arrivals are ranked
 *               behind the window's other voxels and DSVT_STATUS_DUPLICATE_CELL is raised (calls
 *               whose key space exceeds the context's 64 Mi-key bitmap fall back to a stable sort,
 *               which keeps equal keys in index order and raises nothing).
 *   set_table   out, int32 [cap_sets][set_size]: row s = the voxel indices of one set, slot k holding
 *               the voxel of inner-window rank floor((j*set_size + k) * N / (S*set_size)) (exact
 *               integer floor), j = the set's number inside its window.  Rows are ordered by
 *               ascending window id, then j.  Rows [0, *num_sets) are written.
 *   num_sets    out, device int32: total number of sets.
 *   set_rowoff  out, optional (NULL to skip), int32 [4 * cap_sets + 4].  Entries [0, cap_sets]:
 *               set_rowoff[s] = number of distinct voxels in the sets before s; entry [*num_sets] = n.
 *               Entries from [cap_sets + 1] on: a tile plan for the tensor-core layer kernel, which
 *               works on tiles of whole sets with at most 128 distinct rows (the sets of Eq. 3 are
 *               independent of one another, so any of them may share a tile).  Entry [cap_sets + 1]:
 *               -1 = no plan; T = T tiles in table order, tile t holding the sets
 *               [e[t], e[t + 1]) with e = entries [cap_sets + 2, cap_sets + 2 + T];
 *               T | DSVT_PLAN_PACKED = T tiles over a reordering of the sets that fills the tiles
 *               better: tile t holds the sets order[p] for p in [e[t], e[t + 1]), with
 *               order = entries [2 cap_sets + 3, 3 cap_sets + 3) a permutation of the sets and
 *               entries [3 cap_sets + 3, 4 cap_sets + 4) the number of distinct voxels in the sets
 *               before position p of that order.  Passing the buffer on to dsvt_set_attention /
 *               dsvt_layer / dsvt_block / dsvt_layers saves them two passes over the table.  A caller
 *               that fills the row offsets by hand sets entry [cap_sets + 1] to -1 (and may then
 *               pass 2 * cap_sets + 3 entries only).
 *   perm        out, optional, int32 [n]: voxel indices in (window, inner-window) sorted order.
 *   win_start, win_setoff   out, optional, int32 [num_windows + 1]: exclusive prefix sums of the
 *               per-window voxel counts / set counts over ALL windows (empty ones included).
 *   win_count   out, optional, int32 [num_windows].
 *
 * Needs n <= max_voxels, num_windows <= max_windows and num_windows * L*W*H < 2^32
 * (else DSVT_ERR_CAPACITY / DSVT_ERR_UNSUPPORTED).  cap_sets = n is always enough; if *num_sets
 * would exceed cap_sets the excess rows are dropped and DSVT_STATUS_TABLE_OVERFLOW is raised.
 * n = 0 is valid and yields *num_sets = 0.
 */
int dsvt_partition(dsvt_ctx* ctx, const int32_t* coords, int32_t n, int32_t batch, const int32_t grid[3],
                   const int32_t window[3], int32_t set_size, int32_t axis, int32_t* set_table, int32_t cap_sets,
                   int32_t* num_sets, int32_t* set_rowoff, int32_t* perm, int32_t* win_start, int32_t* win_count,
                   int32_t* win_setoff);

/*
 * Both rotated partitions of one DSVT block (Sec. 3.2, "Rotated set attention": X main order for
 * the first layer, Y main order for the second) in one pass: the two axes share the window ids,
 * the per-window counts and the launches.  Arguments as for dsvt_partition; set_table, num_sets,
 * set_rowoff and perm are HOST arrays of two device pointers, entry 0 for axis 0 and entry 1 for
 * axis 1 (set_rowoff, perm or their entries may be NULL; both num_sets entries are required and
 * receive the same value).  The results equal those of two dsvt_partition calls.
 */
int dsvt_partition_rotated(dsvt_ctx* ctx, const int32_t* coords, int32_t n, int32_t batch, const int32_t grid[3],
                           const int32_t window[3], int32_t set_size, int32_t* const set_table[2],
                           int32_t cap_sets, int32_t* const num_sets[2], int32_t* const set_rowoff[2],
                           int32_t* const perm[2], int32_t* win_start, int32_t* win_count, int32_t* win_setoff);

/*
 * dsvt_partition_rotated with the window cut displaced by `shift` cells: Sec. 3.2, "Hybrid window partition"
 * (the windows are re-cut between consecutive blocks with the window shifting of Swin, and with another
 * window size; `window` is a per-call argument anyway).  A voxel at cell (x, y, z) lies in the window that
 * holds cell (x + shift[0], y + shift[1], z + shift[2]) of the unshifted cut: window id =
 * ((b*nWx + (x+sx)/L)*nWy + (y+sy)/W)*nWz + (z+sz)/H with nW* = ceil((grid + shift) / window), in-window
 * offsets ((x+sx) mod L, ...).  0 <= shift[a] < window[a] (else DSVT_ERR_INVALID_ARG); shift NULL = no shift.
 * The window arrays have batch*nWx*nWy*nWz (+ 1) entries, and that count must fit max_windows.  Everything
 * else is dsvt_partition_rotated.
 */
int dsvt_partition_shifted(dsvt_ctx* ctx, const int32_t* coords, int32_t n, int32_t batch, const int32_t grid[3],
                           const int32_t window[3], const int32_t shift[3], int32_t set_size,
                           int32_t* const set_table[2], int32_t cap_sets, int32_t* const num_sets[2],
                           int32_t* const set_rowoff[2], int32_t* const perm[2], int32_t* win_start,
                           int32_t* win_count, int32_t* win_setoff);

/*
 * dsvt_partition_shifted for a frame whose voxel count lives on the device (Sec. 3.2 and Sec. 3.3: the stage after
 * an attention-style pooling partitions the pooled voxels, whose number the pooling has just written to device
 * memory).  The call takes the first min(n, *n_dev) voxels of coords; n is the capacity the launches are sized by.
 * n_dev NULL gives dsvt_partition_shifted exactly.  Everything downstream (num_sets, the tables, the row offsets
 * whose last entry is the voxel count) follows the device count, so dsvt_layers / dsvt_block can run on the tables
 * with n = the capacity and no host read-back in between.  Needs the bitmap route (key space within 64 Mi keys);
 * otherwise DSVT_ERR_UNSUPPORTED.
 */
int dsvt_partition_counted(dsvt_ctx* ctx, const int32_t* coords, int32_t n, const int32_t* n_dev, int32_t batch,
                           const int32_t grid[3], const int32_t window[3], const int32_t shift[3], int32_t set_size,
                           int32_t* const set_table[2], int32_t cap_sets, int32_t* const num_sets[2],
                           int32_t* const set_rowoff[2], int32_t* const perm[2], int32_t* win_start,
                           int32_t* win_count, int32_t* win_setoff);

/*
 * dsvt_partition without any allocation.  (The paper has no counterpart: this is a deployment
 * variant of dsvt_partition, computing exactly the same table.)
 *
 * For callers that may not allocate device memory: a perception loop whose memory was fixed at
 * start-up, a host framework whose allocator owns the device, a plug-in that only receives a
 * stream and buffers.  Such callers cannot use dsvt_create, which reserves its workspace with
 * cudaMalloc.  Here the workspace (sort buffers, digit histograms, per-window arrays) is a fixed
 * array inside the library image, about 1.9 MB, which every GPU that loads the library holds until
 * the process exits.  The call makes no cudaMalloc / cudaFree and uses no allocating library.
 *
 *   cuda_stream   cudaStream_t of the CURRENT device (NULL = legacy default stream); kernels are
 *                 enqueued there and the call does not synchronise.
 *   coords, n, batch, grid, window, set_size, axis, set_table, cap_sets, num_sets, set_rowoff
 *                 exactly as for dsvt_partition (device pointers owned by the caller).
 *   status_bits   optional device int32: receives the DSVT_STATUS_* bits of this call.
 *   cuda_error    optional HOST int32: the cudaError_t behind a DSVT_ERR_CUDA return.
 *
 * Limits: n <= DSVT_NOALLOC_MAX_VOXELS and at most DSVT_NOALLOC_MAX_WINDOWS windows, otherwise
 * DSVT_ERR_CAPACITY is returned and nothing is launched.
 * The first call on each device looks up the array's device address (once, with that device
 * current); make that first call before starting any stream capture.  That first call may also
 * make the driver load the library's code onto the device (the one time the call can change the
 * device's free memory), and the address it caches does not survive a cudaDeviceReset.
 * All calls on a device share the one array, which keeps the previous call's contents (the call
 * clears what has to start at zero): two calls whose kernels overlap on the GPU -- different
 * streams, or threads -- race on it.  Serialise them on one stream.
 */
#define DSVT_NOALLOC_MAX_VOXELS 65536
#define DSVT_NOALLOC_MAX_WINDOWS 65536
int dsvt_partition_noalloc(void* cuda_stream, const int32_t* coords, int32_t n, int32_t batch, const int32_t grid[3],
                           const int32_t window[3], int32_t set_size, int32_t axis, int32_t* set_table,
                           int32_t cap_sets, int32_t* num_sets, int32_t* set_rowoff, int32_t* status_bits,
                           int32_t* cuda_error);

/*
 * Batched set attention: Eq. 4 (INDEX gather of each set's members) followed by the multi-head
 * self attention of Eq. 5 inside every set, output projection, and scatter back to voxels.
 * Slot k of a table row is a duplicate, and is masked as a key and not written back, iff k > 0 and
 * row[k] == row[k-1] (Sec. 3.2: duplicated voxels are masked).
 *
 *   feats, out  float [n][C], 16-byte aligned; out may not alias feats.  Rows of voxels that occur in
 *               no table row are left untouched.  A voxel should occur in at most one set.
 *   set_table   int32 [cap_sets][set_size]; num_sets: device int32, *num_sets <= cap_sets <= max_voxels.
 *   set_rowoff  as produced by dsvt_partition, or NULL (then it is derived from the table).
 *   W_qkv       [3C][C]: rows [0,C) = query map, [C,2C) = key map, [2C,3C) = value map.
 *   W_o         [C][C].  b_qkv float [3C] or NULL, b_o float [C] or NULL.
 *   heads       head h owns channels [h*d, (h+1)*d), d = C / heads; logits are scaled by 1/sqrt(d).
 *   pe          optional float [n][C] positional term, added to the input of the query and key maps only.
 *
 * Needs C % 8 == 0, (C/heads) % 4 == 0, set_size <= 128 (else DSVT_ERR_UNSUPPORTED).
 */
int dsvt_set_attention(dsvt_ctx* ctx, const float* feats, int32_t n, int32_t C, const int32_t* set_table,
                       int32_t cap_sets, const int32_t* num_sets, const int32_t* set_rowoff, int32_t set_size,
                       const void* W_qkv, const float* b_qkv, const void* W_o, const float* b_o, int32_t heads,
                       const float* pe, int precision, float* out);

/*
 * dsvt_set_attention with a relative position bias on the logits (see dsvt_layer_params for the
 * table layout and the meaning of rpb, coords and rpb_extent; rpb_extent is a HOST pointer).
 * rpb == NULL gives dsvt_set_attention exactly.
 */
int dsvt_set_attention_rpb(dsvt_ctx* ctx, const float* feats, int32_t n, int32_t C, const int32_t* set_table,
                           int32_t cap_sets, const int32_t* num_sets, const int32_t* set_rowoff, int32_t set_size,
                           const void* W_qkv, const float* b_qkv, const void* W_o, const float* b_o, int32_t heads,
                           const float* pe, const float* rpb, const int32_t* coords, const int32_t rpb_extent[3],
                           int precision, float* out);

/* Parameters of one DSVT layer (Appendix B.1.1).  hidden == 0 drops the MLP; ln1_g == NULL /
 * ln2_g == NULL drops the corresponding LayerNorm.  hidden <= 2C. */
typedef struct dsvt_layer_params {
  int32_t C, heads, hidden, set_size, precision;
  float ln_eps;
  const void* W_qkv; /* [3C][C] */
  const void* W_o;   /* [C][C] */
  const void* W_1;   /* [hidden][C] */
  const void* W_2;   /* [C][hidden] */
  const float *b_qkv, *b_o, *b_1, *b_2;       /* each may be NULL (= 0) */
  const float *ln1_g, *ln1_b, *ln2_g, *ln2_b; /* float [C]; *_b may be NULL */
  const float* pe;                            /* float [n][C] or NULL */
  /* Relative position bias, the Swin transformer's mechanism that the text after Eq. 5 names for
   * PE(.): rpb float [heads][(2L-1)(2W-1)(2H-1)] or NULL.  The scaled logit of (query, key) in head
   * h gets rpb[h][((dx+L-1)(2W-1) + (dy+W-1))(2H-1) + (dz+H-1)] added, with (dx, dy, dz) =
   * coords[query] - coords[key].  coords: int32 [n][4] = (b, x, y, z), required with rpb.
   * rpb_extent = (L, W, H): the window extent the table covers, at least the window the set
   * table was cut with.  A set whose members are spread wider raises DSVT_STATUS_BAD_INDEX and
   * its out-of-table pairs read a clamped entry. */
  const float* rpb;
  const int32_t* coords;
  int32_t rpb_extent[3];
} dsvt_layer_params;

/*
 * One DSVT layer (Eq. 5 with Appendix B.1.1): x1 = LN1(x + MHSA_sets(x));
 * y = LN2(x1 + W_2 gelu(W_1 x1 + b_1) + b_2), gelu(t) = t/2 (1 + erf(t/sqrt 2)); LayerNorm over the
 * C channels with biased variance.  y may alias x (each voxel belongs to one set, and a set is
 * processed by one thread block).  Rows of voxels in no set are left untouched in y.
 */
int dsvt_layer(dsvt_ctx* ctx, const float* x, int32_t n, const int32_t* set_table, int32_t cap_sets,
               const int32_t* num_sets, const int32_t* set_rowoff, const dsvt_layer_params* params, float* y);

/*
 * One DSVT block (Eq. 5): the layer with the X-axis table, then the layer with the Y-axis table.
 * layers: HOST array of two parameter structs.  y may alias x.  Every voxel must be covered by
 * both tables (true for tables made by dsvt_partition).  Same as dsvt_layers with two layers.
 */
int dsvt_block(dsvt_ctx* ctx, const float* x, int32_t n, const int32_t* table_axis0, int32_t cap_sets0,
               const int32_t* num_sets0, const int32_t* set_rowoff0, const int32_t* table_axis1, int32_t cap_sets1,
               const int32_t* num_sets1, const int32_t* set_rowoff1, const dsvt_layer_params layers[2], float* y);

/*
 * A chain of DSVT layers, e.g. all blocks of a backbone stage (Sec. 3.2: the blocks are stacked, Eq. 5 gives the
 * two layers of one): layer 0 reads x and writes y, every later layer runs in place on y; layer i runs on
 * tables[i] with params[i] (for blocks that share their windows: the X-axis table, the Y-axis table, the X-axis
 * table, ...; with hybrid windows each block brings its own pair).  The result equals num_layers dsvt_layer
 * calls.  Consecutive layers of one shape that the tensor-core kernel covers (bfloat16 weights, see dsvt_layer)
 * run as ONE launch of up to DSVT_MAX_CHAIN_LAYERS layers: thread blocks draw row tiles of layer after layer
 * from a counter, and a tile of layer i starts once the rows it reads carry layer i - 1's completion stamp, so
 * the chain pays a launch's start-up and tail once.  Every voxel that a later layer reads must be covered by the
 * table of the layer before it (true for tables made by dsvt_partition from one set of coordinates; otherwise a
 * bounded wait expires and DSVT_STATUS_TIMEOUT is raised).  All layers have the same C.
 *
 *   tables, params   HOST arrays of num_layers entries; the pointers inside are device pointers.
 *   set_rowoff       as produced by dsvt_partition, or NULL (derived from the table; such a layer runs alone).
 */
#define DSVT_MAX_CHAIN_LAYERS 16
typedef struct dsvt_table_ref {
  const int32_t* set_table; /* int32 [cap_sets][set_size] */
  int32_t cap_sets;
  const int32_t* num_sets;   /* device int32 */
  const int32_t* set_rowoff; /* int32 [4 * cap_sets + 4] or NULL */
} dsvt_table_ref;
int dsvt_layers(dsvt_ctx* ctx, const float* x, int32_t n, int32_t num_layers, const dsvt_table_ref* tables,
                const dsvt_layer_params* params, float* y);

/*
 * Attention-style 3D pooling (Eq. 6, Eq. 7).  Region of voxel (b,x,y,z): (b, x/l, y/w, z/h) with
 * pool = (l, w, h); slot inside the region: ((x%l)*w + y%w)*h + z%h.  Every non-empty region yields
 * one output voxel; outputs are ordered by ascending ((b*GX + X)*GY + Y)*GZ + Z, G* = ceil(grid/pool).
 * The region is padded to l*w*h slots with zero rows; P = channel-wise max over the slots (Eq. 6);
 * output = W_o MHA(q = W_q P + b_q; k_s = W_k (p_s + e_s) + b_k; v_s = W_v (p_s + e_s) + b_v) + b_o
 * (Eq. 7), e_s = slot_pe[s] or 0.  mask_empty = 0: max and keys/values run over all l*w*h padded
 * slots; mask_empty = 1: over the non-empty slots only.
 *
 *   out_coords  int32 [cap_m][4] = (b, X, Y, Z); out_feats float [cap_m][C]; num_out device int32.
 *   region_of   optional int32 [n]: output row of each input voxel; slot_of optional int32 [n].
 *   cap_m = n is always enough; excess outputs are dropped with DSVT_STATUS_TABLE_OVERFLOW.
 *
 * Needs l*w*h <= 32, the number of regions <= max_windows, and the channel limits of
 * dsvt_set_attention.
 */
int dsvt_pool(dsvt_ctx* ctx, const int32_t* coords, const float* feats, int32_t n, int32_t C, int32_t batch,
              const int32_t grid[3], const int32_t pool[3], const void* W_q, const void* W_k, const void* W_v,
              const void* W_o, const float* b_q, const float* b_k, const float* b_v, const float* b_o,
              const float* slot_pe, int32_t heads, int32_t mask_empty, int precision, int32_t* out_coords,
              float* out_feats, int32_t cap_m, int32_t* num_out, int32_t* region_of, int32_t* slot_of);

/*
 * dsvt_pool for an input whose voxel count lives on the device (the second and later poolings of a backbone with
 * several pooled stages, Appendix B.1.1): the first min(n, *n_dev) voxels are pooled; n is the capacity.  n_dev
 * NULL gives dsvt_pool exactly.
 */
int dsvt_pool_counted(dsvt_ctx* ctx, const int32_t* coords, const float* feats, int32_t n, const int32_t* n_dev,
                      int32_t C, int32_t batch, const int32_t grid[3], const int32_t pool[3], const void* W_q,
                      const void* W_k, const void* W_v, const void* W_o, const float* b_q, const float* b_k,
                      const float* b_v, const float* b_o, const float* slot_pe, int32_t heads, int32_t mask_empty,
                      int precision, int32_t* out_coords, float* out_feats, int32_t cap_m, int32_t* num_out,
                      int32_t* region_of, int32_t* slot_of);

/*
 * Projection of the backbone's voxel features to a dense bird's-eye-view map (Sec. 3.1).  The z
 * cells of a column are stacked into channels: channel c*Z + z of cell (b, y, x) is feats[i][c] of
 * the voxel i at (b, x, y, z), and 0 where the grid holds no voxel; (X, Y, Z) = grid.
 *
 *   coords  int32 [n][4] = (b, x, y, z); feats float [n][C], 16-byte aligned, C % 4 == 0.
 *   out     float, 16-byte aligned, written in full:
 *           channels_last == 0: [batch][C*Z][Y][X] (rows of the image run along y, columns along x);
 *           channels_last == 1: [batch][Y][X][C*Z].
 *
 * A voxel outside the grid is skipped with DSVT_STATUS_BAD_COORD; of two voxels in one cell one is
 * kept and DSVT_STATUS_DUPLICATE_CELL is raised.  batch*X*Y*Z must be below 2^31.  The call may
 * grow the context's dense cell map (one cudaMalloc, after a stream synchronise) the first time a
 * grid of that size is seen.
 */
int dsvt_bev_scatter(dsvt_ctx* ctx, const int32_t* coords, const float* feats, int32_t n, int32_t C, int32_t batch,
                     const int32_t grid[3], int32_t channels_last, float* out);

/*
 * A measurement aid (the paper has no counterpart): launches a kernel of `blocks` x `threads` threads that
 * each run `iters` rounds of eight independent fp32 fused multiply-adds and nothing else, on the context's stream.
 * A benchmark times it to learn the FP32 FMA rate of the device, which bounds the fp32 layer path (that path's
 * arithmetic runs on the FMA pipes, not on the tensor cores).  *flops (HOST, optional) receives the number of
 * floating-point operations of the launch (2 per multiply-add); sink is a device float the kernel may write.
 * threads: a multiple of 32, at most 1024.
 */
int dsvt_fma_probe(dsvt_ctx* ctx, int32_t blocks, int32_t threads, int32_t iters, float* sink, int64_t* flops);

#ifdef __cplusplus
}
#endif
#endif /* DSVT_H_ */
