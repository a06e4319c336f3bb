// Attention-style 3D pooling (Eq. 6, Eq. 7) with the four projections on the 5th-generation tensor cores
// (tcgen05 + TMEM), bfloat16 operands, fp32 accumulation.
//
// A tile is 128 padded slot rows = 128 / ns regions of ns slots each (ns a power of two, so a region's rows sit in
// neighbouring lanes of one warp).  Per tile: the compute warps gather the slot rows (zero rows for empty slots,
// plus the slot term), take the Eq. 6 maxima and write two bf16 A operands, the padded slots X~ and the maxima P
// repeated for every slot row of their region; the tensor pipe forms Q = P W_q^T, K = X~ W_k^T (M = 128, N = C) into
// TMEM; each thread reads its row's quarter of Q and K straight from TMEM, takes the scores of its heads, and the
// softmax over the region's slots is a few shuffles between neighbouring lanes; V = X~ W_v^T follows into the
// query's columns, the weighted sum over the slots is again shuffles, and the result (the same in all rows of a
// region) becomes the A operand of the output projection, whose slot-0 rows are the region's output.  No K, V or
// Q tile ever goes through shared memory, and the arithmetic on them is fp32.
//
// Roles (576 threads): warps 0-15 compute; warp 16 streams the four weight matrices through a three-stage ring
// with plain (single-CTA) TMA loads, tile after tile; warp 17 allocates TMEM and issues the tcgen05.mma
// instructions.  Every mbarrier wait is bounded (DSVT_STATUS_TIMEOUT).
#include <cuda.h>

#include "dsvt_common.cuh"
#include "tc_ptx.cuh"

namespace {
using namespace dsvt_tc;

constexpr int kComputeWarps = 16;
constexpr int kComputeThreads = 32 * kComputeWarps;
constexpr int kTmaWarp = kComputeWarps, kMmaWarp = kComputeWarps + 1;
constexpr int kThreads = kComputeThreads + 64;
constexpr int kStages = 3;

struct PoolTcMaps {
  CUtensorMap w[4];  // W_q, W_k, W_v, W_o: boxes of 64 input columns x C rows, 128-byte swizzle
};

struct PoolMisc {
  unsigned long long full[kStages], empty[kStages], acc_full[2], acc_free[2];
  unsigned long long ab_ready;  // compute -> MMA: X~ and P are in place
  unsigned long long ao_ready;  // compute -> MMA: the attention output is in place
  unsigned long long drain;
  uint32_t tmem_base;
  int abort_flag;
  int rowvox[kTM];  // tile row -> voxel (-1: empty slot or no region)
};
__shared__ PoolMisc s_pm;

__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kComputeThreads) : "memory"); }

// fp32 output staging: row r, 16-byte chunk c4, rotated by the row (conflict-free for row-per-thread and
// row-per-warp access alike).
template <int C>
__device__ __forceinline__ uint32_t out_off(int r, int c4) {
  constexpr int NCH = C / 4;
  int idx = c4 + (r % NCH);
  if (idx >= NCH) idx -= NCH;
  return (uint32_t)(r * (C * 4) + (idx << 4));
}

// ================= weight stream (one thread) ===========================================================
template <int C>
__device__ __noinline__ void pool_producer(const PoolTcMaps& maps, uint32_t st_base, int my_tiles) {
  constexpr int NKB = C / 64;
  constexpr uint32_t STAGE_BYTES = C * 128;
  volatile int* abort_flag = &s_pm.abort_flag;
  int stage = 0;
  uint32_t phase = 0;
  int issued[kStages] = {0, 0, 0};
  for (int t = 0; t < my_tiles; ++t) {
    for (int c = 0; c < 4; ++c) {
      for (int kb = 0; kb < NKB; ++kb) {
        if (!mbar_wait(&s_pm.empty[stage], phase ^ 1u, abort_flag)) goto done;
        mbar_expect_tx(&s_pm.full[stage], STAGE_BYTES);
        tma_load_2d(st_base + stage * STAGE_BYTES, &maps.w[c], kb * 64, 0, &s_pm.full[stage]);
        ++issued[stage];
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
    }
  }
done:
  if (*abort_flag) {  // leaving early: no load may still be writing into this CTA's shared memory when it retires
#pragma unroll
    for (int i = 0; i < kStages; ++i)
      if (issued[i] > 0) {
        const uint32_t par = (uint32_t)(issued[i] - 1) & 1u;
        for (int it = 0; it < kMaxPolls && !mbar_try(&s_pm.full[i], par); ++it) {}
      }
  }
}

// ================= MMA issuer (one thread) ==============================================================
// Chunks of a tile: Q (A = P, region 0), K (A = X~, region 1), V (A = X~, region 0 once the scores have read Q),
// O (A = attention output in P's place, region 1 once the scores have read K).
template <int C>
__device__ __noinline__ void pool_mma(uint32_t x_base, uint32_t p_base, uint32_t st_base, uint32_t tmem, int my_tiles) {
  constexpr int NKB = C / 64;
  constexpr uint32_t STAGE_BYTES = C * 128;
  volatile int* abort_flag = &s_pm.abort_flag;
  const uint32_t idesc = umma_idesc(C);
  int stage = 0;
  uint32_t phase = 0;
  uint32_t uses[2] = {0u, 0u};
  for (int t = 0; t < my_tiles; ++t) {
    for (int c = 0; c < 4; ++c) {
      const uint32_t bar = (c == 0 || c == 2) ? 0u : 1u;
      if (c == 0 && !mbar_wait(&s_pm.ab_ready, (uint32_t)t & 1u, abort_flag)) goto done;
      if (c == 3 && !mbar_wait(&s_pm.ao_ready, (uint32_t)t & 1u, abort_flag)) goto done;
      if (!mbar_wait(&s_pm.acc_free[bar], (uses[bar] & 1u) ^ 1u, abort_flag)) goto done;
      ++uses[bar];
      tc_fence_after();
      const uint32_t abase = (c == 0 || c == 3) ? p_base : x_base;
      const uint32_t d_tmem = tmem + bar * C;
      for (int kb = 0; kb < NKB; ++kb) {
        if (!mbar_wait(&s_pm.full[stage], phase, abort_flag)) goto done;
        tc_fence_after();
        const uint32_t sa = abase + kb * (kTM * 128), sb = st_base + stage * STAGE_BYTES;
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
          umma_bf16(d_tmem, umma_desc(sa + k4 * 32), umma_desc(sb + k4 * 32), idesc, (kb | k4) != 0 ? 1u : 0u);
        umma_commit(&s_pm.empty[stage]);
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
      umma_commit(&s_pm.acc_full[bar]);
    }
  }
done:
  if (*abort_flag) {  // the MMAs already issued must have completed before the TMEM columns are returned
    umma_commit(&s_pm.drain);
    for (int it = 0; it < kMaxPolls && !mbar_try(&s_pm.drain, 0u); ++it) {}
  }
}

struct PoolTcArgs {
  const float* feats;
  const int32_t* cell_map;
  const int32_t* region_key;
  const int32_t* num_out;
  int32_t cap_m;
  const float *b_q, *b_k, *b_v, *b_o, *slot_pe;
  float* out_feats;
  int32_t heads, nslots, mask_empty;
  int32_t* status;
};

// ================= compute warps: gather + Eq. 6 ========================================================
// Work item = (region, 16-byte channel chunk): the chunk of every slot row of the region (all loads of a thread's
// items in flight together), the channel-wise maximum, X~ rows and P rows as bf16.
template <int C, int NS>
__device__ __forceinline__ void pool_gather_ns(const PoolTcArgs& a, unsigned char* xs, unsigned char* ps, int nr) {
  constexpr int C4 = C / 4, TR = kTM / NS, ITEMS = TR * C4;
  constexpr int PER = (ITEMS + kComputeThreads - 1) / kComputeThreads;  // items per thread
  constexpr int GROUP = NS <= 4 ? NS : 4;                               // slot rows loaded together
  static_assert(PER * GROUP <= 16, "loads in flight per thread");
  const int tid = threadIdx.x;
  float4 mx[PER];
#pragma unroll
  for (int j = 0; j < PER; ++j) mx[j] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
  for (int s0 = 0; s0 < NS; s0 += GROUP) {
    float4 f[PER][GROUP];
    int vv[PER][GROUP];
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      const int i = tid + j * kComputeThreads, ri = i / C4, c4 = i - ri * C4;
#pragma unroll
      for (int u = 0; u < GROUP; ++u) {
        vv[j][u] = (i < ITEMS && ri < nr) ? s_pm.rowvox[ri * NS + s0 + u] : -1;
        f[j][u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (vv[j][u] >= 0) f[j][u] = __ldg(reinterpret_cast<const float4*>(a.feats + (size_t)vv[j][u] * C) + c4);
      }
    }
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      const int i = tid + j * kComputeThreads, ri = i / C4, c4 = i - ri * C4;
      if (i >= ITEMS) continue;
      const bool live = ri < nr;
#pragma unroll
      for (int u = 0; u < GROUP; ++u) {
        const int s = s0 + u, r = ri * NS + s;
        float4 g = f[j][u];
        if (live && (!a.mask_empty || vv[j][u] >= 0)) {
          mx[j].x = fmaxf(mx[j].x, g.x); mx[j].y = fmaxf(mx[j].y, g.y); mx[j].z = fmaxf(mx[j].z, g.z); mx[j].w = fmaxf(mx[j].w, g.w);
        }
        if (live && a.slot_pe) {
          const float4 e = __ldg(reinterpret_cast<const float4*>(a.slot_pe + (size_t)s * C) + c4);
          g.x += e.x; g.y += e.y; g.z += e.z; g.w += e.w;
        }
        *reinterpret_cast<uint2*>(xs + swz(r, c4 >> 1) + (c4 & 1) * 8) = make_uint2(pack_bf16(g.x, g.y), pack_bf16(g.z, g.w));
      }
    }
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int i = tid + j * kComputeThreads, ri = i / C4, c4 = i - ri * C4;
    if (i >= ITEMS) continue;
    const float4 m4 = ri < nr ? mx[j] : make_float4(0.f, 0.f, 0.f, 0.f);
    const uint2 p2 = make_uint2(pack_bf16(m4.x, m4.y), pack_bf16(m4.z, m4.w));
#pragma unroll
    for (int s = 0; s < NS; ++s)  // the region's maximum, once per slot row
      *reinterpret_cast<uint2*>(ps + swz(ri * NS + s, c4 >> 1) + (c4 & 1) * 8) = p2;
  }
}

template <int C>
__device__ __forceinline__ void pool_gather(const PoolTcArgs& a, unsigned char* xs, unsigned char* ps, int nr, int ns) {
  switch (ns) {
    case 1: pool_gather_ns<C, 1>(a, xs, ps, nr); break;
    case 2: pool_gather_ns<C, 2>(a, xs, ps, nr); break;
    case 4: pool_gather_ns<C, 4>(a, xs, ps, nr); break;
    case 8: pool_gather_ns<C, 8>(a, xs, ps, nr); break;
    case 16: pool_gather_ns<C, 16>(a, xs, ps, nr); break;
    default: pool_gather_ns<C, 32>(a, xs, ps, nr); break;
  }
}

// ================= the kernel ===========================================================================
// Thread (row, quarter): warp w owns TMEM lanes 32 (w % 4) .. + 31 (tile rows) and the column quarter w / 4, which
// holds HQ = (C / 4) / D whole heads.
template <int C, int D>
__global__ void __launch_bounds__(kThreads, 1) pool_tc_kernel(const __grid_constant__ PoolTcArgs a,
                                                              const __grid_constant__ PoolTcMaps maps) {
  constexpr int QC = C / 4, HQ = QC / D;
  constexpr uint32_t TILE_BYTES = kTM * C * 2;
  extern __shared__ unsigned char pool_tc_smem[];
  const uint32_t raw = smem_u32(pool_tc_smem);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* sm = pool_tc_smem + pad;
  const uint32_t sbase = raw + pad;
  unsigned char* xs = sm;                       // X~ (bf16 operand); later the fp32 output staging
  unsigned char* ps = sm + TILE_BYTES;          // P (bf16 operand); later the attention output
  const uint32_t st_base = sbase + 2 * TILE_BYTES;
  float* par = reinterpret_cast<float*>(sm + 2 * TILE_BYTES + kStages * C * 128);  // b_q, b_k, b_v, b_o
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ns = a.nslots, TR = kTM / ns;
  volatile int* abort_flag = &s_pm.abort_flag;
  if (tid == 0) {
    s_pm.abort_flag = 0;
    for (int i = 0; i < kStages; ++i) { mbar_init(&s_pm.full[i], 1); mbar_init(&s_pm.empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&s_pm.acc_full[i], 1); mbar_init(&s_pm.acc_free[i], kComputeThreads); }
    mbar_init(&s_pm.ab_ready, kComputeThreads);
    mbar_init(&s_pm.ao_ready, kComputeThreads);
    mbar_init(&s_pm.drain, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_pm.tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = tid; i < 4 * C; i += kThreads) {
    const int which = i / C;
    const float* v = which == 0 ? a.b_q : which == 1 ? a.b_k : which == 2 ? a.b_v : a.b_o;
    par[i] = v ? __ldg(v + i % C) : 0.f;
  }
  // everything above touched this CTA's own state and the call's weights; what follows reads what the kernels before
  // it in the stream wrote (the region list, the cell map, the number of regions): wait for them if this launch was
  // allowed to start early
  pdl_enter();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_pm.tmem_base;
  const int m = min(*a.num_out, a.cap_m);
  const int num_tiles = (m + TR - 1) / TR;
  const int my_tiles = (int)blockIdx.x < num_tiles ? (num_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  if (warp == kTmaWarp) {
    if (lane == 0) pool_producer<C>(maps, st_base, my_tiles);
    __syncwarp();
  } else if (warp == kMmaWarp) {
    if (lane == 0) pool_mma<C>(sbase, sbase + TILE_BYTES, st_base, tmem, my_tiles);
    __syncwarp();
  } else {
    const int row = 32 * (warp & 3) + lane, hq = warp >> 2;
    const uint32_t taddr = tmem + ((uint32_t)(32 * (warp & 3)) << 16) + hq * QC;
    const float scale = rsqrtf((float)D);
    const int s_of = row & (ns - 1), ri = row / ns;
    uint32_t uses[2] = {0u, 0u};
    bool ok = true;
    auto acc_wait = [&](int bar) {
      ok = mbar_wait(&s_pm.acc_full[bar], uses[bar] & 1u, abort_flag) && ok;
      ++uses[bar];
      tc_fence_after();
    };
    // tile row -> voxel through the region list and the dense cell map: the region's key is looked up two tiles
    // ahead and its cell one tile ahead, so that neither load waits for the other inside a tile
    auto row_key = [&](int tl) {
      const int t = blockIdx.x + tl * gridDim.x, r_lo = t * TR, nr = min(TR, m - r_lo);
      return (tl < my_tiles && tid < kTM && tid / ns < nr) ? __ldg(a.region_key + r_lo + tid / ns) : -1;
    };
    auto row_voxel = [&](int key) {
      return key >= 0 ? __ldg(a.cell_map + (size_t)key * ns + (tid & (ns - 1))) : -1;
    };
    int v_next = row_voxel(row_key(0));
    int key_next = row_key(1);
    for (int tl = 0; tl < my_tiles; ++tl) {
      const int t = blockIdx.x + tl * gridDim.x;
      const int r_lo = t * TR, nr = min(TR, m - r_lo);
      compute_sync();  // the previous tile's staging rows have been stored; its operands are dead
      if (tid < kTM) s_pm.rowvox[tid] = v_next;
      compute_sync();
      v_next = row_voxel(key_next);
      key_next = row_key(tl + 2);
      pool_gather<C>(a, xs, ps, nr, ns);
      fence_proxy_async();
      mbar_arrive(&s_pm.ab_ready);
      // ---- scores: q . k per head of this quarter, softmax over the region's slots (neighbouring lanes) ----
      const bool live = ri < nr;
      const bool key_ok = live && (!a.mask_empty || s_pm.rowvox[row] >= 0);
      float p[HQ];
      float qr[QC];  // this thread's query columns: read at once, so that the value projection can take their region
      acc_wait(0);
      tmem_ld_row(taddr, qr);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&s_pm.acc_free[0]);
      acc_wait(1);
#pragma unroll
      for (int j = 0; j < HQ; ++j) {  // one head at a time: D query and D key columns of this thread's row
        float k[D];
        tmem_ld_row(taddr + C + j * D, k);
        tmem_wait_ld();
        float acc = 0.f;
#pragma unroll
        for (int c = 0; c < D; c += 4) {
          const int cc = hq * QC + j * D + c;
          const float4 bq = *reinterpret_cast<const float4*>(par + cc), bk = *reinterpret_cast<const float4*>(par + C + cc);
          acc = fmaf(qr[j * D + c] + bq.x, k[c] + bk.x, acc);
          acc = fmaf(qr[j * D + c + 1] + bq.y, k[c + 1] + bk.y, acc);
          acc = fmaf(qr[j * D + c + 2] + bq.z, k[c + 2] + bk.z, acc);
          acc = fmaf(qr[j * D + c + 3] + bq.w, k[c + 3] + bk.w, acc);
        }
        const float lg = key_ok ? acc * scale : -INFINITY;
        float mx = lg;
        for (int o = ns >> 1; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float e = key_ok ? __expf(lg - mx) : 0.f;
        float sum = e;
        for (int o = ns >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        p[j] = sum > 0.f ? e / sum : 0.f;
      }
      tc_fence_before();
      mbar_arrive(&s_pm.acc_free[1]);
      // ---- weighted sum of the values over the region's slots -> attention output (bf16 operand, P's place) ----
      {
        float v[QC];
        acc_wait(0);
        tmem_ld_row(taddr, v);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(&s_pm.acc_free[0]);
#pragma unroll
        for (int c4 = 0; c4 < QC; c4 += 4) {
          const float4 bv = *reinterpret_cast<const float4*>(par + 2 * C + hq * QC + c4);
          const float b4[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int cc = c4 + e;
            float t2 = p[cc / D] * v[cc];
            for (int o = ns >> 1; o > 0; o >>= 1) t2 += __shfl_xor_sync(0xffffffffu, t2, o);
            v[cc] = live ? t2 + b4[e] : 0.f;  // the probabilities sum to one: + b_v once
          }
        }
#pragma unroll
        for (int q8 = 0; q8 < QC / 8; ++q8)
          *reinterpret_cast<uint4*>(ps + swz(row, ((hq * QC) >> 3) + q8)) =
              make_uint4(pack_bf16(v[8 * q8], v[8 * q8 + 1]), pack_bf16(v[8 * q8 + 2], v[8 * q8 + 3]),
                         pack_bf16(v[8 * q8 + 4], v[8 * q8 + 5]), pack_bf16(v[8 * q8 + 6], v[8 * q8 + 7]));
      }
      fence_proxy_async();
      mbar_arrive(&s_pm.ao_ready);
      // ---- output projection: the slot-0 rows are the regions' outputs ----
      {
        float o[QC];
        acc_wait(1);
        tmem_ld_row(taddr + C, o);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(&s_pm.acc_free[1]);
        if (live && s_of == 0) {  // (X~ is dead: the value projection has been read)
#pragma unroll
          for (int q4 = 0; q4 < QC / 4; ++q4) {
            const float4 bo = *reinterpret_cast<const float4*>(par + 3 * C + hq * QC + 4 * q4);
            *reinterpret_cast<float4*>(xs + out_off<C>(ri, hq * (QC / 4) + q4)) =
                make_float4(o[4 * q4] + bo.x, o[4 * q4 + 1] + bo.y, o[4 * q4 + 2] + bo.z, o[4 * q4 + 3] + bo.w);
          }
        }
      }
      compute_sync();
      for (int r = warp; r < nr; r += kComputeWarps)
        for (int c4 = lane; c4 < C / 4; c4 += 32)
          reinterpret_cast<float4*>(a.out_feats + (size_t)(r_lo + r) * C)[c4] =
              *reinterpret_cast<const float4*>(xs + out_off<C>(r, c4));
    }
    if (!ok || *abort_flag) {
      if (tid == 0) atomicOr(a.status, DSVT_STATUS_TIMEOUT);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

}  // namespace

bool dsvt_pool_tc_supported(int C, int heads, int nslots) {
  if (heads < 1 || C % heads != 0) return false;
  const int d = C / heads;
  if (!((C == 192 && d == 24) || (C == 128 && (d == 16 || d == 32)) || (C == 64 && d == 16))) return false;
  return nslots >= 1 && nslots <= 32 && (nslots & (nslots - 1)) == 0;
}

namespace {
template <int C, int D>
int launch_pool_tc(dsvt_ctx* ctx, const PoolTcArgs& a, const PoolTcMaps& maps, int grid, unsigned flag) {
  const size_t smem = 2 * (size_t)kTM * C * 2 + kStages * (size_t)C * 128 + 4 * (size_t)C * sizeof(float) + 1024;
  if (!(ctx->attr_flags & flag)) {  // (once per context: the attribute belongs to its device)
    DSVT_CUDA_TRY(ctx, cudaFuncSetAttribute(pool_tc_kernel<C, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    ctx->attr_flags |= flag;
  }
  DSVT_CUDA_TRY(ctx, launch_pdl(pool_tc_kernel<C, D>, dim3(grid), dim3(kThreads), smem, ctx->stream, a, maps));
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}
}  // namespace

int dsvt_launch_pool_tc(dsvt_ctx* ctx, const dsvt_pool_tc_call& c) {
  PoolTcArgs a;
  a.feats = c.feats; a.cell_map = c.cell_map; a.region_key = c.region_key; a.num_out = c.num_out; a.cap_m = c.cap_m;
  a.b_q = c.b_q; a.b_k = c.b_k; a.b_v = c.b_v; a.b_o = c.b_o; a.slot_pe = c.slot_pe;
  a.out_feats = c.out_feats; a.heads = c.heads; a.nslots = c.nslots; a.mask_empty = c.mask_empty;
  a.status = ctx->status;
  PoolTcMaps maps;
  for (int i = 0; i < 4; ++i)
    if (!dsvt_cached_weight_map(ctx, &maps.w[i], c.W[i], c.C, c.C, c.C)) return DSVT_ERR_CUDA;
  const int TR = kTM / c.nslots;
  int64_t tiles = dsvt_ceil_div(c.n < c.cap_m ? c.n : c.cap_m, TR);
  int64_t grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
  if (grid < 1) grid = 1;
  const int d = c.C / c.heads;
  if (c.C == 192) return launch_pool_tc<192, 24>(ctx, a, maps, (int)grid, 16u);
  if (c.C == 128 && d == 16) return launch_pool_tc<128, 16>(ctx, a, maps, (int)grid, 32u);
  if (c.C == 128) return launch_pool_tc<128, 32>(ctx, a, maps, (int)grid, 64u);
  return launch_pool_tc<64, 16>(ctx, a, maps, (int)grid, 128u);
}
