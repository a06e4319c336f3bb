// Fused DSVT layer on the fp32 FMA pipes: gather (Eq. 4) -> QKV projection -> per-set multi-head
// attention (Eq. 5) -> output projection -> residual + LayerNorm -> MLP with GELU -> residual +
// LayerNorm -> scatter (Appendix B.1.1).  One thread block owns a tile of whole sets; because the sets
// partition the voxels (Theorems A.2, A.3), no two blocks touch the same voxel row.
//
// This kernel is the fp32 path (DSVT_FP32) and the general-shape path of DSVT_BF16_FP32ACC: weights
// may be float or bfloat16, all arithmetic is fp32.
//
// Only the distinct members of a set are brought into the tile (a duplicated slot is masked as a key
// and never written back, so it contributes nothing); a set's distinct members occupy consecutive
// tile rows.
#include "dsvt_common.cuh"
#include "fma_tile.cuh"

#include <limits.h>

namespace {
using namespace dsvt_fma;

struct FmaGeom {
  int TM;    // tile rows (multiple of 16)
  int TMn;   // nominal rows per tile: a set belongs to the tile its first row falls in
  int LDQ;   // row stride of the wide buffer (>= 3C, LDQ % 32 == 4)
  int C, hidden, heads, d, tau;
  // relative position bias: entries per head, strides of the x and y offsets, index of the zero offset
  int rb_len, rb_sx, rb_sy, rb_centre;
};

// row[c] = LN(row[c] + add[c]) (gain g == NULL: plain sum).  One warp per row; result left in `row`
// and, if dst != NULL, also written there.
__device__ __forceinline__ void residual_layernorm_row(float* row, const float* add, int C, const float* g,
                                                       const float* b, float eps, float* dst) {
  const int lane = threadIdx.x & 31;
  float s = 0.f;
  for (int c = lane; c < C; c += 32) {
    const float t = row[c] + add[c];
    row[c] = t;
    s += t;
  }
  if (g) {
    const float mean = warp_sum(s) / (float)C;
    float q = 0.f;
    for (int c = lane; c < C; c += 32) {
      const float dlt = row[c] - mean;
      q += dlt * dlt;
    }
    const float inv = rsqrtf(warp_sum(q) / (float)C + eps);
    for (int c = lane; c < C; c += 32) row[c] = (row[c] - mean) * inv * g[c] + (b ? b[c] : 0.f);
  }
  if (dst)
    for (int c = lane; c < C; c += 32) dst[c] = row[c];
}

template <typename WT, int RM>
__global__ void __launch_bounds__(kThreads, 1)
layer_fma_kernel(dsvt_fused_args a, FmaGeom g, int32_t* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int C = g.C, LDQ = g.LDQ, TM = g.TM, tau = g.tau;
  float* Xs = reinterpret_cast<float*>(smem_raw);  // [TM][C]
  float* Bs = Xs + (size_t)TM * C;                  // [TM][LDQ]
  float* Wst = Bs + (size_t)TM * LDQ;               // [kKC][kNC]
  float* pbuf = Wst + kKC * kNC;                    // [kWarps][128]
  int* rowvox = reinterpret_cast<int*>(pbuf + kWarps * 128);  // [TM]
  int* set_lo = rowvox + TM;                                   // [TM + 1]
  int* misc = set_lo + TM + 1;                                 // [4]
  int* rowlin = misc + 4;                                      // [TM] bias: x * rb_sx + y * rb_sy + z of each row
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const dsvt_layer_params& p = a.p;
  const WT* Wqkv = reinterpret_cast<const WT*>(p.W_qkv);
  const WT* Wo = reinterpret_cast<const WT*>(p.W_o);
  const WT* W1 = reinterpret_cast<const WT*>(p.W_1);
  const WT* W2 = reinterpret_cast<const WT*>(p.W_2);

  const int S = min(*a.num_sets, a.cap_sets);
  if (S <= 0) return;
  const int R = a.rowoff[S];
  const int num_tiles = (R + g.TMn - 1) / g.TMn;

  for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
    __syncthreads();
    if (tid == 0) {
      // sets whose first row lies in [t*TMn, (t+1)*TMn)
      const int lo_row = t * g.TMn, hi_row = lo_row + g.TMn;
      int lo = 0, hi = S;
      while (lo < hi) { const int m = (lo + hi) >> 1; if (a.rowoff[m] < lo_row) lo = m + 1; else hi = m; }
      const int s_lo = lo;
      hi = S;
      while (lo < hi) { const int m = (lo + hi) >> 1; if (a.rowoff[m] < hi_row) lo = m + 1; else hi = m; }
      misc[0] = s_lo;
      misc[1] = lo;
      misc[2] = a.rowoff[s_lo];
      misc[3] = a.rowoff[lo] - a.rowoff[s_lo];
    }
    for (int r = tid; r < TM; r += kThreads) rowvox[r] = -1;
    __syncthreads();
    const int s_lo = misc[0], nsets = misc[1] - misc[0], base = misc[2], rows = misc[3];
    if (nsets <= 0) continue;
    if (rows > TM || rows < 0 || nsets > TM) {  // row offsets that do not describe this table
      if (tid == 0) atomicOr(status, DSVT_STATUS_BAD_INDEX);
      continue;
    }
    // ---- distinct slots of each set -> tile rows (Eq. 4) ----
    for (int si = warp; si < nsets; si += kWarps) {
      const int s = s_lo + si;
      const int32_t* row = a.table + (size_t)s * tau;
      const int lb = a.rowoff[s] - base;
      const int cap = a.rowoff[s + 1] - a.rowoff[s];
      int cnt = 0;
      for (int k0 = 0; k0 < tau; k0 += 32) {
        const int k = k0 + lane;
        int v = -1;
        bool uniq = false;
        if (k < tau) {
          v = row[k];
          uniq = (k == 0) || (v != row[k - 1]);
        }
        const unsigned bal = __ballot_sync(0xffffffffu, uniq);
        const int pos = cnt + __popc(bal & ((1u << lane) - 1u));
        if (uniq && pos < cap && lb + pos < TM) {
          if (v < 0 || v >= a.n) { atomicOr(status, DSVT_STATUS_BAD_INDEX); v = -1; }
          rowvox[lb + pos] = v;
        }
        cnt += __popc(bal);
      }
      if (lane == 0) {
        set_lo[si] = lb;
        if (cnt != cap) atomicOr(status, DSVT_STATUS_BAD_INDEX);
      }
    }
    if (tid == 0) set_lo[nsets] = rows;
    __syncthreads();
    const int rm_used = (rows + 15) >> 4;
    const int rows_pad = rm_used << 4;
    const int C4 = C >> 2;
    if (p.rpb) {
      // The bias index is linear in the offset, so one integer per row serves every (query, key) pair.  A set
      // spread wider than the table's extent is reported.
      for (int si = warp; si < nsets; si += kWarps) {
        int lo[3] = {INT_MAX, INT_MAX, INT_MAX}, hi[3] = {INT_MIN, INT_MIN, INT_MIN};
        for (int r = set_lo[si] + lane; r < set_lo[si + 1]; r += 32) {
          const int v = rowvox[r];
          int4 c = make_int4(0, 0, 0, 0);
          if (v >= 0) {
            c = __ldg(reinterpret_cast<const int4*>(p.coords) + v);
            lo[0] = min(lo[0], c.y); hi[0] = max(hi[0], c.y);
            lo[1] = min(lo[1], c.z); hi[1] = max(hi[1], c.z);
            lo[2] = min(lo[2], c.w); hi[2] = max(hi[2], c.w);
          }
          rowlin[r] = c.y * g.rb_sx + c.z * g.rb_sy + c.w;
        }
        bool wide = false;
#pragma unroll
        for (int q = 0; q < 3; ++q) {
          const int l = -warp_max_int(-lo[q]), h = warp_max_int(hi[q]);
          wide |= (h >= l) && (h - l > p.rpb_extent[q] - 1);
        }
        if (wide && lane == 0) atomicOr(status, DSVT_STATUS_BAD_INDEX);
      }
    }
    auto gather = [&](bool with_pe) {
      for (int r = warp; r < rows_pad; r += kWarps) {
        const int v = r < rows ? rowvox[r] : -1;
        for (int c4 = lane; c4 < C4; c4 += 32) {
          float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
          if (v >= 0) {
            f = reinterpret_cast<const float4*>(a.x + (size_t)v * C)[c4];
            if (with_pe) {
              const float4 e = reinterpret_cast<const float4*>(p.pe + (size_t)v * C)[c4];
              f.x += e.x; f.y += e.y; f.z += e.z; f.w += e.w;
            }
          }
          reinterpret_cast<float4*>(Xs + (size_t)r * C)[c4] = f;
        }
      }
      __syncthreads();
    };
    // ---- QKV projection ----
    if (p.pe) {
      gather(true);
      gemm_tile<WT, RM>(Xs, C, rm_used, Wqkv, C, 2 * C, p.b_qkv, Bs, LDQ, false, Wst);
      gather(false);
      gemm_tile<WT, RM>(Xs, C, rm_used, Wqkv + (size_t)2 * C * C, C, C, p.b_qkv ? p.b_qkv + 2 * C : nullptr,
                        Bs + 2 * C, LDQ, false, Wst);
    } else {
      gather(false);
      gemm_tile<WT, RM>(Xs, C, rm_used, Wqkv, C, 3 * C, p.b_qkv, Bs, LDQ, false, Wst);
    }
    // ---- attention inside each set, one warp per (set, head) ----
    {
      const int d = g.d, d4 = d >> 2;
      const float scale = rsqrtf((float)d);
      float* pw = pbuf + warp * 128;
      for (int item = warp; item < nsets * g.heads; item += kWarps) {
        const int si = item / g.heads, h = item - si * g.heads;
        const int r0 = set_lo[si], m = set_lo[si + 1] - r0;
        const float* Qb = Bs + (size_t)r0 * LDQ + h * d;
        const float* Kb = Qb + C;
        const float* Vb = Qb + 2 * C;
        const float* bias = p.rpb ? p.rpb + (size_t)h * g.rb_len : nullptr;
        for (int qa = 0; qa < m; ++qa) {
          const float4* q4 = reinterpret_cast<const float4*>(Qb + (size_t)qa * LDQ);
          float lg[4];
          float mx = -INFINITY;
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int kb = lane + 32 * u;
            lg[u] = -INFINITY;
            if (kb < m) {
              const float4* k4 = reinterpret_cast<const float4*>(Kb + (size_t)kb * LDQ);
              float s = 0.f;
              for (int c = 0; c < d4; ++c) {
                const float4 qv = q4[c], kv = k4[c];
                s = fmaf(qv.x, kv.x, s); s = fmaf(qv.y, kv.y, s); s = fmaf(qv.z, kv.z, s); s = fmaf(qv.w, kv.w, s);
              }
              lg[u] = s * scale;
              if (bias) {
                const int idx = rowlin[r0 + qa] - rowlin[r0 + kb] + g.rb_centre;
                lg[u] += __ldg(bias + min(max(idx, 0), g.rb_len - 1));
              }
              mx = fmaxf(mx, lg[u]);
            }
          }
          mx = warp_max(mx);
          float den = 0.f;
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int kb = lane + 32 * u;
            if (kb < m) {
              const float e = expf(lg[u] - mx);
              pw[kb] = e;
              den += e;
            }
          }
          den = warp_sum(den);
          __syncwarp();
          const float inv = 1.0f / den;
          for (int c = lane; c < d; c += 32) {
            float acc = 0.f;
            for (int kb = 0; kb < m; ++kb) acc = fmaf(pw[kb], Vb[(size_t)kb * LDQ + c], acc);
            // the query row's own slot is dead once its logits exist: reuse it for the attention output
            Bs[(size_t)(r0 + qa) * LDQ + h * d + c] = acc * inv;
          }
          __syncwarp();
        }
      }
    }
    __syncthreads();
    // ---- output projection: Z = Y W_o^T + b_o into the key columns ----
    gemm_tile<WT, RM>(Bs, LDQ, rm_used, Wo, C, C, p.b_o, Bs + C, LDQ, false, Wst);
    if (a.attention_only) {
      for (int r = warp; r < rows; r += kWarps) {
        const int v = rowvox[r];
        if (v < 0) continue;
        for (int c4 = lane; c4 < C4; c4 += 32)
          reinterpret_cast<float4*>(a.y + (size_t)v * C)[c4] =
              *reinterpret_cast<const float4*>(Bs + (size_t)r * LDQ + C + 4 * c4);
      }
      continue;
    }
    // ---- x1 = LN1(x + Z) ----
    const bool mlp = g.hidden > 0;
    for (int r = warp; r < rows; r += kWarps) {
      const int v = rowvox[r];
      float* dst = (!mlp && v >= 0) ? a.y + (size_t)v * C : nullptr;
      residual_layernorm_row(Xs + (size_t)r * C, Bs + (size_t)r * LDQ + C, C, p.ln1_g, p.ln1_b, p.ln_eps, dst);
    }
    __syncthreads();
    if (!mlp) continue;
    // ---- MLP: H = gelu(x1 W_1^T + b_1) into columns [0, hidden); M = H W_2^T + b_2 into [2C, 3C) ----
    gemm_tile<WT, RM>(Xs, C, rm_used, W1, C, g.hidden, p.b_1, Bs, LDQ, true, Wst);
    gemm_tile<WT, RM>(Bs, LDQ, rm_used, W2, g.hidden, C, p.b_2, Bs + 2 * C, LDQ, false, Wst);
    // ---- y = LN2(x1 + M) ----
    for (int r = warp; r < rows; r += kWarps) {
      const int v = rowvox[r];
      float* dst = v >= 0 ? a.y + (size_t)v * C : nullptr;
      residual_layernorm_row(Xs + (size_t)r * C, Bs + (size_t)r * LDQ + 2 * C, C, p.ln2_g, p.ln2_b, p.ln_eps, dst);
    }
  }
}

size_t fma_smem_bytes(const FmaGeom& g) {
  size_t fl = (size_t)g.TM * g.C + (size_t)g.TM * g.LDQ + kKC * kNC + kWarps * 128;
  size_t in = (size_t)g.TM + (g.TM + 1) + 4 + g.TM;
  return fl * 4 + in * 4 + 16;
}

template <typename WT, int RM>
int launch_one(dsvt_ctx* ctx, const dsvt_fused_args& a, const FmaGeom& g, int grid) {
  const size_t smem = fma_smem_bytes(g);
  cudaError_t e = cudaFuncSetAttribute(layer_fma_kernel<WT, RM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return DSVT_ERR_CUDA; }
  layer_fma_kernel<WT, RM><<<grid, kThreads, smem, ctx->stream>>>(a, g, ctx->status);
  DSVT_LAUNCHED(ctx);
  return DSVT_OK;
}

template <typename WT>
int launch_rm(dsvt_ctx* ctx, const dsvt_fused_args& a, const FmaGeom& g, int grid) {
  switch (g.TM / 16) {
    case 1: return launch_one<WT, 1>(ctx, a, g, grid);
    case 2: return launch_one<WT, 2>(ctx, a, g, grid);
    case 3: return launch_one<WT, 3>(ctx, a, g, grid);
    case 4: return launch_one<WT, 4>(ctx, a, g, grid);
    case 6: return launch_one<WT, 6>(ctx, a, g, grid);
    case 8: return launch_one<WT, 8>(ctx, a, g, grid);
  }
  return DSVT_ERR_UNSUPPORTED;
}

}  // namespace

int dsvt_launch_layer_fma(dsvt_ctx* ctx, const dsvt_fused_args& a) {
  const dsvt_layer_params& p = a.p;
  FmaGeom g;
  g.C = p.C; g.hidden = a.attention_only ? 0 : p.hidden; g.heads = p.heads; g.d = p.C / p.heads; g.tau = p.set_size;
  g.rb_len = g.rb_sx = g.rb_sy = g.rb_centre = 0;
  if (p.rpb) {
    const int L = p.rpb_extent[0], W = p.rpb_extent[1], H = p.rpb_extent[2];
    g.rb_sy = 2 * H - 1;
    g.rb_sx = (2 * W - 1) * g.rb_sy;
    g.rb_len = (2 * L - 1) * g.rb_sx;
    g.rb_centre = (L - 1) * g.rb_sx + (W - 1) * g.rb_sy + (H - 1);
  }
  g.LDQ = 3 * p.C + (36 - (3 * p.C) % 32) % 32;  // LDQ % 32 == 4: conflict-free 128-bit row-strided loads
  static const int kTiles[] = {128, 96, 64, 48, 32, 16};
  g.TM = 0;
  for (int tm : kTiles) {
    FmaGeom t = g;
    t.TM = tm;
    if (tm >= g.tau && fma_smem_bytes(t) <= 227 * 1024) { g.TM = tm; break; }
  }
  if (g.TM == 0) return DSVT_ERR_UNSUPPORTED;
  g.TMn = g.TM - g.tau + 1;
  int64_t rmax = (int64_t)a.cap_sets * g.tau;
  if (rmax > a.n) rmax = a.n;
  int64_t grid = dsvt_ceil_div(rmax, g.TMn);
  if (grid < 1) grid = 1;
  const int64_t gmax = (int64_t)ctx->sm_count * 16;
  if (grid > gmax) grid = gmax;
  if (p.precision == DSVT_FP32) return launch_rm<float>(ctx, a, g, (int)grid);
  return launch_rm<__nv_bfloat16>(ctx, a, g, (int)grid);
}
