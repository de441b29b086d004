// PowerSGD rank-r step with error feedback over W workers (compressor of Section 5.2).
//
// Because every product of the step is linear in the workers' matrices, the factors only depend on
// the mean matrix  Mbar = (1/W) sum_w (g_w + e_w):   P = Mbar Q,  Q' = Mbar^T P^,  A = P^ Q'^T.
// The project pass therefore reads every worker's g and e once, writes M_w back over e_w, and keeps
// Mbar (1/W of the data) in `out` for the second product; only the residual pass touches the
// per-worker data again.
#include "acc_internal.cuh"

namespace acc {

// One row of an item (columns [col0, col0 + ncols) of the layer's row): scalar head up to the first
// 16-byte boundary, aligned float4 body, scalar tail.  Column indices below are relative to col0.
struct RowGeom {
  long long start;  // element index of the first column of the chunk inside a worker's slice
  int head, nbody4, tail;
};

__device__ __forceinline__ RowGeom row_geom(const DevLayer& L, const RowItem& it, int row) {
  RowGeom g;
  g.start = L.offset + (long long)row * L.cols + it.col0;
  int h = (int)((4 - (g.start & 3)) & 3);
  g.head = h < it.ncols ? h : it.ncols;
  g.nbody4 = (it.ncols - g.head) >> 2;
  g.tail = it.ncols - g.head - 4 * g.nbody4;
  return g;
}

// out = mean_w g_w on one tile of a VECTOR layer; delta += g_decider.
__device__ void vector_mean_tile(const Tile& t, const DevLayer& L, const float* __restrict__ grads,
                                 float* __restrict__ out, float* __restrict__ delta, long long stride, int W,
                                 int decider, float inv_w) {
  const long long base = L.offset + t.elem0;
  for (int i = threadIdx.x; i < t.nelem; i += blockDim.x) {
    float acc = 0.f;
    for (int w = 0; w < W; ++w) {
      const float g = grads[(long long)w * stride + base + i];
      acc += g;
      if (delta != nullptr && w == decider) delta[base + i] += g;
    }
    out[base + i] = acc * inv_w;
  }
}

__device__ __forceinline__ float lowrank_entry(const float4& pv, const float4& qv, int r) {
  float a = pv.x * qv.x;
  if (r > 1) a = fmaf(pv.y, qv.y, a);
  if (r > 2) a = fmaf(pv.z, qv.z, a);
  if (r > 3) a = fmaf(pv.w, qv.w, a);
  return a;
}

// Sum over the `lpr` consecutive lanes of a row group (lpr = 8, 16 or 32); every lane of the warp calls it.
__device__ __forceinline__ float group_sum(float v, int lpr) {
  for (int o = lpr >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Pass 1.  One block per row slab, all workers.  A group of `lpr` lanes owns a row (8*32/lpr rows in
// flight per block):
//   e_w = err_w                               (eager: err holds the error memory)
//   e_w = err_w - P^_prev Q^T  (first rp ranks) (lazy: err holds last step's M_w, residual still pending)
//   M_w = g_w + e_w -> err;  Mbar = mean_w M_w -> out;  P[row, :] = Mbar[row, :] . Q   (first r ranks);
//   delta += g_decider.  Blocks beyond the row items handle the VECTOR tiles.
template <int WB, bool LAZY>
__global__ void __launch_bounds__(256, 3)
psgd_project_kernel(const DevLayer* __restrict__ layers, const RowItem* __restrict__ items, int n_items,
                    const Tile* __restrict__ tiles, const int* __restrict__ vec_tiles,
                    const float* __restrict__ grads, float* __restrict__ err, const float* __restrict__ q,
                    float* __restrict__ p, float4* __restrict__ p_part, const uint8_t* __restrict__ level,
                    const int* __restrict__ pending, float* __restrict__ out, float* __restrict__ delta,
                    long long stride, int W, int decider, float inv_w, int rank_low, int rank_high) {
  if ((int)blockIdx.x >= n_items) {
    const Tile t = tiles[vec_tiles[blockIdx.x - n_items]];
    vector_mean_tile(t, layers[t.layer], grads, out, delta, stride, W, decider, inv_w);
    return;
  }
  const RowItem it = items[blockIdx.x];
  const DevLayer L = layers[it.layer];
  const int r = level[it.layer] ? rank_low : rank_high;
  const int rp = LAZY ? pending[it.layer] : 0;
  const float4* __restrict__ Q4 = reinterpret_cast<const float4*>(q) + L.q_row + it.col0;
  float4* __restrict__ P4 = reinterpret_cast<float4*>(p) + L.p_row;
  const int lpr = L.lpr, groups = 32 / lpr;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane / lpr, gl = lane - g * lpr;
  const int row_end = it.row0 + it.nrows;
  for (int r0 = it.row0 + warp * groups; r0 < row_end; r0 += 8 * groups) {
    const int row = r0 + g;
    const bool valid = row < row_end;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    if (valid) {
      const RowGeom rg = row_geom(L, it, row);
      float4 pp = make_float4(0.f, 0.f, 0.f, 0.f);
      if (LAZY && rp > 0) pp = P4[row];
      for (int t = gl; t < rg.nbody4; t += lpr) {
        const int col = rg.head + 4 * t;
        const long long idx = rg.start + col;
        const float4 q0 = __ldg(Q4 + col), q1 = __ldg(Q4 + col + 1), q2 = __ldg(Q4 + col + 2), q3 = __ldg(Q4 + col + 3);
        float4 corr = make_float4(0.f, 0.f, 0.f, 0.f);
        if (LAZY && rp > 0) {
          corr.x = lowrank_entry(pp, q0, rp); corr.y = lowrank_entry(pp, q1, rp);
          corr.z = lowrank_entry(pp, q2, rp); corr.w = lowrank_entry(pp, q3, rp);
        }
        float4 mb = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int w0 = 0; w0 < W; w0 += WB) {
          float4 gv[WB], ev[WB];
#pragma unroll
          for (int b = 0; b < WB; ++b)
            if (w0 + b < W) {
              gv[b] = ld_stream4(grads + (long long)(w0 + b) * stride + idx);
              ev[b] = ld_stream4(err + (long long)(w0 + b) * stride + idx);
            }
#pragma unroll
          for (int b = 0; b < WB; ++b)
            if (w0 + b < W) {
              float4 e = ev[b];
              if (LAZY && rp > 0) { e.x -= corr.x; e.y -= corr.y; e.z -= corr.z; e.w -= corr.w; }
              const float4 m = make_float4(gv[b].x + e.x, gv[b].y + e.y, gv[b].z + e.z, gv[b].w + e.w);
              if (LAZY) st_stream4(err + (long long)(w0 + b) * stride + idx, m);
              else *reinterpret_cast<float4*>(err + (long long)(w0 + b) * stride + idx) = m;
              mb.x += m.x; mb.y += m.y; mb.z += m.z; mb.w += m.w;
              if (delta != nullptr && w0 + b == decider) {
                float4 d = *reinterpret_cast<const float4*>(delta + idx);
                d.x += gv[b].x; d.y += gv[b].y; d.z += gv[b].z; d.w += gv[b].w;
                *reinterpret_cast<float4*>(delta + idx) = d;
              }
            }
        }
        mb.x *= inv_w; mb.y *= inv_w; mb.z *= inv_w; mb.w *= inv_w;
        *reinterpret_cast<float4*>(out + idx) = mb;
        a0 = fmaf(mb.x, q0.x, a0); a1 = fmaf(mb.x, q0.y, a1); a2 = fmaf(mb.x, q0.z, a2); a3 = fmaf(mb.x, q0.w, a3);
        a0 = fmaf(mb.y, q1.x, a0); a1 = fmaf(mb.y, q1.y, a1); a2 = fmaf(mb.y, q1.z, a2); a3 = fmaf(mb.y, q1.w, a3);
        a0 = fmaf(mb.z, q2.x, a0); a1 = fmaf(mb.z, q2.y, a1); a2 = fmaf(mb.z, q2.z, a2); a3 = fmaf(mb.z, q2.w, a3);
        a0 = fmaf(mb.w, q3.x, a0); a1 = fmaf(mb.w, q3.y, a1); a2 = fmaf(mb.w, q3.z, a2); a3 = fmaf(mb.w, q3.w, a3);
      }
      if (gl < rg.head + rg.tail) {  // the unaligned ends of the row, one element per lane
        const int col = gl < rg.head ? gl : rg.head + 4 * rg.nbody4 + (gl - rg.head);
        const long long idx = rg.start + col;
        const float4 q0 = __ldg(Q4 + col);
        const float corr = (LAZY && rp > 0) ? lowrank_entry(pp, q0, rp) : 0.f;
        float mb = 0.f;
        for (int w = 0; w < W; ++w) {
          const float gv = grads[(long long)w * stride + idx];
          float e = err[(long long)w * stride + idx];
          if (LAZY && rp > 0) e -= corr;
          const float m = gv + e;
          err[(long long)w * stride + idx] = m;
          mb += m;
          if (delta != nullptr && w == decider) delta[idx] += gv;
        }
        mb *= inv_w;
        out[idx] = mb;
        a0 = fmaf(mb, q0.x, a0); a1 = fmaf(mb, q0.y, a1); a2 = fmaf(mb, q0.z, a2); a3 = fmaf(mb, q0.w, a3);
      }
    }
    a0 = group_sum(a0, lpr); a1 = group_sum(a1, lpr); a2 = group_sum(a2, lpr); a3 = group_sum(a3, lpr);
    if (valid && gl == 0) {
      if (L.nchunks > 1) {  // partial row of this column chunk; summed over chunks before orthonormalising
        p_part[L.ppart_base + (long long)row * L.nchunks + it.chunk] = make_float4(a0, a1, a2, a3);
      } else {
        float4 pv = P4[row];
        pv.x = a0;
        if (r > 1) pv.y = a1;
        if (r > 2) pv.z = a2;
        if (r > 3) pv.w = a3;
        P4[row] = pv;
      }
    }
  }
}

// Deterministic block-wide sum of doubles; every thread gets the result.
__device__ __forceinline__ double block_sum(double v, double* sm) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
  __syncthreads();
  double s = 0.0;
  const int nw = blockDim.x >> 5;
  for (int i = 0; i < nw; ++i) s += sm[i];
  return s;
}

// Pass 2.  One block per MATRIX layer: modified Gram-Schmidt on the first r columns of P, in place.
__global__ void __launch_bounds__(1024)
psgd_orthonormalise_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers,
                           float* __restrict__ p, const float4* __restrict__ p_part,
                           const uint8_t* __restrict__ level, int* __restrict__ pending, int rank_low, int rank_high,
                           float eps) {
  __shared__ double sm[32];
  const int l = mat_layers[blockIdx.x];
  const DevLayer L = layers[l];
  const int r = level[l] ? rank_low : rank_high;
  if (pending != nullptr && threadIdx.x == 0) pending[l] = r;  // lazy mode: this step's residual stays pending
  float* P = p + 4ll * L.p_row;
  const int n = L.rows;
  if (L.nchunks > 1) {  // rows split into column chunks: P = sum of the chunk partials, in chunk order
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      const float4* pp = p_part + L.ppart_base + (long long)i * L.nchunks;
      float4 acc = pp[0];
      for (int ch = 1; ch < L.nchunks; ++ch) { acc.x += pp[ch].x; acc.y += pp[ch].y; acc.z += pp[ch].z; acc.w += pp[ch].w; }
      P[4 * i] = acc.x;
      if (r > 1) P[4 * i + 1] = acc.y;
      if (r > 2) P[4 * i + 2] = acc.z;
      if (r > 3) P[4 * i + 3] = acc.w;
    }
  }
  for (int c = 0; c < r; ++c) {
    for (int j = 0; j < c; ++j) {
      double part = 0.0;
      for (int i = threadIdx.x; i < n; i += blockDim.x) part += (double)P[4 * i + j] * (double)P[4 * i + c];
      const float dot = (float)block_sum(part, sm);
      for (int i = threadIdx.x; i < n; i += blockDim.x) P[4 * i + c] = fmaf(-dot, P[4 * i + j], P[4 * i + c]);
    }
    double part = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) part += (double)P[4 * i + c] * (double)P[4 * i + c];
    const double nrm = sqrt(block_sum(part, sm));
    const float inv = (float)(1.0 / (nrm + (double)eps));
    for (int i = threadIdx.x; i < n; i += blockDim.x) P[4 * i + c] *= inv;
  }
}

template <int VEC>
struct VecT;
template <> struct VecT<4> { using type = float4; };
template <> struct VecT<2> { using type = float2; };
template <> struct VecT<1> { using type = float; };

template <int VEC>
__device__ __forceinline__ void qpart_cols(const ColItem& it, const DevLayer& L, const float* __restrict__ mbar,
                                           const float4* __restrict__ P4, float4* __restrict__ part) {
  using V = typename VecT<VEC>::type;
  const int col = it.col0 + (int)threadIdx.x * VEC;
  if (col >= L.cols) return;
  float acc[VEC][4];
#pragma unroll
  for (int e = 0; e < VEC; ++e) acc[e][0] = acc[e][1] = acc[e][2] = acc[e][3] = 0.f;
  const float* base = mbar + L.offset + (long long)it.row0 * L.cols + col;
  const float4* pr = P4 + it.row0;
#pragma unroll 8
  for (int i = 0; i < it.nrows; ++i) {
    const V mv = *reinterpret_cast<const V*>(base + (long long)i * L.cols);
    const float4 pv = __ldg(pr + i);
    const float* m = reinterpret_cast<const float*>(&mv);
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
      acc[e][0] = fmaf(m[e], pv.x, acc[e][0]);
      acc[e][1] = fmaf(m[e], pv.y, acc[e][1]);
      acc[e][2] = fmaf(m[e], pv.z, acc[e][2]);
      acc[e][3] = fmaf(m[e], pv.w, acc[e][3]);
    }
  }
  float4* dst = part + L.part_base + (long long)it.slab * L.cols + col;
#pragma unroll
  for (int e = 0; e < VEC; ++e) dst[e] = make_float4(acc[e][0], acc[e][1], acc[e][2], acc[e][3]);
}

// Pass 3.  One block per (row slab, column block): partial Q' = Mbar[slab]^T P^[slab]; each thread owns
// `vec` adjacent columns and walks the slab's rows.
__global__ void __launch_bounds__(kColBlockThreads)
psgd_qpartial_kernel(const DevLayer* __restrict__ layers, const ColItem* __restrict__ items,
                     const float* __restrict__ mbar, const float* __restrict__ p, float4* __restrict__ part) {
  const ColItem it = items[blockIdx.x];
  const DevLayer L = layers[it.layer];
  const float4* P4 = reinterpret_cast<const float4*>(p) + L.p_row;
  if (L.vec == 4) qpart_cols<4>(it, L, mbar, P4, part);
  else if (L.vec == 2) qpart_cols<2>(it, L, mbar, P4, part);
  else qpart_cols<1>(it, L, mbar, P4, part);
}

// Pass 4.  Sums the slab partials of 32 columns in a fixed order and stores the first r ranks of Q'.
__global__ void __launch_bounds__(256)
psgd_qreduce_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers,
                    const float4* __restrict__ part, float* __restrict__ q, const uint8_t* __restrict__ level,
                    int rank_low, int rank_high) {
  __shared__ float4 sm[8][32];
  const int l = mat_layers[blockIdx.y];
  const DevLayer L = layers[l];
  if ((int)blockIdx.x * 32 >= L.cols) return;
  const int cx = threadIdx.x & 31, gy = threadIdx.x >> 5;
  const int col = blockIdx.x * 32 + cx;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  if (col < L.cols) {
    for (int s = gy; s < L.nslabs; s += 8) {
      const float4 v = part[L.part_base + (long long)s * L.cols + col];
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
  }
  sm[gy][cx] = acc;
  __syncthreads();
  if (gy == 0 && col < L.cols) {
    float4 t = sm[0][cx];
    for (int g = 1; g < 8; ++g) { t.x += sm[g][cx].x; t.y += sm[g][cx].y; t.z += sm[g][cx].z; t.w += sm[g][cx].w; }
    const int r = level[l] ? rank_low : rank_high;
    float4* Q4 = reinterpret_cast<float4*>(q) + L.q_row;
    float4 qv = Q4[col];
    qv.x = t.x;
    if (r > 1) qv.y = t.y;
    if (r > 2) qv.z = t.z;
    if (r > 3) qv.w = t.w;
    Q4[col] = qv;
  }
}

// Pass 5.  One block per row slab, a group of `lpr` lanes per row:  A = P^ Q'^T (first r ranks);
//   WRITE_OUT: out = A;   UPDATE_ERR: err_w -= A for every worker.
// Eager step: both (r from the level).  Lazy step: WRITE_OUT only.  Flush: UPDATE_ERR only, r = pending rank.
template <int WB, bool WRITE_OUT, bool UPDATE_ERR>
__global__ void __launch_bounds__(256)
psgd_residual_kernel(const DevLayer* __restrict__ layers, const RowItem* __restrict__ items,
                     float* __restrict__ err, const float* __restrict__ q, const float* __restrict__ p,
                     const uint8_t* __restrict__ level, const int* __restrict__ pending, float* __restrict__ out,
                     long long stride, int W, int rank_low, int rank_high) {
  const RowItem it = items[blockIdx.x];
  const DevLayer L = layers[it.layer];
  const int r = pending != nullptr ? pending[it.layer] : (level[it.layer] ? rank_low : rank_high);
  if (r == 0) return;
  const float4* __restrict__ Q4 = reinterpret_cast<const float4*>(q) + L.q_row + it.col0;
  const float4* __restrict__ P4 = reinterpret_cast<const float4*>(p) + L.p_row;
  const int lpr = L.lpr, groups = 32 / lpr;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane / lpr, gl = lane - g * lpr;
  const int row_end = it.row0 + it.nrows;
  for (int row = it.row0 + warp * groups + g; row < row_end; row += 8 * groups) {
    const RowGeom rg = row_geom(L, it, row);
    const float4 pv = __ldg(P4 + row);
    for (int t = gl; t < rg.nbody4; t += lpr) {
      const int col = rg.head + 4 * t;
      const long long idx = rg.start + col;
      float4 a;
      a.x = lowrank_entry(pv, __ldg(Q4 + col), r);
      a.y = lowrank_entry(pv, __ldg(Q4 + col + 1), r);
      a.z = lowrank_entry(pv, __ldg(Q4 + col + 2), r);
      a.w = lowrank_entry(pv, __ldg(Q4 + col + 3), r);
      if (UPDATE_ERR) {
        for (int w0 = 0; w0 < W; w0 += WB) {
          float4 m[WB];
#pragma unroll
          for (int b = 0; b < WB; ++b)
            if (w0 + b < W) m[b] = ld_stream4(err + (long long)(w0 + b) * stride + idx);
#pragma unroll
          for (int b = 0; b < WB; ++b)
            if (w0 + b < W)
              st_stream4(err + (long long)(w0 + b) * stride + idx,
                         make_float4(m[b].x - a.x, m[b].y - a.y, m[b].z - a.z, m[b].w - a.w));
        }
      }
      if (WRITE_OUT) st_stream4(out + idx, a);
    }
    if (gl < rg.head + rg.tail) {
      const int col = gl < rg.head ? gl : rg.head + 4 * rg.nbody4 + (gl - rg.head);
      const long long idx = rg.start + col;
      const float a = lowrank_entry(pv, __ldg(Q4 + col), r);
      if (UPDATE_ERR)
        for (int w = 0; w < W; ++w) err[(long long)w * stride + idx] -= a;
      if (WRITE_OUT) out[idx] = a;
    }
  }
}

// Lazy mode only: after a flush no residual is pending.
__global__ void psgd_clear_pending_kernel(int* __restrict__ pending, int n_layers) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l < n_layers) pending[l] = 0;
}

cudaError_t launch_powersgd(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                            const uint8_t* level, float* out, float* delta, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const int n_items = (int)pl.row_items.size();
  const int n_vec = (int)pl.vec_tiles.size();
  const float inv_w = 1.0f / (float)c.n_workers;
  const bool lazy = (c.flags & ACC_FLAG_LAZY_RESIDUAL) != 0;
  if (n_items + n_vec > 0) {
    PhaseTimer pt(ctx, PH_PSGD_PROJECT, s);
    if (lazy)
      psgd_project_kernel<4, true><<<n_items + n_vec, 256, 0, s>>>(
          ctx->d_layers, ctx->d_row_items, n_items, ctx->d_tiles, ctx->d_vec_tiles, grads, err, q, p_hat, ctx->d_ppart,
          level, ctx->d_pending, out, delta, c.worker_stride, c.n_workers, c.decider, inv_w, c.rank_low, c.rank_high);
    else
      psgd_project_kernel<4, false><<<n_items + n_vec, 256, 0, s>>>(
          ctx->d_layers, ctx->d_row_items, n_items, ctx->d_tiles, ctx->d_vec_tiles, grads, err, q, p_hat, ctx->d_ppart,
          level, nullptr, out, delta, c.worker_stride, c.n_workers, c.decider, inv_w, c.rank_low, c.rank_high);
  }
  if (pl.n_mat > 0) {
    {
      PhaseTimer pt(ctx, PH_PSGD_ORTHO, s);
      psgd_orthonormalise_kernel<<<pl.n_mat, 1024, 0, s>>>(ctx->d_layers, ctx->d_mat_layers, p_hat, ctx->d_ppart, level,
                                                          lazy ? ctx->d_pending : nullptr, c.rank_low, c.rank_high,
                                                          c.gs_eps);
    }
    {
      PhaseTimer pt(ctx, PH_PSGD_QPARTIAL, s);
      psgd_qpartial_kernel<<<(unsigned)pl.col_items.size(), kColBlockThreads, 0, s>>>(
          ctx->d_layers, ctx->d_col_items, out, p_hat, ctx->d_part);
    }
    int max_cols = 0;
    for (int l : pl.mat_layers) max_cols = max_cols > pl.layers[l].cols ? max_cols : pl.layers[l].cols;
    {
      PhaseTimer pt(ctx, PH_PSGD_QREDUCE, s);
      psgd_qreduce_kernel<<<dim3((max_cols + 31) / 32, pl.n_mat), 256, 0, s>>>(
          ctx->d_layers, ctx->d_mat_layers, ctx->d_part, q, level, c.rank_low, c.rank_high);
    }
    {
      PhaseTimer pt(ctx, PH_PSGD_RESIDUAL, s);
      if (lazy)
        psgd_residual_kernel<4, true, false><<<n_items, 256, 0, s>>>(
            ctx->d_layers, ctx->d_row_items, err, q, p_hat, level, nullptr, out, c.worker_stride, c.n_workers,
            c.rank_low, c.rank_high);
      else
        psgd_residual_kernel<4, true, true><<<n_items, 256, 0, s>>>(
            ctx->d_layers, ctx->d_row_items, err, q, p_hat, level, nullptr, out, c.worker_stride, c.n_workers,
            c.rank_low, c.rank_high);
    }
  }
  return cudaGetLastError();
}

cudaError_t launch_powersgd_flush(acc_ctx* ctx, float* err, const float* q, const float* p_hat, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const int n_items = (int)pl.row_items.size();
  if (n_items > 0) {
    {
      PhaseTimer pt(ctx, PH_PSGD_FLUSH, s);
      psgd_residual_kernel<4, false, true><<<n_items, 256, 0, s>>>(
          ctx->d_layers, ctx->d_row_items, err, q, p_hat, nullptr, ctx->d_pending, nullptr, c.worker_stride,
          c.n_workers, c.rank_low, c.rank_high);
    }
    ctx->last_launches += 1;
    psgd_clear_pending_kernel<<<(c.n_layers + 127) / 128, 128, 0, s>>>(ctx->d_pending, c.n_layers);
  }
  return cudaGetLastError();
}

}  // namespace acc
