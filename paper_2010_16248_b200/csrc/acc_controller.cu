// Error-feedback add, detector accumulation, per-layer norms and the regime test (Section 4.2, Algorithm 1).
#include "acc_internal.cuh"

namespace acc {

// One block per (tile, worker): err <- g + err on MATRIX tiles; delta += g for the deciding worker.
__global__ void __launch_bounds__(256) ef_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles,
                                                 const float* __restrict__ grads, float* __restrict__ err,
                                                 float* __restrict__ delta, long long stride, int decider) {
  const Tile t = tiles[blockIdx.x];
  const int w = blockIdx.y;
  const DevLayer L = layers[t.layer];
  const bool is_mat = L.kind == ACC_MATRIX;
  const bool acc_delta = (delta != nullptr) && (w == decider);
  if (!is_mat && !acc_delta) return;
  const long long base = L.offset + t.elem0;
  const float* g = grads + (long long)w * stride + base;
  float* e = err + (long long)w * stride + base;
  float* d = delta + base;
  const int n4 = t.nelem >> 2;
  // four float4 per thread at a time: all loads of a group before its first store, so that they are in flight
  // together (a store in between would hold the later loads of the same buffer back)
  constexpr int kGroup = 4, kThreads = 256;
  for (int i0 = 0; i0 < n4; i0 += kGroup * kThreads) {
    float4 gv[kGroup], ev[kGroup], dv[kGroup];
#pragma unroll
    for (int k = 0; k < kGroup; ++k) {
      const int i = i0 + k * kThreads + (int)threadIdx.x;
      if (i < n4) {
        gv[k] = ld_stream4(g + 4 * i);
        if (is_mat) ev[k] = ld_stream4(e + 4 * i);
        if (acc_delta) dv[k] = *reinterpret_cast<const float4*>(d + 4 * i);
      }
    }
#pragma unroll
    for (int k = 0; k < kGroup; ++k) {
      const int i = i0 + k * kThreads + (int)threadIdx.x;
      if (i < n4) {
        if (is_mat)
          st_stream4(e + 4 * i, make_float4(gv[k].x + ev[k].x, gv[k].y + ev[k].y, gv[k].z + ev[k].z, gv[k].w + ev[k].w));
        if (acc_delta)
          *reinterpret_cast<float4*>(d + 4 * i) =
              make_float4(dv[k].x + gv[k].x, dv[k].y + gv[k].y, dv[k].z + gv[k].z, dv[k].w + gv[k].w);
      }
    }
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
    const float gv = g[i];
    if (is_mat) e[i] = gv + e[i];
    if (acc_delta) d[i] += gv;
  }
}

// One block per (tile, buffer): fp64 sum of squares of the tile, reduced in a fixed order.
__global__ void __launch_bounds__(256) norm_partial_kernel(const DevLayer* __restrict__ layers,
                                                           const Tile* __restrict__ tiles,
                                                           const float* __restrict__ buf, long long stride,
                                                           const float* __restrict__ minus,
                                                           double* __restrict__ part, int n_tiles) {
  __shared__ double sm[8];
  const Tile t = tiles[blockIdx.x];
  const int b = blockIdx.y;
  const long long base = layers[t.layer].offset + t.elem0;
  const float* x = buf + (long long)b * stride + base;
  const float* y = minus != nullptr ? minus + base : nullptr;  // norms of (buf - minus), one buffer only
  double acc = 0.0;
  const int n4 = t.nelem >> 2;
  for (int i = threadIdx.x; i < n4; i += blockDim.x) {
    float4 v = ld_stream4(x + 4 * i);
    if (y != nullptr) {
      const float4 u = ld_stream4(y + 4 * i);
      v.x -= u.x; v.y -= u.y; v.z -= u.z; v.w -= u.w;
    }
    acc += (double)v.x * v.x;
    acc += (double)v.y * v.y;
    acc += (double)v.z * v.z;
    acc += (double)v.w * v.w;
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
    const float v = y != nullptr ? x[i] - y[i] : x[i];
    acc += (double)v * v;
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += sm[i];
    part[(long long)b * n_tiles + blockIdx.x] = s;
  }
}

// One warp per (layer, buffer): sums the layer's tile partials in a fixed order.
__global__ void norm_final_kernel(const DevLayer* __restrict__ layers, const double* __restrict__ part,
                                  double* __restrict__ norm2, int n_layers, int n_tiles) {
  const int l = blockIdx.x, b = blockIdx.y;
  const DevLayer L = layers[l];
  double acc = 0.0;
  for (int i = threadIdx.x; i < L.ntiles; i += 32) acc += part[(long long)b * n_tiles + L.tile0 + i];
  acc = warp_sum(acc);
  if (threadIdx.x == 0) norm2[(long long)b * n_layers + l] = acc;
}

// One block per (tile, buffer): fp64 sum and sum of squares of the tile (the two moments behind the
// mean-to-standard-deviation ratio; the sum of squares is also the tile's share of the layer norm of Section 4.2),
// reduced in a fixed order.  part holds [buffer][tile][2].
__global__ void __launch_bounds__(256) moments_partial_kernel(const DevLayer* __restrict__ layers,
                                                              const Tile* __restrict__ tiles,
                                                              const float* __restrict__ buf, long long stride,
                                                              double* __restrict__ part, int n_tiles) {
  __shared__ double sm[2][8];
  const Tile t = tiles[blockIdx.x];
  const int b = blockIdx.y;
  const float* x = buf + (long long)b * stride + layers[t.layer].offset + t.elem0;
  double s1 = 0.0, s2 = 0.0;
  const int n4 = t.nelem >> 2;
  for (int i = threadIdx.x; i < n4; i += blockDim.x) {
    const float4 v = ld_stream4(x + 4 * i);
    s1 += (double)v.x; s2 += (double)v.x * v.x;
    s1 += (double)v.y; s2 += (double)v.y * v.y;
    s1 += (double)v.z; s2 += (double)v.z * v.z;
    s1 += (double)v.w; s2 += (double)v.w * v.w;
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
    const float v = x[i];
    s1 += (double)v; s2 += (double)v * v;
  }
  s1 = warp_sum(s1);
  s2 = warp_sum(s2);
  if ((threadIdx.x & 31) == 0) { sm[0][threadIdx.x >> 5] = s1; sm[1][threadIdx.x >> 5] = s2; }
  __syncthreads();
  if (threadIdx.x < 2) {
    double s = 0.0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += sm[threadIdx.x][i];
    part[2 * ((long long)b * n_tiles + blockIdx.x) + threadIdx.x] = s;
  }
}

// One warp per (layer, buffer): the layer's moments from its tile partials in a fixed order, then
//   mean = S1 / n,  var = max(S2 / n - mean^2, 0),  msdr = |mean| / sqrt(var)   (0 when mean = 0, +inf when var = 0).
__global__ void moments_final_kernel(const DevLayer* __restrict__ layers, const double* __restrict__ part,
                                     double* __restrict__ moments, double* __restrict__ msdr, int n_layers,
                                     int n_tiles) {
  const int l = blockIdx.x, b = blockIdx.y;
  const DevLayer L = layers[l];
  double s1 = 0.0, s2 = 0.0;
  for (int i = threadIdx.x; i < L.ntiles; i += 32) {
    const double* p = part + 2 * ((long long)b * n_tiles + L.tile0 + i);
    s1 += p[0]; s2 += p[1];
  }
  s1 = warp_sum(s1);
  s2 = warp_sum(s2);
  if (threadIdx.x == 0) {
    const double n = (double)L.rows * (double)L.cols;
    const double mean = s1 / n;
    double var = s2 / n - mean * mean;
    var = var > 0.0 ? var : 0.0;
    const long long o = (long long)b * n_layers + l;
    moments[2 * o] = s1;
    moments[2 * o + 1] = s2;
    msdr[o] = mean == 0.0 ? 0.0 : fabs(mean) / sqrt(var);  // var == 0: +inf
  }
}

// Algorithm 1 per layer, in product form so that a zero previous norm needs no division.
// With n2d (squared norms of the difference of the two accumulated gradients) the variant criterion
// ||D_prev - D_curr|| >= eta ||D_prev|| is used instead of | ||D_prev|| - ||D_curr|| | >= eta ||D_prev||.
// With lr_dev (two DEVICE floats: current and next learning rate) the rates are read from there instead of the
// arguments, so that a captured graph follows a learning-rate schedule.
__global__ void detect_kernel(const double* __restrict__ n2c, double* __restrict__ n2p,
                              const double* __restrict__ n2d, float lr_curr, float lr_next,
                              const float* __restrict__ lr_dev, double eta, uint8_t* __restrict__ level,
                              int n_layers) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l >= n_layers) return;
  if (lr_dev != nullptr) { lr_curr = lr_dev[0]; lr_next = lr_dev[1]; }
  const double cur = n2c[l], prev = n2p[l];
  uint8_t lv;
  if (prev < 0.0) {
    lv = 1;
  } else {
    const double a = sqrt(prev), b = sqrt(cur);
    const double change = n2d != nullptr ? sqrt(n2d[l]) : fabs(a - b);
    lv = (change >= eta * a || lr_next < lr_curr) ? 1 : 0;
  }
  level[l] = lv;
  n2p[l] = cur;
}

cudaError_t launch_error_feedback(acc_ctx* ctx, const float* grads, float* err, float* delta, cudaStream_t s) {
  dim3 grid((unsigned)ctx->plan.tiles.size(), (unsigned)ctx->cfg.n_workers);
  {
    PhaseTimer pt(ctx, PH_EF, s);
    ef_kernel<<<grid, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, grads, err, delta, ctx->cfg.worker_stride,
                                   ctx->cfg.decider);
  }
  return cudaGetLastError();
}

cudaError_t launch_layer_norms(acc_ctx* ctx, const float* buf, long long stride, int n_bufs, const float* minus,
                               double* norm2, cudaStream_t s) {
  const int nt = (int)ctx->plan.tiles.size();
  {
    PhaseTimer pt(ctx, PH_NORM_PARTIAL, s);
    norm_partial_kernel<<<dim3((unsigned)nt, (unsigned)n_bufs), 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, buf, stride,
                                                                            minus, ctx->d_norm_part, nt);
  }
  {
    PhaseTimer pt(ctx, PH_NORM_FINAL, s);
    norm_final_kernel<<<dim3((unsigned)ctx->cfg.n_layers, (unsigned)n_bufs), 32, 0, s>>>(
        ctx->d_layers, ctx->d_norm_part, norm2, ctx->cfg.n_layers, nt);
  }
  return cudaGetLastError();
}

cudaError_t launch_layer_msdr(acc_ctx* ctx, const float* buf, long long stride, int n_bufs, double* moments,
                              double* msdr, cudaStream_t s) {
  const int nt = (int)ctx->plan.tiles.size();
  {
    PhaseTimer pt(ctx, PH_MOMENTS_PARTIAL, s);
    moments_partial_kernel<<<dim3((unsigned)nt, (unsigned)n_bufs), 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, buf,
                                                                               stride, ctx->d_norm_part, nt);
  }
  {
    PhaseTimer pt(ctx, PH_MOMENTS_FINAL, s);
    moments_final_kernel<<<dim3((unsigned)ctx->cfg.n_layers, (unsigned)n_bufs), 32, 0, s>>>(
        ctx->d_layers, ctx->d_norm_part, moments, msdr, ctx->cfg.n_layers, nt);
  }
  return cudaGetLastError();
}

cudaError_t launch_detect(acc_ctx* ctx, const double* n2c, double* n2p, const double* n2d, float lr_curr,
                          float lr_next, const float* lr_dev, uint8_t* level, cudaStream_t s) {
  const int L = ctx->cfg.n_layers;
  {
    PhaseTimer pt(ctx, PH_DETECT, s);
    detect_kernel<<<(L + 127) / 128, 128, 0, s>>>(n2c, n2p, n2d, lr_curr, lr_next, lr_dev, (double)ctx->cfg.eta, level,
                                                  L);
  }
  return cudaGetLastError();
}

}  // namespace acc
