// Batch-size mode of the controller (Section 4.2: the same algorithm switches between B_low and B_high at the
// granularity of the whole model; Appendix A: large batches are simulated by accumulating the gradients of
// several backward passes before they are exchanged, and the batch size is only ever increased).
#include "acc_internal.cuh"

namespace acc {

// One block per (tile, worker), every layer:  acc_w <- (first ? 0 : acc_w) + g_w;  delta += g_decider.
__global__ void __launch_bounds__(256)
batch_accumulate_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles,
                        const float* __restrict__ grads, float* __restrict__ acc, float* __restrict__ delta,
                        long long stride, int decider, int first) {
  const Tile t = tiles[blockIdx.x];
  const int w = blockIdx.y;
  const long long base = layers[t.layer].offset + t.elem0;
  const float* g = grads + (long long)w * stride + base;
  float* a = acc + (long long)w * stride + base;
  const bool acc_delta = delta != nullptr && w == decider;
  float* d = delta + base;
  const int n4 = t.nelem >> 2;
  for (int i = threadIdx.x; i < n4; i += blockDim.x) {
    const float4 gv = ld_stream4(g + 4 * i);
    float4 av = gv;
    if (!first) {
      const float4 o = ld_stream4(a + 4 * i);
      av = make_float4(o.x + gv.x, o.y + gv.y, o.z + gv.z, o.w + gv.w);
    }
    st_stream4(a + 4 * i, av);
    if (acc_delta) {
      float4 dv = *reinterpret_cast<const float4*>(d + 4 * i);
      dv.x += gv.x; dv.y += gv.y; dv.z += gv.z; dv.w += gv.w;
      *reinterpret_cast<float4*>(d + 4 * i) = dv;
    }
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
    const float gv = g[i];
    a[i] = first ? gv : a[i] + gv;
    if (acc_delta) d[i] += gv;
  }
}

// One block per tile, every layer:  out = scale * sum_w acc_w, workers added in order (bit-reproducible),
// scale = 1 / (W * n_accum).  SGD: the optimiser tail is applied where out is written.
template <bool SGD>
__global__ void __launch_bounds__(256)
batch_average_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles,
                     const float* __restrict__ acc, float* __restrict__ out, long long stride, int W, float scale,
                     const SgdTail tail) {
  const Tile t = tiles[blockIdx.x];
  const long long base = layers[t.layer].offset + t.elem0;
  SgdHyper h = {0.f, 0.f, 0.f};
  if (SGD) h = sgd_hyper(tail);
  const int n4 = t.nelem >> 2;
  for (int i = threadIdx.x; i < n4; i += blockDim.x) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int w = 0; w < W; ++w) {
      const float4 v = ld_stream4(acc + (long long)w * stride + base + 4 * i);
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    s.x *= scale; s.y *= scale; s.z *= scale; s.w *= scale;
    st_stream4(out + base + 4 * i, s);
    if (SGD) sgd_apply4(tail, h, base + 4 * i, s);
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
    float s = 0.f;
    for (int w = 0; w < W; ++w) s += acc[(long long)w * stride + base + i];
    s *= scale;
    out[base + i] = s;
    if (SGD) sgd_apply1(tail, h, base + i, s);
  }
}

// One block.  Whole-model squared norm = sum of the per-layer squared norms (fp64, fixed order), then
// Algorithm 1 on it with B_low / B_high in place of the two compression levels; the batch size never decreases.
__global__ void __launch_bounds__(256)
detect_batch_kernel(const double* __restrict__ n2_layers, int n_layers, double* __restrict__ n2_prev, float lr_curr,
                    float lr_next, double eta, int b_low, int b_high, int32_t* __restrict__ batch,
                    float* __restrict__ lr_scale) {
  __shared__ double sm[256];
  double acc = 0.0;
  for (int l = threadIdx.x; l < n_layers; l += 256) acc += n2_layers[l];
  sm[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double cur = sm[0], prev = *n2_prev;
    bool critical = true;
    if (prev >= 0.0) {
      const double a = sqrt(prev), b = sqrt(cur);
      critical = fabs(a - b) >= eta * a || lr_next < lr_curr;
    }
    const int want = critical ? b_low : b_high;
    const int now = *batch;
    const int next = now > want ? now : want;
    *batch = next;
    *lr_scale = (float)next / (float)b_low;
    *n2_prev = cur;
  }
}

cudaError_t launch_batch_accumulate(acc_ctx* ctx, const float* grads, float* acc, float* delta, int first,
                                    cudaStream_t s) {
  dim3 grid((unsigned)ctx->plan.tiles.size(), (unsigned)ctx->cfg.n_workers);
  {
    PhaseTimer pt(ctx, PH_BATCH_ACCUMULATE, s);
    batch_accumulate_kernel<<<grid, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, grads, acc, delta,
                                                 ctx->cfg.worker_stride, ctx->cfg.decider, first);
  }
  return cudaGetLastError();
}

cudaError_t launch_batch_average(acc_ctx* ctx, const float* acc, int n_accum, float* out, SgdTail tail,
                                 cudaStream_t s) {
  const unsigned nt = (unsigned)ctx->plan.tiles.size();
  const float scale = 1.0f / ((float)ctx->cfg.n_workers * (float)n_accum);
  {
    PhaseTimer pt(ctx, PH_BATCH_AVERAGE, s);
    if (tail.params)
      batch_average_kernel<true><<<nt, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, acc, out, ctx->cfg.worker_stride,
                                                    ctx->cfg.n_workers, scale, tail);
    else
      batch_average_kernel<false><<<nt, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, acc, out, ctx->cfg.worker_stride,
                                                     ctx->cfg.n_workers, scale, tail);
  }
  return cudaGetLastError();
}

cudaError_t launch_detect_batch(acc_ctx* ctx, const double* n2_layers, double* n2_prev, float lr_curr, float lr_next,
                                int b_low, int b_high, int32_t* batch, float* lr_scale, cudaStream_t s) {
  {
    PhaseTimer pt(ctx, PH_DETECT_BATCH, s);
    detect_batch_kernel<<<1, 256, 0, s>>>(n2_layers, ctx->cfg.n_layers, n2_prev, lr_curr, lr_next,
                                          (double)ctx->cfg.eta, b_low, b_high, batch, lr_scale);
  }
  return cudaGetLastError();
}

}  // namespace acc
