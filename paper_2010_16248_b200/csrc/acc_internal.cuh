// Internal declarations shared by the CUDA translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "acc.h"

namespace acc {

constexpr int kTile = 8192;        // elements per flat tile (TopK / EF / norms); multiple of 4
constexpr int kBins1 = 4096;       // radix-select level 1: key bits [30:19]
constexpr int kBins2 = 4096;       // level 2: key bits [18:7]
constexpr int kBins3 = 128;        // level 3: key bits [6:0]
constexpr int kColBlockThreads = 256;
constexpr int kMaxWorkers = 1024;  // workers per context

// One layer, device-side view.
struct DevLayer {
  long long offset;   // element offset inside a worker's slice
  int rows, cols, kind;
  double inv_cols;    // 1.0 / cols, for row = index / cols without an integer division
  int q_row, p_row;   // first row of the layer's block in q / p_hat (MATRIX), else -1
  int vec;            // widest vector width (4, 2, 1) at which every row start is aligned
  int nslots;         // tiles a row of this layer can touch: (cols - 1) / 8192 + 2
  long long ppart_base;  // first float4 of the layer's partial P rows, [rows][nslots]
  int mat;            // index among MATRIX layers, else -1
  int tile0, ntiles;  // flat tiles of this layer: [tile0, tile0 + ntiles)
  int k_low, k_high;  // TopK counts
  long long seg_off;  // first packed entry of the layer inside a worker's packed region
  long long cand_base;  // first slot of the layer's candidate keys inside a worker's candidate region
  int cand_cap;         // slots of that list (the list path is taken when bucket b1 fits)
  long long part_base;  // first float4 of the layer's Q partials
  int slab_rows, nslabs;  // row slabs of the Q-partial pass
  long long vec_off;      // VECTOR layers: first float of the layer inside the packed exchange region, else -1
};

struct ColItem { int layer, slab, row0, nrows, col0; };  // (row slab, column block) of a MATRIX layer
struct Tile { int layer, elem0, nelem; };              // flat tile, never spans layers

// Per (worker, MATRIX layer) state of the radix select.
struct Select {
  unsigned b1, b2;      // chosen buckets of level 1 and 2
  unsigned tau;         // 31-bit key of the k-th largest magnitude
  int k, k1, k2, need;  // k wanted; still wanted inside bucket b1 / (b1,b2); ties (key == tau) to keep
  int mode;             // kSelDense: levels 2-3 read M;  kSelList: they read the collected keys of bucket b1
};
constexpr int kSelDense = 0, kSelList = 1, kSelListPred = 2, kSelStaged = 3, kSelZeroFill = 4;
// ListPred: the key list was filled by pass A;  Staged: pass A staged whole (value, index) entries;
// ZeroFill: the threshold is 0 (k exceeds the non-zero entries): settled from the first pass's per-tile counts
// Work lists of (worker, tile) pairs, rebuilt every step on the device, so that the passes that serve only some
// segments launch as many blocks as there is work: tiles of segments whose bucket is collected by the collect
// pass, tiles of dense segments, tiles the select pass must read, tiles served from staged entries.
constexpr int kListCollect = 0, kListDense = 1, kListSelect = 2, kListStaged = 3, kNumLists = 4;
constexpr int kListCountWord = 8;  // the lists' lengths live at words 8..11 of the per-step word block
constexpr int kTicketWord = 16;    // tile ticket of the decompress pass, same block (cleared at the start of a step)
constexpr unsigned kNoPendingTau = 0xffffffffu;  // no key is larger: nothing pending
constexpr int kPredTileCap = 2048;  // keys one tile may hand to a predicted list (more: overflow, fall back)

// Kernels of the library, for per-kernel timing (acc_profile_*).
enum Phase {
  PH_EF = 0, PH_NORM_PARTIAL, PH_NORM_FINAL, PH_DETECT,
  PH_PSGD_PROJECT, PH_PSGD_ORTHO, PH_PSGD_QPARTIAL, PH_PSGD_QREDUCE, PH_PSGD_RESIDUAL,
  PH_TOPK_EF_HIST1, PH_TOPK_PICK1, PH_TOPK_HIST2, PH_TOPK_PICK2, PH_TOPK_HIST3, PH_TOPK_PICK3_SCAN, PH_TOPK_SELECT,
  PH_TOPK_DECOMPRESS, PH_PSGD_FLUSH, PH_TOPK_COLLECT, PH_TOPK_PICK3, PH_TOPK_TILE_COUNTS, PH_TOPK_HIST2_LIST, PH_TOPK_HIST3_LIST, PH_TOPK_FINALIZE_STAGED, PH_PSGD_ORTHO_BLOCK, PH_SGD_TILES, PH_BATCH_ACCUMULATE, PH_BATCH_AVERAGE, PH_DETECT_BATCH,
  PH_PSGD_PFOLD, PH_VEC_EXCHANGE, PH_PSGD_QMERGE, PH_TOPK_DECOMPRESS_PACKED, PH_TOPK_FLUSH,
  PH_MOMENTS_PARTIAL, PH_MOMENTS_FINAL,
  PH_COUNT
};

struct ProfSlot { int phase; cudaEvent_t a, b; };

struct Plan {
  std::vector<DevLayer> layers;
  std::vector<ColItem> col_items;
  std::vector<int2> qred_items;  // (layer, block of 32 columns) of every MATRIX layer: the grid of the Q-reduce pass
  std::vector<Tile> tiles;
  std::vector<int> mat_layers;   // layer index of each MATRIX layer
  std::vector<int> vec_tiles;    // tile indices that belong to VECTOR layers
  std::vector<int> mat_tiles;    // tile indices that belong to MATRIX layers, in order
  long long q_rows = 0, p_rows = 0, capacity = 0, part_f4 = 0, cand_total = 0, ppart_f4 = 0;
  int n_mat = 0;
  int max_rows = 0;  // most rows of any MATRIX layer
  int max_cols = 0;  // most columns of any MATRIX layer
  long long vec_floats = 0;  // packed VECTOR elements (each layer starts at a multiple of 4)
  // workspace offsets (bytes)
  size_t o_qred_items = 0;
  size_t o_layers = 0, o_col_items = 0, o_tiles = 0, o_mat_layers = 0, o_vec_tiles = 0, o_mat_tiles = 0, o_status = 0,
         o_part = 0, o_ppart = 0, o_pending = 0, o_norm_part = 0, o_hist = 0, o_sel = 0, o_pred = 0, o_cand = 0, o_tile_cand = 0, o_tile_cnt = 0, o_tile_h3 = 0, o_tile_pre = 0, o_tile_rng = 0, o_lists = 0, o_pend_tau = 0,
         hist_bytes = 0, total = 0;
};

}  // namespace acc

struct acc_ctx {
  acc_config cfg;
  std::vector<acc_layer_desc> host_layers;
  acc::Plan plan;
  char* ws = nullptr;
  int sm_count = 148;
  int occ_topk_first_pass = 3;       // resident blocks per SM of topk_ef_hist1_kernel (queried at creation)
  int last_launches = 0;
  bool prof = false;                 // per-kernel event timing on
  std::vector<acc::ProfSlot> prof_slots;
  size_t prof_used = 0;
  // device views into the workspace
  acc::DevLayer* d_layers = nullptr;
  acc::ColItem* d_col_items = nullptr;
  int2* d_qred_items = nullptr;
  acc::Tile* d_tiles = nullptr;
  int* d_mat_layers = nullptr;
  int* d_vec_tiles = nullptr;
  int* d_mat_tiles = nullptr;
  int* d_status = nullptr;           // 64 words: [0] device-side error flag (0 = none), see acc_device_status;
                                     // [8], [9] tile ticket and finished-block count of the pipelined first PowerSGD pass
  float4* d_part = nullptr;
  float4* d_ppart = nullptr;         // partial rows of P, one slot per tile a row touches
  int* d_pending = nullptr;          // lazy PowerSGD: rank of the residual not yet applied to err, per layer
  double* d_norm_part = nullptr;
  unsigned* d_hist1 = nullptr;
  unsigned* d_hist2 = nullptr;
  unsigned* d_hist3 = nullptr;
  acc::Select* d_sel = nullptr;
  unsigned* d_seg_cand = nullptr;    // per (worker, layer): candidate slots handed out this step
  unsigned* d_any_list = nullptr;    // per-step word block, cleared with the histograms; words 8..11: lengths of the work lists
  unsigned* d_seg_flag = nullptr;    // per (worker, layer): 1 if pass A's collection overflowed this step
  unsigned* d_pred = nullptr;        // [6][W * n_mat]: prediction word, last threshold bucket, last move of the bucket, each per level; kept across steps
  unsigned* d_cand = nullptr;        // candidate keys, [W][cand_total]
  int2* d_tile_cand = nullptr;       // per (worker, tile): (first slot, count) inside the segment's list
  int2* d_tile_cnt = nullptr;
  unsigned short* d_tile_h3 = nullptr;
  int2* d_tile_pre = nullptr;
  int2* d_tile_rng = nullptr;        // per (worker, tile): the tile's entries [first, end) inside the worker's packed segment
  int2* d_lists = nullptr;           // [kNumLists][W * tiles] work lists of (worker, tile)
  unsigned* d_pend_tau = nullptr;    // lazy TopK: per (worker, layer) threshold of the last step whose kept entries
                                     // (key > threshold) are still to be zeroed in err; kNoPendingTau: none
};

namespace acc {

// Optimiser tail (Nesterov momentum, Appendix A) applied by the kernels that produce `out`, at the element
// they have just computed.  params == nullptr: no tail.  hyper: three DEVICE floats (learning rate, momentum,
// weight decay), read by the kernels so that a captured graph follows a learning-rate schedule.
struct SgdTail { float* params; float* mom; const float* hyper; };

// Kernel launchers (one per translation unit).  Each returns a cudaError_t from cudaGetLastError and
// adds the number of kernels it launched to ctx->last_launches.
cudaError_t launch_error_feedback(acc_ctx* ctx, const float* grads, float* err, float* delta, cudaStream_t s);
cudaError_t launch_layer_norms(acc_ctx* ctx, const float* buf, long long stride, int n_bufs, const float* minus,
                               double* norm2, cudaStream_t s);
cudaError_t launch_layer_msdr(acc_ctx* ctx, const float* buf, long long stride, int n_bufs, double* moments,
                              double* msdr, cudaStream_t s);
cudaError_t launch_detect(acc_ctx* ctx, const double* n2c, double* n2p, const double* n2d, float lr_curr,
                          float lr_next, const float* lr_dev, uint8_t* level, cudaStream_t s);
cudaError_t launch_powersgd(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                            const uint8_t* level, float* out, float* delta, SgdTail tail, cudaStream_t s);
cudaError_t prepare_powersgd();
cudaError_t launch_selftest_wait(acc_ctx* ctx, cudaStream_t s);
// Real workers: the step in three parts, around the two exchanges (x1: P rows + packed VECTOR means, x2: Q' rows).
cudaError_t launch_powersgd_phase1(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                                   const uint8_t* level, float* out, float* delta, float* x1, cudaStream_t s);
cudaError_t launch_powersgd_phase2(acc_ctx* ctx, const float* x1, float scale, float* p_hat, const uint8_t* level,
                                   const float* out, float* x2, cudaStream_t s);
cudaError_t launch_powersgd_phase3(acc_ctx* ctx, float* err, float* q, const float* p_hat, const uint8_t* level,
                                   const float* x1, const float* x2, float scale, float* out, SgdTail tail,
                                   cudaStream_t s);
cudaError_t launch_powersgd_flush(acc_ctx* ctx, float* err, const float* q, const float* p_hat, cudaStream_t s);
cudaError_t launch_topk(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals,
                        int32_t* idx, int32_t* counts, float* out, float* delta, SgdTail tail, cudaStream_t s);
// Real workers: the TopK step in two halves around the all-gather of the packed sets.
cudaError_t launch_topk_flush(acc_ctx* ctx, float* err, cudaStream_t s);
cudaError_t prepare_topk(acc_ctx* ctx);
cudaError_t launch_topk_compress(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals,
                                 int32_t* idx, int32_t* counts, float* delta, float* vec_packed, cudaStream_t s);
cudaError_t launch_topk_decompress_packed(acc_ctx* ctx, const float* vals, const int32_t* idx, const int32_t* counts,
                                          int n_sets, const float* vec_packed, float vec_scale, float* out,
                                          SgdTail tail, cudaStream_t s);
// Optimiser tail on its own over the given tiles (tile_ids == nullptr: all tiles, in order).
cudaError_t launch_sgd_tiles(acc_ctx* ctx, const int* tile_ids, int n, const float* d, SgdTail tail, cudaStream_t s);
cudaError_t launch_batch_accumulate(acc_ctx* ctx, const float* grads, float* acc, float* delta, int first,
                                    cudaStream_t s);
cudaError_t launch_batch_average(acc_ctx* ctx, const float* acc, int n_accum, float* out, SgdTail tail,
                                 cudaStream_t s);
cudaError_t launch_detect_batch(acc_ctx* ctx, const double* n2_layers, double* n2_prev, float lr_curr, float lr_next,
                                int b_low, int b_high, int32_t* batch, float* lr_scale, cudaStream_t s);

// Brackets one kernel launch with CUDA events on its stream when profiling is on; counts the launch.
struct PhaseTimer {
  acc_ctx* ctx; cudaStream_t s; ProfSlot* slot = nullptr;
  PhaseTimer(acc_ctx* c, int phase, cudaStream_t st) : ctx(c), s(st) {
    ctx->last_launches += 1;
    if (!ctx->prof) return;
    if (ctx->prof_used == ctx->prof_slots.size()) {
      ProfSlot n{phase, nullptr, nullptr};
      if (cudaEventCreate(&n.a) != cudaSuccess || cudaEventCreate(&n.b) != cudaSuccess) return;
      ctx->prof_slots.push_back(n);
    }
    slot = &ctx->prof_slots[ctx->prof_used++];
    slot->phase = phase;
    cudaEventRecord(slot->a, s);
  }
  ~PhaseTimer() { if (slot) cudaEventRecord(slot->b, s); }
};

// ---- small device helpers -------------------------------------------------------------------------
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
__device__ __forceinline__ float4 ld_stream4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float ld_stream1(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

struct SgdHyper { float lr, mu, wd; };
__device__ __forceinline__ SgdHyper sgd_hyper(const SgdTail& t) {
  SgdHyper h;
  h.lr = __ldg(t.hyper); h.mu = __ldg(t.hyper + 1); h.wd = __ldg(t.hyper + 2);
  return h;
}
// d' = d + wd x;  u <- mu u + d';  x <- x - lr (d' + mu u).  One fixed fp32 operation order everywhere, so the
// fused tails and the stand-alone kernel give the same bits.
__device__ __forceinline__ void sgd_update(float d, float& x, float& u, const SgdHyper& h) {
  const float dd = fmaf(h.wd, x, d);
  u = fmaf(h.mu, u, dd);
  x = fmaf(-h.lr, fmaf(h.mu, u, dd), x);
}
__device__ __forceinline__ void sgd_apply1(const SgdTail& t, const SgdHyper& h, long long i, float d) {
  float x = t.params[i], u = t.mom[i];
  sgd_update(d, x, u, h);
  t.params[i] = x; t.mom[i] = u;
}
__device__ __forceinline__ void sgd_apply4(const SgdTail& t, const SgdHyper& h, long long i, const float4 d) {
  float4 x = *reinterpret_cast<const float4*>(t.params + i), u = *reinterpret_cast<const float4*>(t.mom + i);
  sgd_update(d.x, x.x, u.x, h); sgd_update(d.y, x.y, u.y, h);
  sgd_update(d.z, x.z, u.z, h); sgd_update(d.w, x.w, u.w, h);
  *reinterpret_cast<float4*>(t.params + i) = x;
  *reinterpret_cast<float4*>(t.mom + i) = u;
}

// One VECTOR tile: mean over the workers of the tile's gradients, four elements per thread and step, the W loads
// of a step in flight together; the deciding worker's values are added to delta after the loop (no
// read-modify-write between the loads).  emit4(i, v) / emit1(i, v) receive the means of elements [i, i+4) / i.
template <typename Emit4, typename Emit1>
__device__ __forceinline__ void vector_tile_mean(const float* __restrict__ g /* worker 0, first element */,
                                                 long long stride, int W, int decider, float inv_w, int nelem,
                                                 float* __restrict__ delta /* first element, or nullptr */,
                                                 Emit4 emit4, Emit1 emit1) {
  const int n4 = nelem >> 2;
  for (int f = threadIdx.x; f < n4; f += blockDim.x) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), gd = a;
#pragma unroll 8
    for (int w = 0; w < W; ++w) {
      const float4 v = ld_stream4(g + (long long)w * stride + 4 * f);
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
      if (w == decider) gd = v;
    }
    if (delta != nullptr) {
      float4 d = *reinterpret_cast<const float4*>(delta + 4 * f);
      d.x += gd.x; d.y += gd.y; d.z += gd.z; d.w += gd.w;
      *reinterpret_cast<float4*>(delta + 4 * f) = d;
    }
    emit4(4 * f, make_float4(a.x * inv_w, a.y * inv_w, a.z * inv_w, a.w * inv_w));
  }
  for (int i = 4 * n4 + threadIdx.x; i < nelem; i += blockDim.x) {
    float a = 0.f, gd = 0.f;
    for (int w = 0; w < W; ++w) {
      const float v = g[(long long)w * stride + i];
      a += v;
      gd = w == decider ? v : gd;
    }
    if (delta != nullptr) delta[i] += gd;
    emit1(i, a * inv_w);
  }
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace acc
