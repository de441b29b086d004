// C-ABI entry points: configuration checks, launch-table planning, workspace layout.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>

#include "acc_internal.cuh"

namespace acc {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static int topk_count(long long size, int bp) {
  long long k = size * (long long)bp / 10000;
  return (int)std::max<long long>(1, k);
}

static int validate(const acc_config* cfg) {
  if (!cfg || !cfg->layers) return ACC_EINVAL;
  if (cfg->n_workers < 1 || cfg->n_workers > kMaxWorkers || cfg->n_layers < 1) return ACC_EINVAL;
  if (cfg->flags & ~(ACC_FLAG_LAZY_RESIDUAL | ACC_FLAG_PIPELINE_ALWAYS | ACC_FLAG_PIPELINE_NEVER | ACC_FLAG_SHARE_SMS))
    return ACC_EINVAL;
  if ((cfg->flags & ACC_FLAG_PIPELINE_ALWAYS) && (cfg->flags & ACC_FLAG_PIPELINE_NEVER)) return ACC_EINVAL;
  if (cfg->rank_high < 1 || cfg->rank_low < cfg->rank_high || cfg->rank_low > ACC_MAX_RANK) return ACC_EINVAL;
  if (cfg->topk_high_bp < 1 || cfg->topk_low_bp < cfg->topk_high_bp || cfg->topk_low_bp > 10000) return ACC_EINVAL;
  if (!(cfg->eta >= 0.f) || !(cfg->gs_eps >= 0.f)) return ACC_EINVAL;
  if (cfg->decider < 0 || cfg->decider >= cfg->n_workers) return ACC_EINVAL;
  if (cfg->worker_stride < 4) return ACC_EINVAL;
  if (cfg->worker_stride % 4 != 0) return ACC_EALIGN;
  long long prev_end = 0;
  long long rows_total = 0, cols_total = 0;
  for (int l = 0; l < cfg->n_layers; ++l) {
    const acc_layer_desc& d = cfg->layers[l];
    if (d.kind != ACC_MATRIX && d.kind != ACC_VECTOR) return ACC_EINVAL;
    if (d.rows < 1 || d.cols < 1) return ACC_EINVAL;
    if (d.kind == ACC_VECTOR && d.rows != 1) return ACC_EINVAL;
    if (d.offset < 0) return ACC_EINVAL;
    if (d.offset % 4 != 0) return ACC_EALIGN;
    long long size = (long long)d.rows * d.cols;
    if (size >= (1ll << 31) - kTile) return ACC_EINVAL;          // layer-local indices are int32
    if (d.offset < prev_end) return ACC_EINVAL;                  // layers in order, no overlap
    prev_end = d.offset + size;
    if (prev_end > cfg->worker_stride) return ACC_EINVAL;
    if (d.kind == ACC_MATRIX) { rows_total += d.rows; cols_total += d.cols; }
  }
  if (rows_total >= (1ll << 31) || cols_total >= (1ll << 31)) return ACC_EINVAL;
  return ACC_OK;
}

static int make_plan(const acc_config* cfg, Plan& p) {
  int st = validate(cfg);
  if (st != ACC_OK) return st;
  const int L = cfg->n_layers, W = cfg->n_workers;
  p.layers.resize(L);
  for (int l = 0; l < L; ++l) {
    const acc_layer_desc& d = cfg->layers[l];
    DevLayer& o = p.layers[l];
    memset(&o, 0, sizeof(o));
    o.offset = d.offset; o.rows = d.rows; o.cols = d.cols; o.kind = d.kind;
    o.inv_cols = 1.0 / (double)d.cols;
    o.q_row = o.p_row = o.mat = -1; o.seg_off = -1; o.part_base = -1; o.vec_off = -1;
    o.vec = (d.cols % 4 == 0) ? 4 : (d.cols % 2 == 0) ? 2 : 1;
    const long long size = (long long)d.rows * d.cols;
    // flat tiles
    o.tile0 = (int)p.tiles.size();
    for (long long e = 0; e < size; e += kTile) {
      Tile t{l, (int)e, (int)std::min<long long>(kTile, size - e)};
      if (d.kind == ACC_VECTOR) p.vec_tiles.push_back((int)p.tiles.size());
      else p.mat_tiles.push_back((int)p.tiles.size());
      p.tiles.push_back(t);
    }
    o.ntiles = (int)p.tiles.size() - o.tile0;
    if (d.kind != ACC_MATRIX) {
      o.vec_off = p.vec_floats;
      p.vec_floats += (size + 3) / 4 * 4;
      continue;
    }
    o.mat = p.n_mat++;
    p.max_rows = std::max(p.max_rows, d.rows);
    p.max_cols = std::max(p.max_cols, d.cols);
    p.mat_layers.push_back(l);
    o.q_row = (int)p.q_rows; p.q_rows += d.cols;
    o.p_row = (int)p.p_rows; p.p_rows += d.rows;
    o.k_low = topk_count(size, cfg->topk_low_bp);
    o.k_high = topk_count(size, cfg->topk_high_bp);
    o.seg_off = p.capacity; p.capacity += o.k_low;
    o.cand_cap = (int)std::max<long long>(64, (size / 4 + 3) / 4 * 4);
    o.cand_base = p.cand_total; p.cand_total += o.cand_cap;
    // row slabs of the row-wise passes: about kRowSlabElems elements per worker, whole rows,
    // a multiple of 8 rows (one row per warp of a 256-thread block) where the layer allows it
    // partial rows of P: one slot per tile a row can touch
    o.nslots = (d.cols - 1) / kTile + 2;
    o.ppart_base = p.ppart_f4; p.ppart_f4 += (long long)d.rows * o.nslots;
    // row slabs x column blocks of the Q-partial pass (each thread owns `vec` adjacent columns)
    o.slab_rows = std::min(d.rows, std::min(64, std::max(32, (d.rows + 511) / 512)));
    o.nslabs = (d.rows + o.slab_rows - 1) / o.slab_rows;
    o.part_base = p.part_f4; p.part_f4 += (long long)o.nslabs * d.cols;
    const int cb = kColBlockThreads * o.vec;
    for (int s = 0; s < o.nslabs; ++s)
      for (int c0 = 0; c0 < d.cols; c0 += cb)
        p.col_items.push_back(ColItem{l, s, s * o.slab_rows, std::min(o.slab_rows, d.rows - s * o.slab_rows), c0});
    for (int c0 = 0; c0 < d.cols; c0 += 32) p.qred_items.push_back(make_int2(l, c0 / 32));
  }
  const size_t nt = p.tiles.size();
  const size_t seg = (size_t)W * std::max(p.n_mat, 1);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  p.o_layers = take(sizeof(DevLayer) * L);
  p.o_col_items = take(sizeof(ColItem) * std::max<size_t>(1, p.col_items.size()));
  p.o_qred_items = take(sizeof(int2) * std::max<size_t>(1, p.qred_items.size()));
  p.o_tiles = take(sizeof(Tile) * nt);
  p.o_mat_layers = take(sizeof(int) * std::max<size_t>(1, p.mat_layers.size()));
  p.o_vec_tiles = take(sizeof(int) * std::max<size_t>(1, p.vec_tiles.size()));
  p.o_mat_tiles = take(sizeof(int) * std::max<size_t>(1, p.mat_tiles.size()));
  p.o_status = take(sizeof(int) * 64);
  p.o_part = take(sizeof(float4) * std::max<long long>(1, p.part_f4));
  p.o_ppart = take(sizeof(float4) * std::max<long long>(1, p.ppart_f4));
  p.o_pending = take(sizeof(int) * L);
  p.o_norm_part = take(sizeof(double) * 2 * (size_t)W * nt);  // per (buffer, tile): sum of squares, or (sum, sum of squares)
  p.o_hist = o;
  take(sizeof(unsigned) * seg * kBins1);
  take(sizeof(unsigned) * seg * kBins2);
  take(sizeof(unsigned) * seg * kBins3);
  take(sizeof(unsigned) * seg);  // candidate counters, cleared with the histograms
  take(sizeof(unsigned) * seg);  // overflow flags of the predicted collection, likewise
  take(sizeof(unsigned) * 64);   // "some segment needs the collect pass" flag, likewise
  p.o_tile_cnt = take(sizeof(int2) * (size_t)W * nt);  // per-tile counters (atomically added to), likewise
  p.hist_bytes = o - p.o_hist;
  p.o_sel = take(sizeof(Select) * seg);
  p.o_pred = take(sizeof(unsigned) * 6 * seg);  // [2] prediction words, [2] last buckets, [2] last moves, per level
  p.o_cand = take(sizeof(unsigned) * (size_t)W * std::max<long long>(1, p.cand_total));
  p.o_tile_cand = take(sizeof(int2) * (size_t)W * nt);
  p.o_tile_h3 = take(sizeof(unsigned short) * (size_t)W * nt * kBins3);
  p.o_tile_pre = take(sizeof(int2) * (size_t)W * nt);
  p.o_tile_rng = take(sizeof(int2) * (size_t)W * nt);
  p.o_lists = take(sizeof(int2) * (size_t)kNumLists * W * nt);
  p.o_pend_tau = take(sizeof(unsigned) * seg);
  p.total = o;
  return ACC_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace acc

using namespace acc;

extern "C" {

int acc_workspace_bytes(const acc_config* cfg, size_t* bytes) {
  if (!bytes) return ACC_EINVAL;
  Plan p;
  int st = make_plan(cfg, p);
  if (st != ACC_OK) return st;
  *bytes = p.total;
  return ACC_OK;
}

int acc_create(const acc_config* cfg, void* workspace, size_t workspace_bytes, acc_ctx** out) {
  if (!out) return ACC_EINVAL;
  *out = nullptr;
  acc_ctx* ctx = new (std::nothrow) acc_ctx();
  if (!ctx) return ACC_EINVAL;
  int st = make_plan(cfg, ctx->plan);
  if (st != ACC_OK) { delete ctx; return st; }
  if (!workspace || workspace_bytes < ctx->plan.total) { delete ctx; return ACC_EWORKSPACE; }
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) { delete ctx; return ACC_EALIGN; }
  ctx->cfg = *cfg;
  ctx->host_layers.assign(cfg->layers, cfg->layers + cfg->n_layers);
  ctx->cfg.layers = ctx->host_layers.data();
  ctx->ws = static_cast<char*>(workspace);
  Plan& p = ctx->plan;
  char* ws = ctx->ws;
  ctx->d_layers = reinterpret_cast<DevLayer*>(ws + p.o_layers);
  ctx->d_col_items = reinterpret_cast<ColItem*>(ws + p.o_col_items);
  ctx->d_qred_items = reinterpret_cast<int2*>(ws + p.o_qred_items);
  ctx->d_tiles = reinterpret_cast<Tile*>(ws + p.o_tiles);
  ctx->d_mat_layers = reinterpret_cast<int*>(ws + p.o_mat_layers);
  ctx->d_vec_tiles = reinterpret_cast<int*>(ws + p.o_vec_tiles);
  ctx->d_mat_tiles = reinterpret_cast<int*>(ws + p.o_mat_tiles);
  ctx->d_status = reinterpret_cast<int*>(ws + p.o_status);
  ctx->d_part = reinterpret_cast<float4*>(ws + p.o_part);
  ctx->d_ppart = reinterpret_cast<float4*>(ws + p.o_ppart);
  ctx->d_pending = reinterpret_cast<int*>(ws + p.o_pending);
  ctx->d_norm_part = reinterpret_cast<double*>(ws + p.o_norm_part);
  const size_t seg = (size_t)cfg->n_workers * std::max(p.n_mat, 1);
  ctx->d_hist1 = reinterpret_cast<unsigned*>(ws + p.o_hist);
  ctx->d_hist2 = ctx->d_hist1 + (align_up(sizeof(unsigned) * seg * kBins1, 256) / sizeof(unsigned));
  ctx->d_hist3 = ctx->d_hist2 + (align_up(sizeof(unsigned) * seg * kBins2, 256) / sizeof(unsigned));
  ctx->d_seg_cand = ctx->d_hist3 + (align_up(sizeof(unsigned) * seg * kBins3, 256) / sizeof(unsigned));
  ctx->d_seg_flag = ctx->d_seg_cand + (align_up(sizeof(unsigned) * seg, 256) / sizeof(unsigned));
  ctx->d_any_list = ctx->d_seg_flag + (align_up(sizeof(unsigned) * seg, 256) / sizeof(unsigned));
  ctx->d_pred = reinterpret_cast<unsigned*>(ws + p.o_pred);
  ctx->d_sel = reinterpret_cast<Select*>(ws + p.o_sel);
  ctx->d_cand = reinterpret_cast<unsigned*>(ws + p.o_cand);
  ctx->d_tile_cand = reinterpret_cast<int2*>(ws + p.o_tile_cand);
  ctx->d_tile_cnt = reinterpret_cast<int2*>(ws + p.o_tile_cnt);
  ctx->d_tile_h3 = reinterpret_cast<unsigned short*>(ws + p.o_tile_h3);
  ctx->d_tile_pre = reinterpret_cast<int2*>(ws + p.o_tile_pre);
  ctx->d_tile_rng = reinterpret_cast<int2*>(ws + p.o_tile_rng);
  ctx->d_lists = reinterpret_cast<int2*>(ws + p.o_lists);
  ctx->d_pend_tau = reinterpret_cast<unsigned*>(ws + p.o_pend_tau);

  cudaError_t e = cudaSuccess;
  auto up = [&](void* dst, const void* src, size_t bytes) {
    if (e == cudaSuccess && bytes) e = cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice);
  };
  up(ctx->d_layers, p.layers.data(), sizeof(DevLayer) * p.layers.size());
  up(ctx->d_col_items, p.col_items.data(), sizeof(ColItem) * p.col_items.size());
  up(ctx->d_qred_items, p.qred_items.data(), sizeof(int2) * p.qred_items.size());
  up(ctx->d_tiles, p.tiles.data(), sizeof(Tile) * p.tiles.size());
  up(ctx->d_mat_layers, p.mat_layers.data(), sizeof(int) * p.mat_layers.size());
  up(ctx->d_vec_tiles, p.vec_tiles.data(), sizeof(int) * p.vec_tiles.size());
  up(ctx->d_mat_tiles, p.mat_tiles.data(), sizeof(int) * p.mat_tiles.size());
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, sizeof(int) * 64);
  if (e == cudaSuccess) e = cudaMemset(ctx->d_pending, 0, sizeof(int) * cfg->n_layers);
  if (e == cudaSuccess) e = cudaMemset(ctx->d_pred, 0xff, sizeof(unsigned) * 6 * seg);  // no prediction yet
  if (e == cudaSuccess) e = cudaMemset(ctx->d_pend_tau, 0xff, sizeof(unsigned) * seg);  // nothing pending
  if (e == cudaSuccess) e = prepare_powersgd();
  if (e == cudaSuccess) e = prepare_topk(ctx);
  int dev = 0;
  if (e == cudaSuccess) e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) { delete ctx; return ACC_ECUDA; }
  *out = ctx;
  return ACC_OK;
}

int acc_destroy(acc_ctx* ctx) {
  if (!ctx) return ACC_EINVAL;
  for (ProfSlot& sl : ctx->prof_slots) { cudaEventDestroy(sl.a); cudaEventDestroy(sl.b); }
  delete ctx;
  return ACC_OK;
}

int acc_factor_layout(const acc_ctx* ctx, int64_t* q_row, int64_t* p_row, int64_t* q_rows, int64_t* p_rows) {
  if (!ctx) return ACC_EINVAL;
  for (int l = 0; l < ctx->cfg.n_layers; ++l) {
    if (q_row) q_row[l] = ctx->plan.layers[l].q_row;
    if (p_row) p_row[l] = ctx->plan.layers[l].p_row;
  }
  if (q_rows) *q_rows = ctx->plan.q_rows;
  if (p_rows) *p_rows = ctx->plan.p_rows;
  return ACC_OK;
}

int acc_topk_layout(const acc_ctx* ctx, int64_t* seg_offset, int64_t* k_low, int64_t* k_high, int64_t* capacity) {
  if (!ctx) return ACC_EINVAL;
  for (int l = 0; l < ctx->cfg.n_layers; ++l) {
    const DevLayer& d = ctx->plan.layers[l];
    if (seg_offset) seg_offset[l] = d.seg_off;
    if (k_low) k_low[l] = d.kind == ACC_MATRIX ? d.k_low : 0;
    if (k_high) k_high[l] = d.kind == ACC_MATRIX ? d.k_high : 0;
  }
  if (capacity) *capacity = ctx->plan.capacity;
  return ACC_OK;
}

static int finish(cudaError_t e) { return e == cudaSuccess ? ACC_OK : ACC_ECUDA; }

int acc_error_feedback(acc_ctx* ctx, const float* grads, float* err, float* delta, void* stream) {
  if (!ctx || !grads || !err) return ACC_EINVAL;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(delta)) return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_error_feedback(ctx, grads, err, delta, static_cast<cudaStream_t>(stream)));
}

int acc_layer_norms(acc_ctx* ctx, const float* buf, int64_t buf_stride, int32_t n_bufs, double* norm2, void* stream) {
  if (!ctx || !buf || !norm2 || n_bufs < 1 || n_bufs > ctx->cfg.n_workers) return ACC_EINVAL;
  if (n_bufs > 1 && buf_stride < ctx->cfg.worker_stride) return ACC_EINVAL;
  if (!aligned16(buf) || (n_bufs > 1 && buf_stride % 4 != 0) || (reinterpret_cast<uintptr_t>(norm2) & 7u)) return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_layer_norms(ctx, buf, buf_stride, n_bufs, nullptr, norm2, static_cast<cudaStream_t>(stream)));
}

int acc_layer_msdr(acc_ctx* ctx, const float* buf, int64_t buf_stride, int32_t n_bufs, double* moments, double* msdr,
                   void* stream) {
  if (!ctx || !buf || !moments || !msdr || n_bufs < 1 || n_bufs > ctx->cfg.n_workers) return ACC_EINVAL;
  if (n_bufs > 1 && buf_stride < ctx->cfg.worker_stride) return ACC_EINVAL;
  if (!aligned16(buf) || (n_bufs > 1 && buf_stride % 4 != 0) || (reinterpret_cast<uintptr_t>(moments) & 7u) ||
      (reinterpret_cast<uintptr_t>(msdr) & 7u))
    return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_layer_msdr(ctx, buf, buf_stride, n_bufs, moments, msdr, static_cast<cudaStream_t>(stream)));
}

int acc_layer_diff_norms(acc_ctx* ctx, const float* a, const float* b, double* norm2, void* stream) {
  if (!ctx || !a || !b || !norm2) return ACC_EINVAL;
  if (!aligned16(a) || !aligned16(b) || (reinterpret_cast<uintptr_t>(norm2) & 7u)) return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_layer_norms(ctx, a, 0, 1, b, norm2, static_cast<cudaStream_t>(stream)));
}

int acc_detect_regime(acc_ctx* ctx, const double* norm2_curr, double* norm2_prev, float lr_curr, float lr_next,
                      uint8_t* level, float* delta, void* stream) {
  if (!ctx || !norm2_curr || !norm2_prev || !level) return ACC_EINVAL;
  if (!aligned16(delta)) return ACC_EALIGN;
  ctx->last_launches = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_detect(ctx, norm2_curr, norm2_prev, nullptr, lr_curr, lr_next, nullptr, level, s);
  if (e == cudaSuccess && delta) e = cudaMemsetAsync(delta, 0, sizeof(float) * (size_t)ctx->cfg.worker_stride, s);
  return finish(e);
}

int acc_detect_regime_lr(acc_ctx* ctx, const double* norm2_curr, double* norm2_prev, const float* lr_pair,
                         uint8_t* level, float* delta, void* stream) {
  if (!ctx || !norm2_curr || !norm2_prev || !lr_pair || !level) return ACC_EINVAL;
  if (!aligned16(delta) || (reinterpret_cast<uintptr_t>(lr_pair) & 3u)) return ACC_EALIGN;
  ctx->last_launches = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_detect(ctx, norm2_curr, norm2_prev, nullptr, 0.f, 0.f, lr_pair, level, s);
  if (e == cudaSuccess && delta) e = cudaMemsetAsync(delta, 0, sizeof(float) * (size_t)ctx->cfg.worker_stride, s);
  return finish(e);
}

int acc_detect_regime_diff(acc_ctx* ctx, const double* norm2_diff, const double* norm2_curr, double* norm2_prev,
                           float lr_curr, float lr_next, uint8_t* level, float* delta, float* delta_prev,
                           void* stream) {
  if (!ctx || !norm2_diff || !norm2_curr || !norm2_prev || !level || !delta || !delta_prev) return ACC_EINVAL;
  if (!aligned16(delta) || !aligned16(delta_prev)) return ACC_EALIGN;
  ctx->last_launches = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t bytes = sizeof(float) * (size_t)ctx->cfg.worker_stride;
  cudaError_t e = launch_detect(ctx, norm2_curr, norm2_prev, norm2_diff, lr_curr, lr_next, nullptr, level, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(delta_prev, delta, bytes, cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(delta, 0, bytes, s);
  return finish(e);
}

int acc_powersgd_step(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat, const uint8_t* level,
                      float* out, float* delta, void* stream) {
  if (!ctx || !grads || !err || !q || !p_hat || !level || !out) return ACC_EINVAL;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(q) || !aligned16(p_hat) || !aligned16(out) ||
      !aligned16(delta))
    return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_powersgd(ctx, grads, err, q, p_hat, level, out, delta, SgdTail{nullptr, nullptr, nullptr},
                                static_cast<cudaStream_t>(stream)));
}

static int check_tail(const float* params, const float* mom, const float* hyper) {
  if (!params || !mom || !hyper) return ACC_EINVAL;
  if (!aligned16(params) || !aligned16(mom) || (reinterpret_cast<uintptr_t>(hyper) & 3u)) return ACC_EALIGN;
  return ACC_OK;
}

int acc_powersgd_step_sgd(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat, const uint8_t* level,
                          float* out, float* delta, float* params, float* mom, const float* hyper, void* stream) {
  if (!ctx || !grads || !err || !q || !p_hat || !level || !out) return ACC_EINVAL;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(q) || !aligned16(p_hat) || !aligned16(out) ||
      !aligned16(delta))
    return ACC_EALIGN;
  const int st = check_tail(params, mom, hyper);
  if (st != ACC_OK) return st;
  ctx->last_launches = 0;
  return finish(launch_powersgd(ctx, grads, err, q, p_hat, level, out, delta, SgdTail{params, mom, hyper},
                                static_cast<cudaStream_t>(stream)));
}

int acc_exchange_layout(const acc_ctx* ctx, int64_t* x1_floats, int64_t* x2_floats, int64_t* vec_floats) {
  if (!ctx) return ACC_EINVAL;
  if (x1_floats) *x1_floats = 4 * ctx->plan.p_rows + ctx->plan.vec_floats;
  if (x2_floats) *x2_floats = 4 * ctx->plan.q_rows;
  if (vec_floats) *vec_floats = ctx->plan.vec_floats;
  return ACC_OK;
}

int acc_powersgd_phase1(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat, const uint8_t* level,
                        float* out, float* delta, float* x1, void* stream) {
  if (!ctx || !grads || !err || !q || !p_hat || !level || !out || !x1) return ACC_EINVAL;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(q) || !aligned16(p_hat) || !aligned16(out) ||
      !aligned16(delta) || !aligned16(x1))
    return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_powersgd_phase1(ctx, grads, err, q, p_hat, level, out, delta, x1,
                                       static_cast<cudaStream_t>(stream)));
}

int acc_powersgd_phase2(acc_ctx* ctx, const float* x1, float scale, float* p_hat, const uint8_t* level,
                        const float* out, float* x2, void* stream) {
  if (!ctx || !x1 || !p_hat || !level || !out || !x2) return ACC_EINVAL;
  if (!aligned16(x1) || !aligned16(p_hat) || !aligned16(out) || !aligned16(x2)) return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_powersgd_phase2(ctx, x1, scale, p_hat, level, out, x2, static_cast<cudaStream_t>(stream)));
}

int acc_powersgd_phase3(acc_ctx* ctx, float* err, float* q, const float* p_hat, const uint8_t* level,
                        const float* x1, const float* x2, float scale, float* out, float* params, float* mom,
                        const float* hyper, void* stream) {
  if (!ctx || !err || !q || !p_hat || !level || !x1 || !x2 || !out) return ACC_EINVAL;
  if (!aligned16(err) || !aligned16(q) || !aligned16(p_hat) || !aligned16(x1) || !aligned16(x2) || !aligned16(out))
    return ACC_EALIGN;
  SgdTail tail{nullptr, nullptr, nullptr};
  if (params) {
    const int st = check_tail(params, mom, hyper);
    if (st != ACC_OK) return st;
    tail = SgdTail{params, mom, hyper};
  }
  ctx->last_launches = 0;
  return finish(launch_powersgd_phase3(ctx, err, q, p_hat, level, x1, x2, scale, out, tail,
                                       static_cast<cudaStream_t>(stream)));
}

int acc_upload_grads(acc_ctx* ctx, const float* grads_host, float* grads_dev, void* stream) {
  if (!ctx || !grads_host || !grads_dev) return ACC_EINVAL;
  if (!aligned16(grads_dev)) return ACC_EALIGN;
  const size_t bytes = sizeof(float) * (size_t)ctx->cfg.n_workers * (size_t)ctx->cfg.worker_stride;
  return finish(cudaMemcpyAsync(grads_dev, grads_host, bytes, cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream)));
}

int acc_download_out(acc_ctx* ctx, const float* out_dev, float* out_host, void* stream) {
  if (!ctx || !out_dev || !out_host) return ACC_EINVAL;
  const size_t bytes = sizeof(float) * (size_t)ctx->cfg.worker_stride;
  return finish(cudaMemcpyAsync(out_host, out_dev, bytes, cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream)));
}

int acc_topk_flush(acc_ctx* ctx, float* err, void* stream) {
  if (!ctx || !err) return ACC_EINVAL;
  if (!(ctx->cfg.flags & ACC_FLAG_LAZY_RESIDUAL)) return ACC_EINVAL;
  if (!aligned16(err)) return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_topk_flush(ctx, err, static_cast<cudaStream_t>(stream)));
}

int acc_topk_compress(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals, int32_t* idx,
                      int32_t* counts, float* delta, float* vec_packed, void* stream) {
  if (!ctx || !grads || !err || !level || !vals || !idx || !counts) return ACC_EINVAL;
  if (!vec_packed && ctx->plan.vec_floats > 0) return ACC_EINVAL;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(vals) || !aligned16(idx) || !aligned16(delta) ||
      !aligned16(vec_packed))
    return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_topk_compress(ctx, grads, err, level, vals, idx, counts, delta, vec_packed,
                                     static_cast<cudaStream_t>(stream)));
}

int acc_topk_decompress(acc_ctx* ctx, const float* vals_all, const int32_t* idx_all, const int32_t* counts_all,
                        int32_t n_sets, const float* vec_packed, float vec_scale, float* out, float* params,
                        float* mom, const float* hyper, void* stream) {
  if (!ctx || !vals_all || !idx_all || !counts_all || !out || n_sets < 1) return ACC_EINVAL;
  if (!vec_packed && ctx->plan.vec_floats > 0) return ACC_EINVAL;
  if (!aligned16(vals_all) || !aligned16(idx_all) || !aligned16(out) || !aligned16(vec_packed)) return ACC_EALIGN;
  SgdTail tail{nullptr, nullptr, nullptr};
  if (params) {
    const int st = check_tail(params, mom, hyper);
    if (st != ACC_OK) return st;
    tail = SgdTail{params, mom, hyper};
  }
  ctx->last_launches = 0;
  return finish(launch_topk_decompress_packed(ctx, vals_all, idx_all, counts_all, n_sets, vec_packed, vec_scale, out,
                                              tail, static_cast<cudaStream_t>(stream)));
}

int acc_sgd_nesterov(acc_ctx* ctx, const float* d, float* params, float* mom, const float* hyper, void* stream) {
  if (!ctx || !d) return ACC_EINVAL;
  if (!aligned16(d)) return ACC_EALIGN;
  const int st = check_tail(params, mom, hyper);
  if (st != ACC_OK) return st;
  ctx->last_launches = 0;
  return finish(launch_sgd_tiles(ctx, nullptr, (int)ctx->plan.tiles.size(), d, SgdTail{params, mom, hyper},
                                 static_cast<cudaStream_t>(stream)));
}

int acc_batch_accumulate(acc_ctx* ctx, const float* grads, float* acc, float* delta, int32_t first, void* stream) {
  if (!ctx || !grads || !acc) return ACC_EINVAL;
  if (!aligned16(grads) || !aligned16(acc) || !aligned16(delta)) return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_batch_accumulate(ctx, grads, acc, delta, first != 0, static_cast<cudaStream_t>(stream)));
}

int acc_batch_average(acc_ctx* ctx, const float* acc, int32_t n_accum, float* out, float* params, float* mom,
                      const float* hyper, void* stream) {
  if (!ctx || !acc || !out || n_accum < 1) return ACC_EINVAL;
  if (!aligned16(acc) || !aligned16(out)) return ACC_EALIGN;
  SgdTail tail{nullptr, nullptr, nullptr};
  if (params) {
    const int st = check_tail(params, mom, hyper);
    if (st != ACC_OK) return st;
    tail = SgdTail{params, mom, hyper};
  }
  ctx->last_launches = 0;
  return finish(launch_batch_average(ctx, acc, n_accum, out, tail, static_cast<cudaStream_t>(stream)));
}

int acc_detect_batch(acc_ctx* ctx, const double* norm2_layers, double* norm2_prev, float lr_curr, float lr_next,
                     int32_t b_low, int32_t b_high, int32_t* batch, float* lr_scale, float* delta, void* stream) {
  if (!ctx || !norm2_layers || !norm2_prev || !batch || !lr_scale) return ACC_EINVAL;
  if (b_low < 1 || b_high < b_low) return ACC_EINVAL;
  if (!aligned16(delta)) return ACC_EALIGN;
  ctx->last_launches = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_detect_batch(ctx, norm2_layers, norm2_prev, lr_curr, lr_next, b_low, b_high, batch, lr_scale, s);
  if (e == cudaSuccess && delta) e = cudaMemsetAsync(delta, 0, sizeof(float) * (size_t)ctx->cfg.worker_stride, s);
  return finish(e);
}

int acc_powersgd_flush(acc_ctx* ctx, float* err, const float* q, const float* p_hat, void* stream) {
  if (!ctx || !err || !q || !p_hat) return ACC_EINVAL;
  if (!(ctx->cfg.flags & ACC_FLAG_LAZY_RESIDUAL)) return ACC_EINVAL;
  if (!aligned16(err) || !aligned16(q) || !aligned16(p_hat)) return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_powersgd_flush(ctx, err, q, p_hat, static_cast<cudaStream_t>(stream)));
}

int acc_topk_step(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals, int32_t* idx,
                  int32_t* counts, float* out, float* delta, void* stream) {
  if (!ctx || !grads || !err || !level || !vals || !idx || !counts || !out) return ACC_EINVAL;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(vals) || !aligned16(idx) || !aligned16(out) ||
      !aligned16(delta))
    return ACC_EALIGN;
  ctx->last_launches = 0;
  return finish(launch_topk(ctx, grads, err, level, vals, idx, counts, out, delta, SgdTail{nullptr, nullptr, nullptr},
                            static_cast<cudaStream_t>(stream)));
}

int acc_topk_step_sgd(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals, int32_t* idx,
                      int32_t* counts, float* out, float* delta, float* params, float* mom, const float* hyper,
                      void* stream) {
  if (!ctx || !grads || !err || !level || !vals || !idx || !counts || !out) return ACC_EINVAL;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(vals) || !aligned16(idx) || !aligned16(out) ||
      !aligned16(delta))
    return ACC_EALIGN;
  const int st = check_tail(params, mom, hyper);
  if (st != ACC_OK) return st;
  ctx->last_launches = 0;
  return finish(launch_topk(ctx, grads, err, level, vals, idx, counts, out, delta, SgdTail{params, mom, hyper},
                            static_cast<cudaStream_t>(stream)));
}

int64_t acc_floats_sent(const acc_config* cfg, const uint8_t* level_host, int32_t compressor) {
  if (!level_host || validate(cfg) != ACC_OK) return -1;
  if (compressor != ACC_COMPRESSOR_POWERSGD && compressor != ACC_COMPRESSOR_TOPK) return -1;
  int64_t total = 0;
  for (int l = 0; l < cfg->n_layers; ++l) {
    const acc_layer_desc& d = cfg->layers[l];
    const long long size = (long long)d.rows * d.cols;
    if (d.kind == ACC_VECTOR) { total += size; continue; }
    if (compressor == ACC_COMPRESSOR_POWERSGD) {
      total += (int64_t)(level_host[l] ? cfg->rank_low : cfg->rank_high) * (d.rows + d.cols);
    } else {
      total += 2ll * topk_count(size, level_host[l] ? cfg->topk_low_bp : cfg->topk_high_bp) * cfg->n_workers;
    }
  }
  return total;
}

int acc_profile_enable(acc_ctx* ctx, int32_t enable) {
  if (!ctx) return ACC_EINVAL;
  ctx->prof = enable != 0;
  ctx->prof_used = 0;
  return ACC_OK;
}

int acc_profile_read(acc_ctx* ctx, double* ms, int32_t* launches, int32_t n) {
  if (!ctx || !ms || !launches || n < PH_COUNT) return ACC_EINVAL;
  for (int i = 0; i < n; ++i) { ms[i] = 0.0; launches[i] = 0; }
  for (size_t i = 0; i < ctx->prof_used; ++i) {
    const ProfSlot& sl = ctx->prof_slots[i];
    float t = 0.f;
    if (cudaEventSynchronize(sl.b) != cudaSuccess || cudaEventElapsedTime(&t, sl.a, sl.b) != cudaSuccess)
      return ACC_ECUDA;
    ms[sl.phase] += (double)t;
    launches[sl.phase] += 1;
  }
  ctx->prof_used = 0;
  return ACC_OK;
}

int32_t acc_profile_kernel_count(void) { return PH_COUNT; }

const char* acc_profile_kernel_name(int32_t i) {
  static const char* names[PH_COUNT] = {
      "ef_kernel", "norm_partial_kernel", "norm_final_kernel", "detect_kernel",
      "psgd_project_kernel", "psgd_orthonormalise_kernel", "psgd_qpartial_kernel", "psgd_qreduce_kernel",
      "psgd_residual_kernel",
      "topk_ef_hist1_kernel", "topk_pick1_kernel", "topk_hist2_kernel", "topk_pick2_kernel", "topk_hist3_kernel",
      "topk_tile_scan_kernel", "topk_select_kernel", "topk_decompress_kernel", "psgd_flush_kernel",
      "topk_collect_kernel", "topk_pick3_kernel", "topk_tile_counts_kernel",
      "topk_hist2_list_kernel", "topk_hist3_list_kernel", "topk_finalize_staged_kernel",
      "psgd_orthonormalise_block_kernel", "sgd_tiles_kernel", "batch_accumulate_kernel", "batch_average_kernel",
      "detect_batch_kernel", "psgd_pfold_kernel", "vec_exchange_kernel", "psgd_qmerge_kernel",
      "topk_decompress_packed_kernel", "topk_flush_kernel", "moments_partial_kernel", "moments_final_kernel"};
  return (i >= 0 && i < PH_COUNT) ? names[i] : "";
}

int acc_topk_last_paths(acc_ctx* ctx, int32_t* paths, int32_t n) {
  if (!ctx || !paths) return ACC_EINVAL;
  const int n_seg = ctx->cfg.n_workers * ctx->plan.n_mat;
  if (n < n_seg) return ACC_EINVAL;
  std::vector<Select> host((size_t)std::max(n_seg, 1));
  if (n_seg > 0 &&
      cudaMemcpy(host.data(), ctx->d_sel, sizeof(Select) * (size_t)n_seg, cudaMemcpyDeviceToHost) != cudaSuccess)
    return ACC_ECUDA;
  for (int i = 0; i < n_seg; ++i) paths[i] = host[i].mode;
  return ACC_OK;
}

int acc_device_status(acc_ctx* ctx, int32_t* status) {
  if (!ctx || !status) return ACC_EINVAL;
  int v = 0;
  if (cudaMemcpy(&v, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return ACC_ECUDA;
  *status = v;
  return ACC_OK;
}

int acc_selftest_wait_timeout(acc_ctx* ctx, void* stream) {
  if (!ctx) return ACC_EINVAL;
  ctx->last_launches = 0;
  return finish(launch_selftest_wait(ctx, static_cast<cudaStream_t>(stream)));
}

int acc_reset_device_status(acc_ctx* ctx, void* stream) {
  if (!ctx) return ACC_EINVAL;
  return finish(cudaMemsetAsync(ctx->d_status, 0, sizeof(int), static_cast<cudaStream_t>(stream)));
}

int32_t acc_last_launch_count(const acc_ctx* ctx) { return ctx ? ctx->last_launches : -1; }

const char* acc_strerror(int status) {
  switch (status) {
    case ACC_OK: return "ok";
    case ACC_EINVAL: return "invalid argument or configuration";
    case ACC_EALIGN: return "pointer, offset or stride not 16-byte aligned";
    case ACC_EWORKSPACE: return "workspace missing or too small";
    case ACC_ECUDA: return "CUDA runtime or launch error";
    case ACC_ETIMEOUT: return "a bounded device-side wait gave up (asynchronous copy did not complete)";
    case ACC_ETOOBIG: return "size exceeds the capacity of the built-in scratch array (ACC_STATIC_NORM_MAX_ELEMS)";
    default: return "unknown status";
  }
}

}  // extern "C"
