// PowerSGD rank-r step with error feedback over W workers (compressor of the Section "Accordion with PowerSGD").
//
// Because every product of the step is linear in the workers' matrices, the factors only depend on
// the mean matrix  Mbar = (1/W) sum_w (g_w + e_w):   P = Mbar Q,  Q' = Mbar^T P^,  A = P^ Q'^T.
// The project pass therefore reads every worker's g and e once, writes M_w back over e_w, and keeps
// Mbar (1/W of the data) in `out` for the second product.
//
// The streaming passes work on flat 8192-element tiles of a layer (the same tiles as the TopK path):
// every access is a fully coalesced, 16-byte aligned float4 whatever the row length, and all blocks carry
// the same load.  Row structure only enters through the factors: element i of a layer sits in row i / m,
// column i % m, and the rows a tile cuts are reduced from shared memory afterwards.
#include <cooperative_groups.h>

#include "acc_async.cuh"
#include "acc_internal.cuh"

namespace acc {

namespace cg = cooperative_groups;

__device__ __forceinline__ float lowrank_entry(const float4& pv, const float4& qv, int r) {
  float a = pv.x * qv.x;
  if (r > 1) a = fmaf(pv.y, qv.y, a);
  if (r > 2) a = fmaf(pv.z, qv.z, a);
  if (r > 3) a = fmaf(pv.w, qv.w, a);
  return a;
}

// A = P^[row] . Q[col] (first r ranks) for the four consecutive elements that start at layer element e_idx.
// row = e_idx / m without an integer division: the double-precision reciprocal is exact to within one.
__device__ __forceinline__ int row_of(int e_idx, int m, double inv_m) {
  int row = (int)((double)e_idx * inv_m);
  const int col = e_idx - row * m;
  row += (col >= m) - (col < 0);
  return row;
}

__device__ __forceinline__ float4 lowrank4(const float4* __restrict__ P4, const float4* __restrict__ Q4, int m,
                                           double inv_m, int e_idx, int r) {
  int row = row_of(e_idx, m, inv_m), col = e_idx - row * m;
  float4 pv = __ldg(P4 + row);
  float a[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    a[e] = lowrank_entry(pv, __ldg(Q4 + col), r);
    if (++col == m && e < 3) { col = 0; ++row; pv = __ldg(P4 + row); }
  }
  return make_float4(a[0], a[1], a[2], a[3]);
}

// out = mean_w g_w on one tile of a VECTOR layer; delta += g_decider.
__device__ void vector_mean_tile(const Tile& t, const DevLayer& L, const float* __restrict__ grads,
                                 float* __restrict__ out, float* __restrict__ delta, long long stride, int W,
                                 int decider, float inv_w) {
  const long long base = L.offset + t.elem0;
  float* o = out + base;
  vector_tile_mean(grads + base, stride, W, decider, inv_w, t.nelem, delta != nullptr ? delta + base : nullptr,
                   [&](int i, float4 v) { *reinterpret_cast<float4*>(o + i) = v; }, [&](int i, float v) { o[i] = v; });
}

// Partial rows of P from a tile's mean matrix in shared memory: for every row the tile cuts, the dot products of
// Mbar[row, columns inside the tile] with the columns of Q go to the row's slot for this tile in p_part.  Both
// first-pass kernels end a tile with it (NWARPS warps, all threads of the block; s_mbar complete and visible),
// so they give the same bits.  s_pp: 2 * kTile / kSpan float4 of shared memory.
constexpr int kSpan = 512;
constexpr int kSpans = kTile / kSpan;
template <int NWARPS>
__device__ __forceinline__ void tile_p_partials(const float* s_mbar, float4* s_pp, const Tile& t, const DevLayer& L,
                                                const float4* __restrict__ Q4, float4* __restrict__ p_part) {
  const int m = L.cols;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int first_row = t.elem0 / m, last_row = (t.elem0 + t.nelem - 1) / m;
  const int tile_in_layer = t.elem0 / kTile;
  if (m >= 2 * kSpan) {
    // long rows (too few row pieces to occupy the warps): the tile is cut into 512-element spans, a warp reduces
    // a span at a time (a span meets at most two rows); the spans of a row are then added in span order
    for (int sp = warp; sp < kSpans; sp += NWARPS) {
      const int s0 = sp * kSpan, s1 = min(s0 + kSpan, t.nelem);
      const int r_lo = (t.elem0 + s0) / m;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int row_begin = (r_lo + j) * m;
        const int lo = max(row_begin - t.elem0, s0), hi = min(row_begin + m - t.elem0, s1);
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        for (int i = lo + lane; i < hi; i += 32) {
          const float v = s_mbar[i];
          const float4 qv = __ldg(Q4 + (t.elem0 + i - row_begin));
          a0 = fmaf(v, qv.x, a0); a1 = fmaf(v, qv.y, a1); a2 = fmaf(v, qv.z, a2); a3 = fmaf(v, qv.w, a3);
        }
        a0 = warp_sum(a0); a1 = warp_sum(a1); a2 = warp_sum(a2); a3 = warp_sum(a3);
        if (lane == 0) s_pp[2 * sp + j] = make_float4(a0, a1, a2, a3);
      }
    }
    __syncthreads();
    const int row = first_row + (int)threadIdx.x;
    if (row <= last_row) {
      const int row_begin = row * m;
      const int lo = max(row_begin, t.elem0) - t.elem0, hi = min(row_begin + m, t.elem0 + t.nelem) - t.elem0;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int sp = lo / kSpan; sp <= (hi - 1) / kSpan; ++sp) {
        const float4 v = s_pp[2 * sp + (row - (t.elem0 + sp * kSpan) / m)];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      p_part[L.ppart_base + (long long)row * L.nslots + (tile_in_layer - row_begin / kTile)] = acc;
    }
  } else {
    // short rows: one warp per row piece
    for (int row = first_row + warp; row <= last_row; row += NWARPS) {
      const int row_begin = row * m;
      const int lo = max(row_begin, t.elem0) - t.elem0, hi = min(row_begin + m, t.elem0 + t.nelem) - t.elem0;
      const float4* qr = Q4 + (t.elem0 + lo - row_begin);
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
      for (int i = lo + lane; i < hi; i += 32) {
        const float v = s_mbar[i];
        const float4 qv = __ldg(qr + (i - lo));
        a0 = fmaf(v, qv.x, a0); a1 = fmaf(v, qv.y, a1); a2 = fmaf(v, qv.z, a2); a3 = fmaf(v, qv.w, a3);
      }
      a0 = warp_sum(a0); a1 = warp_sum(a1); a2 = warp_sum(a2); a3 = warp_sum(a3);
      if (lane == 0)
        p_part[L.ppart_base + (long long)row * L.nslots + (tile_in_layer - row_begin / kTile)] =
            make_float4(a0, a1, a2, a3);
    }
  }
}

constexpr int kProjThreads = 256;

// The same for a tile whose shared memory holds, per group of four consecutive elements, the group's dot products
// with its four rows of Q (rows whose length is a multiple of four: a group never meets two rows).  Only adds are
// left: a quarter of the shared-memory reads of the element version and no loads of Q.
template <int NWARPS>
__device__ __forceinline__ void tile_p_partials_grouped(const float4* s_grp, float4* s_pp, const Tile& t,
                                                        const DevLayer& L, float4* __restrict__ p_part) {
  const int m = L.cols;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int first_row = t.elem0 / m, last_row = (t.elem0 + t.nelem - 1) / m;
  const int tile_in_layer = t.elem0 / kTile;
  if (m >= 2 * kSpan) {
    for (int sp = warp; sp < kSpans; sp += NWARPS) {
      const int s0 = sp * kSpan, s1 = min(s0 + kSpan, t.nelem);
      const int r_lo = (t.elem0 + s0) / m;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int row_begin = (r_lo + j) * m;
        const int lo = max(row_begin - t.elem0, s0), hi = min(row_begin + m - t.elem0, s1);
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int i = (lo >> 2) + lane; i < (hi >> 2); i += 32) {
          const float4 v = s_grp[i];
          a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
        a.x = warp_sum(a.x); a.y = warp_sum(a.y); a.z = warp_sum(a.z); a.w = warp_sum(a.w);
        if (lane == 0) s_pp[2 * sp + j] = a;
      }
    }
    __syncthreads();
    const int row = first_row + (int)threadIdx.x;
    if (row <= last_row) {
      const int row_begin = row * m;
      const int lo = max(row_begin, t.elem0) - t.elem0, hi = min(row_begin + m, t.elem0 + t.nelem) - t.elem0;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int sp = lo / kSpan; sp <= (hi - 1) / kSpan; ++sp) {
        const float4 v = s_pp[2 * sp + (row - (t.elem0 + sp * kSpan) / m)];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      p_part[L.ppart_base + (long long)row * L.nslots + (tile_in_layer - row_begin / kTile)] = acc;
    }
  } else {
    for (int row = first_row + warp; row <= last_row; row += NWARPS) {
      const int row_begin = row * m;
      const int lo = max(row_begin, t.elem0) - t.elem0, hi = min(row_begin + m, t.elem0 + t.nelem) - t.elem0;
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int i = (lo >> 2) + lane; i < (hi >> 2); i += 32) {
        const float4 v = s_grp[i];
        a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
      }
      a.x = warp_sum(a.x); a.y = warp_sum(a.y); a.z = warp_sum(a.z); a.w = warp_sum(a.w);
      if (lane == 0) p_part[L.ppart_base + (long long)row * L.nslots + (tile_in_layer - row_begin / kTile)] = a;
    }
  }
}

// The streaming part of pass 1 on one MATRIX tile (all threads of the block).  GROUPED (rows of a multiple of four
// elements): the thread that holds four consecutive means multiplies them with their rows of Q at once and leaves
// the four-rank sum in shared memory, and the pending residual comes from one row of P^ and the same rows of Q,
// with no branch between the loads; otherwise the means themselves go to shared memory.
template <int WB, bool LAZY, bool GROUPED>
__device__ __forceinline__ void project_tile_stream(const Tile& t, const DevLayer& L, int rp,
                                                    const float4* __restrict__ Q4, const float4* __restrict__ P4,
                                                    const float* __restrict__ grads, float* __restrict__ err,
                                                    float* __restrict__ out, float* __restrict__ delta,
                                                    long long stride, int W, int decider, float inv_w,
                                                    float* s_mbar) {
  const int m = L.cols;
  const long long base = L.offset + t.elem0;
  const int n4 = t.nelem >> 2;
  for (int f = threadIdx.x; f < n4; f += blockDim.x) {
    const long long idx = base + 4 * f;
    float4 corr = make_float4(0.f, 0.f, 0.f, 0.f);
    int col = 0;
    if (GROUPED) {
      const int e_idx = t.elem0 + 4 * f, row = row_of(e_idx, m, L.inv_cols);
      col = e_idx - row * m;
      if (LAZY && rp > 0) {
        const float4 pv = __ldg(P4 + row);
        corr.x = lowrank_entry(pv, __ldg(Q4 + col), rp);
        corr.y = lowrank_entry(pv, __ldg(Q4 + col + 1), rp);
        corr.z = lowrank_entry(pv, __ldg(Q4 + col + 2), rp);
        corr.w = lowrank_entry(pv, __ldg(Q4 + col + 3), rp);
      }
    } else if (LAZY && rp > 0) {
      corr = lowrank4(P4, Q4, m, L.inv_cols, t.elem0 + 4 * f, rp);
    }
    float4 mb = make_float4(0.f, 0.f, 0.f, 0.f);
    // the detector's accumulator is asked for together with the first batch
    float4 dv = make_float4(0.f, 0.f, 0.f, 0.f);
    if (delta != nullptr) dv = *reinterpret_cast<const float4*>(delta + idx);
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
          const float4 mw = make_float4(gv[b].x + e.x, gv[b].y + e.y, gv[b].z + e.z, gv[b].w + e.w);
          if (LAZY) st_stream4(err + (long long)(w0 + b) * stride + idx, mw);
          else *reinterpret_cast<float4*>(err + (long long)(w0 + b) * stride + idx) = mw;
          mb.x += mw.x; mb.y += mw.y; mb.z += mw.z; mb.w += mw.w;
          if (delta != nullptr && w0 + b == decider) {
            dv.x += gv[b].x; dv.y += gv[b].y; dv.z += gv[b].z; dv.w += gv[b].w;
            *reinterpret_cast<float4*>(delta + idx) = dv;
          }
        }
    }
    mb.x *= inv_w; mb.y *= inv_w; mb.z *= inv_w; mb.w *= inv_w;
    *reinterpret_cast<float4*>(out + idx) = mb;
    if (GROUPED) {
      const float4 q0 = __ldg(Q4 + col), q1 = __ldg(Q4 + col + 1), q2 = __ldg(Q4 + col + 2), q3 = __ldg(Q4 + col + 3);
      float4 g;
      g.x = fmaf(mb.w, q3.x, fmaf(mb.z, q2.x, fmaf(mb.y, q1.x, mb.x * q0.x)));
      g.y = fmaf(mb.w, q3.y, fmaf(mb.z, q2.y, fmaf(mb.y, q1.y, mb.x * q0.y)));
      g.z = fmaf(mb.w, q3.z, fmaf(mb.z, q2.z, fmaf(mb.y, q1.z, mb.x * q0.z)));
      g.w = fmaf(mb.w, q3.w, fmaf(mb.z, q2.w, fmaf(mb.y, q1.w, mb.x * q0.w)));
      *reinterpret_cast<float4*>(s_mbar + 4 * f) = g;
    } else {
      *reinterpret_cast<float4*>(s_mbar + 4 * f) = mb;
    }
  }
}

// Pass 1.  One block per tile, all workers:
//   e_w = err_w                                 (eager: err holds the error memory)
//   e_w = err_w - P^_prev Q^T  (first rp ranks) (lazy: err holds last step's M_w, residual still pending)
//   M_w = g_w + e_w -> err;  Mbar = mean_w M_w -> out and shared memory;  delta += g_decider;
// then, for every row the tile cuts, the partial dot products Mbar[row, cols in tile] . Q go to the row's
// slot for this tile in p_part (a row touches (m-1)/8192 + 2 tiles at most; the orthonormalise pass adds
// the slots in order).
template <int WB, bool LAZY>
__global__ void __launch_bounds__(kProjThreads, 768 / kProjThreads)
psgd_project_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles,
                    const float* __restrict__ grads, float* __restrict__ err, const float* __restrict__ q,
                    const float* __restrict__ p, float4* __restrict__ p_part, const uint8_t* __restrict__ level,
                    const int* __restrict__ pending, float* __restrict__ out, float* __restrict__ delta,
                    long long stride, int W, int decider, float inv_w) {
  __shared__ __align__(16) float s_mbar[kTile];
  __shared__ float4 s_pp[2 * kSpans];
  const Tile t = tiles[blockIdx.x];
  const DevLayer L = layers[t.layer];
  if (L.kind != ACC_MATRIX) {
    vector_mean_tile(t, L, grads, out, delta, stride, W, decider, inv_w);
    return;
  }
  const int rp = LAZY ? pending[t.layer] : 0;
  const int m = L.cols;
  const float4* __restrict__ Q4 = reinterpret_cast<const float4*>(q) + L.q_row;
  const float4* __restrict__ P4 = reinterpret_cast<const float4*>(p) + L.p_row;
  if ((m & 3) == 0) {
    project_tile_stream<WB, LAZY, true>(t, L, rp, Q4, P4, grads, err, out, delta, stride, W, decider, inv_w, s_mbar);
    __syncthreads();
    tile_p_partials_grouped<kProjThreads / 32>(reinterpret_cast<const float4*>(s_mbar), s_pp, t, L, p_part);
    return;
  }
  project_tile_stream<WB, LAZY, false>(t, L, rp, Q4, P4, grads, err, out, delta, stride, W, decider, inv_w, s_mbar);
  const long long base = L.offset + t.elem0;
  const int n4 = t.nelem >> 2;
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {  // last 1-3 elements of the layer
    const long long idx = base + i;
    const int e_idx = t.elem0 + i, row = e_idx / m, col = e_idx - row * m;
    const float corr = (LAZY && rp > 0) ? lowrank_entry(__ldg(P4 + row), __ldg(Q4 + col), rp) : 0.f;
    float mb = 0.f;
    for (int w = 0; w < W; ++w) {
      const float gv = grads[(long long)w * stride + idx];
      float e = err[(long long)w * stride + idx];
      if (LAZY && rp > 0) e -= corr;
      const float mw = gv + e;
      err[(long long)w * stride + idx] = mw;
      mb += mw;
      if (delta != nullptr && w == decider) delta[idx] += gv;
    }
    mb *= inv_w;
    out[idx] = mb;
    s_mbar[i] = mb;
  }
  __syncthreads();
  tile_p_partials<kProjThreads / 32>(s_mbar, s_pp, t, L, Q4, p_part);
}

// Pass 1, pipelined.  Persistent blocks (one per SM, 512 threads), each with a contiguous range of MATRIX
// tiles and, at the end, a few tiles drawn by ticket.  The sequence of (tile, worker) stages of a block is streamed
// through two shared-memory stage buffers by bulk asynchronous copies: while the threads consume stage i (g_w and
// e_w of one tile, 2 x 32 KB), the copy of stage i+1 is in flight and, once everybody has left stage i's buffer,
// stage i+2 is issued into it -- 64-128 KB per SM are in flight at all times without costing registers.
// The arithmetic is that of the direct kernel's element path (same operations in the same order).
constexpr int kPipeThreads = 512;
constexpr int kPipePos = kTile / 4 / kPipeThreads;  // float4 positions per thread and tile
constexpr int kPipeStages = 2;
constexpr int kPipeMinStagesPerSm = 200;  // below this the direct kernel is used
constexpr int kPipeWarps = kPipeThreads / 32;
constexpr int kPipeDynamicTiles = 3;  // tiles per block handed out by ticket instead of the even split (LSTM set, W = 8:
                                      // 0.858 ms with 0, 0.851 with 1, 0.838 with 2, 0.835 with 3, 0.832-0.839 with 4 to all)
constexpr int kPipeTicketWord = 8;    // status block, words 8-9: ticket and count of finished blocks
// stage buffers, the mean matrix of the tile, the detector accumulator of the tile
constexpr size_t kPipeSmemBytes = sizeof(float) * kTile * (2 * kPipeStages + 2) + sizeof(float4) * 2 * kPipeWarps + 64;

template <bool LAZY>
__global__ void __launch_bounds__(kPipeThreads, 1)
psgd_project_pipe_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles,
                         const int* __restrict__ mat_tiles, int n_mat_tiles, const int* __restrict__ vec_tiles,
                         int n_vec_tiles, const float* __restrict__ grads, float* __restrict__ err,
                         const float* __restrict__ q, const float* __restrict__ p, float4* __restrict__ p_part,
                         const int* __restrict__ pending, float* __restrict__ out, float* __restrict__ delta,
                         long long stride, int W, int decider, float inv_w, int* __restrict__ status,
                         int dyn_tiles) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* stage = reinterpret_cast<float*>(smem_raw);                  // [kPipeStages buffers][g, e][kTile]
  float* s_mbar = stage + 2 * kPipeStages * kTile;                    // [kTile]
  float* s_delta = s_mbar + kTile;                                    // [kTile] detector accumulator of the tile
  float4* s_pp = reinterpret_cast<float4*>(s_delta + kTile);          // [kPipeWarps][2] partial rows of P
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_pp + 2 * kPipeWarps);  // [kPipeStages]
  for (int i = blockIdx.x; i < n_vec_tiles; i += gridDim.x) {
    const Tile t = tiles[vec_tiles[i]];
    vector_mean_tile(t, layers[t.layer], grads, out, delta, stride, W, decider, inv_w);
  }
  // The tiles of a block: a contiguous range of the first n_static tiles (an even split), then tiles of the rest
  // handed out one at a time by ticket -- blocks do not take the same time per tile (ragged tiles, rows of the
  // factor tables in L1 or not, the SM's share of DRAM), and with an even split of everything the SMs were idle for
  // 5 % of the kernel on average (8 % on the VGG set) while the slowest blocks finished.  ticket[0] hands out the
  // tiles, ticket[1] counts the blocks that are through; the last one clears both for the next launch.
  int* ticket = status + kPipeTicketWord;
  const int n_dynamic = min(n_mat_tiles, (int)gridDim.x * dyn_tiles);
  const int n_static = n_mat_tiles - n_dynamic;
  const int t0 = (int)((long long)n_static * blockIdx.x / gridDim.x);
  const int n_own = (int)((long long)n_static * (blockIdx.x + 1) / gridDim.x) - t0;
  int* s_seq = reinterpret_cast<int*>(bars + kPipeStages);  // [4] ring: the block's i-th tile (index into mat_tiles), -1 = none
  if (threadIdx.x == 0) {
    for (int b = 0; b < kPipeStages; ++b) mbar_init(&bars[b], 1);
    fence_mbar_init();
  }
  __syncthreads();
  const bool delta_by_copy = delta != nullptr && W >= 2;
  // thread 0 only: the tile whose stages are being issued is kept in registers, so that issuing a stage costs
  // no dependent global loads (they would sit on the critical path of every stage)
  int is_ti = -1;
  long long is_base = 0;
  unsigned is_bytes = 0;
  bool ended = false;  // the block's sequence of tiles is complete (a ticket beyond the last tile was drawn)
  auto issue = [&](int it) {
    if (ended) return;
    const int ti = it / W, w = it - ti * W;
    if (ti != is_ti) {
      int g = t0 + ti;
      if (ti >= n_own) {
        const int k = atomicAdd(&ticket[0], 1);
        g = k < n_dynamic ? n_static + k : -1;
      }
      s_seq[ti & 3] = g;  // read by everybody at the first stage of the tile, at least one barrier later
      if (g < 0) { ended = true; return; }
      const Tile tt = tiles[mat_tiles[g]];
      is_ti = ti;
      is_base = layers[tt.layer].offset + tt.elem0;
      is_bytes = (unsigned)((tt.nelem + 3) / 4) * 16u;  // a ragged tile reads into the layer's padding
    }
    const long long base = (long long)w * stride + is_base;
    const int buf = it % kPipeStages;
    // the deciding worker's stage also brings the tile of the detector's accumulator (single buffer: it is
    // read once per tile, W stages apart; with W == 1 the next copy would overtake the read, so that case
    // reads the accumulator with plain loads)
    const bool with_delta = delta_by_copy && w == decider;
    mbar_arrive_expect_tx(&bars[buf], (with_delta ? 3 : 2) * is_bytes);
    bulk_copy_g2s(stage + (2 * buf) * kTile, grads + base, is_bytes, &bars[buf]);
    bulk_copy_g2s(stage + (2 * buf + 1) * kTile, err + base, is_bytes, &bars[buf]);
    if (with_delta) bulk_copy_g2s(s_delta, delta + is_base, is_bytes, &bars[buf]);
  };
  auto leave = [&]() {  // thread 0, once per block
    __threadfence();
    if (atomicAdd(&ticket[1], 1) == (int)gridDim.x - 1) { ticket[0] = 0; ticket[1] = 0; }
  };
  if (threadIdx.x == 0)
    for (int it = 0; it < kPipeStages; ++it) issue(it);
  __syncthreads();  // s_seq of the first tile(s) is in place
  int gt = 0;  // the tile's index among all tiles
  Tile t;
  DevLayer L;
  t.layer = -1; t.elem0 = 0; t.nelem = 0;
  float4 corr[kPipePos], mb[kPipePos];
  int rp = 0;
  int last_g = -2;
  for (int it = 0, ti = 0, w = 0;; ++it) {
    const int buf = it % kPipeStages;
    if (w == 0) {  // new tile: factors of the pending residual at this thread's positions
      const int g = s_seq[ti & 3];
      if (g < 0) break;  // (uniform over the block)
      if (g == last_g + 1 && gt + 1 < L.tile0 + L.ntiles) {  // next tile of the same layer: no table look-ups
        gt += 1;
        t.elem0 += kTile;
        t.nelem = (int)min((long long)kTile, (long long)L.rows * L.cols - t.elem0);
      } else {
        gt = mat_tiles[g];
        t = tiles[gt];
        L = layers[t.layer];
        rp = LAZY ? pending[t.layer] : 0;
      }
      last_g = g;
      const float4* Q4 = reinterpret_cast<const float4*>(q) + L.q_row;
      const float4* P4 = reinterpret_cast<const float4*>(p) + L.p_row;
#pragma unroll
      for (int k = 0; k < kPipePos; ++k) {
        const int e0 = 4 * (k * kPipeThreads + (int)threadIdx.x);
        mb[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        corr[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (LAZY && rp > 0 && e0 + 3 < t.nelem) corr[k] = lowrank4(P4, Q4, L.cols, L.inv_cols, t.elem0 + e0, rp);
        else if (LAZY && rp > 0 && e0 < t.nelem) {  // ragged last float4 of a layer
          float c[4] = {0.f, 0.f, 0.f, 0.f};
          for (int e = 0; e0 + e < t.nelem; ++e) {
            const int ei = t.elem0 + e0 + e, row = ei / L.cols;
            c[e] = lowrank_entry(__ldg(P4 + row), __ldg(Q4 + (ei - row * L.cols)), rp);
          }
          corr[k] = make_float4(c[0], c[1], c[2], c[3]);
        }
      }
    }
    const bool arrived = __syncthreads_and(mbar_wait_bounded(&bars[buf], (unsigned)(it / kPipeStages) & 1u));
    if (!arrived) {  // a copy never completed: report and leave (uniformly for the whole block)
      if (threadIdx.x == 0) { atomicExch(status, ACC_ETIMEOUT); leave(); }
      return;
    }
    const float* sg = stage + (2 * buf) * kTile;
    const float* se = sg + kTile;
    const long long gbase = (long long)w * stride + L.offset + t.elem0;
    const bool acc_delta = delta != nullptr && w == decider;
#pragma unroll
    for (int k = 0; k < kPipePos; ++k) {
      const int e0 = 4 * (k * kPipeThreads + (int)threadIdx.x);
      if (e0 >= t.nelem) continue;
      const float4 gv = *reinterpret_cast<const float4*>(sg + e0);
      float4 e = *reinterpret_cast<const float4*>(se + e0);
      if (LAZY && rp > 0) { e.x -= corr[k].x; e.y -= corr[k].y; e.z -= corr[k].z; e.w -= corr[k].w; }
      const float4 mw = make_float4(gv.x + e.x, gv.y + e.y, gv.z + e.z, gv.w + e.w);
      mb[k].x += mw.x; mb[k].y += mw.y; mb[k].z += mw.z; mb[k].w += mw.w;
      if (e0 + 3 < t.nelem) {
        st_stream4(err + gbase + e0, mw);
        if (acc_delta) {
          float4 d = delta_by_copy ? *reinterpret_cast<const float4*>(s_delta + e0)
                                   : *reinterpret_cast<const float4*>(delta + L.offset + t.elem0 + e0);
          d.x += gv.x; d.y += gv.y; d.z += gv.z; d.w += gv.w;
          st_stream4(delta + L.offset + t.elem0 + e0, d);
        }
      } else {
        const float mm[4] = {mw.x, mw.y, mw.z, mw.w}, gg[4] = {gv.x, gv.y, gv.z, gv.w};
        for (int e2 = 0; e0 + e2 < t.nelem; ++e2) {
          err[gbase + e0 + e2] = mm[e2];
          if (acc_delta)
            delta[L.offset + t.elem0 + e0 + e2] = (delta_by_copy ? s_delta[e0 + e2] : delta[L.offset + t.elem0 + e0 + e2]) + gg[e2];
        }
      }
    }
    __syncthreads();  // everybody has left this stage buffer
    if (threadIdx.x == 0 && !ended) {
      fence_proxy_async_smem();
      issue(it + kPipeStages);
    }
    if (w == W - 1) {  // tile complete: mean matrix out, partial rows of P from shared memory
      const long long obase = L.offset + t.elem0;
#pragma unroll
      for (int k = 0; k < kPipePos; ++k) {
        const int e0 = 4 * (k * kPipeThreads + (int)threadIdx.x);
        if (e0 >= t.nelem) continue;
        const float4 v = make_float4(mb[k].x * inv_w, mb[k].y * inv_w, mb[k].z * inv_w, mb[k].w * inv_w);
        *reinterpret_cast<float4*>(s_mbar + e0) = v;
        if (e0 + 3 < t.nelem) {
          *reinterpret_cast<float4*>(out + obase + e0) = v;
        } else {
          const float vv[4] = {v.x, v.y, v.z, v.w};
          for (int e2 = 0; e0 + e2 < t.nelem; ++e2) out[obase + e0 + e2] = vv[e2];
        }
      }
      __syncthreads();
      tile_p_partials<kPipeWarps>(s_mbar, s_pp, t, L, reinterpret_cast<const float4*>(q) + L.q_row, p_part);
    }
    if (++w == W) { w = 0; ++ti; }
  }
  if (threadIdx.x == 0) leave();
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

// Pass 2, cluster version.  One thread-block cluster of 8 blocks per MATRIX layer: modified Gram-Schmidt on
// the first r columns of P.  Every block keeps its eighth of the rows in registers (up to kOrthoRowsPerThread
// per thread) for all passes; a pass is a block-level sum, an exchange of the eight partial sums through
// distributed shared memory and one cluster barrier.  The eight partials are added in rank order by every
// block, so all blocks see the same value and the result does not depend on scheduling.
constexpr int kOrthoCluster = 8;
constexpr int kOrthoThreads = 512;
constexpr int kOrthoRowsPerThread = 12;
constexpr int kOrthoMaxRows = kOrthoCluster * kOrthoThreads * kOrthoRowsPerThread;  // 49152; beyond: block kernel
constexpr int kOrthoMinRows = 2048;  // below this one block is faster than a cluster (block barriers are cheaper)
__host__ __device__ inline bool ortho_by_cluster(int rows) { return rows > kOrthoMinRows && rows <= kOrthoMaxRows; }

__device__ __forceinline__ double cluster_sum(double v, double* sm_warp, double* slots, int phase,
                                              cg::cluster_group& cluster) {
  // block-level sum (fixed order), published in this block's slot of the current phase parity
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sm_warp[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int i = 0; i < kOrthoThreads / 32; ++i) s += sm_warp[i];
    slots[phase & 1] = s;
  }
  cluster.sync();
  double total = 0.0;
  for (int r = 0; r < kOrthoCluster; ++r) total += cluster.map_shared_rank(slots, r)[phase & 1];
  return total;
}

// Row i of the unnormalised P of layer L: the sum, in tile order, of the partial rows the project pass left for
// the tiles the row touches -- or, when the rows were exchanged between GPUs (p_in != nullptr: the summed rows
// of all ranks, [p_rows] float4), p_scale times the exchanged row.
__device__ __forceinline__ float4 load_p_row(const DevLayer& L, int i, const float4* __restrict__ p_part,
                                             const float4* __restrict__ p_in, float p_scale) {
  if (p_in != nullptr) {
    const float4 v = p_in[L.p_row + i];
    return make_float4(v.x * p_scale, v.y * p_scale, v.z * p_scale, v.w * p_scale);
  }
  const int first_tile = (i * L.cols) / kTile, last_tile = (i * L.cols + L.cols - 1) / kTile;
  const float4* pp = p_part + L.ppart_base + (long long)i * L.nslots;
  float4 acc = pp[0];
  for (int sl = 1; sl <= last_tile - first_tile; ++sl) {
    acc.x += pp[sl].x; acc.y += pp[sl].y; acc.z += pp[sl].z; acc.w += pp[sl].w;
  }
  return acc;
}

__global__ void __cluster_dims__(kOrthoCluster, 1, 1) __launch_bounds__(kOrthoThreads)
psgd_orthonormalise_cluster_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers,
                                   float* __restrict__ p, const float4* __restrict__ p_part,
                                   const uint8_t* __restrict__ level, int* __restrict__ pending, int rank_low,
                                   int rank_high, float eps, const float4* __restrict__ p_in, float p_scale) {
  __shared__ double sm_warp[kOrthoThreads / 32];
  __shared__ double slots[2];
  cg::cluster_group cluster = cg::this_cluster();
  const int l = mat_layers[blockIdx.x / kOrthoCluster];
  const DevLayer L = layers[l];
  if (!ortho_by_cluster(L.rows)) return;  // uniform over the cluster: such layers go to the block kernel
  const int rank = (int)cluster.block_rank();
  const int r = level[l] ? rank_low : rank_high;
  if (pending != nullptr && rank == 0 && threadIdx.x == 0) pending[l] = r;
  float4* P4 = reinterpret_cast<float4*>(p) + L.p_row;
  const int per = (L.rows + kOrthoCluster - 1) / kOrthoCluster;
  const int row_lo = rank * per, row_hi = min(L.rows, row_lo + per);
  float4 v[kOrthoRowsPerThread];
#pragma unroll
  for (int k = 0; k < kOrthoRowsPerThread; ++k) {
    const int i = row_lo + k * kOrthoThreads + (int)threadIdx.x;
    v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < row_hi) {
      // ranks beyond r keep their value
      const float4 acc = load_p_row(L, i, p_part, p_in, p_scale);
      const float4 old = P4[i];
      v[k] = make_float4(acc.x, r > 1 ? acc.y : old.y, r > 2 ? acc.z : old.z, r > 3 ? acc.w : old.w);
    }
  }
  // columns as separate register arrays so that every index below is a compile-time constant
  float col[ACC_MAX_RANK][kOrthoRowsPerThread];
#pragma unroll
  for (int k = 0; k < kOrthoRowsPerThread; ++k) { col[0][k] = v[k].x; col[1][k] = v[k].y; col[2][k] = v[k].z; col[3][k] = v[k].w; }
  int phase = 0;
#pragma unroll
  for (int c = 0; c < ACC_MAX_RANK; ++c) {
    if (c < r) {  // uniform over the cluster
#pragma unroll
      for (int j = 0; j < c; ++j) {
        double part = 0.0;
#pragma unroll
        for (int k = 0; k < kOrthoRowsPerThread; ++k) part += (double)col[j][k] * (double)col[c][k];  // zeros outside the range
        const float dot = (float)cluster_sum(part, sm_warp, slots, phase++, cluster);
#pragma unroll
        for (int k = 0; k < kOrthoRowsPerThread; ++k) col[c][k] = fmaf(-dot, col[j][k], col[c][k]);
      }
      double part = 0.0;
#pragma unroll
      for (int k = 0; k < kOrthoRowsPerThread; ++k) part += (double)col[c][k] * (double)col[c][k];
      const double nrm = sqrt(cluster_sum(part, sm_warp, slots, phase++, cluster));
      const float inv = (float)(1.0 / (nrm + (double)eps));
#pragma unroll
      for (int k = 0; k < kOrthoRowsPerThread; ++k) col[c][k] *= inv;
    }
  }
#pragma unroll
  for (int k = 0; k < kOrthoRowsPerThread; ++k) v[k] = make_float4(col[0][k], col[1][k], col[2][k], col[3][k]);
#pragma unroll
  for (int k = 0; k < kOrthoRowsPerThread; ++k) {
    const int i = row_lo + k * kOrthoThreads + (int)threadIdx.x;
    if (i < row_hi) P4[i] = v[k];
  }
  cluster.sync();  // no block may exit while another still reads its shared memory
}

// Pass 2, block version, for layers with few rows (or with more than the cluster version holds in registers).
// One block per MATRIX layer: modified Gram-Schmidt on the first r columns of P, in place.
__global__ void __launch_bounds__(1024)
psgd_orthonormalise_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers,
                           float* __restrict__ p, const float4* __restrict__ p_part,
                           const uint8_t* __restrict__ level, int* __restrict__ pending, int rank_low, int rank_high,
                           float eps, const float4* __restrict__ p_in, float p_scale) {
  __shared__ double sm[32];
  const int l = mat_layers[blockIdx.x];
  const DevLayer L = layers[l];
  if (ortho_by_cluster(L.rows)) return;  // served by the cluster kernel
  const int r = level[l] ? rank_low : rank_high;
  if (pending != nullptr && threadIdx.x == 0) pending[l] = r;  // lazy mode: this step's residual stays pending
  float* P = p + 4ll * L.p_row;
  const int n = L.rows;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const float4 acc = load_p_row(L, i, p_part, p_in, p_scale);
    P[4 * i] = acc.x;
    if (r > 1) P[4 * i + 1] = acc.y;
    if (r > 2) P[4 * i + 2] = acc.z;
    if (r > 3) P[4 * i + 3] = acc.w;
  }
  __syncthreads();
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
  // rows in batches of kRows: the batch's loads of the mean matrix go out together (the rows are added in order)
  constexpr int kRows = 16 / VEC;  // 64 bytes of every row batch per thread
  for (int i0 = 0; i0 < it.nrows; i0 += kRows) {
    V mv[kRows];
#pragma unroll
    for (int k = 0; k < kRows; ++k)
      if (i0 + k < it.nrows) mv[k] = *reinterpret_cast<const V*>(base + (long long)(i0 + k) * L.cols);
#pragma unroll
    for (int k = 0; k < kRows; ++k)
      if (i0 + k < it.nrows) {
        const float4 pv = __ldg(pr + i0 + k);
        const float* m = reinterpret_cast<const float*>(&mv[k]);
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
          acc[e][0] = fmaf(m[e], pv.x, acc[e][0]);
          acc[e][1] = fmaf(m[e], pv.y, acc[e][1]);
          acc[e][2] = fmaf(m[e], pv.z, acc[e][2]);
          acc[e][3] = fmaf(m[e], pv.w, acc[e][3]);
        }
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

// Pass 5, lazy mode (out = A only).  Same items as the Q-partial pass: a thread owns `vec` adjacent columns,
// keeps their rows of Q' in registers and walks the slab's rows, so the factor tables are read once per
// (slab, column) instead of once per element; entries use the same lowrank_entry as every other pass.
// SGD: the optimiser tail is applied to the element just computed (params and mom laid out like out).
template <int VEC, bool SGD>
__device__ __forceinline__ void decompress_cols(const ColItem& it, const DevLayer& L, const float4* __restrict__ Q4,
                                                const float4* __restrict__ P4, float* __restrict__ out, int r,
                                                const SgdTail& tail) {
  using V = typename VecT<VEC>::type;
  const int col = it.col0 + (int)threadIdx.x * VEC;
  if (col >= L.cols) return;
  float4 qv[VEC];
#pragma unroll
  for (int e = 0; e < VEC; ++e) qv[e] = __ldg(Q4 + col + e);
  const long long first = L.offset + (long long)it.row0 * L.cols + col;
  float* base = out + first;
  const float4* pr = P4 + it.row0;
  if (!SGD) {
#pragma unroll 8
    for (int i = 0; i < it.nrows; ++i) {
      const float4 pv = __ldg(pr + i);
      float a[VEC];
#pragma unroll
      for (int e = 0; e < VEC; ++e) a[e] = lowrank_entry(pv, qv[e], r);
      __stcs(reinterpret_cast<V*>(base + (long long)i * L.cols), *reinterpret_cast<const V*>(a));
    }
    return;
  }
  // with the optimiser tail: rows in groups of kRows, the parameters and momenta of a group loaded before the
  // group's first store (a store in between would hold the later loads back)
  const SgdHyper h = sgd_hyper(tail);
  constexpr int kRows = 4;
  for (int i0 = 0; i0 < it.nrows; i0 += kRows) {
    V xv[kRows], uv[kRows];
#pragma unroll
    for (int k = 0; k < kRows; ++k)
      if (i0 + k < it.nrows) {
        const long long at = first + (long long)(i0 + k) * L.cols;
        xv[k] = *reinterpret_cast<const V*>(tail.params + at);
        uv[k] = *reinterpret_cast<const V*>(tail.mom + at);
      }
#pragma unroll
    for (int k = 0; k < kRows; ++k)
      if (i0 + k < it.nrows) {
        const long long at = first + (long long)(i0 + k) * L.cols;
        const float4 pv = __ldg(pr + i0 + k);
        float a[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) a[e] = lowrank_entry(pv, qv[e], r);
        __stcs(reinterpret_cast<V*>(out + at), *reinterpret_cast<const V*>(a));
        float* x = reinterpret_cast<float*>(&xv[k]);
        float* u = reinterpret_cast<float*>(&uv[k]);
#pragma unroll
        for (int e = 0; e < VEC; ++e) sgd_update(a[e], x[e], u[e], h);
        *reinterpret_cast<V*>(tail.params + at) = xv[k];
        *reinterpret_cast<V*>(tail.mom + at) = uv[k];
      }
  }
}

template <bool SGD>
__global__ void __launch_bounds__(kColBlockThreads)
psgd_decompress_kernel(const DevLayer* __restrict__ layers, const ColItem* __restrict__ items,
                       const float* __restrict__ q, const float* __restrict__ p, const uint8_t* __restrict__ level,
                       float* __restrict__ out, int rank_low, int rank_high, const SgdTail tail) {
  const ColItem it = items[blockIdx.x];
  const DevLayer L = layers[it.layer];
  const int r = level[it.layer] ? rank_low : rank_high;
  const float4* Q4 = reinterpret_cast<const float4*>(q) + L.q_row;
  const float4* P4 = reinterpret_cast<const float4*>(p) + L.p_row;
  if (L.vec == 4) decompress_cols<4, SGD>(it, L, Q4, P4, out, r, tail);
  else if (L.vec == 2) decompress_cols<2, SGD>(it, L, Q4, P4, out, r, tail);
  else decompress_cols<1, SGD>(it, L, Q4, P4, out, r, tail);
}

// Pass 4.  Sums the slab partials of 32 columns in a fixed order and stores the first r ranks of Q'.
__global__ void __launch_bounds__(256)
psgd_qreduce_kernel(const DevLayer* __restrict__ layers, const int2* __restrict__ items,
                    const float4* __restrict__ part, float* __restrict__ q, const uint8_t* __restrict__ level,
                    int rank_low, int rank_high, float4* __restrict__ q_sum) {
  __shared__ float4 sm[8][32];
  const int2 it = items[blockIdx.x];  // (layer, block of 32 columns)
  const int l = it.x;
  const DevLayer L = layers[l];
  const int cx = threadIdx.x & 31, gy = threadIdx.x >> 5;
  const int col = it.y * 32 + cx;
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
    if (q_sum != nullptr) {  // real workers: this GPU's share goes to the exchange buffer, ranks beyond r as zeros
      q_sum[L.q_row + col] = make_float4(t.x, r > 1 ? t.y : 0.f, r > 2 ? t.z : 0.f, r > 3 ? t.w : 0.f);
      return;
    }
    float4* Q4 = reinterpret_cast<float4*>(q) + L.q_row;
    float4 qv = Q4[col];
    qv.x = t.x;
    if (r > 1) qv.y = t.y;
    if (r > 2) qv.z = t.z;
    if (r > 3) qv.w = t.w;
    Q4[col] = qv;
  }
}

// Pass 5.  One block per tile:  A = P^ Q'^T (first r ranks) at every element of the tile;
//   WRITE_OUT: out = A;   UPDATE_ERR: err_w -= A for every worker.
// Eager step: both (r from the level).  Lazy step: WRITE_OUT only.  Flush: UPDATE_ERR only, r = pending rank.
// SGD (with WRITE_OUT): the optimiser tail is applied to A where it is written.
template <int WB, bool WRITE_OUT, bool UPDATE_ERR, bool SGD>
__global__ void __launch_bounds__(256)
psgd_residual_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, float* __restrict__ err,
                     const float* __restrict__ q, const float* __restrict__ p, const uint8_t* __restrict__ level,
                     const int* __restrict__ pending, float* __restrict__ out, long long stride, int W,
                     int rank_low, int rank_high, const SgdTail tail) {
  const Tile t = tiles[blockIdx.x];
  const DevLayer L = layers[t.layer];
  if (L.kind != ACC_MATRIX) return;
  const int r = pending != nullptr ? pending[t.layer] : (level[t.layer] ? rank_low : rank_high);
  if (r == 0) return;
  const int m = L.cols;
  const float4* __restrict__ Q4 = reinterpret_cast<const float4*>(q) + L.q_row;
  const float4* __restrict__ P4 = reinterpret_cast<const float4*>(p) + L.p_row;
  const long long base = L.offset + t.elem0;
  const int n4 = t.nelem >> 2;
  SgdHyper h = {0.f, 0.f, 0.f};
  if (SGD) h = sgd_hyper(tail);
  for (int f = threadIdx.x; f < n4; f += blockDim.x) {
    const long long idx = base + 4 * f;
    const float4 a = lowrank4(P4, Q4, m, L.inv_cols, t.elem0 + 4 * f, r);
    if (UPDATE_ERR) {
      for (int w0 = 0; w0 < W; w0 += WB) {
        float4 mw[WB];
#pragma unroll
        for (int b = 0; b < WB; ++b)
          if (w0 + b < W) mw[b] = ld_stream4(err + (long long)(w0 + b) * stride + idx);
#pragma unroll
        for (int b = 0; b < WB; ++b)
          if (w0 + b < W)
            st_stream4(err + (long long)(w0 + b) * stride + idx,
                       make_float4(mw[b].x - a.x, mw[b].y - a.y, mw[b].z - a.z, mw[b].w - a.w));
      }
    }
    if (WRITE_OUT) st_stream4(out + idx, a);
    if (SGD) sgd_apply4(tail, h, idx, a);
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
    const int e_idx = t.elem0 + i, row = e_idx / m, col = e_idx - row * m;
    const float a = lowrank_entry(__ldg(P4 + row), __ldg(Q4 + col), r);
    if (UPDATE_ERR)
      for (int w = 0; w < W; ++w) err[(long long)w * stride + base + i] -= a;
    if (WRITE_OUT) out[base + i] = a;
    if (SGD) sgd_apply1(tail, h, base + i, a);
  }
}

// Optimiser tail on its own: x, u updated from d over the given flat tiles (tile_ids == nullptr: tile
// blockIdx.x).  Used for the VECTOR layers of a fused PowerSGD step (their `out` comes from the first pass)
// and as the stand-alone tail.
__global__ void __launch_bounds__(256)
sgd_tiles_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, const int* __restrict__ tile_ids,
                 const float* __restrict__ d, const SgdTail tail) {
  const Tile t = tiles[tile_ids != nullptr ? tile_ids[blockIdx.x] : (int)blockIdx.x];
  const DevLayer L = layers[t.layer];
  const long long base = L.offset + t.elem0;
  const SgdHyper h = sgd_hyper(tail);
  const int n4 = t.nelem >> 2;
  // four float4 per thread at a time: all loads of a group before its first store
  constexpr int kGroup = 4, kThreads = 256;
  for (int f0 = 0; f0 < n4; f0 += kGroup * kThreads) {
    float4 dv[kGroup], xv[kGroup], uv[kGroup];
#pragma unroll
    for (int k = 0; k < kGroup; ++k) {
      const int f = f0 + k * kThreads + (int)threadIdx.x;
      if (f < n4) {
        dv[k] = ld_stream4(d + base + 4 * f);
        xv[k] = *reinterpret_cast<const float4*>(tail.params + base + 4 * f);
        uv[k] = *reinterpret_cast<const float4*>(tail.mom + base + 4 * f);
      }
    }
#pragma unroll
    for (int k = 0; k < kGroup; ++k) {
      const int f = f0 + k * kThreads + (int)threadIdx.x;
      if (f < n4) {
        sgd_update(dv[k].x, xv[k].x, uv[k].x, h); sgd_update(dv[k].y, xv[k].y, uv[k].y, h);
        sgd_update(dv[k].z, xv[k].z, uv[k].z, h); sgd_update(dv[k].w, xv[k].w, uv[k].w, h);
        *reinterpret_cast<float4*>(tail.params + base + 4 * f) = xv[k];
        *reinterpret_cast<float4*>(tail.mom + base + 4 * f) = uv[k];
      }
    }
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) sgd_apply1(tail, h, base + i, d[base + i]);
}

cudaError_t launch_sgd_tiles(acc_ctx* ctx, const int* tile_ids, int n, const float* d, SgdTail tail, cudaStream_t s) {
  if (n > 0) {
    PhaseTimer pt(ctx, PH_SGD_TILES, s);
    sgd_tiles_kernel<<<n, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, tile_ids, d, tail);
  }
  return cudaGetLastError();
}

// Lazy mode only: after a flush no residual is pending.
__global__ void psgd_clear_pending_kernel(int* __restrict__ pending, int n_layers) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l < n_layers) pending[l] = 0;
}

// Exercises the bounded wait: a barrier nobody arrives at, a short poll limit; the block reports ACC_ETIMEOUT in
// the status word and returns normally (what a pipelined kernel does if a copy never completes).
__global__ void selftest_wait_kernel(int* __restrict__ status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_mbar_init();
  }
  __syncthreads();
  const bool arrived = __syncthreads_and(mbar_wait_bounded(&bar, 0u, 2048u));
  if (!arrived && threadIdx.x == 0) atomicExch(status, ACC_ETIMEOUT);
}

cudaError_t launch_selftest_wait(acc_ctx* ctx, cudaStream_t s) {
  ctx->last_launches += 1;
  selftest_wait_kernel<<<1, 64, 0, s>>>(ctx->d_status);
  return cudaGetLastError();
}

// Once per context, at creation (not a stream operation): the pipelined kernels need more than 48 KB of
// dynamic shared memory.
cudaError_t prepare_powersgd() {
  cudaError_t e = cudaFuncSetAttribute(psgd_project_pipe_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kPipeSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(psgd_project_pipe_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kPipeSmemBytes);
  return e;
}

// ---- real workers: the factors cross GPUs between the passes ---------------------------------------------
// Exchange buffer 1: [p_rows] float4 rows of the unnormalised P (ranks beyond r as zeros), then the VECTOR
// layers' means packed one after the other.  Exchange buffer 2: [q_rows] float4 rows of Q' (same convention).

// One thread per row of P: folds the row's partials into exchange buffer 1.
__global__ void __launch_bounds__(256)
psgd_pfold_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers,
                  const float4* __restrict__ p_part, const uint8_t* __restrict__ level, int rank_low, int rank_high,
                  float4* __restrict__ p_sum) {
  const int l = mat_layers[blockIdx.y];
  const DevLayer L = layers[l];
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= L.rows) return;
  const int r = level[l] ? rank_low : rank_high;
  const float4 a = load_p_row(L, i, p_part, nullptr, 1.f);
  p_sum[L.p_row + i] = make_float4(a.x, r > 1 ? a.y : 0.f, r > 2 ? a.z : 0.f, r > 3 ? a.w : 0.f);
}

// VECTOR tiles: packed <- out (PACK) or out <- scale * packed.
template <bool PACK>
__global__ void __launch_bounds__(256)
vec_exchange_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles,
                    const int* __restrict__ vec_tiles, float* __restrict__ out, float* __restrict__ packed,
                    float scale) {
  const Tile t = tiles[vec_tiles[blockIdx.x]];
  const DevLayer L = layers[t.layer];
  float* o = out + L.offset + t.elem0;
  float* x = packed + L.vec_off + t.elem0;
  for (int i = threadIdx.x; i < t.nelem; i += blockDim.x) {
    if (PACK) x[i] = o[i];
    else o[i] = scale * x[i];
  }
}

// One thread per column of Q: the first r ranks of Q' <- scale * exchanged sum.
__global__ void __launch_bounds__(256)
psgd_qmerge_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers,
                   const float4* __restrict__ q_in, float scale, float* __restrict__ q,
                   const uint8_t* __restrict__ level, int rank_low, int rank_high) {
  const int l = mat_layers[blockIdx.y];
  const DevLayer L = layers[l];
  const int col = blockIdx.x * 256 + threadIdx.x;
  if (col >= L.cols) return;
  const int r = level[l] ? rank_low : rank_high;
  const float4 t = q_in[L.q_row + col];
  float4* Q4 = reinterpret_cast<float4*>(q) + L.q_row;
  float4 qv = Q4[col];
  qv.x = t.x * scale;
  if (r > 1) qv.y = t.y * scale;
  if (r > 2) qv.z = t.z * scale;
  if (r > 3) qv.w = t.w * scale;
  Q4[col] = qv;
}

// Pass 1 (both implementations of it; same arithmetic, same results).
static void launch_psgd_project(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                                const uint8_t* level, float* out, float* delta, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const int nt = (int)pl.tiles.size();
  const float inv_w = 1.0f / (float)c.n_workers;
  const bool lazy = (c.flags & ACC_FLAG_LAZY_RESIDUAL) != 0;
  // The persistent pipelined kernel wins once every SM has a long queue of stages (measured: 330 stages/SM ->
  // 0.95 ms against 1.11 ms); on small sets its one-block-per-SM static split loses a few percent to tile
  // quantisation.
  const long long stages_per_sm = (long long)pl.mat_tiles.size() * c.n_workers / (ctx->sm_count > 0 ? ctx->sm_count : 1);
  const bool pipelined = (c.flags & ACC_FLAG_PIPELINE_ALWAYS) ||
                         (!(c.flags & ACC_FLAG_PIPELINE_NEVER) && stages_per_sm >= kPipeMinStagesPerSm);
  PhaseTimer pt(ctx, PH_PSGD_PROJECT, s);
  if (pipelined && pl.n_mat > 0) {
    const int n_mt = (int)pl.mat_tiles.size(), n_vt = (int)pl.vec_tiles.size();
    // one block fills an SM; when a TopK step runs beside this one, half of the SMs are left to it (measured on the
    // LSTM set, W = 8, both steps replayed from one graph: 2.15 -> 2.09 ms at the high level, 2.52 -> 2.46 ms at the
    // low level; with every SM taken, the TopK step's short kernels wait for this pass to end)
    const int sms = (c.flags & ACC_FLAG_SHARE_SMS) ? std::max(ctx->sm_count / 2, 1) : ctx->sm_count;
    const int grid = n_mt < sms ? n_mt : sms;
    const int dyn_tiles = kPipeDynamicTiles;
    if (lazy) {
      psgd_project_pipe_kernel<true><<<grid, kPipeThreads, kPipeSmemBytes, s>>>(
          ctx->d_layers, ctx->d_tiles, ctx->d_mat_tiles, n_mt, ctx->d_vec_tiles, n_vt, grads, err, q, p_hat,
          ctx->d_ppart, ctx->d_pending, out, delta, c.worker_stride, c.n_workers, c.decider, inv_w, ctx->d_status,
          dyn_tiles);
    } else {
      psgd_project_pipe_kernel<false><<<grid, kPipeThreads, kPipeSmemBytes, s>>>(
          ctx->d_layers, ctx->d_tiles, ctx->d_mat_tiles, n_mt, ctx->d_vec_tiles, n_vt, grads, err, q, p_hat,
          ctx->d_ppart, nullptr, out, delta, c.worker_stride, c.n_workers, c.decider, inv_w, ctx->d_status, dyn_tiles);
    }
  } else if (lazy) {
    psgd_project_kernel<4, true><<<nt, kProjThreads, 0, s>>>(ctx->d_layers, ctx->d_tiles, grads, err, q, p_hat, ctx->d_ppart,
                                                    level, ctx->d_pending, out, delta, c.worker_stride,
                                                    c.n_workers, c.decider, inv_w);
  } else {
    psgd_project_kernel<4, false><<<nt, kProjThreads, 0, s>>>(ctx->d_layers, ctx->d_tiles, grads, err, q, p_hat,
                                                     ctx->d_ppart, level, nullptr, out, delta, c.worker_stride,
                                                     c.n_workers, c.decider, inv_w);
  }
}

// Passes 2-4: P^ from the partial rows (or from exchanged rows p_in), Q' partials from Mbar (held in out),
// their reduction into q (or into the exchange buffer q_sum).
static void launch_psgd_ortho_q(acc_ctx* ctx, float* q, float* p_hat, const uint8_t* level, const float* out,
                                const float4* p_in, float p_scale, float4* q_sum, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const bool lazy = (c.flags & ACC_FLAG_LAZY_RESIDUAL) != 0;
  bool any_cluster = false, any_block = false;
  for (int l : pl.mat_layers) (ortho_by_cluster(pl.layers[l].rows) ? any_cluster : any_block) = true;
  if (any_cluster) {
    PhaseTimer pt(ctx, PH_PSGD_ORTHO, s);
    psgd_orthonormalise_cluster_kernel<<<pl.n_mat * kOrthoCluster, kOrthoThreads, 0, s>>>(
        ctx->d_layers, ctx->d_mat_layers, p_hat, ctx->d_ppart, level, lazy ? ctx->d_pending : nullptr, c.rank_low,
        c.rank_high, c.gs_eps, p_in, p_scale);
  }
  if (any_block) {
    PhaseTimer pt(ctx, PH_PSGD_ORTHO_BLOCK, s);
    psgd_orthonormalise_kernel<<<pl.n_mat, 1024, 0, s>>>(ctx->d_layers, ctx->d_mat_layers, p_hat, ctx->d_ppart,
                                                        level, lazy ? ctx->d_pending : nullptr, c.rank_low,
                                                        c.rank_high, c.gs_eps, p_in, p_scale);
  }
  {
    PhaseTimer pt(ctx, PH_PSGD_QPARTIAL, s);
    psgd_qpartial_kernel<<<(unsigned)pl.col_items.size(), kColBlockThreads, 0, s>>>(
        ctx->d_layers, ctx->d_col_items, out, p_hat, ctx->d_part);
  }
  {
    PhaseTimer pt(ctx, PH_PSGD_QREDUCE, s);
    psgd_qreduce_kernel<<<(unsigned)pl.qred_items.size(), 256, 0, s>>>(
        ctx->d_layers, ctx->d_qred_items, ctx->d_part, q, level, c.rank_low, c.rank_high, q_sum);
  }
}

// Pass 5 (+ the optimiser tail): out = A, and in eager mode err_w -= A.
static cudaError_t launch_psgd_finish(acc_ctx* ctx, float* err, const float* q, const float* p_hat,
                                      const uint8_t* level, float* out, SgdTail tail, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const int nt = (int)pl.tiles.size();
  const bool lazy = (c.flags & ACC_FLAG_LAZY_RESIDUAL) != 0;
  if (pl.n_mat > 0) {
    PhaseTimer pt(ctx, PH_PSGD_RESIDUAL, s);
    const unsigned n_items = (unsigned)pl.col_items.size();
    if (lazy && tail.params)
      psgd_decompress_kernel<true><<<n_items, kColBlockThreads, 0, s>>>(
          ctx->d_layers, ctx->d_col_items, q, p_hat, level, out, c.rank_low, c.rank_high, tail);
    else if (lazy)
      psgd_decompress_kernel<false><<<n_items, kColBlockThreads, 0, s>>>(
          ctx->d_layers, ctx->d_col_items, q, p_hat, level, out, c.rank_low, c.rank_high, tail);
    else if (tail.params)
      psgd_residual_kernel<4, true, true, true><<<nt, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, err, q, p_hat, level,
                                                                   nullptr, out, c.worker_stride, c.n_workers,
                                                                   c.rank_low, c.rank_high, tail);
    else
      psgd_residual_kernel<4, true, true, false><<<nt, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, err, q, p_hat,
                                                                    level, nullptr, out, c.worker_stride,
                                                                    c.n_workers, c.rank_low, c.rank_high, tail);
  }
  // VECTOR layers: their out (the plain mean) was written by the first pass
  if (tail.params && !pl.vec_tiles.empty()) {
    const cudaError_t e = launch_sgd_tiles(ctx, ctx->d_vec_tiles, (int)pl.vec_tiles.size(), out, tail, s);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

cudaError_t launch_powersgd(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                            const uint8_t* level, float* out, float* delta, SgdTail tail, cudaStream_t s) {
  launch_psgd_project(ctx, grads, err, q, p_hat, level, out, delta, s);
  if (ctx->plan.n_mat > 0) launch_psgd_ortho_q(ctx, q, p_hat, level, out, nullptr, 1.f, nullptr, s);
  return launch_psgd_finish(ctx, err, q, p_hat, level, out, tail, s);
}

cudaError_t launch_powersgd_phase1(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                                   const uint8_t* level, float* out, float* delta, float* x1, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  launch_psgd_project(ctx, grads, err, q, p_hat, level, out, delta, s);
  if (pl.n_mat > 0) {
    PhaseTimer pt(ctx, PH_PSGD_PFOLD, s);
    psgd_pfold_kernel<<<dim3((pl.max_rows + 255) / 256, pl.n_mat), 256, 0, s>>>(
        ctx->d_layers, ctx->d_mat_layers, ctx->d_ppart, level, c.rank_low, c.rank_high,
        reinterpret_cast<float4*>(x1));
  }
  if (!pl.vec_tiles.empty()) {
    PhaseTimer pt(ctx, PH_VEC_EXCHANGE, s);
    vec_exchange_kernel<true><<<(unsigned)pl.vec_tiles.size(), 256, 0, s>>>(
        ctx->d_layers, ctx->d_tiles, ctx->d_vec_tiles, out, x1 + 4 * pl.p_rows, 1.f);
  }
  return cudaGetLastError();
}

cudaError_t launch_powersgd_phase2(acc_ctx* ctx, const float* x1, float scale, float* p_hat, const uint8_t* level,
                                   const float* out, float* x2, cudaStream_t s) {
  if (ctx->plan.n_mat > 0)
    launch_psgd_ortho_q(ctx, nullptr, p_hat, level, out, reinterpret_cast<const float4*>(x1), scale,
                        reinterpret_cast<float4*>(x2), s);
  return cudaGetLastError();
}

cudaError_t launch_powersgd_phase3(acc_ctx* ctx, float* err, float* q, const float* p_hat, const uint8_t* level,
                                   const float* x1, const float* x2, float scale, float* out, SgdTail tail,
                                   cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  if (pl.n_mat > 0) {
    PhaseTimer pt(ctx, PH_PSGD_QMERGE, s);
    psgd_qmerge_kernel<<<dim3((pl.max_cols + 255) / 256, pl.n_mat), 256, 0, s>>>(
        ctx->d_layers, ctx->d_mat_layers, reinterpret_cast<const float4*>(x2), scale, q, level, c.rank_low,
        c.rank_high);
  }
  if (!pl.vec_tiles.empty()) {
    PhaseTimer pt(ctx, PH_VEC_EXCHANGE, s);
    vec_exchange_kernel<false><<<(unsigned)pl.vec_tiles.size(), 256, 0, s>>>(
        ctx->d_layers, ctx->d_tiles, ctx->d_vec_tiles, out, const_cast<float*>(x1) + 4 * pl.p_rows, scale);
  }
  return launch_psgd_finish(ctx, err, q, p_hat, level, out, tail, s);
}

cudaError_t launch_powersgd_flush(acc_ctx* ctx, float* err, const float* q, const float* p_hat, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const int nt = (int)pl.tiles.size();
  if (pl.n_mat > 0) {
    {
      PhaseTimer pt(ctx, PH_PSGD_FLUSH, s);
      psgd_residual_kernel<4, false, true, false><<<nt, 256, 0, s>>>(
          ctx->d_layers, ctx->d_tiles, err, q, p_hat, nullptr, ctx->d_pending, nullptr, c.worker_stride, c.n_workers,
          c.rank_low, c.rank_high, SgdTail{nullptr, nullptr, nullptr});
    }
    ctx->last_launches += 1;
    psgd_clear_pending_kernel<<<(c.n_layers + 127) / 128, 128, 0, s>>>(ctx->d_pending, c.n_layers);
  }
  return cudaGetLastError();
}

}  // namespace acc
