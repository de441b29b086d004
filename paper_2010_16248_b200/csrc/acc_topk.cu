// TopK-K% sparsification with error feedback (sparsifier of the Section "Accordion with TopK"), exact and order-preserving.
//
// Selection is a three-level radix select on the 31-bit magnitude pattern key = bits(M) & 0x7fffffff
// (12 + 12 + 7 bits, shared-memory histograms), followed by an ordered compaction:
//   ef_hist1   M = g + e -> err, level-1 histogram per (worker, layer)                [reads g, e; writes M]
//              (+ keys of the buckets around the predicted threshold bucket -> candidate list)
//              (+ per-tile counts of non-zero keys)
//   pick1      bucket b1 holding the k-th largest key; zero fill if the threshold falls among exact zeros (every
//              non-zero kept, the zeros of lowest index fill up: settled from the non-zero counts, levels 2-3 skipped);
//              predicted-list / staged path if pass A's prediction held, else list path if the keys of b1 fit the
//              candidate list, else dense path
//   collect    (list path) keys of bucket b1 -> per-tile ranges of the segment's candidate list,
//              per-tile count of keys above b1                                                  [reads M]
//   hist2      level-2 histogram of the keys inside b1 (dense path: reads M and also counts the keys
//              above b1 per tile; list path, topk_hist_list_kernel: reads the segment's collected keys)
//   pick2      bucket b2
//   hist3      level-3 histogram of the keys with prefix (b1,b2) (dense path: reads M, keeps it per tile
//              together with the per-tile count above; list path: per segment from the collected keys)
//   pick3      threshold tau and the number of ties to keep
//   tilecounts per tile (keys above tau, keys equal to tau), from the tile's level-3 histogram (dense), its collected
//              keys (list) or its non-zero count (zero fill);  tilescan: their exclusive prefix per layer, every
//              tile's range inside the packed segment, and the work lists of select / finalize
//   select     keep key > tau and the lowest-index `need` of key == tau; write (val, idx) in index
//              order, zero the kept entries of err                                              [reads M]
//   finalize   the same for segments whose pass A staged whole entries: from the list, M is not read
//   decompress out = (1/W) sum_w scatter(idx_w, val_w), accumulated per tile in shared memory from the workers'
//              entries staged there by asynchronous copies                                      [reads packed]
// No floating-point atomics and no inter-block waiting: same input, same bits.
#include <algorithm>

#include "acc_async.cuh"
#include "acc_internal.cuh"

namespace acc {

__device__ __forceinline__ unsigned key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

// A prediction word: level-1 bucket expected for the threshold, extrapolated from the segment's last two steps
// at this level (bits 0-15),
// the half-width in buckets of the band collected around it (bits 16-23), and whether the next pass A may
// stage whole entries instead of keys (bit 24, see below; bit 25 forbids it for good).
constexpr unsigned kPredInvalid = 0xffffffffu;
__device__ __forceinline__ bool pred_band(unsigned word, unsigned* lo, unsigned* hi, bool* staged) {
  *staged = false;
  if (word == kPredInvalid) return false;
  const unsigned b = word & 0xffffu, hw = (word >> 16) & 0xffu;
  *staged = (word >> 24) & 1u;
  *lo = b > hw ? b - hw : 1u;  // bucket 0 (zeros, denormals) is never collected
  *hi = b + hw < (unsigned)kBins1 ? b + hw : (unsigned)kBins1 - 1u;
  return *lo <= *hi;
}

// Pass A.  Persistent blocks over (worker, tile) in worker-major order; the shared histogram is flushed
// when the (worker, layer) segment changes.  Where a prediction of the threshold's level-1 bucket exists
// (the bucket of the previous step at the same level), the keys of the buckets around it are collected
// on the fly into the segment's candidate list, so that no further pass over M is needed to refine the
// threshold when the prediction holds (checked exactly by pick1).
// When few entries are expected at or above the band (high compression level), pass A stages them whole --
// (value bits, layer-local index) for every key in a bucket >= the band's lowest -- so that, if the
// prediction holds, the kept entries are produced from this list and M is never read again for the
// segment (topk_finalize_staged_kernel instead of topk_select_kernel).
__global__ void __launch_bounds__(256)
topk_ef_hist1_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_tiles, int n_mat,
                     const float* __restrict__ grads, float* __restrict__ err, float* __restrict__ delta,
                     long long stride, int W, int decider, const uint8_t* __restrict__ level,
                     const unsigned* __restrict__ pred, unsigned* __restrict__ hist1,
                     unsigned* __restrict__ seg_cand, unsigned* __restrict__ seg_flag, unsigned* __restrict__ cand,
                     int2* __restrict__ tile_cand, long long cand_total, int2* __restrict__ tile_cnt,
                     const unsigned* __restrict__ pend_tau) {
  __shared__ unsigned h[kBins1];
  // three staging buffers for the collected keys: a tile's keys are copied out while the next tile is
  // being processed and the buffer is reused two tiles later, so one barrier per tile is enough
  __shared__ unsigned s_buf[3][kPredTileCap];
  __shared__ unsigned s_cnt[3], s_n[3];
  __shared__ int s_above[3];
  __shared__ long long s_dst[3];
  for (int b = threadIdx.x; b < kBins1; b += blockDim.x) h[b] = 0;
  if (threadIdx.x < 3) { s_cnt[threadIdx.x] = 0; s_above[threadIdx.x] = 0; s_n[threadIdx.x] = 0; }
  __syncthreads();
  const long long V = (long long)W * n_tiles;
  const long long v0 = V * blockIdx.x / gridDim.x, v1 = V * (blockIdx.x + 1) / gridDim.x;
  int cur = -1;
  int cb = 0, pend = -1;  // staging buffer in use; buffer waiting to be copied out
  bool collect = false, staged = false;
  unsigned blo = 1, bhi = 0;
  unsigned ptau = kNoPendingTau;  // lazy residual: entries of err above this key were kept by the last step
  // the layer record is kept while the tiles stay inside the layer (a tile's extent follows from its index), so
  // that a tile does not start with a chain of dependent loads
  DevLayer L;
  int cur_layer = -1;
  for (long long v = v0; v < v1; ++v) {
    const int w = (int)(v / n_tiles), ti = (int)(v % n_tiles);
    if (cur_layer < 0 || ti < L.tile0 || ti >= L.tile0 + L.ntiles) {
      cur_layer = tiles[ti].layer;
      L = layers[cur_layer];
    }
    if (L.kind != ACC_MATRIX) continue;
    Tile t;
    t.layer = cur_layer;
    t.elem0 = (ti - L.tile0) * kTile;
    t.nelem = (int)min((long long)kTile, (long long)L.rows * L.cols - t.elem0);
    const int seg = w * n_mat + L.mat;
    if (seg != cur) {
      __syncthreads();
      if (cur >= 0)
        for (int b = threadIdx.x; b < kBins1; b += blockDim.x) {
          const unsigned c = h[b];
          if (c) { atomicAdd(&hist1[(long long)cur * kBins1 + b], c); h[b] = 0; }
        }
      __syncthreads();
      cur = seg;
      collect = pred_band(pred[(level[t.layer] ? 1 : 0) * W * n_mat + seg], &blo, &bhi, &staged);
      ptau = pend_tau != nullptr ? pend_tau[seg] : kNoPendingTau;
    }
    const long long base = L.offset + t.elem0;
    const float* g = grads + (long long)w * stride + base;
    float* e = err + (long long)w * stride + base;
    const bool acc_delta = delta != nullptr && w == decider;
    const int n4 = t.nelem >> 2;
    const unsigned span = bhi - blo;
    unsigned* buf = s_buf[cb];
    unsigned* cnt = &s_cnt[cb];
    int above = 0;
    int nz = 0;  // non-zero keys of the tile seen by this thread (settles a threshold that falls among the zeros)
    // batches of kBatch float4 per thread: all loads of a batch are issued before the first store, so that
    // they are in flight together (a store to err in between would pin the later loads of err behind it)
    constexpr int kBatch = 4, kThreads = 256;
    for (int i0 = 0; i0 < n4; i0 += kBatch * kThreads) {
      float4 gb[kBatch], eb[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * kThreads + (int)threadIdx.x;
        if (i < n4) { gb[u] = ld_stream4(g + 4 * i); eb[u] = ld_stream4(e + 4 * i); }
      }
      // the next batch's lines are asked into L2 meanwhile (one request per 128-byte line)
      if ((threadIdx.x & 7) == 0) {
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int i = i0 + (kBatch + u) * kThreads + (int)threadIdx.x;
          if (i < n4) { prefetch_l2(g + 4 * i); prefetch_l2(e + 4 * i); }
        }
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * kThreads + (int)threadIdx.x;
        if (i >= n4) break;
        const float4 gv = gb[u];
        float4 ev = eb[u];
        // lazy residual: what the last step kept (key above its threshold) counts as +0.0
        ev.x = key_of(ev.x) > ptau ? 0.f : ev.x;
        ev.y = key_of(ev.y) > ptau ? 0.f : ev.y;
        ev.z = key_of(ev.z) > ptau ? 0.f : ev.z;
        ev.w = key_of(ev.w) > ptau ? 0.f : ev.w;
        const float4 m = make_float4(gv.x + ev.x, gv.y + ev.y, gv.z + ev.z, gv.w + ev.w);
        *reinterpret_cast<float4*>(e + 4 * i) = m;
        const unsigned k[4] = {key_of(m.x), key_of(m.y), key_of(m.z), key_of(m.w)};
        const float mm[4] = {m.x, m.y, m.z, m.w};
        nz += (k[0] != 0u) + (k[1] != 0u) + (k[2] != 0u) + (k[3] != 0u);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const unsigned bin = k[q] >> 19;
          atomicAdd(&h[bin], 1u);
          if (staged) {
            if (bin >= blo) {
              const unsigned slot = atomicAdd(cnt, 1u);
              if (slot < (unsigned)kPredTileCap / 2) {
                buf[2 * slot] = __float_as_uint(mm[q]);
                buf[2 * slot + 1] = (unsigned)(t.elem0 + 4 * i + q);
              }
            }
          } else if (collect) {
            above += bin > bhi;
            if (bin - blo <= span) {
              const unsigned slot = atomicAdd(cnt, 1u);
              if (slot < (unsigned)kPredTileCap) buf[slot] = k[q];
            }
          }
        }
      }
      if (acc_delta) {  // detector accumulator of the batch: its loads together too (err's registers are free now)
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int i = i0 + u * kThreads + (int)threadIdx.x;
          if (i < n4) eb[u] = *reinterpret_cast<const float4*>(delta + base + 4 * i);
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int i = i0 + u * kThreads + (int)threadIdx.x;
          if (i < n4)
            *reinterpret_cast<float4*>(delta + base + 4 * i) =
                make_float4(eb[u].x + gb[u].x, eb[u].y + gb[u].y, eb[u].z + gb[u].z, eb[u].w + gb[u].w);
        }
      }
    }
    for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
      const float gv = g[i];
      const float ev = e[i];
      const float m = gv + (key_of(ev) > ptau ? 0.f : ev);
      e[i] = m;
      const unsigned kk = key_of(m), bin = kk >> 19;
      nz += kk != 0u;
      atomicAdd(&h[bin], 1u);
      if (staged) {
        if (bin >= blo) {
          const unsigned slot = atomicAdd(cnt, 1u);
          if (slot < (unsigned)kPredTileCap / 2) {
            buf[2 * slot] = __float_as_uint(m);
            buf[2 * slot + 1] = (unsigned)(t.elem0 + i);
          }
        }
      } else if (collect) {
        above += bin > bhi;
        if (bin - blo <= span) {
          const unsigned slot = atomicAdd(cnt, 1u);
          if (slot < (unsigned)kPredTileCap) buf[slot] = kk;
        }
      }
      if (acc_delta) delta[base + i] += gv;
    }
    nz = __reduce_add_sync(0xffffffffu, nz);
    if ((threadIdx.x & 31) == 0 && nz) atomicAdd(&tile_cnt[(long long)w * n_tiles + ti].y, nz);  // cleared per step
    if (collect) {  // hand the tile's collected keys over to the segment's list
      above = __reduce_add_sync(0xffffffffu, above);
      if ((threadIdx.x & 31) == 0 && above) atomicAdd(&s_above[cb], above);
      const int nb = cb == 2 ? 0 : cb + 1;
      if (threadIdx.x == 0) { s_cnt[nb] = 0; s_above[nb] = 0; }  // free since the barrier of the previous tile
      __syncthreads();
      if (pend >= 0) {  // copy out the previous tile's keys (its range was published before this barrier)
        unsigned* dst = cand + s_dst[pend];
        const unsigned n = s_n[pend];  // in 4-byte words
        for (unsigned i = threadIdx.x; i < n; i += blockDim.x) dst[i] = s_buf[pend][i];
      }
      if (threadIdx.x == 0) {
        const unsigned words = staged ? 2u : 1u;  // list slots are keys (one word) or entries (two words)
        unsigned n = s_cnt[cb], start = 0;
        if (n * words > (unsigned)kPredTileCap) {
          atomicOr(&seg_flag[seg], 1u);
          n = 0;
        } else if (n) {
          start = atomicAdd(&seg_cand[seg], n);
          if ((start + n) * words > (unsigned)L.cand_cap) { atomicOr(&seg_flag[seg], 1u); n = 0; }
        }
        s_n[cb] = n * words;
        s_dst[cb] = (long long)w * cand_total + L.cand_base + (long long)start * words;
        tile_cand[(long long)w * n_tiles + ti] = make_int2((int)start, (int)n);
        tile_cnt[(long long)w * n_tiles + ti].x = s_above[cb];
      }
      pend = cb;
      cb = nb;
    }
  }
  __syncthreads();
  if (pend >= 0) {
    unsigned* dst = cand + s_dst[pend];
    const unsigned n = s_n[pend];
    for (unsigned i = threadIdx.x; i < n; i += blockDim.x) dst[i] = s_buf[pend][i];
  }
  if (cur >= 0)
    for (int b = threadIdx.x; b < kBins1; b += blockDim.x) {
      const unsigned c = h[b];
      if (c) atomicAdd(&hist1[(long long)cur * kBins1 + b], c);
    }
}

// Finds, scanning from the top bin, the bin that holds the `want`-th largest key (1-based).
// Single-thread helper over `nbins` counters; returns the bin and the count of keys in higher bins.
__device__ void pick_from_top(const unsigned* __restrict__ hist, int nbins, long long want, unsigned* bin,
                              long long* above) {
  long long cum = 0;
  int b = nbins - 1;
  for (; b > 0; --b) {
    const long long c = hist[b];
    if (cum + c >= want) break;
    cum += c;
  }
  *bin = (unsigned)b;
  *above = cum;
}

// Block-parallel version for the 4096-bin levels: each of 256 threads owns 16 consecutive bins; a suffix scan
// over the threads' sums finds the thread whose bins hold the `want`-th largest key, and that thread walks
// its own 16 counters.  (want >= 1 and the histogram holds at least `want` keys.)
__device__ void pick_from_top_block(const unsigned* __restrict__ hist, long long want, unsigned* bin,
                                    long long* above, unsigned* sm_sums) {
  const int tid = threadIdx.x;
  unsigned c[16];
  unsigned s = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) { c[i] = hist[tid * 16 + i]; s += c[i]; }
  sm_sums[tid] = s;
  if (tid == 0) { *bin = 0; *above = 0; }
  __syncthreads();
  for (int o = 1; o < 256; o <<= 1) {  // inclusive suffix sums: sm_sums[t] = keys in the bins of threads t..255
    const unsigned v = tid + o < 256 ? sm_sums[tid + o] : 0u;
    __syncthreads();
    sm_sums[tid] += v;
    __syncthreads();
  }
  const long long incl = sm_sums[tid], excl = incl - s;
  if (excl < want && want <= incl) {
    long long cum = excl;
    int b = 15;
    for (; b > 0; --b) {
      if (cum + c[b] >= want) break;
      cum += c[b];
    }
    *bin = (unsigned)(tid * 16 + b);
    *above = cum;
  }
  __syncthreads();
}

// One block per (worker, MATRIX layer): level-1 bucket b1 of the threshold, and how levels 2-3 will read
// the keys of that bucket: from the list collected by pass A if its prediction held (b1 inside the collected
// band, no overflow), else from a list the collect pass builds if the bucket fits, else from M itself.
// Also records b1 as the next prediction for this (level, segment).
__global__ void __launch_bounds__(256)
topk_pick1_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers, int n_mat, int n_layers,
                  int W, const uint8_t* __restrict__ level, const unsigned* __restrict__ hist1,
                  Select* __restrict__ sel, int32_t* __restrict__ counts, unsigned* __restrict__ pred,
                  unsigned* __restrict__ seg_cand, const unsigned* __restrict__ seg_flag,
                  unsigned* __restrict__ any_list, int2* __restrict__ lists, int n_tiles,
                  const int2* __restrict__ tile_cnt, unsigned* __restrict__ pend_tau) {
  __shared__ unsigned sums[256];
  __shared__ unsigned bin;
  __shared__ long long above;
  __shared__ int s_list;
  __shared__ unsigned s_base;
  __shared__ unsigned s_nz;
  const int seg = blockIdx.x, w = seg / n_mat, l = mat_layers[seg % n_mat];
  const DevLayer L = layers[l];
  const int lv = level[l] ? 1 : 0;
  const int k = lv ? L.k_low : L.k_high;
  if (threadIdx.x == 0) s_nz = 0;
  pick_from_top_block(hist1 + (long long)seg * kBins1, k, &bin, &above, sums);
  // The threshold falls into the lowest bucket (k exceeds the keys of all other buckets -- a row-sparse layer at a
  // large K): when that bucket holds nothing but exact zeros, which the first pass's per-tile counts of non-zero
  // keys tell, the answer needs no further look at M: every non-zero is kept and the first k - nnz zeros, tau = 0.
  bool zero_fill = false;
  if (bin == 0) {
    // (a layer holds fewer than 2^31 elements, so 32 bits do; the loads of a thread are independent and go out
    // together, the warps add their sums with one native shared-memory atomic each)
    const int2* tc = tile_cnt + (long long)w * n_tiles + L.tile0;
    unsigned part = 0;
#pragma unroll 4
    for (int i = threadIdx.x; i < L.ntiles; i += blockDim.x) part += (unsigned)__ldg(&tc[i].y);
    part = __reduce_add_sync(0xffffffffu, part);
    if ((threadIdx.x & 31) == 0 && part) atomicAdd(&s_nz, part);
    __syncthreads();
    zero_fill = (long long)s_nz == above;  // no non-zero key below the second bucket
  }
  if (threadIdx.x == 0) {
    Select s;
    s.b1 = bin; s.b2 = 0; s.tau = 0; s.k = k; s.k1 = k - (int)above; s.k2 = 0; s.need = 0;
    unsigned* pw = pred + (long long)lv * W * n_mat + seg;
    const unsigned word = *pw;
    unsigned blo, bhi;
    bool was_staged;
    const bool had_band = pred_band(word, &blo, &bhi, &was_staged);
    const bool overflow = seg_flag[seg] != 0;
    const unsigned* hs = hist1 + (long long)seg * kBins1;
    const bool fits = hs[bin] <= (unsigned)L.cand_cap;
    if (had_band && !overflow && bin >= blo && bin <= bhi) {
      s.mode = was_staged ? kSelStaged : kSelListPred;
    } else {
      seg_cand[seg] = 0;  // whatever pass A collected is of no use
      s.mode = fits ? kSelList : kSelDense;
    }
    if (zero_fill) {
      s.mode = kSelZeroFill;
      s.k2 = s.k1;
      s.need = s.k1;  // zeros to keep, lowest indices first
      if (pend_tau != nullptr) pend_tau[seg] = 0u;  // lazy residual: every non-zero entry was kept
    }
    // next prediction: narrow the band after an overflow; none for the zero bucket or for buckets that
    // do not fit the list
    unsigned hw = had_band ? ((word >> 16) & 0xffu) : 1u;
    if (had_band && overflow && !was_staged) hw = 0;
    // staging whole entries pays when few keys lie at or above the band: the entries of buckets >= b1 - hw,
    // with a margin, must fit half the list (two words each); after a staged overflow keys are collected again
    long long n_ge = above;
    for (unsigned b = bin > hw ? bin - hw : 1u; b <= bin; ++b) n_ge += hs[b];
    // (bit 25, sticky: staging overflowed once for this segment and level -- e.g. a row-sparse layer whose
    // non-zero rows fill whole tiles -- and is not tried again
    // -- only when the prediction itself was right: a band that lay too low overflows for that reason alone)
    const bool no_stage = (word != kPredInvalid && ((word >> 25) & 1u)) ||
                          (had_band && overflow && was_staged && bin >= blo && bin <= bhi);
    const bool stage_next = !no_stage && n_ge * 5 / 2 <= (long long)L.cand_cap &&
                            n_ge * 3 / 2 <= (long long)L.ntiles * (kPredTileCap / 2);
    // the band is centred on the bucket extrapolated from the last two steps at this level: under error
    // feedback the threshold drifts steadily (it climbs for tens of steps after a switch to the high level)
    unsigned* lb = pred + (long long)(2 + lv) * W * n_mat + seg;
    const unsigned last = *lb;
    int drift = last != kPredInvalid ? (int)bin - (int)last : 0;
    drift = drift < -12 ? -12 : drift > 12 ? 12 : drift;
    // the mean of the last two moves (rounded toward zero): a threshold that hops between two neighbouring buckets
    // keeps its band, a climb of one to two buckets a step with some jitter stays inside it, steady faster
    // moves are followed
    int* ld = reinterpret_cast<int*>(pred + (long long)(4 + lv) * W * n_mat + seg);
    const int prev_drift = last != kPredInvalid ? *ld : 0;
    *ld = drift;
    int centre = (int)bin + (drift + prev_drift) / 2;
    centre = centre < 1 ? 1 : centre > kBins1 - 1 ? kBins1 - 1 : centre;
    *lb = bin;
    *pw = (!fits || bin == 0) ? kPredInvalid
                              : ((unsigned)centre | (hw << 16) | ((stage_next ? 1u : 0u) << 24) |
                                 ((no_stage ? 1u : 0u) << 25));
    sel[seg] = s;
    counts[w * n_layers + l] = k;
    // the segment's tiles join the work list of the pass that will read M for levels 2-3, as one run
    s_list = s.mode == kSelList ? kListCollect : s.mode == kSelDense ? kListDense : -1;
    if (s_list >= 0) s_base = atomicAdd(&any_list[kListCountWord + s_list], (unsigned)L.ntiles);
  }
  __syncthreads();
  if (s_list >= 0) {
    int2* dst = lists + (long long)s_list * W * n_tiles + s_base;
    for (int i = threadIdx.x; i < L.ntiles; i += blockDim.x) dst[i] = make_int2(w, L.tile0 + i);
  }
}

__global__ void __launch_bounds__(256)
topk_pick2_kernel(int n_mat, const unsigned* __restrict__ hist2, Select* __restrict__ sel) {
  __shared__ unsigned sums[256];
  __shared__ unsigned bin;
  __shared__ long long above;
  const int seg = blockIdx.x;
  if (sel[seg].mode == kSelZeroFill) return;  // settled by pick1
  const int k1 = sel[seg].k1;
  pick_from_top_block(hist2 + (long long)seg * kBins2, k1, &bin, &above, sums);
  if (threadIdx.x == 0) { sel[seg].b2 = bin; sel[seg].k2 = k1 - (int)above; }
}

// List path.  One block per (tile, worker) of a segment in list mode: the tile's keys of bucket b1 go to a
// range of the segment's candidate list (reserved with one atomic per tile; the order of the ranges does
// not matter, the keys are only counted later), and the keys above b1 are counted.
template <bool FULL>
__device__ __forceinline__ void collect_tile(const Tile& t, const Select& s, const float* __restrict__ m,
                                             unsigned* __restrict__ seg_counter, unsigned* __restrict__ seg_list,
                                             int2* __restrict__ tile_cand_out, int2* __restrict__ tile_cnt_out,
                                             unsigned* wsum, unsigned* s_start) {
  const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float4 mv[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e0 = 4 * (j * 256 + (int)threadIdx.x);
    if (FULL || e0 + 3 < t.nelem) {
      mv[j] = ld_stream4(m + e0);
    } else {  // ragged end of the layer: absent elements are masked out by `valid` below
      mv[j].x = e0 < t.nelem ? m[e0] : 0.f;
      mv[j].y = e0 + 1 < t.nelem ? m[e0 + 1] : 0.f;
      mv[j].z = e0 + 2 < t.nelem ? m[e0 + 2] : 0.f;
      mv[j].w = 0.f;
    }
  }
  unsigned inb = 0;  // one bit per element of this thread: key in bucket b1
  int above = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e0 = 4 * (j * 256 + (int)threadIdx.x);
    const float v[4] = {mv[j].x, mv[j].y, mv[j].z, mv[j].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const unsigned b = key_of(v[e]) >> 19;
      const bool valid = FULL || e0 + e < t.nelem;
      above += valid && b > s.b1;
      inb |= (unsigned)(valid && b == s.b1) << (4 * j + e);
    }
  }
  // block-wide exclusive prefix of (candidates | above << 16)
  const unsigned own = (unsigned)__popc(inb) | ((unsigned)above << 16);
  unsigned c = own;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, c, o);
    if (lane >= o) c += n;
  }
  if (lane == 31) wsum[wi] = c;
  __syncthreads();
  unsigned wbase = 0, total = 0;
  for (int i = 0; i < 8; ++i) {
    if (i < wi) wbase += wsum[i];
    total += wsum[i];
  }
  if (threadIdx.x == 0) {
    const unsigned n_cand = total & 0xffffu;
    const unsigned start = n_cand ? atomicAdd(seg_counter, n_cand) : 0u;
    *s_start = start;
    *tile_cand_out = make_int2((int)start, (int)n_cand);
    tile_cnt_out->x = (int)(total >> 16);
  }
  __syncthreads();
  if (inb != 0) {
    unsigned* dst = seg_list + *s_start + ((wbase + c - own) & 0xffffu);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float v[4] = {mv[j].x, mv[j].y, mv[j].z, mv[j].w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if ((inb >> (4 * j + e)) & 1u) *dst++ = key_of(v[e]);
    }
  }
  __syncthreads();  // wsum and s_start are reused by the block's next tile
}

// Blocks walk the (worker, tile) pairs with a grid stride; when no segment of this step is in list mode
// (every prediction of pass A held, or only dense segments remain) the kernel ends at once.
__global__ void __launch_bounds__(256, 3)
topk_collect_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_tiles, int n_mat,
                    int W, const float* __restrict__ err, long long stride, const Select* __restrict__ sel,
                    const unsigned* __restrict__ any_list, unsigned* __restrict__ seg_cand,
                    unsigned* __restrict__ cand, int2* __restrict__ tile_cand, long long cand_total,
                    int2* __restrict__ tile_cnt, const int2* __restrict__ lists) {
  __shared__ unsigned wsum[8];
  __shared__ unsigned s_start;
  const unsigned n_work = any_list[kListCountWord + kListCollect];
  const int2* work = lists + (long long)kListCollect * W * n_tiles;
  for (unsigned b = blockIdx.x; b < n_work; b += gridDim.x) {
    __syncthreads();  // the shared words of the previous tile are no longer read
    const int w = work[b].x, ti = work[b].y;
    const long long v = (long long)w * n_tiles + ti;
    const Tile t = tiles[ti];
    const DevLayer L = layers[t.layer];
    const int seg = w * n_mat + L.mat;
    const Select s = sel[seg];
    const float* m = err + (long long)w * stride + L.offset + t.elem0;
    unsigned* list = cand + (long long)w * cand_total + L.cand_base;
    if (t.nelem == kTile) collect_tile<true>(t, s, m, seg_cand + seg, list, tile_cand + v, tile_cnt + v, wsum, &s_start);
    else collect_tile<false>(t, s, m, seg_cand + seg, list, tile_cand + v, tile_cnt + v, wsum, &s_start);
  }
}

// Pass C.  Level-2 histogram of the keys whose level-1 bin is b1; per tile, how many keys lie in higher bins.
__global__ void __launch_bounds__(256)
topk_hist2_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_tiles, int n_mat,
                  const float* __restrict__ err, long long stride, int W, const Select* __restrict__ sel,
                  const unsigned* __restrict__ any_list, unsigned* __restrict__ hist2,
                  int2* __restrict__ tile_cnt, const int2* __restrict__ lists) {
  __shared__ unsigned h[kBins2];
  __shared__ int cnt;
  // the dense segments' tiles, each segment one contiguous run of the list; a block takes a contiguous share
  const long long V = any_list[kListCountWord + kListDense];
  const long long v0 = V * blockIdx.x / gridDim.x, v1 = V * (blockIdx.x + 1) / gridDim.x;
  if (v0 >= v1) return;
  const int2* work = lists + (long long)kListDense * W * n_tiles;
  for (int b = threadIdx.x; b < kBins2; b += blockDim.x) h[b] = 0;
  if (threadIdx.x == 0) cnt = 0;
  __syncthreads();
  int cur = -1;
  unsigned b1 = 0;
  for (long long v = v0; v < v1; ++v) {
    const int w = work[v].x, ti = work[v].y;
    const Tile t = tiles[ti];
    const DevLayer L = layers[t.layer];
    const int seg = w * n_mat + L.mat;
    if (seg != cur) {
      __syncthreads();
      if (cur >= 0)
        for (int b = threadIdx.x; b < kBins2; b += blockDim.x) {
          const unsigned c = h[b];
          if (c) { atomicAdd(&hist2[(long long)cur * kBins2 + b], c); h[b] = 0; }
        }
      __syncthreads();
      cur = seg;
      b1 = sel[seg].b1;
    }
    const float* m = err + (long long)w * stride + L.offset + t.elem0;
    int above = 0;
    const int n4 = t.nelem >> 2;
#pragma unroll 4
    for (int i = threadIdx.x; i < n4; i += blockDim.x) {
      const float4 mv = ld_stream4(m + 4 * i);
      const unsigned k0 = key_of(mv.x), k1 = key_of(mv.y), k2 = key_of(mv.z), k3 = key_of(mv.w);
      above += ((k0 >> 19) > b1) + ((k1 >> 19) > b1) + ((k2 >> 19) > b1) + ((k3 >> 19) > b1);
      if ((k0 >> 19) == b1) atomicAdd(&h[(k0 >> 7) & 0xfffu], 1u);
      if ((k1 >> 19) == b1) atomicAdd(&h[(k1 >> 7) & 0xfffu], 1u);
      if ((k2 >> 19) == b1) atomicAdd(&h[(k2 >> 7) & 0xfffu], 1u);
      if ((k3 >> 19) == b1) atomicAdd(&h[(k3 >> 7) & 0xfffu], 1u);
    }
    for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
      const unsigned k0 = key_of(m[i]);
      above += (k0 >> 19) > b1;
      if ((k0 >> 19) == b1) atomicAdd(&h[(k0 >> 7) & 0xfffu], 1u);
    }
    above = __reduce_add_sync(0xffffffffu, above);
    if ((threadIdx.x & 31) == 0 && above) atomicAdd(&cnt, above);
    __syncthreads();
    if (threadIdx.x == 0) { tile_cnt[(long long)w * n_tiles + ti].x = cnt; cnt = 0; }
    __syncthreads();
  }
  __syncthreads();
  if (cur >= 0)
    for (int b = threadIdx.x; b < kBins2; b += blockDim.x) {
      const unsigned c = h[b];
      if (c) atomicAdd(&hist2[(long long)cur * kBins2 + b], c);
    }
}

// Pass C'.  One block per (tile, worker): level-3 histogram of the keys with 24-bit prefix (b1, b2), kept
// per tile (16-bit counters) and summed per segment; per-tile count of keys in bin b1 above b2.
__global__ void __launch_bounds__(256)
topk_hist3_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_tiles, int n_mat,
                  const float* __restrict__ err, long long stride, const Select* __restrict__ sel,
                  const unsigned* __restrict__ any_list, unsigned* __restrict__ hist3,
                  int2* __restrict__ tile_cnt, unsigned short* __restrict__ tile_h3, const int2* __restrict__ lists,
                  int W) {
  __shared__ unsigned h[kBins3];
  __shared__ int cnt;
  const unsigned n_work = any_list[kListCountWord + kListDense];
  const int2* work = lists + (long long)kListDense * W * n_tiles;
  for (unsigned b = blockIdx.x; b < n_work; b += gridDim.x) {
    const int w = work[b].x, ti = work[b].y;
    const Tile t = tiles[ti];
    const DevLayer L = layers[t.layer];
    const int seg = w * n_mat + L.mat;
    const Select s = sel[seg];
    __syncthreads();  // the previous tile's counters have been read
    if (threadIdx.x < kBins3) h[threadIdx.x] = 0;
    if (threadIdx.x == 0) cnt = 0;
    __syncthreads();
    const unsigned prefix = (s.b1 << 12) | s.b2;
    const float* m = err + (long long)w * stride + L.offset + t.elem0;
    int above = 0;
    {
      const int n4 = t.nelem >> 2;
#pragma unroll 4
      for (int i = threadIdx.x; i < n4; i += blockDim.x) {
        const float4 mv = ld_stream4(m + 4 * i);
        const unsigned k[4] = {key_of(mv.x), key_of(mv.y), key_of(mv.z), key_of(mv.w)};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned p = k[e] >> 7;
          above += ((p >> 12) == s.b1) && (p > prefix);
          if (p == prefix) atomicAdd(&h[k[e] & 127u], 1u);
        }
      }
      for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
        const unsigned k0 = key_of(m[i]), p = k0 >> 7;
        above += ((p >> 12) == s.b1) && (p > prefix);
        if (p == prefix) atomicAdd(&h[k0 & 127u], 1u);
      }
    }
    above = __reduce_add_sync(0xffffffffu, above);
    if ((threadIdx.x & 31) == 0 && above) atomicAdd(&cnt, above);
    __syncthreads();
    if (threadIdx.x == 0) tile_cnt[(long long)w * n_tiles + ti].y = cnt;
    if (threadIdx.x < kBins3) {
      const unsigned c = h[threadIdx.x];
      tile_h3[((long long)w * n_tiles + ti) * kBins3 + threadIdx.x] = (unsigned short)c;
      if (c) atomicAdd(&hist3[(long long)seg * kBins3 + threadIdx.x], c);
    }
  }
}

// List path, levels 2 and 3.  The keys collected for a segment (by pass A or by the collect pass) sit in one
// contiguous list; blocks (chunk, segment) histogram them.  LEVEL 2: keys of bucket b1 by their next 12 bits;
// LEVEL 3: keys with the 24-bit prefix (b1, b2) by their last 7 bits.
template <int LEVEL>
__global__ void __launch_bounds__(256)
topk_hist_list_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers, int n_mat,
                      const Select* __restrict__ sel, const unsigned* __restrict__ seg_cand,
                      const unsigned* __restrict__ cand, long long cand_total, unsigned* __restrict__ hist) {
  constexpr int kBins = LEVEL == 2 ? kBins2 : kBins3;
  constexpr unsigned kChunk = 4096;
  __shared__ unsigned h[kBins];
  const int seg = blockIdx.y;
  const Select s = sel[seg];
  if (s.mode == kSelDense || s.mode == kSelZeroFill) return;
  const unsigned n = seg_cand[seg] << (s.mode == kSelStaged ? 1 : 0);  // in 4-byte words
  if (blockIdx.x * kChunk >= n) return;
  for (int b = threadIdx.x; b < kBins; b += blockDim.x) h[b] = 0;
  __syncthreads();
  const DevLayer L = layers[mat_layers[seg % n_mat]];
  const unsigned* keys = cand + (long long)(seg / n_mat) * cand_total + L.cand_base;
  const unsigned prefix = (s.b1 << 12) | s.b2;
  const bool staged = s.mode == kSelStaged;  // the list holds (value bits, index) pairs instead of keys
  auto count = [&](unsigned kk) {
    if (LEVEL == 2) {
      if ((kk >> 19) == s.b1) atomicAdd(&h[(kk >> 7) & 0xfffu], 1u);
    } else {
      if ((kk >> 7) == prefix) atomicAdd(&h[kk & 127u], 1u);
    }
  };
  for (unsigned c0 = blockIdx.x * kChunk; c0 < n; c0 += gridDim.x * kChunk) {
    const unsigned c1 = min(c0 + kChunk, n);  // the list starts 16-byte aligned and kChunk is a multiple of 4
    const unsigned n4 = (c1 - c0) >> 2;
    const uint4* k4 = reinterpret_cast<const uint4*>(keys + c0);
    // (the chunk's loads of a thread -- four 16-byte words -- go out together, then the counting)
    constexpr int kLoads = kChunk / 4 / 256;
    uint4 kb[kLoads];
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const unsigned i = threadIdx.x + u * 256u;
      if (i < n4) kb[u] = __ldcs(k4 + i);
    }
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const unsigned i = threadIdx.x + u * 256u;
      if (i < n4) {
        const uint4 kk = kb[u];
        if (staged) {
          count(kk.x & 0x7fffffffu); count(kk.z & 0x7fffffffu);
        } else {
          count(kk.x); count(kk.y); count(kk.z); count(kk.w);
        }
      }
    }
    for (unsigned i = c0 + 4 * n4 + threadIdx.x; i < c1; i += blockDim.x)
      if (!staged) count(keys[i]);
      else if ((i & 1u) == 0) count(keys[i] & 0x7fffffffu);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kBins; b += blockDim.x) {
    const unsigned c = h[b];
    if (c) atomicAdd(&hist[(long long)seg * kBins + b], c);
  }
}

// One warp per (worker, MATRIX layer): bucket b3 of level 3, hence the threshold tau and the number of ties
// (key == tau) to keep.  Lane l owns bins 4l..4l+3; a suffix sum over the lanes locates the bin.
__global__ void __launch_bounds__(256)
topk_pick3_kernel(int n_seg, const unsigned* __restrict__ hist3, Select* __restrict__ sel,
                  unsigned* __restrict__ pend_tau) {
  const int seg = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (seg >= n_seg || sel[seg].mode == kSelZeroFill) return;
  const uint4 c4 = *reinterpret_cast<const uint4*>(hist3 + (long long)seg * kBins3 + 4 * lane);
  const unsigned c[4] = {c4.x, c4.y, c4.z, c4.w};
  const unsigned own = c[0] + c[1] + c[2] + c[3];
  const unsigned want = (unsigned)sel[seg].k2;
  unsigned suf = own;  // sum over lanes >= this one
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned n = __shfl_down_sync(0xffffffffu, suf, o);
    if (lane + o < 32) suf += n;
  }
  const unsigned hit = __ballot_sync(0xffffffffu, suf >= want);
  const int top = hit ? 31 - __clz((int)hit) : 0;  // highest lane whose suffix reaches `want`
  if (lane == top) {
    unsigned cum = suf - own;
    int i = 3;
    for (; i > 0; --i) {
      if (cum + c[i] >= want) break;
      cum += c[i];
    }
    Select s = sel[seg];
    s.tau = (s.b1 << 19) | (s.b2 << 7) | (unsigned)(4 * lane + i);
    s.need = s.k2 - (int)cum;
    sel[seg] = s;
    if (pend_tau != nullptr) pend_tau[seg] = s.tau;  // lazy residual: keys above tau stay in err until the next load
  }
}

// One warp per (tile, worker): (keys above tau, keys equal to tau) of the tile, from its counters and its
// level-3 histogram.
__global__ void __launch_bounds__(256)
topk_tile_counts_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_tiles, int n_mat,
                        int W, const Select* __restrict__ sel, const int2* __restrict__ tile_cnt,
                        const unsigned short* __restrict__ tile_h3, const unsigned* __restrict__ cand,
                        const int2* __restrict__ tile_cand, long long cand_total, int2* __restrict__ tile_pre) {
  const long long v = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (v >= (long long)W * n_tiles) return;
  const int w = (int)(v / n_tiles), ti = (int)(v % n_tiles);
  const DevLayer L = layers[tiles[ti].layer];
  if (L.kind != ACC_MATRIX) return;
  const Select s = sel[w * n_mat + L.mat];
  if (s.mode == kSelZeroFill) {  // tau = 0: the non-zeros lie above it, the zeros tie with it
    if (lane == 0) {
      const int nz = tile_cnt[v].y;
      tile_pre[v] = make_int2(nz, tiles[ti].nelem - nz);
    }
    return;
  }
  if (s.mode != kSelDense) {  // list segment: count the tile's collected keys against the final threshold
    const int2 tc = tile_cand[v];
    const bool staged = s.mode == kSelStaged;
    const unsigned* keys = cand + (long long)w * cand_total + L.cand_base + (staged ? 2 * tc.x : tc.x);
    int above = 0, ties = 0;
    for (int i = lane; i < tc.y; i += 32) {
      const unsigned kk = staged ? (keys[2 * i] & 0x7fffffffu) : keys[i];
      above += kk > s.tau;
      ties += kk == s.tau;
    }
    above = __reduce_add_sync(0xffffffffu, above);
    ties = __reduce_add_sync(0xffffffffu, ties);
    if (lane == 0) tile_pre[v] = make_int2(tile_cnt[v].x + above, ties);
    return;
  }
  const unsigned b3 = s.tau & 127u;
  const unsigned short* h = tile_h3 + v * kBins3;
  const uint2 raw = *reinterpret_cast<const uint2*>(h + 4 * lane);  // bins 4*lane .. 4*lane+3
  const unsigned c[4] = {raw.x & 0xffffu, raw.x >> 16, raw.y & 0xffffu, raw.y >> 16};
  int above = 0, ties = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const unsigned b = 4 * lane + i;
    above += b > b3 ? (int)c[i] : 0;
    ties += b == b3 ? (int)c[i] : 0;
  }
  above = __reduce_add_sync(0xffffffffu, above);
  ties = __reduce_add_sync(0xffffffffu, ties);
  if (lane == 0) {
    const int2 c0 = tile_cnt[v];
    tile_pre[v] = make_int2(c0.x + c0.y + above, ties);
  }
}

// Exclusive prefix of v over the 256 threads of the block (warp shuffles + the eight warp totals); *total = sum.
__device__ __forceinline__ int block_excl_scan_256(int v, int* wsum, int* total) {
  const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) wsum[wi] = incl;
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = wsum[i];
    base += i < wi ? c : 0;
    tot += c;
  }
  __syncthreads();  // wsum may be reused
  *total = tot;
  return base + incl - v;
}

// One block per (worker, MATRIX layer): exclusive prefix, over the layer's tiles in index order, of the
// per-tile (above, ties) counts, in place.  The tiles that hold something to keep -- a key above the threshold, or a
// tie while fewer than `need` ties precede the tile -- join the work list of the pass that will write their
// entries: the staged list or the select list.
__global__ void __launch_bounds__(256)
topk_tile_scan_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ mat_layers, int n_mat,
                      int n_tiles, int W, const Select* __restrict__ sel, int2* __restrict__ tile_pre,
                      int2* __restrict__ tile_own, int2* __restrict__ tile_rng, unsigned* __restrict__ any_list,
                      int2* __restrict__ lists) {
  __shared__ int wsum[8];
  __shared__ unsigned s_base;
  const int seg = blockIdx.x, w = seg / n_mat, l = mat_layers[seg % n_mat];
  const DevLayer L = layers[l];
  const Select s = sel[seg];
  const int which = s.mode == kSelStaged ? kListStaged : kListSelect;
  const long long tb = (long long)w * n_tiles + L.tile0;
  const int per = (L.ntiles + 255) / 256;
  const int t0 = min(L.ntiles, (int)threadIdx.x * per), t1 = min(L.ntiles, t0 + per);
  int2 sum = make_int2(0, 0);
  for (int t = t0; t < t1; ++t) {
    const int2 c = tile_pre[tb + t];
    sum.x += c.x; sum.y += c.y;
  }
  int total;
  int2 run;
  run.x = block_excl_scan_256(sum.x, wsum, &total);
  run.y = block_excl_scan_256(sum.y, wsum, &total);
  int act = 0;
  {
    int ties_before = run.y;
    for (int t = t0; t < t1; ++t) {
      const int2 c = tile_pre[tb + t];
      act += c.x != 0 || (c.y != 0 && ties_before < s.need);
      ties_before += c.y;
    }
  }
  const int slot = block_excl_scan_256(act, wsum, &total);
  if (threadIdx.x == 0) s_base = total ? atomicAdd(&any_list[kListCountWord + which], (unsigned)total) : 0u;
  __syncthreads();
  int2* dst = lists + (long long)which * W * n_tiles + s_base + slot;
  for (int t = t0; t < t1; ++t) {
    const int2 c = tile_pre[tb + t];
    tile_pre[tb + t] = run;
    tile_own[tb + t] = c;  // the tile's own (above, ties), for the select pass
    if (c.x != 0 || (c.y != 0 && run.y < s.need)) *dst++ = make_int2(w, L.tile0 + t);
    const int lo = min(run.x + min(run.y, s.need), s.k);  // (the clamps hold by construction)
    run.x += c.x; run.y += c.y;
    // the tile's entries inside the worker's packed segment, for the decompress pass
    tile_rng[tb + t] = make_int2(lo, min(run.x + min(run.y, s.need), s.k));
  }
}

__device__ __forceinline__ unsigned warp_incl_scan(unsigned c, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, c, o);
    if (lane >= o) c += n;
  }
  return c;
}

// Pass E.  One block per (tile, worker).  Warp `wi` owns float4s [wi*256, wi*256+256) of the tile; lane
// handles float4 j*32+lane of that range for j = 0..7, so (j, lane, element) is index order.  Writes the
// kept (value, index) pairs at their final positions and zeroes them in err.
// Per-j lane counts are at most 4 and their warp prefixes at most 128, so four j share one 32-bit scan.
// LAZY: entries above the threshold are not zeroed in err (the next first pass, or the flush, treats them as zero);
// the kept ties are.
template <bool FULL, bool LAZY>
__device__ __forceinline__ void select_tile(const Tile& t, const unsigned tau, const int need, const int k,
                                            const int2 pre, float* __restrict__ m, float* __restrict__ vals,
                                            int32_t* __restrict__ idx, long long seg, unsigned* wtot) {
  const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float4 mv[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e0 = 4 * (wi * 256 + j * 32 + lane);
    if (FULL || e0 + 3 < t.nelem) {
      mv[j] = ld_stream4(m + e0);
    } else {
      mv[j].x = e0 < t.nelem ? m[e0] : 0.f;
      mv[j].y = e0 + 1 < t.nelem ? m[e0 + 1] : 0.f;
      mv[j].z = e0 + 2 < t.nelem ? m[e0 + 2] : 0.f;
      mv[j].w = 0.f;
    }
  }
  unsigned am = 0, tm = 0;                   // 4 bits per j: key > tau, key == tau
  unsigned ca[2] = {0, 0}, ct[2] = {0, 0};   // one byte per j: counts of this lane
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e0 = 4 * (wi * 256 + j * 32 + lane);
    const unsigned k[4] = {key_of(mv[j].x), key_of(mv[j].y), key_of(mv[j].z), key_of(mv[j].w)};
    unsigned a = 0, tt = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool valid = FULL || e0 + e < t.nelem;
      a |= (unsigned)(valid && k[e] > tau) << e;
      tt |= (unsigned)(valid && k[e] == tau) << e;
    }
    am |= a << (4 * j);
    tm |= tt << (4 * j);
    ca[j >> 2] |= (unsigned)__popc(a) << (8 * (j & 3));
    ct[j >> 2] |= (unsigned)__popc(tt) << (8 * (j & 3));
  }
  unsigned ia[2], it[2] = {0, 0};
  ia[0] = warp_incl_scan(ca[0], lane);
  ia[1] = warp_incl_scan(ca[1], lane);
  const bool any_tie = __any_sync(0xffffffffu, tm != 0);
  if (any_tie) {
    it[0] = warp_incl_scan(ct[0], lane);
    it[1] = warp_incl_scan(ct[1], lane);
  }
  const unsigned ta0 = __shfl_sync(0xffffffffu, ia[0], 31), ta1 = __shfl_sync(0xffffffffu, ia[1], 31);
  const unsigned tt0 = __shfl_sync(0xffffffffu, it[0], 31), tt1 = __shfl_sync(0xffffffffu, it[1], 31);
  // byte sums: totals of the warp
  const unsigned wa = __dp4a(ta0, 0x01010101u, 0u) + __dp4a(ta1, 0x01010101u, 0u);
  const unsigned wt = __dp4a(tt0, 0x01010101u, 0u) + __dp4a(tt1, 0x01010101u, 0u);
  if (lane == 0) wtot[wi] = wa | (wt << 16);
  __syncthreads();
  if ((am | tm) == 0) return;
  unsigned wbase = 0;
  for (int i = 0; i < wi; ++i) wbase += wtot[i];
  int base_a = pre.x + (int)(wbase & 0xffffu), base_t = pre.y + (int)(wbase >> 16);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const unsigned a = (am >> (4 * j)) & 15u, tt = (tm >> (4 * j)) & 15u;
    const unsigned sh = 8 * (j & 3);
    const unsigned tot_a = ((j < 4 ? ta0 : ta1) >> sh) & 0xffu, tot_t = ((j < 4 ? tt0 : tt1) >> sh) & 0xffu;
    if (a | tt) {
      const int e0 = 4 * (wi * 256 + j * 32 + lane);
      int above_before = base_a + (int)((ia[j >> 2] >> sh) & 0xffu) - __popc(a);
      int ties_before = base_t + (int)((it[j >> 2] >> sh) & 0xffu) - __popc(tt);
      const float v[4] = {mv[j].x, mv[j].y, mv[j].z, mv[j].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool is_a = (a >> e) & 1u, is_t = (tt >> e) & 1u;
        if (is_a || (is_t && ties_before < need)) {
          const int pos = above_before + min(ties_before, need);
          if ((unsigned)pos < (unsigned)k) {  // always true for consistent counts; keeps a write inside the segment
            vals[seg + pos] = v[e];
            idx[seg + pos] = t.elem0 + e0 + e;
            if (!LAZY || !is_a) m[e0 + e] = 0.f;
          }
        }
        above_before += is_a;
        ties_before += is_t;
      }
    }
    base_a += (int)tot_a;
    base_t += (int)tot_t;
  }
}

// The same for a tile in which the ties need no counting: either every key equal to tau is kept (the tie budget
// outlasts the tile) or none is (no tie in the tile, or the budget ran out before it) -- every tile of a segment but
// the one where the budget runs out.  An entry is then kept iff its key >= thr (tau or tau + 1), one mask and one
// scan instead of two, and the positions follow from the count of kept entries alone.
template <bool FULL, bool LAZY>
__device__ __forceinline__ void select_tile_simple(const Tile& t, unsigned thr, unsigned tau, bool zero_ties,
                                                   int base, int k, float* __restrict__ m,
                                                   float* __restrict__ vals, int32_t* __restrict__ idx, long long seg,
                                                   unsigned* wtot) {
  const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float4 mv[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e0 = 4 * (wi * 256 + j * 32 + lane);
    if (FULL || e0 + 3 < t.nelem) {
      mv[j] = ld_stream4(m + e0);
    } else {
      mv[j].x = e0 < t.nelem ? m[e0] : 0.f;
      mv[j].y = e0 + 1 < t.nelem ? m[e0 + 1] : 0.f;
      mv[j].z = e0 + 2 < t.nelem ? m[e0 + 2] : 0.f;
      mv[j].w = 0.f;
    }
  }
  unsigned km = 0;            // 4 bits per j: entry kept
  unsigned c[2] = {0, 0};     // one byte per j: kept entries of this lane
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e0 = 4 * (wi * 256 + j * 32 + lane);
    const unsigned kk[4] = {key_of(mv[j].x), key_of(mv[j].y), key_of(mv[j].z), key_of(mv[j].w)};
    unsigned nib = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) nib |= (unsigned)((FULL || e0 + e < t.nelem) && kk[e] >= thr) << e;
    km |= nib << (4 * j);
    c[j >> 2] |= (unsigned)__popc(nib) << (8 * (j & 3));
  }
  const unsigned i0 = warp_incl_scan(c[0], lane), i1 = warp_incl_scan(c[1], lane);
  const unsigned t0 = __shfl_sync(0xffffffffu, i0, 31), t1 = __shfl_sync(0xffffffffu, i1, 31);
  if (lane == 0) wtot[wi] = __dp4a(t0, 0x01010101u, 0u) + __dp4a(t1, 0x01010101u, 0u);
  __syncthreads();
  if (km == 0) return;
  int pos0 = base;
  for (int i = 0; i < wi; ++i) pos0 += (int)wtot[i];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const unsigned nib = (km >> (4 * j)) & 15u;
    const unsigned sh = 8 * (j & 3);
    if (nib) {
      const int e0 = 4 * (wi * 256 + j * 32 + lane);
      int pos = pos0 + (int)(((j < 4 ? i0 : i1) >> sh) & 0xffu) - __popc(nib);
      const float v[4] = {mv[j].x, mv[j].y, mv[j].z, mv[j].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if ((nib >> e) & 1u) {
          if ((unsigned)pos < (unsigned)k) {  // always true for consistent counts; keeps a write inside the segment
            vals[seg + pos] = v[e];
            idx[seg + pos] = t.elem0 + e0 + e;
            // eager: every kept entry becomes +0.0; lazy: only the kept ties (entries above tau are dropped by the
            // next load), and of those only the ones that are not +0.0 already (tau = 0: the negative zeros)
            if (!LAZY) m[e0 + e] = 0.f;
            else if (zero_ties && key_of(v[e]) == tau && __float_as_uint(v[e]) != 0u) m[e0 + e] = 0.f;
          }
          ++pos;
        }
      }
    }
    pos0 += (int)(((j < 4 ? t0 : t1) >> sh) & 0xffu);
  }
}

// The same for a full tile with few entries to keep (the usual case: K of 1 % to 10 %), every lane owning 32
// CONSECUTIVE elements: the warp's 1024 elements go through shared memory (coalesced 16-byte loads in, one padded
// row of 32 per lane out), so that an entry's position is the lane's exclusive prefix plus a running count -- the
// kept entries are found by walking the set bits of one 32-bit mask, a dozen instructions each, instead of deriving
// the position of every entry from per-row prefixes (the walk was half of the pass).  A warp runs as many rounds
// as its busiest lane has kept entries.
constexpr int kRowWords = 36;  // 32 elements + 4 words of padding: 16-byte reads of consecutive rows hit distinct banks
template <bool LAZY>
__device__ __forceinline__ void select_tile_rows(const Tile& t, unsigned thr, unsigned tau, bool zero_ties, int base,
                                                 int k, float* __restrict__ m, float* __restrict__ vals,
                                                 int32_t* __restrict__ idx, long long seg, unsigned* wtot,
                                                 float* rows) {
  const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* wr = rows + wi * (32 * kRowWords);
  float4 mv[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) mv[j] = ld_stream4(m + 4 * (wi * 256 + j * 32 + lane));
#pragma unroll
  for (int j = 0; j < 8; ++j)  // float4 number j * 32 + lane of the warp: row 4 j + lane / 8, column 4 (lane % 8)
    *reinterpret_cast<float4*>(wr + kRowWords * (4 * j + (lane >> 3)) + 4 * (lane & 7)) = mv[j];
  __syncwarp();
  const float* my = wr + kRowWords * lane;
  unsigned km = 0;  // bit i: element 32 * lane + i of the warp's share is kept
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const float4 v = *reinterpret_cast<const float4*>(my + 4 * q);
    km |= ((unsigned)(key_of(v.x) >= thr) | ((unsigned)(key_of(v.y) >= thr) << 1) |
           ((unsigned)(key_of(v.z) >= thr) << 2) | ((unsigned)(key_of(v.w) >= thr) << 3)) << (4 * q);
  }
  const unsigned cnt = __popc(km);
  unsigned incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) wtot[wi] = incl;
  __syncthreads();
  if (km == 0) return;
  int pos = base + (int)(incl - cnt);
  for (int i = 0; i < wi; ++i) pos += (int)wtot[i];
  const int ebase = wi * 1024 + 32 * lane;
  unsigned rem = km;
  while (rem) {
    const int b = __ffs((int)rem) - 1;
    rem &= rem - 1;
    if ((unsigned)pos < (unsigned)k) {  // always true for consistent counts; keeps a write inside the segment
      const float v = my[b];
      vals[seg + pos] = v;
      idx[seg + pos] = t.elem0 + ebase + b;
      if (!LAZY) m[ebase + b] = 0.f;
      else if (zero_ties && key_of(v) == tau && __float_as_uint(v) != 0u) m[ebase + b] = 0.f;
    }
    ++pos;
  }
}

// Persistent blocks, each over a contiguous share of the select work list (the tiles of the non-staged segments
// that hold something to keep; a segment's tiles are consecutive entries, so the layer and threshold records are
// re-read only when the segment changes).  The list entry and the counters of the next tile are fetched while
// the current one is processed, and its lines are asked into L2.
template <bool LAZY>
__global__ void __launch_bounds__(256, 4)
topk_select_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_tiles, int n_mat,
                   float* __restrict__ err, const Select* __restrict__ sel, const int2* __restrict__ tile_pre,
                   const int2* __restrict__ tile_own, const unsigned* __restrict__ any_list,
                   float* __restrict__ vals, int32_t* __restrict__ idx,
                   long long stride, long long capacity, const int2* __restrict__ lists, int W) {
  __shared__ unsigned wtot[8];
  __shared__ __align__(16) float rows[8 * 32 * kRowWords];
  const unsigned long long n_work = any_list[kListCountWord + kListSelect];
  const unsigned b0 = (unsigned)(n_work * blockIdx.x / gridDim.x), b1 = (unsigned)(n_work * (blockIdx.x + 1) / gridDim.x);
  if (b0 >= b1) return;
  const int2* work = lists + (long long)kListSelect * W * n_tiles;
  int2 wk = work[b0];
  int2 pre = tile_pre[(long long)wk.x * n_tiles + wk.y], own = tile_own[(long long)wk.x * n_tiles + wk.y];
  int2 wk_next = b0 + 1 < b1 ? work[b0 + 1] : wk;
  int cur_w = -1, tile0 = 0, tile1 = 0;  // the segment whose records are held: worker, tiles [tile0, tile1)
  long long l_size = 0, l_offset = 0, l_seg_off = 0;
  unsigned tau = 0;
  int need = 0, k = 0;
  for (unsigned b = b0; b < b1; ++b) {
    __syncthreads();  // wtot of the previous tile is no longer read
    const int w = wk.x, ti = wk.y;
    const int2 p = pre, o = own;
    if (w != cur_w || ti < tile0 || ti >= tile1) {
      const DevLayer& L = layers[tiles[ti].layer];
      cur_w = w; tile0 = L.tile0; tile1 = L.tile0 + L.ntiles;
      l_size = (long long)L.rows * L.cols; l_offset = L.offset; l_seg_off = L.seg_off;
      const Select& ss = sel[w * n_mat + L.mat];
      tau = ss.tau; need = ss.need; k = ss.k;
    }
    Tile t;
    t.layer = 0;
    t.elem0 = (ti - tile0) * kTile;
    t.nelem = (int)min((long long)kTile, l_size - t.elem0);
    float* m = err + (long long)w * stride + l_offset + t.elem0;
    const long long seg = (long long)w * capacity + l_seg_off;
    // the next tile: its lines into L2 now, its counters and the list entry after it while this tile is worked on
    wk = wk_next;
    if (b + 1 < b1) {
      const Tile tn = tiles[wk.y];
      prefetch_l2(err + (long long)wk.x * stride + layers[tn.layer].offset + tn.elem0 + 32 * (int)threadIdx.x);
      pre = tile_pre[(long long)wk.x * n_tiles + wk.y];
      own = tile_own[(long long)wk.x * n_tiles + wk.y];
      if (b + 2 < b1) wk_next = work[b + 2];
    }
    const bool all_ties = p.y + o.y <= need, no_ties = o.y == 0 || p.y >= need;
    if (all_ties || no_ties) {
      const unsigned thr = all_ties ? tau : tau + 1u;
      const int base = p.x + min(p.y, need);
      const bool zt = all_ties && o.y != 0;
      const int kept = o.x + (all_ties ? o.y : 0);  // entries of the tile that will be written
      if (t.nelem != kTile) select_tile_simple<false, LAZY>(t, thr, tau, zt, base, k, m, vals, idx, seg, wtot);
      else if (kept <= kTile / 5) select_tile_rows<LAZY>(t, thr, tau, zt, base, k, m, vals, idx, seg, wtot, rows);
      else select_tile_simple<true, LAZY>(t, thr, tau, zt, base, k, m, vals, idx, seg, wtot);
    } else {
      if (t.nelem == kTile) select_tile<true, LAZY>(t, tau, need, k, p, m, vals, idx, seg, wtot);
      else select_tile<false, LAZY>(t, tau, need, k, p, m, vals, idx, seg, wtot);
    }
  }
}

// Pass E', staged segments.  One warp per (tile, worker): the tile's staged entries (every element whose key
// lies in a bucket at or above the predicted band) already hold all candidates, so the kept ones are written
// from them and M is not read.  Index order inside the tile comes from two 8192-bit maps in shared memory
// (keys above tau, keys equal to tau) with per-word prefix counts: an entry's rank is the number of set bits
// below its index.
template <bool LAZY>
__global__ void __launch_bounds__(256)
topk_finalize_staged_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_tiles,
                            int n_mat, int W, float* __restrict__ err, const Select* __restrict__ sel,
                            const int2* __restrict__ tile_pre, const unsigned* __restrict__ cand,
                            const int2* __restrict__ tile_cand, long long cand_total, float* __restrict__ vals,
                            int32_t* __restrict__ idx, long long stride, long long capacity,
                            const unsigned* __restrict__ any_list, const int2* __restrict__ lists) {
  constexpr int kWords = kTile / 32;  // 256
  __shared__ unsigned bits_a[8][kWords], bits_t[8][kWords];
  __shared__ unsigned short pref_a[8][kWords], pref_t[8][kWords];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned n_work = any_list[kListCountWord + kListStaged];
  const int2* work = lists + (long long)kListStaged * W * n_tiles;
  for (unsigned b = blockIdx.x * 8 + warp; b < n_work; b += gridDim.x * 8) {
  __syncwarp();  // the maps of the previous tile are no longer read
  const int w = work[b].x, ti = work[b].y;
  const long long v = (long long)w * n_tiles + ti;
  const Tile t = tiles[ti];
  const DevLayer L = layers[t.layer];
  const Select s = sel[w * n_mat + L.mat];
  const int2 tc = tile_cand[v];
  const int2 pre = tile_pre[v];
  const uint2* ent = reinterpret_cast<const uint2*>(cand + (long long)w * cand_total + L.cand_base) + tc.x;
  unsigned* ba = bits_a[warp];
  unsigned* bt = bits_t[warp];
  for (int i = lane; i < kWords; i += 32) { ba[i] = 0; bt[i] = 0; }
  __syncwarp();
  // entries are read four per lane at a time, so that the loads are in flight together (an absent entry reads
  // as key 0, which lies below every staged threshold)
  for (int i0 = 0; i0 < tc.y; i0 += 128) {
    uint2 eb[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + 32 * u + lane;
      eb[u] = i < tc.y ? ent[i] : make_uint2(0u, (unsigned)t.elem0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const unsigned kk = eb[u].x & 0x7fffffffu, li = eb[u].y - (unsigned)t.elem0;
      if (kk > s.tau) atomicOr(&ba[li >> 5], 1u << (li & 31u));
      else if (kk == s.tau) atomicOr(&bt[li >> 5], 1u << (li & 31u));
    }
  }
  __syncwarp();
  {  // per-word exclusive prefix counts: lane l owns words 8l .. 8l+7
    unsigned ca = 0, ct = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) { ca += __popc(ba[8 * lane + j]); ct += __popc(bt[8 * lane + j]); }
    unsigned c = ca | (ct << 16), incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    unsigned run = incl - c;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      pref_a[warp][8 * lane + j] = (unsigned short)(run & 0xffffu);
      pref_t[warp][8 * lane + j] = (unsigned short)(run >> 16);
      run += __popc(ba[8 * lane + j]) | (__popc(bt[8 * lane + j]) << 16);
    }
  }
  __syncwarp();
  const long long seg = (long long)w * capacity + L.seg_off;
  float* m = err + (long long)w * stride + L.offset;
  for (int i0 = 0; i0 < tc.y; i0 += 128) {
    uint2 eb[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + 32 * u + lane;
      eb[u] = i < tc.y ? ent[i] : make_uint2(0u, (unsigned)t.elem0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint2 e = eb[u];
      const unsigned kk = e.x & 0x7fffffffu, li = e.y - (unsigned)t.elem0;
      const bool is_a = kk > s.tau, is_t = kk == s.tau;
      if (!is_a && !is_t) continue;
      const unsigned wd = li >> 5, below = (1u << (li & 31u)) - 1u;
      const int above_before = pre.x + (int)pref_a[warp][wd] + __popc(ba[wd] & below);
      const int ties_before = pre.y + (int)pref_t[warp][wd] + __popc(bt[wd] & below);
      if (is_a || ties_before < s.need) {
        const int pos = above_before + min(ties_before, s.need);
        if ((unsigned)pos < (unsigned)s.k && li < (unsigned)t.nelem) {  // always true for consistent lists
          vals[seg + pos] = __uint_as_float(e.x);
          idx[seg + pos] = (int32_t)e.y;
          if (!LAZY || !is_a) m[e.y] = 0.f;
        }
      }
    }
  }
  }
}

// Pass F.  Scatter-decompress and average: the tile of `out` is accumulated in shared memory from every worker's
// packed entries that fall into it (their ranges come from the tile scan), workers in order (fixed fp32 order), then
// scaled by 1/W.  VECTOR tiles: out = mean_w g_w, delta += g_decider.
// The entries of all workers (as many as the staging area holds: always all of them for W <= 8 at K <= 12 %) are
// brought into shared memory by asynchronous 4-byte copies issued back to back, so that a tile pays one memory
// latency whatever the number of workers and entries; the adds then run from shared memory, one worker after the
// other (an element may be kept by several workers and the order of its sum is fixed).
// Persistent blocks take tiles by ticket (one atomic per tile, requested two tiles ahead), and the ranges of a
// block's next tile are fetched while the current one is worked on.
// SGD: the optimiser tail is applied to every element of out where it is written.
constexpr int kDecStage = kTile / 2;  // staged entries per round
constexpr int kDecWide = 256;         // tiles in which worker 0 has this many entries move them in 16-byte copies
constexpr size_t kDecSmemBytes = sizeof(float) * kTile + (sizeof(int) + sizeof(float)) * kDecStage +
                                 sizeof(int) * 2 * kMaxWorkers + 16;

__device__ __forceinline__ void cp_async4(void* dst_smem, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(__cvta_generic_to_global(src))
               : "memory");
}
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(__cvta_generic_to_global(src))
               : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

template <bool SGD>
__global__ void __launch_bounds__(256, 3)
topk_decompress_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_tiles,
                       const float* __restrict__ grads, const int2* __restrict__ tile_rng,
                       const float* __restrict__ vals, const int32_t* __restrict__ idx, float* __restrict__ out,
                       float* __restrict__ delta, long long stride, long long capacity, int W, int decider,
                       float inv_w, unsigned* __restrict__ ticket, const SgdTail tail) {
  extern __shared__ __align__(16) unsigned char dec_smem[];
  float* acc = reinterpret_cast<float*>(dec_smem);             // [kTile]
  int* s_idx = reinterpret_cast<int*>(acc + kTile);            // [kDecStage]
  float* s_val = reinterpret_cast<float*>(s_idx + kDecStage);  // [kDecStage]
  int* r_lo = reinterpret_cast<int*>(s_val + kDecStage);       // [kMaxWorkers]
  int* r_hi = r_lo + kMaxWorkers;                              // [kMaxWorkers]
  int* s_tile = r_hi + kMaxWorkers;                            // [2]
  constexpr int kRng = kMaxWorkers / 256;  // ranges a thread holds for the block's next tile
  SgdHyper h = {0.f, 0.f, 0.f};
  if (SGD) h = sgd_hyper(tail);
  if (threadIdx.x == 0) {
    s_tile[0] = (int)atomicAdd(ticket, 1u);
    s_tile[1] = (int)atomicAdd(ticket, 1u);
  }
  __syncthreads();
  int cur = s_tile[0], nxt = s_tile[1];
  int2 rn[kRng];
#pragma unroll
  for (int u = 0; u < kRng; ++u) {
    const int w = u * 256 + (int)threadIdx.x;
    rn[u] = (w < W && cur < n_tiles) ? tile_rng[(long long)w * n_tiles + cur] : make_int2(0, 0);
  }
  int l_tile0 = 0, l_tile1 = 0, l_kind = ACC_VECTOR;  // the layer whose record is held: tiles [l_tile0, l_tile1)
  long long l_size = 0, l_offset = 0, l_seg_off = 0;
  while (cur < n_tiles) {
    __syncthreads();  // acc, the ranges and s_tile of the previous tile are no longer read
    unsigned tick = 0;
    if (threadIdx.x == 0) tick = atomicAdd(ticket, 1u);  // the tile after the next one
    if (cur < l_tile0 || cur >= l_tile1) {
      const DevLayer& L = layers[tiles[cur].layer];
      l_tile0 = L.tile0; l_tile1 = L.tile0 + L.ntiles; l_kind = L.kind;
      l_size = (long long)L.rows * L.cols; l_offset = L.offset; l_seg_off = L.seg_off;
    }
    const int elem0 = (cur - l_tile0) * kTile;
    const int nelem = (int)min((long long)kTile, l_size - elem0);
    const long long base = l_offset + elem0;
#pragma unroll
    for (int u = 0; u < kRng; ++u) {
      const int w = u * 256 + (int)threadIdx.x;
      if (w < W) { r_lo[w] = rn[u].x; r_hi[w] = rn[u].y; }
      rn[u] = (w < W && nxt < n_tiles) ? tile_rng[(long long)w * n_tiles + nxt] : make_int2(0, 0);
    }
    if (l_kind != ACC_MATRIX) {
      vector_tile_mean(grads + base, stride, W, decider, inv_w, nelem, delta != nullptr ? delta + base : nullptr,
                       [&](int i, float4 v) {
                         *reinterpret_cast<float4*>(out + base + i) = v;
                         if (SGD) sgd_apply4(tail, h, base + i, v);
                       },
                       [&](int i, float v) {
                         out[base + i] = v;
                         if (SGD) sgd_apply1(tail, h, base + i, v);
                       });
    } else {
      for (int i = threadIdx.x; i < kTile / 4; i += blockDim.x)
        reinterpret_cast<float4*>(acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      __syncthreads();  // the ranges are in place (and acc is clear)
      // Long ranges (a low compression level; told by worker 0's range): a piece is placed so that its first entry
      // on a 16-byte boundary of the packed arrays also lies on one in shared memory; everything between the
      // boundaries then moves in 16-byte copies (four entries each), at most three entries at either end in 4-byte
      // copies.  Short ranges are not worth the placement arithmetic.
      if (r_hi[0] - r_lo[0] >= kDecWide) {
        const int cap3 = (int)(capacity & 3), seg3 = (int)(l_seg_off & 3);
        auto piece = [&](int w, int off, int o, int* lo, int* take, int* os, int* lead, bool* whole) {
          *lo = r_lo[w] + off;
          const int rem = r_hi[w] - *lo;
          // (the last two bits of the piece's first position, w * capacity + seg_off + lo, in 32-bit arithmetic)
          *lead = -((w & 3) * cap3 + seg3 + *lo) & 3;
          *os = o + (-(o + *lead) & 3);
          *take = rem > 0 ? max(0, min(rem, kDecStage - *os)) : 0;
          *whole = *take == rem;  // (an empty range is whole; a range that finds the area full is not)
        };
        int w0 = 0, off0 = 0;  // first worker of the round and how many of its entries earlier rounds have taken
        while (w0 < W) {
          int w = w0, off = off0, o = 0;
          while (w < W) {
            int lo, take, os, lead;
            bool whole;
            piece(w, off, o, &lo, &take, &os, &lead, &whole);
            if (take > 0) {
              const long long g0 = (long long)w * capacity + l_seg_off + lo;
              const int32_t* gi = idx + g0;
              const float* gv = vals + g0;
              const int ld = min(lead, take), nq = (take - ld) >> 2, tail0 = ld + 4 * nq;
              for (int i = threadIdx.x; i < nq; i += 256) {
                cp_async16(s_idx + os + ld + 4 * i, gi + ld + 4 * i);
                cp_async16(s_val + os + ld + 4 * i, gv + ld + 4 * i);
              }
              const int ne = ld + (take - tail0);  // the entries outside the boundaries: at most six
              if ((int)threadIdx.x < ne) {
                const int j = (int)threadIdx.x < ld ? (int)threadIdx.x : tail0 + ((int)threadIdx.x - ld);
                cp_async4(s_idx + os + j, gi + j);
                cp_async4(s_val + os + j, gv + j);
              }
              o = os + take;
            }
            if (!whole) { off += take; break; }
            ++w;
            off = 0;
          }
          cp_async_wait_all();
          __syncthreads();
          int w2 = w0, off2 = off0;
          o = 0;
          while (w2 < W) {
            int lo, take, os, lead;
            bool whole;
            piece(w2, off2, o, &lo, &take, &os, &lead, &whole);
            for (int i = threadIdx.x; i < take; i += 256) {
              const unsigned li = (unsigned)(s_idx[os + i] - elem0);
              if (li < (unsigned)kTile) acc[li] += s_val[os + i];
            }
            if (take > 0) o = os + take;
            __syncthreads();  // the next worker may add to the same elements; the last piece frees the staging area
            if (!whole) break;
            ++w2;
            off2 = 0;
          }
          w0 = w;
          off0 = off;
        }
      } else {
        // rounds: the staging area is filled with the entries of as many workers as fit, in worker order (a worker
        // with more entries in the tile than the area holds is cut into pieces that take a round each)
        int w0 = 0, off0 = 0;  // first worker of the round and how many of its entries earlier rounds have taken
        while (w0 < W) {
          int w = w0, off = off0, o = 0;
          while (w < W && o < kDecStage) {
            const int lo = r_lo[w] + off, n = min(r_hi[w] - lo, kDecStage - o);
            const long long seg = (long long)w * capacity + l_seg_off;
            for (int i = threadIdx.x; i < n; i += 256) {
              cp_async4(s_idx + o + i, idx + seg + lo + i);
              cp_async4(s_val + o + i, vals + seg + lo + i);
            }
            o += n;
            if (lo + n == r_hi[w]) { ++w; off = 0; } else { off += n; }
          }
          cp_async_wait_all();
          __syncthreads();
          int w2 = w0, off2 = off0;
          o = 0;
          while (w2 < W && o < kDecStage) {
            const int lo = r_lo[w2] + off2, n = min(r_hi[w2] - lo, kDecStage - o);
            for (int i = threadIdx.x; i < n; i += 256) {
              const unsigned li = (unsigned)(s_idx[o + i] - elem0);
              if (li < (unsigned)kTile) acc[li] += s_val[o + i];
            }
            o += n;
            if (lo + n == r_hi[w2]) { ++w2; off2 = 0; } else { off2 += n; }
            __syncthreads();  // the next worker may add to the same elements; the last piece frees the staging area
          }
          w0 = w;
          off0 = off;
        }
      }
      const int n4 = nelem >> 2;
      for (int i = threadIdx.x; i < n4; i += blockDim.x) {
        const float4 a = reinterpret_cast<const float4*>(acc)[i];
        const float4 v = make_float4(a.x * inv_w, a.y * inv_w, a.z * inv_w, a.w * inv_w);
        st_stream4(out + base + 4 * i, v);
        if (SGD) sgd_apply4(tail, h, base + 4 * i, v);
      }
      for (int i = 4 * n4 + threadIdx.x; i < nelem; i += blockDim.x) {
        out[base + i] = acc[i] * inv_w;
        if (SGD) sgd_apply1(tail, h, base + i, acc[i] * inv_w);
      }
    }
    if (threadIdx.x == 0) s_tile[0] = (int)tick;
    __syncthreads();
    cur = nxt;
    nxt = s_tile[0];
  }
}

// Real workers.  VECTOR tiles of the compress half: this GPU's mean of the workers' gradients goes to the packed
// exchange region; delta += g_decider.
__global__ void __launch_bounds__(256)
topk_vec_local_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles,
                      const int* __restrict__ vec_tiles, const float* __restrict__ grads,
                      float* __restrict__ packed, float* __restrict__ delta, long long stride, int W, int decider,
                      float inv_w) {
  const Tile t = tiles[vec_tiles[blockIdx.x]];
  const DevLayer L = layers[t.layer];
  const long long base = L.offset + t.elem0;
  float* x = packed + L.vec_off + t.elem0;
  vector_tile_mean(grads + base, stride, W, decider, inv_w, t.nelem, delta != nullptr ? delta + base : nullptr,
                   [&](int i, float4 v) { *reinterpret_cast<float4*>(x + i) = v; }, [&](int i, float v) { x[i] = v; });
}

// First position in the ascending array a[0..n) whose value is >= key.
__device__ __forceinline__ int lower_bound_i32(const int32_t* __restrict__ a, int n, int key) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (a[mid] < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// Real workers, decompress half.  One block per tile, from the gathered packed sets of all n_sets workers
// (set j = worker j of the whole job: GPU-major, then the GPU's workers): each set's entries are in ascending
// index order, so the tile's entries are a contiguous range found by binary search.  Sets are added in order
// (bit-reproducible, and the same order as the single-GPU step), then scaled by 1/n_sets.
// VECTOR tiles: out = vec_scale * (summed packed means).
template <bool SGD>
__global__ void __launch_bounds__(256)
topk_decompress_packed_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_layers,
                              const float* __restrict__ vals, const int32_t* __restrict__ idx,
                              const int32_t* __restrict__ counts, int n_sets, long long capacity,
                              const float* __restrict__ packed, float vec_scale, float* __restrict__ out,
                              const SgdTail tail) {
  __shared__ float acc[kTile];
  __shared__ int range[256];
  const Tile t = tiles[blockIdx.x];
  const DevLayer L = layers[t.layer];
  const long long base = L.offset + t.elem0;
  SgdHyper h = {0.f, 0.f, 0.f};
  if (SGD) h = sgd_hyper(tail);
  if (L.kind != ACC_MATRIX) {
    for (int i = threadIdx.x; i < t.nelem; i += blockDim.x) {
      const float v = vec_scale * packed[L.vec_off + t.elem0 + i];
      out[base + i] = v;
      if (SGD) sgd_apply1(tail, h, base + i, v);
    }
    return;
  }
  for (int i = threadIdx.x; i < kTile; i += blockDim.x) acc[i] = 0.f;
  // the tile's range in every set: 128 sets at a time, one thread per bound, all searches in flight together
  for (int j0 = 0; j0 < n_sets; j0 += 128) {
    const int nj = min(128, n_sets - j0);
    __syncthreads();  // acc cleared / previous chunk consumed
    if ((int)threadIdx.x < 2 * nj) {
      const int j = j0 + ((int)threadIdx.x >> 1);
      const long long seg = (long long)j * capacity + L.seg_off;
      const int n = counts[(long long)j * n_layers + t.layer];
      range[threadIdx.x] = lower_bound_i32(idx + seg, n, (threadIdx.x & 1) ? t.elem0 + t.nelem : t.elem0);
    }
    __syncthreads();
    for (int jj = 0; jj < nj; ++jj) {  // sets in order: the sum of an element's contributions has a fixed order
      const long long seg = (long long)(j0 + jj) * capacity + L.seg_off;
      const int lo = range[2 * jj], hi = range[2 * jj + 1];
      for (int i = lo + (int)threadIdx.x; i < hi; i += blockDim.x) {
        const unsigned li = (unsigned)(idx[seg + i] - t.elem0);
        if (li < (unsigned)kTile) acc[li] += vals[seg + i];
      }
      if (lo < hi) __syncthreads();  // lo, hi are uniform over the block
    }
  }
  __syncthreads();
  const float inv = 1.0f / (float)n_sets;
  const int n4 = t.nelem >> 2;
  for (int i = threadIdx.x; i < n4; i += blockDim.x) {
    const float4 v = make_float4(acc[4 * i] * inv, acc[4 * i + 1] * inv, acc[4 * i + 2] * inv, acc[4 * i + 3] * inv);
    st_stream4(out + base + 4 * i, v);
    if (SGD) sgd_apply4(tail, h, base + 4 * i, v);
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x) {
    out[base + i] = acc[i] * inv;
    if (SGD) sgd_apply1(tail, h, base + i, acc[i] * inv);
  }
}

// Everything of the TopK step up to the packed sets (threshold, selection, error memory).
static cudaError_t launch_topk_select_part(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level,
                                           float* vals, int32_t* idx, int32_t* counts, float* delta, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const int nt = (int)pl.tiles.size(), W = c.n_workers, n_mat = pl.n_mat;
  const bool lazy = (c.flags & ACC_FLAG_LAZY_RESIDUAL) != 0;
  cudaError_t e = cudaMemsetAsync(ctx->ws + pl.o_hist, 0, pl.hist_bytes, s);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(counts, 0, sizeof(int32_t) * (size_t)W * c.n_layers, s);
  if (e != cudaSuccess) return e;
  if (n_mat > 0) {
    // blocks per segment of the list histograms: the longest possible list in 16 K-word pieces, 8..128
    int max_cap = 0;
    for (int l : pl.mat_layers) max_cap = std::max(max_cap, pl.layers[l].cand_cap);
    const int list_chunks = std::min(128, std::max(8, max_cap / 16384));
    const long long V = (long long)W * nt;
    // grids of the passes that usually find an empty work list: the blocks resident at once and no more (an idle
    // block costs about 5 ns: 1776 of them were 10 us of an otherwise empty launch)
    const int grid = (int)(V < (long long)ctx->sm_count * 4 ? V : (long long)ctx->sm_count * 4);
    // first pass: a whole number of waves of resident blocks (a grid that is not a multiple of what fits leaves the
    // last wave of the static split short: 8 blocks per SM with 3 resident cost 4 %), two to six of them (finer
    // shares even out the deciding worker's tiles, which also carry the detector's accumulator)
    const long long per_wave = (long long)ctx->sm_count * ctx->occ_topk_first_pass;
    const long long waves = std::min<long long>(6, std::max<long long>(2, V / (per_wave * 4)));
    const int grid_a = (int)std::min(V, per_wave * waves);
    {
      PhaseTimer pt(ctx, PH_TOPK_EF_HIST1, s);
      topk_ef_hist1_kernel<<<grid_a, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, nt, n_mat, grads, err, delta,
                                                c.worker_stride, W, c.decider, level, ctx->d_pred, ctx->d_hist1,
                                                ctx->d_seg_cand, ctx->d_seg_flag, ctx->d_cand, ctx->d_tile_cand,
                                                pl.cand_total, ctx->d_tile_cnt, lazy ? ctx->d_pend_tau : nullptr);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_PICK1, s);
      topk_pick1_kernel<<<W * n_mat, 256, 0, s>>>(ctx->d_layers, ctx->d_mat_layers, n_mat, c.n_layers, W, level,
                                                  ctx->d_hist1, ctx->d_sel, counts, ctx->d_pred, ctx->d_seg_cand,
                                                  ctx->d_seg_flag, ctx->d_any_list, ctx->d_lists, nt, ctx->d_tile_cnt,
                                                  lazy ? ctx->d_pend_tau : nullptr);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_COLLECT, s);
      const long long cap = (long long)ctx->sm_count * 3;
      topk_collect_kernel<<<(unsigned)(V < cap ? V : cap), 256, 0, s>>>(
          ctx->d_layers, ctx->d_tiles, nt, n_mat, W, err, c.worker_stride, ctx->d_sel, ctx->d_any_list,
          ctx->d_seg_cand, ctx->d_cand, ctx->d_tile_cand, pl.cand_total, ctx->d_tile_cnt, ctx->d_lists);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_HIST2, s);
      topk_hist2_kernel<<<grid, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, nt, n_mat, err, c.worker_stride, W,
                                             ctx->d_sel, ctx->d_any_list, ctx->d_hist2, ctx->d_tile_cnt,
                                             ctx->d_lists);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_HIST2_LIST, s);
      topk_hist_list_kernel<2><<<dim3(list_chunks, W * n_mat), 256, 0, s>>>(ctx->d_layers, ctx->d_mat_layers, n_mat, ctx->d_sel,
                                                                   ctx->d_seg_cand, ctx->d_cand, pl.cand_total,
                                                                   ctx->d_hist2);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_PICK2, s);
      topk_pick2_kernel<<<W * n_mat, 256, 0, s>>>(n_mat, ctx->d_hist2, ctx->d_sel);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_HIST3, s);
      topk_hist3_kernel<<<grid, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, nt, n_mat, err, c.worker_stride,
                                             ctx->d_sel, ctx->d_any_list, ctx->d_hist3, ctx->d_tile_cnt,
                                             ctx->d_tile_h3, ctx->d_lists, W);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_HIST3_LIST, s);
      topk_hist_list_kernel<3><<<dim3(list_chunks, W * n_mat), 256, 0, s>>>(ctx->d_layers, ctx->d_mat_layers, n_mat, ctx->d_sel,
                                                                   ctx->d_seg_cand, ctx->d_cand, pl.cand_total,
                                                                   ctx->d_hist3);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_PICK3, s);
      topk_pick3_kernel<<<(W * n_mat + 7) / 8, 256, 0, s>>>(W * n_mat, ctx->d_hist3, ctx->d_sel,
                                                            lazy ? ctx->d_pend_tau : nullptr);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_TILE_COUNTS, s);
      topk_tile_counts_kernel<<<(unsigned)(((long long)W * nt + 7) / 8), 256, 0, s>>>(
          ctx->d_layers, ctx->d_tiles, nt, n_mat, W, ctx->d_sel, ctx->d_tile_cnt, ctx->d_tile_h3, ctx->d_cand,
          ctx->d_tile_cand, pl.cand_total, ctx->d_tile_pre);
    }
    {
      PhaseTimer pt(ctx, PH_TOPK_PICK3_SCAN, s);
      topk_tile_scan_kernel<<<W * n_mat, 256, 0, s>>>(ctx->d_layers, ctx->d_mat_layers, n_mat, nt, W, ctx->d_sel,
                                                      ctx->d_tile_pre, ctx->d_tile_cnt, ctx->d_tile_rng,
                                                      ctx->d_any_list, ctx->d_lists);
    }
  }
  if (n_mat > 0) {
    {
      PhaseTimer pt(ctx, PH_TOPK_FINALIZE_STAGED, s);
      const long long warps = (long long)W * nt, cap = (long long)ctx->sm_count * 32;
      const unsigned fgrid = (unsigned)std::min((warps + 7) / 8, cap);
      if (lazy)
        topk_finalize_staged_kernel<true><<<fgrid, 256, 0, s>>>(
            ctx->d_layers, ctx->d_tiles, nt, n_mat, W, err, ctx->d_sel, ctx->d_tile_pre, ctx->d_cand,
            ctx->d_tile_cand, pl.cand_total, vals, idx, c.worker_stride, pl.capacity, ctx->d_any_list, ctx->d_lists);
      else
        topk_finalize_staged_kernel<false><<<fgrid, 256, 0, s>>>(
            ctx->d_layers, ctx->d_tiles, nt, n_mat, W, err, ctx->d_sel, ctx->d_tile_pre, ctx->d_cand,
            ctx->d_tile_cand, pl.cand_total, vals, idx, c.worker_stride, pl.capacity, ctx->d_any_list, ctx->d_lists);
    }
    PhaseTimer pt(ctx, PH_TOPK_SELECT, s);
    // contiguous shares of the select work list.  Large sets: shares of about four tiles, fine enough that a run of
    // expensive tiles (the fully kept head of a zero-filled layer) spreads over many blocks (config 5 at K = 10 %:
    // 0.68 ms with 592 blocks, 0.51 ms with 1776, 0.46 ms with 4736).  Small sets: the blocks resident at once,
    // so that a launch which finds an empty list stays cheap (an idle block costs about 5 ns).
    const long long blocks = (long long)W * nt;
    const long long sm = ctx->sm_count;
    const long long want = blocks >= sm * 128 ? std::min(blocks / 4, sm * 64) : sm * 4;
    const unsigned sgrid = (unsigned)std::min(blocks, want);
    if (lazy)
      topk_select_kernel<true><<<sgrid, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, nt, n_mat, err, ctx->d_sel,
                                                     ctx->d_tile_pre, ctx->d_tile_cnt, ctx->d_any_list, vals, idx,
                                                     c.worker_stride, pl.capacity, ctx->d_lists, W);
    else
      topk_select_kernel<false><<<sgrid, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, nt, n_mat, err, ctx->d_sel,
                                                      ctx->d_tile_pre, ctx->d_tile_cnt, ctx->d_any_list, vals, idx,
                                                      c.worker_stride, pl.capacity, ctx->d_lists, W);
  }
  return cudaGetLastError();
}

cudaError_t launch_topk(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals,
                        int32_t* idx, int32_t* counts, float* out, float* delta, SgdTail tail, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const int nt = (int)pl.tiles.size(), W = c.n_workers;
  const float inv_w = 1.0f / (float)W;
  const cudaError_t e = launch_topk_select_part(ctx, grads, err, level, vals, idx, counts, delta, s);
  if (e != cudaSuccess) return e;
  {
    PhaseTimer pt(ctx, PH_TOPK_DECOMPRESS, s);
    // persistent blocks (two fit an SM), tiles handed out by ticket; the ticket word was cleared with the
    // histograms at the start of the step
    const int dgrid = std::min(nt, ctx->sm_count * 3);
    unsigned* ticket = ctx->d_any_list + kTicketWord;
    if (tail.params)
      topk_decompress_kernel<true><<<dgrid, 256, kDecSmemBytes, s>>>(ctx->d_layers, ctx->d_tiles, nt, grads, ctx->d_tile_rng, vals,
                                                         idx, out, delta, c.worker_stride, pl.capacity, W, c.decider,
                                                         inv_w, ticket, tail);
    else
      topk_decompress_kernel<false><<<dgrid, 256, kDecSmemBytes, s>>>(ctx->d_layers, ctx->d_tiles, nt, grads, ctx->d_tile_rng, vals,
                                                          idx, out, delta, c.worker_stride, pl.capacity, W, c.decider,
                                                          inv_w, ticket, tail);
  }
  return cudaGetLastError();
}

// Lazy mode: err_w <- err_w with the entries the last step kept (key above the segment's pending threshold) set to
// +0.0; afterwards nothing is pending.  One block per (tile, worker).
__global__ void __launch_bounds__(256)
topk_flush_kernel(const DevLayer* __restrict__ layers, const Tile* __restrict__ tiles, int n_mat,
                  float* __restrict__ err, long long stride, const unsigned* __restrict__ pend_tau) {
  const Tile t = tiles[blockIdx.x];
  const int w = blockIdx.y;
  const DevLayer L = layers[t.layer];
  if (L.kind != ACC_MATRIX) return;
  const unsigned ptau = pend_tau[w * n_mat + L.mat];
  if (ptau == kNoPendingTau) return;
  float* e = err + (long long)w * stride + L.offset + t.elem0;
  const int n4 = t.nelem >> 2;
  for (int i = threadIdx.x; i < n4; i += blockDim.x) {
    float4 v = ld_stream4(e + 4 * i);
    const bool any = key_of(v.x) > ptau || key_of(v.y) > ptau || key_of(v.z) > ptau || key_of(v.w) > ptau;
    if (any) {
      v.x = key_of(v.x) > ptau ? 0.f : v.x;
      v.y = key_of(v.y) > ptau ? 0.f : v.y;
      v.z = key_of(v.z) > ptau ? 0.f : v.z;
      v.w = key_of(v.w) > ptau ? 0.f : v.w;
      *reinterpret_cast<float4*>(e + 4 * i) = v;
    }
  }
  for (int i = 4 * n4 + threadIdx.x; i < t.nelem; i += blockDim.x)
    if (key_of(e[i]) > ptau) e[i] = 0.f;
}

__global__ void topk_clear_pending_kernel(unsigned* __restrict__ pend_tau, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) pend_tau[i] = kNoPendingTau;
}

// Once per context, at creation: how many blocks of the first pass fit an SM.
cudaError_t prepare_topk(acc_ctx* ctx) {
  int occ = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, topk_ef_hist1_kernel, 256, 0);
  ctx->occ_topk_first_pass = occ > 0 ? occ : 1;
  // the decompress pass stages its entries in more than 48 KB of dynamic shared memory
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(topk_decompress_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kDecSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(topk_decompress_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kDecSmemBytes);
  return e;
}

cudaError_t launch_topk_flush(acc_ctx* ctx, float* err, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  if (pl.n_mat > 0) {
    {
      PhaseTimer pt(ctx, PH_TOPK_FLUSH, s);
      topk_flush_kernel<<<dim3((unsigned)pl.tiles.size(), (unsigned)c.n_workers), 256, 0, s>>>(
          ctx->d_layers, ctx->d_tiles, pl.n_mat, err, c.worker_stride, ctx->d_pend_tau);
    }
    const int n = c.n_workers * pl.n_mat;
    ctx->last_launches += 1;
    topk_clear_pending_kernel<<<(n + 127) / 128, 128, 0, s>>>(ctx->d_pend_tau, n);
  }
  return cudaGetLastError();
}

cudaError_t launch_topk_compress(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals,
                                 int32_t* idx, int32_t* counts, float* delta, float* vec_packed, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const acc_config& c = ctx->cfg;
  const cudaError_t e = launch_topk_select_part(ctx, grads, err, level, vals, idx, counts, delta, s);
  if (e != cudaSuccess) return e;
  if (!pl.vec_tiles.empty()) {
    PhaseTimer pt(ctx, PH_VEC_EXCHANGE, s);
    topk_vec_local_kernel<<<(unsigned)pl.vec_tiles.size(), 256, 0, s>>>(
        ctx->d_layers, ctx->d_tiles, ctx->d_vec_tiles, grads, vec_packed, delta, c.worker_stride, c.n_workers,
        c.decider, 1.0f / (float)c.n_workers);
  }
  return cudaGetLastError();
}

cudaError_t launch_topk_decompress_packed(acc_ctx* ctx, const float* vals, const int32_t* idx, const int32_t* counts,
                                          int n_sets, const float* vec_packed, float vec_scale, float* out,
                                          SgdTail tail, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  const unsigned nt = (unsigned)pl.tiles.size();
  PhaseTimer pt(ctx, PH_TOPK_DECOMPRESS_PACKED, s);
  if (tail.params)
    topk_decompress_packed_kernel<true><<<nt, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, ctx->cfg.n_layers, vals, idx,
                                                           counts, n_sets, pl.capacity, vec_packed, vec_scale, out,
                                                           tail);
  else
    topk_decompress_packed_kernel<false><<<nt, 256, 0, s>>>(ctx->d_layers, ctx->d_tiles, ctx->cfg.n_layers, vals, idx,
                                                            counts, n_sets, pl.capacity, vec_packed, vec_scale, out,
                                                            tail);
  return cudaGetLastError();
}

}  // namespace acc
