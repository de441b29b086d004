/*
 * acc.h -- C ABI of the Accordion gradient-compression step for NVIDIA B200 (sm_100a).
 *
 * The library runs, for W simulated data-parallel workers whose gradients sit in one GPU's
 * memory, the per-iteration step that Accordion (arXiv 2010.16248) drives:
 *
 *   - error-feedback accumulation          M_w = g_w + e_w           (the "memory term", Section "Accordion with PowerSGD")
 *   - gradient accumulation + layer norms  for the critical-regime test (Section 4.2)
 *   - the regime test itself               Algorithm 1
 *   - the compressor at the chosen level   PowerSGD rank r, or TopK K%   (Section "Experimental evaluation", first paragraph)
 *   - the mean over workers of the compressed gradients   (update rule of Section 3)
 *
 * General rules, valid for every entry point unless it says otherwise:
 *   * Pointers named in "Device pointers" below are DEVICE pointers owned by the caller; the library
 *     never allocates or frees device memory.  `cfg`, `layers`, and every `int64_t*` / `size_t*`
 *     out-parameter are HOST pointers.
 *   * Every device buffer of floats or indices must be 16-byte aligned (ACC_EALIGN otherwise); arrays of doubles
 *     need 8 bytes, level arrays (bytes) no alignment at all.
 *   * Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream),
 *     never synchronise the device, and return an int status: ACC_OK or one of the ACC_E* codes.
 *     Calls on one context must be ordered on one stream (or otherwise serialised by the caller):
 *     they share the context's scratch memory.  One exception: the PowerSGD calls and the TopK calls use
 *     disjoint parts of it, so a PowerSGD step and a TopK step of the same iteration (different error
 *     memories and outputs, the same gradients and levels) may run concurrently on two streams.
 *   * Layout.  All per-parameter buffers use one flat per-worker layout given by the layer table:
 *     layer l occupies elements [offset_l, offset_l + rows_l*cols_l) of each worker's slice, each
 *     offset a multiple of 4 elements; worker w's slice starts at element w*worker_stride
 *     (worker_stride a multiple of 4).  MATRIX layers are row-major rows x cols (convolution weights
 *     viewed as out x (in*k*k), the view that reproduces the "Data Sent" columns of Tables 1-2);
 *     VECTOR layers (1-D tensors) are never compressed and carry no error memory (Appendix F).
 *   * level[l] = 1 selects the low-compression level l_low (rank_low / topk_low_bp),
 *     level[l] = 0 the high-compression level l_high (rank_high / topk_high_bp)  (Section 4.2).
 */
#ifndef ACC_H_
#define ACC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ACC_OK 0
#define ACC_EINVAL 1      /* bad argument / inconsistent configuration            */
#define ACC_EALIGN 2      /* a pointer, offset or stride is not 16-byte aligned    */
#define ACC_EWORKSPACE 3  /* workspace missing or too small                        */
#define ACC_ECUDA 4       /* a CUDA runtime call or kernel launch reported an error */
#define ACC_ETOOBIG 5     /* size beyond the fixed capacity of acc_sumsq_static    */
#define ACC_ETIMEOUT 6    /* device side: a bounded wait on an asynchronous copy gave up (acc_device_status) */

#define ACC_MATRIX 0
#define ACC_VECTOR 1
#define ACC_MAX_RANK 4    /* ranks are interleaved in groups of ACC_MAX_RANK floats  */

/* acc_config.flags */
#define ACC_FLAG_LAZY_RESIDUAL 1 /* err keeps M_w after a step; the compressed part is removed on the next load
                                   (see acc_powersgd_step and acc_topk_step) */
/* The first PowerSGD pass exists as a direct kernel and as a persistent kernel fed by bulk asynchronous
 * copies; both compute the same values up to the rounding order of a few additions (the last bits of P).
 * By default the library picks by problem size (the pipelined one needs a long queue of tiles per SM to
 * pay off).  These two flags force the choice (tests, tuning). */
#define ACC_FLAG_PIPELINE_ALWAYS 2
#define ACC_FLAG_PIPELINE_NEVER 4
/* The caller issues this context's PowerSGD step and TopK step at the same time on two streams.  The pipelined
 * first PowerSGD pass then starts half as many persistent blocks as the GPU has SMs (a block fills an SM, so
 * nothing else runs beside it): the TopK step's kernels get the other SMs instead of waiting for the pass to end.
 * Same results bit for bit; a PowerSGD step that runs alone is slower with it.  No effect on the direct kernel. */
#define ACC_FLAG_SHARE_SMS 8

#define ACC_COMPRESSOR_POWERSGD 0
#define ACC_COMPRESSOR_TOPK 1

typedef struct {
  int64_t offset; /* first element of the layer inside a worker's slice; multiple of 4 */
  int32_t rows;   /* MATRIX: rows; VECTOR: 1                                           */
  int32_t cols;   /* MATRIX: cols; VECTOR: length                                      */
  int32_t kind;   /* ACC_MATRIX or ACC_VECTOR                                          */
  int32_t reserved;
} acc_layer_desc;

typedef struct {
  int32_t n_workers;            /* W >= 1                                                        */
  int32_t n_layers;             /* L >= 1                                                        */
  const acc_layer_desc* layers; /* HOST array [L], copied by acc_create                          */
  int64_t worker_stride;        /* elements between consecutive workers' slices                  */
  int32_t rank_low, rank_high;  /* PowerSGD ranks, 1 <= rank_high <= rank_low <= ACC_MAX_RANK    */
  int32_t topk_low_bp;          /* TopK fraction at l_low in basis points (1000 = 10 %)          */
  int32_t topk_high_bp;         /* TopK fraction at l_high; 1 <= high <= low <= 10000            */
  float eta;                    /* detection threshold of Algorithm 1 (the paper uses 0.5)       */
  float gs_eps;                 /* Gram-Schmidt divides by (norm + gs_eps)                       */
  int32_t decider;              /* worker whose raw gradient is accumulated for the detector     */
  int32_t flags;                /* 0 or an OR of ACC_FLAG_* values                               */
} acc_config;

typedef struct acc_ctx acc_ctx;

/* Bytes of device scratch memory acc_create needs for this configuration (HOST out-parameter). */
int acc_workspace_bytes(const acc_config* cfg, size_t* bytes);

/* Validates cfg, copies the layer table and the launch tables into `workspace` (DEVICE memory of at
 * least acc_workspace_bytes bytes, 256-byte aligned, owned by the caller and kept alive until
 * acc_destroy) and returns a context.  Synchronous (blocking copies on the current device).        */
int acc_create(const acc_config* cfg, void* workspace, size_t workspace_bytes, acc_ctx** out);
int acc_destroy(acc_ctx* ctx);

/* Factor layout of PowerSGD.  q holds, for every MATRIX layer, cols_l rows of ACC_MAX_RANK floats
 * (row j = Q[j, 0..3], rank-interleaved); p_hat holds rows_l rows of ACC_MAX_RANK floats.  The block
 * of layer l starts at row q_row[l] / p_row[l] (-1 for VECTOR layers).  Any out-pointer may be NULL.
 * q_rows / p_rows: total rows, i.e. the buffers hold 4*q_rows and 4*p_rows floats.                 */
int acc_factor_layout(const acc_ctx* ctx, int64_t* q_row /*[L]*/, int64_t* p_row /*[L]*/,
                      int64_t* q_rows, int64_t* p_rows);

/* Packed TopK layout.  A worker's packed region has `capacity` entries; the segment of MATRIX layer l
 * starts at seg_offset[l] (-1 for VECTOR layers) and has room for k_low[l] entries.  Worker w's
 * region starts at entry w*capacity of `vals` and `idx`.                                          */
int acc_topk_layout(const acc_ctx* ctx, int64_t* seg_offset /*[L]*/, int64_t* k_low /*[L]*/,
                    int64_t* k_high /*[L]*/, int64_t* capacity);

/* Error-feedback accumulation on its own (Section "Accordion with PowerSGD": the compressors run "with memory"):
 *   err_w <- g_w + err_w  on MATRIX layers, in fp32 (one IEEE add), for every worker;
 *   delta <- delta + g_decider on every layer when delta != NULL (gradient accumulation of the
 *   detector, Section 4.2 "Computational and memory overhead").
 * Device pointers: grads [W][worker_stride] (read), err [W][worker_stride] (in: e, out: M),
 * delta [worker_stride] or NULL.                                                                   */
int acc_error_feedback(acc_ctx* ctx, const float* grads, float* err, float* delta, void* stream);

/* Per-layer squared L2 norms (Section 4.2: "After each epoch, norms are calculated"):
 *   norm2[b*L + l] = sum of squares of layer l in buffer b, b < n_bufs <= W, accumulated in fp64 in a
 *   fixed order (bit-reproducible).  Device pointers: buf [n_bufs][buf_stride] (read),
 *   norm2 [n_bufs*L] doubles (written).                                                            */
int acc_layer_norms(acc_ctx* ctx, const float* buf, int64_t buf_stride, int32_t n_bufs, double* norm2,
                    void* stream);

/* Second detector statistic: the mean-to-standard-deviation ratio (MSDR) per layer, the quantity the adaptive scheme
 * of the Section "Comparison with Prior Work" switches on (that scheme lowers the compression when the ratio of its
 * gradients has dropped; the paper names the statistic and no formula).  Taken over the coordinates of a layer:
 *   S1 = sum_i x_i, S2 = sum_i x_i^2 (fp64, fixed order);  mean = S1/n;  var = max(S2/n - mean^2, 0);
 *   msdr = |mean| / sqrt(var), 0 when mean = 0, +inf when var = 0 and mean != 0.
 *   moments[2*(b*L + l)] = S1, moments[2*(b*L + l) + 1] = S2 (= the squared norm acc_layer_norms returns, so one pass
 *   over the detector's accumulated gradient serves Algorithm 1 and this statistic);  msdr[b*L + l].
 * Only the statistic is built; the switching rule of that scheme is not.
 * Device pointers: buf [n_bufs][buf_stride] (read), moments [2*n_bufs*L] doubles, msdr [n_bufs*L] doubles (written);
 * n_bufs <= W.                                                                                       */
int acc_layer_msdr(acc_ctx* ctx, const float* buf, int64_t buf_stride, int32_t n_bufs, double* moments, double* msdr,
                   void* stream);

/* Critical-regime test, Algorithm 1, per layer, on the device:
 *   a = sqrt(norm2_prev[l]), b = sqrt(norm2_curr[l]);
 *   level[l] = 1 (l_low)  if norm2_prev[l] < 0 (no earlier window), or |a - b| >= eta*a, or
 *              lr_next < lr_curr;  else 0 (l_high).
 *   Then norm2_prev[l] <- norm2_curr[l] and, when delta != NULL, delta <- 0 (new window).
 * Device pointers: norm2_curr [L] doubles (read), norm2_prev [L] doubles (in/out), level [L] bytes
 * (written), delta [worker_stride] or NULL (cleared).                                              */
int acc_detect_regime(acc_ctx* ctx, const double* norm2_curr, double* norm2_prev, float lr_curr,
                      float lr_next, uint8_t* level, float* delta, void* stream);

/* acc_detect_regime with the two learning rates read from DEVICE memory (lr_pair[0] = current, lr_pair[1] = next) at
 * the time the kernel runs, instead of from the arguments: a CUDA graph that captured the call then follows a
 * learning-rate schedule -- the second condition of Algorithm 1 -- when the caller rewrites the two floats between
 * replays.  Otherwise identical.  Device pointers: lr_pair 2 floats (read); the others as above.        */
int acc_detect_regime_lr(acc_ctx* ctx, const double* norm2_curr, double* norm2_prev, const float* lr_pair,
                         uint8_t* level, float* delta, void* stream);

/* Variant of the regime test with the norm of the DIFFERENCE of the two accumulated gradients,
 *   || D_prev - D_curr || >= eta * || D_prev ||,
 * in place of the difference of their norms that the display equation of Section 4.2 and Algorithm 1 print.
 * It needs the previous accumulated gradient itself (a second model-sized buffer), which Section 4.2 says the
 * method does not keep; it is offered because the criterion is sometimes quoted in this form.
 *   acc_layer_diff_norms:   norm2[l] = sum over layer l of (a - b)^2, fp64, fixed order (a, b: [worker_stride]).
 *   acc_detect_regime_diff: level as in acc_detect_regime with sqrt(norm2_diff[l]) as the change; then
 *                           norm2_prev <- norm2_curr, delta_prev <- delta, delta <- 0.
 * Device pointers: a, b, delta, delta_prev [worker_stride] floats; norm2, norm2_diff, norm2_curr, norm2_prev
 * [L] doubles; level [L] bytes.                                                                      */
int acc_layer_diff_norms(acc_ctx* ctx, const float* a, const float* b, double* norm2, void* stream);
int acc_detect_regime_diff(acc_ctx* ctx, const double* norm2_diff, const double* norm2_curr, double* norm2_prev,
                           float lr_curr, float lr_next, uint8_t* level, float* delta, float* delta_prev,
                           void* stream);

/* One PowerSGD step with error feedback (the compressor of the Section "Accordion with PowerSGD", applied per MATRIX layer at
 * rank r = rank_low if level[l] else rank_high), all workers, mean over workers (Section 3):
 *   M_w = g_w + e_w;  P = mean_w M_w Q[:, :r];  P^ = modified Gram-Schmidt(P) (divide by norm + gs_eps);
 *   Q[:, :r] <- mean_w M_w^T P^;  A = P^ Q[:, :r]^T;  out[l] = A;  e_w <- M_w - A.
 *   VECTOR layers: out[l] = mean_w g_w[l].  delta != NULL: delta += g_decider (all layers).
 * Columns r..3 of q and p_hat keep their previous contents.
 * Device pointers: grads [W][worker_stride] (read), err [W][worker_stride] (in/out),
 * q [4*q_rows] (in: warm start, out: new Q), p_hat [4*p_rows] (out: P^), level [L] bytes (read),
 * out [worker_stride] (written), delta [worker_stride] or NULL.
 *
 * With ACC_FLAG_LAZY_RESIDUAL the subtraction e_w <- M_w - A is deferred: after the call err holds M_w,
 * and the next acc_powersgd_step subtracts the A of this step (recomputed from p_hat and q, in the same
 * fp32 operation order) while it loads err, so every later result is bit-identical to the eager mode's
 * and one full read + write of err per step is saved.  Between steps the caller must leave err, q and
 * p_hat untouched; acc_powersgd_flush materialises the error memory.                                 */
int acc_powersgd_step(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                      const uint8_t* level, float* out, float* delta, void* stream);

/* Lazy mode only (ACC_EINVAL otherwise): err_w <- err_w - P^ Q^T for the residual still pending from the
 * last acc_powersgd_step, for every MATRIX layer and worker; afterwards err is the error memory e_w of
 * the eager mode and nothing is pending.  A no-op per layer when nothing is pending.
 * Device pointers: err [W][worker_stride] (in/out), q, p_hat (read).                                */
int acc_powersgd_flush(acc_ctx* ctx, float* err, const float* q, const float* p_hat, void* stream);

/* One TopK step with error feedback (the sparsifier of the Section "Accordion with TopK", per MATRIX layer and worker,
 * k = max(1, floor(rows*cols*K_bp/10000)), K_bp = topk_low_bp if level[l] else topk_high_bp):
 *   M_w = g_w + e_w (fp32);  keep the k entries of largest |M_w| -- compared as 31-bit patterns,
 *   ties broken by lower index --;  vals/idx <- kept values (bit copies) and layer-local indices in
 *   ascending index order;  counts[w*L + l] = k;  e_w <- M_w with the kept entries set to +0.0;
 *   out[l] = (1/W) sum_w scatter(idx_w, val_w)  (workers added in order, bit-reproducible).
 *   VECTOR layers: out[l] = mean_w g_w[l], counts = 0.  delta != NULL: delta += g_decider.
 * Device pointers: grads, err, level, out, delta as above; vals [W*capacity] floats,
 * idx [W*capacity] int32, counts [W*L] int32 (see acc_topk_layout).
 *
 * With ACC_FLAG_LAZY_RESIDUAL the kept entries above the threshold are not zeroed in err by the call: err keeps
 * M_w there, the context remembers the threshold per (worker, layer), and the next acc_topk_step (or
 * acc_topk_compress) reads every entry of err whose key lies above that threshold as +0.0 while it loads
 * err -- the same value the eager mode would have stored -- so every later result is bit-identical and the
 * scattered 4-byte stores into err (a DRAM sector read-modify-write each) are saved.  Kept entries equal to
 * the threshold are zeroed at once in both modes.  Between steps the caller must leave err untouched;
 * acc_topk_flush materialises the error memory (ACC_EINVAL without the flag).                         */
int acc_topk_step(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals,
                  int32_t* idx, int32_t* counts, float* out, float* delta, void* stream);
int acc_topk_flush(acc_ctx* ctx, float* err, void* stream);

/* ---- Optimiser tail (Appendix A, hyper-parameter table: Nesterov momentum 0.9; the paper gives the name
 * and the momentum only, the update below is the usual statement of it, without dampening) -------------
 *   d' = d + weight_decay * x;   u <- momentum * u + d';   x <- x - lr * (d' + momentum * u)
 * on every element of every layer (padding between layers is left alone), in fp32 with one fixed
 * operation order.  hyper is a DEVICE array of three floats {lr, momentum, weight_decay}: the kernels read
 * it, so a captured graph follows a learning-rate schedule by rewriting those floats.  (The paper lists no
 * weight decay; 0 reproduces its setting.)
 *
 * acc_sgd_nesterov applies the tail on its own from a gradient d [worker_stride].
 * acc_powersgd_step_sgd / acc_topk_step_sgd are acc_powersgd_step / acc_topk_step with the tail applied by the
 * kernels that produce `out`, at each element as it is written, which saves a later pass over `out`;
 * every other result (out, err, q, p_hat, vals, idx, counts, delta) is bit-identical to the plain step's,
 * and params / mom are bit-identical to running acc_sgd_nesterov(out) after the plain step.
 * Device pointers: params, mom [worker_stride] floats (in/out), 16-byte aligned; hyper 3 floats.       */
int acc_sgd_nesterov(acc_ctx* ctx, const float* d, float* params, float* mom, const float* hyper, void* stream);
int acc_powersgd_step_sgd(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                          const uint8_t* level, float* out, float* delta, float* params, float* mom,
                          const float* hyper, void* stream);
int acc_topk_step_sgd(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals,
                      int32_t* idx, int32_t* counts, float* out, float* delta, float* params, float* mom,
                      const float* hyper, void* stream);

/* ---- Batch-size mode (Section 4.2: "For batch size we use the same algorithm", switching between B_low and
 * B_high at the granularity of the whole model; Section 5.1: the learning rate scales in the same ratio;
 * Appendix A: large batches are simulated by accumulating several backward passes before the exchange, and
 * the batch size is only ever increased) ---------------------------------------------------------------
 * acc_batch_accumulate: acc_w <- (first ? 0 : acc_w) + g_w for every worker and layer (fp32);
 *   delta += g_decider when delta != NULL.  grads, acc [W][worker_stride]; delta [worker_stride] or NULL.
 * acc_batch_average: the uncompressed exchange, out = (1 / (W * n_accum)) * sum_w acc_w, workers added in
 *   order; with params != NULL the optimiser tail above is applied to out as it is written.
 * acc_detect_batch: whole-model statistic n2 = sum_l norm2_layers[l] (fp64, fixed order), then Algorithm 1:
 *   critical = *norm2_prev < 0, or | sqrt(prev) - sqrt(n2) | >= eta * sqrt(prev), or lr_next < lr_curr;
 *   *batch <- max(*batch, critical ? b_low : b_high);  *lr_scale <- *batch / b_low;  *norm2_prev <- n2;
 *   delta <- 0 when delta != NULL (new window).
 *   Device pointers: norm2_layers [L] doubles (e.g. from acc_layer_norms on delta), norm2_prev one double
 *   (in/out, < 0 = none yet), batch one int32 (in/out), lr_scale one float (out).
 *   1 <= b_low <= b_high, otherwise ACC_EINVAL.                                                        */
int acc_batch_accumulate(acc_ctx* ctx, const float* grads, float* acc, float* delta, int32_t first, void* stream);
int acc_batch_average(acc_ctx* ctx, const float* acc, int32_t n_accum, float* out, float* params, float* mom,
                      const float* hyper, void* stream);
int acc_detect_batch(acc_ctx* ctx, const double* norm2_layers, double* norm2_prev, float lr_curr, float lr_next,
                     int32_t b_low, int32_t b_high, int32_t* batch, float* lr_scale, float* delta, void* stream);

/* ---- Real workers (Section 3: every worker computes its gradient on its own GPU; Section 5.1: the PowerSGD
 * factors are exchanged by all-reduce, TopK's values and indices by all-gather) ------------------------------
 * A context then holds this GPU's workers only (n_workers = workers on this GPU, the same on every GPU), and a
 * step is split around the exchanges, which the caller performs with its collective library between the calls
 * (sum over GPUs, in place):
 *   acc_powersgd_phase1: first pass of acc_powersgd_step over this GPU's workers; then x1 <- this GPU's rows of
 *                        the unnormalised P (ranks beyond r as zeros) followed by the VECTOR layers' local means.
 *       -- all-reduce(sum) x1 --
 *   acc_powersgd_phase2: P^ = Gram-Schmidt(scale * x1 rows); x2 <- this GPU's rows of Q' = Mbar^T P^.
 *       -- all-reduce(sum) x2 --
 *   acc_powersgd_phase3: Q[:, :r] <- scale * x2;  VECTOR out <- scale * x1 tail;  out = P^ Q^T and the residual as in
 *                        acc_powersgd_step; with params != NULL the optimiser tail as in acc_powersgd_step_sgd.
 * scale = 1 / (number of GPUs).  With one GPU and scale 1 the three calls give the results of acc_powersgd_step
 * up to fp32 rounding (the fold of P changes the order of a few additions).
 * acc_exchange_layout: lengths in floats of x1 (4*p_rows + packed VECTOR elements) and x2 (4*q_rows), and the
 * length of the packed VECTOR region alone (each VECTOR layer, in order, starts at a multiple of 4 floats).
 * Device pointers: x1, x2 16-byte aligned, caller-owned; the others as in acc_powersgd_step.                */
int acc_exchange_layout(const acc_ctx* ctx, int64_t* x1_floats, int64_t* x2_floats, int64_t* vec_floats);
int acc_powersgd_phase1(acc_ctx* ctx, const float* grads, float* err, float* q, float* p_hat,
                        const uint8_t* level, float* out, float* delta, float* x1, void* stream);
int acc_powersgd_phase2(acc_ctx* ctx, const float* x1, float scale, float* p_hat, const uint8_t* level,
                        const float* out, float* x2, void* stream);
int acc_powersgd_phase3(acc_ctx* ctx, float* err, float* q, const float* p_hat, const uint8_t* level,
                        const float* x1, const float* x2, float scale, float* out, float* params, float* mom,
                        const float* hyper, void* stream);

/* TopK with real workers: values and indices are gathered from every worker (Section 5.1).
 *   acc_topk_compress: acc_topk_step without its last pass, over this GPU's workers: vals / idx / counts and the
 *                      error memories as in acc_topk_step; vec_packed <- this GPU's means of the VECTOR layers
 *                      (packed as in acc_exchange_layout, vec_floats floats); delta += g_decider when != NULL.
 *       -- all-gather vals, idx, counts (every GPU contributes its whole buffers); all-reduce(sum) vec_packed --
 *   acc_topk_decompress: out[l] = (1/n_sets) sum_j scatter(idx_j, val_j) over the n_sets gathered packed sets
 *                      (set j at entry j*capacity of vals_all / idx_all, its counts at counts_all[j*L ..]), sets
 *                      added in order; VECTOR layers: out = vec_scale * vec_packed.  Each set's entries must be in
 *                      ascending index order per layer (as acc_topk_compress writes them).  With params != NULL
 *                      the optimiser tail is applied to out as it is written.
 * With the sets of one GPU (n_sets = n_workers, vec_scale = 1) the pair gives the bits of acc_topk_step.    */
int acc_topk_compress(acc_ctx* ctx, const float* grads, float* err, const uint8_t* level, float* vals,
                      int32_t* idx, int32_t* counts, float* delta, float* vec_packed, void* stream);
int acc_topk_decompress(acc_ctx* ctx, const float* vals_all, const int32_t* idx_all, const int32_t* counts_all,
                        int32_t n_sets, const float* vec_packed, float vec_scale, float* out, float* params,
                        float* mom, const float* hyper, void* stream);

/* Host-fed operation (no counterpart in the paper: there the gradients are produced on the GPU).  For callers whose
 * gradients arrive in HOST memory -- and for the end-to-end leg of the benchmark --
 *   acc_upload_grads:  grads_dev [W][worker_stride] <- grads_host, one asynchronous copy on `stream`;
 *   acc_download_out:  out_host [worker_stride] <- out_dev, likewise.
 * grads_host / out_host are HOST pointers and should be page-locked (pinned), otherwise the copies are staged by
 * the driver and block; grads_dev / out_dev are DEVICE pointers.  Issue the upload on a copy stream and order
 * the step after it with an event to overlap it with the previous step's kernels.                     */
int acc_upload_grads(acc_ctx* ctx, const float* grads_host, float* grads_dev, void* stream);
int acc_download_out(acc_ctx* ctx, const float* out_dev, float* out_host, void* stream);

/* Device-side condition of the kernels launched so far on this context (no counterpart in the paper).
 * The pipelined kernels wait for their asynchronous shared-memory copies with a bounded number of polls;
 * should a wait ever give up, the block stores ACC_ETIMEOUT in a status word and returns instead of
 * hanging, and the results of that call are undefined.  This call copies the status word to *status
 * (HOST pointer; 0 = no such event) and blocks until the device has finished the work queued before it. */
int acc_device_status(acc_ctx* ctx, int32_t* status);

/* Failure-detection self-test (no counterpart in the paper).  acc_selftest_wait_timeout launches one small kernel
 * that waits, with a short poll limit, on a barrier at which nothing ever arrives; the wait gives up, the kernel
 * stores ACC_ETIMEOUT in the status word and returns normally -- the path a pipelined kernel takes should one of
 * its copies never complete.  Nothing faults or hangs, and the context stays usable.  acc_reset_device_status
 * clears the status word (asynchronously on `stream`).                                                 */
int acc_selftest_wait_timeout(acc_ctx* ctx, void* stream);
int acc_reset_device_status(acc_ctx* ctx, void* stream);

/* Diagnostic (no counterpart in the paper): which selection path the last acc_topk_step took for every
 * (worker, MATRIX layer) pair, in worker-major order, n >= W * (number of MATRIX layers) HOST ints:
 *   0 dense (levels 2-3 of the radix select read M), 1 list built by the collect pass, 2 list built by the
 *   first pass from a held prediction, 3 whole entries staged by the first pass (M not read again),
 *   4 zero fill (k exceeds the non-zero entries, e.g. a row-sparse embedding gradient at a large K: the threshold
 *   is 0, every non-zero is kept and the zeros of lowest index fill up; settled from counts of the first pass).
 * Blocks until the device has finished the queued work.  All paths give identical results; tests use
 * this to make sure each one is exercised.                                                          */
#define ACC_TOPK_PATH_DENSE 0
#define ACC_TOPK_PATH_LIST 1
#define ACC_TOPK_PATH_LIST_PREDICTED 2
#define ACC_TOPK_PATH_STAGED 3
#define ACC_TOPK_PATH_ZERO_FILL 4
int acc_topk_last_paths(acc_ctx* ctx, int32_t* paths, int32_t n);

/* Floats one iteration communicates at the given HOST level array, following the "Data Sent"
 * accounting of Tables 1-4: PowerSGD r*(rows+cols) per MATRIX layer, TopK 2*k*W per MATRIX layer
 * (values + indices gathered from every worker), plus every VECTOR element once.  Returns -1 on a
 * bad argument.  Host-only helper.                                                                 */
int64_t acc_floats_sent(const acc_config* cfg, const uint8_t* level_host, int32_t compressor);

/* Number of kernels the last *_step / acc_error_feedback / acc_layer_norms / acc_detect_regime call
 * on this context launched (for launch accounting in benchmarks).                                  */
int32_t acc_last_launch_count(const acc_ctx* ctx);

/* Squared L2 norm of one flat fp32 buffer without any caller-provided scratch (the paper has no
 * counterpart; the value is what acc_layer_norms returns for a single layer covering the buffer,
 * e.g. the whole-model gradient norm).
 *
 * Who needs it: callers that cannot allocate device memory and have no workspace to pass -- code
 * that runs inside another framework's fixed memory budget, a plugin that is only handed tensors,
 * a loop that cannot afford the device-wide synchronisation an allocation implies.  Every other
 * entry point needs the workspace given to acc_create; this one keeps its reduction scratch in a
 * device array built into the library (256 KB on every GPU that loads the library, held until the
 * process exits).  It performs no allocation of any kind.
 *
 *   *norm2 = sum_i buf[i]^2, i < n, accumulated in fp64 in a fixed order (bit-reproducible).
 *
 * Device pointers: buf [n] floats, 16-byte aligned (read); norm2: one double (written).
 * Limits and rules:
 *   - 1 <= n <= ACC_STATIC_NORM_MAX_ELEMS, otherwise ACC_ETOOBIG (nothing is launched).
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's partial sums.
 *     Nothing in it needs clearing (each call overwrites every slot it later reads), but two calls
 *     that overlap on the GPU -- different streams, no ordering between them -- race on it and
 *     return garbage: order them on one stream or with events.                                      */
#define ACC_STATIC_NORM_MAX_ELEMS (1 << 28)
int acc_sumsq_static(const float* buf, int64_t n, double* norm2, void* stream);

/* Per-kernel timing aid (no counterpart in the paper).  While enabled, every kernel the library
 * launches on this context is bracketed by CUDA events on its stream.  acc_profile_read waits for the
 * recorded events (blocks the host until those kernels finished), writes per kernel the summed
 * duration in milliseconds and the number of launches since the last read into HOST arrays of
 * n >= acc_profile_kernel_count() entries, and clears the record.  Kernel i is named
 * acc_profile_kernel_name(i).  Event records cost about a microsecond each: leave profiling off
 * when timing whole steps.                                                                          */
int acc_profile_enable(acc_ctx* ctx, int32_t enable);
int acc_profile_read(acc_ctx* ctx, double* ms, int32_t* launches, int32_t n);
int32_t acc_profile_kernel_count(void);
const char* acc_profile_kernel_name(int32_t i);

const char* acc_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* ACC_H_ */
