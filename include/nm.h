/*
 * nm.h — C ABI of the column-wise N:M sparse convolution library for NVIDIA B200 (sm_100a).
 *
 * The library implements the inference hot path of "Efficient Column-Wise N:M Pruning on
 * RISC-V CPU" (arXiv 2507.17301) on one GPU:
 *
 *   nm_prune      column-wise N:M pruning at tile level (Sec. 3.1) into the compressed
 *                 weight + index-array form (Sec. 2.1, inputs of Algorithm 1);
 *   nm_conv2d     convolution with those weights as a sparse implicit GEMM: the fused
 *                 im2col + packing pass (Sec. 3.2, Algorithm 2) becomes an index-driven gather
 *                 of the retained (kh, kw, c) slices from NHWC activations into shared memory,
 *                 and the tiled outer-product micro-kernel (Algorithm 1) becomes a dense TF32
 *                 tensor-core sub-GEMM per output-channel tile with fp32 accumulation;
 *   nm_autotune   on-device profiling of candidate launch plans, keeping the fastest
 *                 (Sec. 3.3).
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, fp32 unless stated,
 *     contiguous, 16-byte aligned.  The library never frees or reallocates caller memory.
 *     Entry points whose name ends in _host take HOST pointers instead and say so.
 *   - Activations are NHWC  x[batch][h][w][c_in];  outputs NHWC  y[batch][ho][wo][c_out] with
 *       ho = (h + 2*pad_h - dil_h*(kh-1) - 1) / stride_h + 1   (floor; same for wo).
 *   - Dense weights are OHWI  w[c_out][kh][kw][c_in]; reduction column k = (kh*Kw + kw)*c_in + c
 *     (Fig. 4: kernel layout OHWI), K = kh*kw*c_in <= 65535.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work
 *     is enqueued on it; calls return without synchronising unless stated.
 *   - All functions return an nm_status_t; nothing throws, aborts or exits.  A human-readable
 *     description of the calling thread's last failure is available from nm_last_error().
 *   - Handles (nm_weights_t) are owned by the library and released only by nm_weights_free.
 *   - There is no CPU fallback: without a CUDA device every compute entry point fails with
 *     NM_ERR_CUDA.
 */
#ifndef NM_H_
#define NM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NM_OK = 0,
    NM_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, N > M, misaligned pointer, ... */
    NM_ERR_UNSUPPORTED = -2, /* valid but outside what the kernels cover (K > 65535, tile > 256, ...) */
    NM_ERR_CUDA = -3,        /* a CUDA runtime / driver call failed (text in nm_last_error) */
    NM_ERR_ALLOC = -4,       /* host or device allocation failed */
    NM_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired (reported by nm_weights_check) */
    NM_ERR_INTERNAL = -6
} nm_status_t;

/* Opaque compressed-weight handle: compacted values, per-tile column indices and the
 * library's internal copies (TF32-rounded, padded weight tiles; decoded tap table). */
typedef struct nm_weights nm_weights_t;

/*
 * Launch plan for nm_conv2d (the analogue of the paper's per-layer template parameters, Sec. 3.3).
 *   variant  0 = let the library choose;
 *            1 = direct-gather kernel (any shape);
 *            2 = slab kernel (dense activation slab staged once per CTA, kept columns picked by
 *                4-byte loads; needs c_in % 4 == 0 and whole N:M groups per slab);
 *            3 = stream kernel (persistent; slab read once with 16-byte loads, kept columns of
 *                every tile selected in registers; needs c_in % 32 == 0, tile_t % 16 == 0,
 *                c_out % tile_t == 0, N:M one of 1:4 2:4 3:4 1:8 2:8 4:8 or N = M, an input of at
 *                least 128 KiB);
 *            4 = expanded-operand kernel (persistent; the slab feeds the tensor core directly and
 *                zero weights stand for the pruned columns: M/N times the kept FLOPs, no
 *                per-element work; needs c_in % 32 == 0 (pointwise layers, kh = kw = 1: c_in % 4 == 0,
 *                the last 32-channel block is filled up with zeros), c_out % 4 == 0, an input of at
 *                least 128 KiB; any tile_t, any N:M);
 *            5 = row-run kernel for few input channels (c_in % 32 != 0, dil_w = 1, output rows of
 *                at most 128 pixels, K <= 512, c_out % 32 == 0 and <= 256, w * c_in * 4 a multiple
 *                of 16).
 *            6 = window kernel for stride-1 convolutions with a spatial kernel (3x3 and the like): one
 *                input patch per 32-channel block in shared memory, every tap a shifted view of it
 *                (needs stride 1, c_in % 32 == 0, c_out % 32 == 0, w + 2 * pad_w <= 256; expanded
 *                weights as in variant 4).
 *            7 = pair kernel: variant 4 run by clusters of two CTAs (tcgen05 cta_group::2), each SM
 *                staging its own 128 pixels and half of the weight rows of a 256 x bn MMA, which
 *                halves the shared-memory traffic per FLOP on reduction-heavy layers (needs the
 *                conditions of variant 4, bn 128 or 256, c_out % bn == 0).
 *            8 = select kernel (persistent; contracts over the retained columns only: the dense
 *                activations of a chunk are staged once per CTA, each thread reads its pixel's row with
 *                16-byte loads and picks every tile's retained columns with M - N bitwise selects per
 *                column under precomputed masks; up to four MMA issuer threads; needs N:M one of
 *                1:4 2:4 3:4 1:8 2:8 4:8, K % M == 0, c_in a multiple of the chunk's 64 (3:4: 32) source
 *                columns, tile_t % 16 == 0, c_out % tile_t == 0, an input of at least 128 KiB).  Activation
 *                loads (`loads`): im2col-mode TMA loads (any stride / dilation), or, for stride-1 layers
 *                whose output has the input's size, "patch" loads that fetch a pixel block and its halo
 *                once for all kh * kw taps.  `stages` = activation ring depth; `ksplit` > 1 splits the
 *                reduction axis like variant 4's split (same scratch, same second pass).
 *            9 = plane kernel for at most four input channels and a horizontal stride of 1 or 2 (the 7x7 / 2
 *                stem): the input rows of a band of output rows are held in shared memory with the channels
 *                padded to four and, for stride 2, even and odd columns in separate planes, so that the tensor
 *                core reads every tap's operand straight out of them (unswizzled K-major core matrices) and no
 *                patch matrix is built (needs c_in <= 4, kw <= 8, dil_w = 1, stride_w 1 or 2, output rows of at
 *                most 128 pixels, c_out % 32 == 0 and <= 256; any tile_t, any N:M).  `split` = output rows per
 *                work item (1-4, 0 = as many as tensor memory holds), `stages` = row-band buffers (2 or 3).
 *   bn       output channels per CTA / work item (variants 2, 3, 8: a multiple of tile_t; variant 4: a
 *            multiple of 32 up to 256 that divides c_out rounded up to a multiple of 32; variant 6: a multiple
 *            of 32 up to 256 that divides c_out; variant 7: 128 or 256), 0 = default
 *   stages   depth of the shared-memory ring, 0 = default
 *   split    variant 2: 1 = cp.async producer, 2 = direct-store epilogue; variant 4: 0 = keep a CTA's weight
 *            slice resident in shared memory when it fits, 1 = stream the weights with the activations,
 *            2-8 = number of CTAs the reduction axis is split over ( partial sums go through scratch memory that nm_autotune
 *            reserves on the handle, so such a plan works only on a handle nm_autotune has seen with a
 *            layer at least as large), -1 = balanced: the (work item, stage) pairs of the layer are cut into
 *            one equal contiguous range per SM, an item shared by several CTAs is completed by the CTA
 *            that holds its first stage from the others' partial sums (per-SM slots in the same
 *            scratch; for layers with too few work items to fill every SM evenly);
 *            variant 6: M-tiles per work item (1-4); variant 8: 1 = four epilogue warps, 2 = eight (0 = eight where a
 *            work item has at most four chunks); variant 9: output rows per work item (1-4, 0 = most);
 *            otherwise 0
 *   kblk     variants 4 and 7: 32-column blocks of the reduction axis per pipeline stage, 1 or 2 (0 = 1);
 *            two blocks halve the barrier round trips per MMA, which pays where the MMAs are short
 *            (few channels per work item) or the layer is small; K / 32 (per split) must be a multiple
 * A plan the layer does not admit gives NM_ERR_UNSUPPORTED.
 */
typedef struct {
    int variant;
    int bn;
    int stages;
    int split;
    int kblk;
    int loads;    /* variant 8: 0 = the library's choice, 1 = im2col loads, 2 = patch loads */
    int issuers;  /* MMA issuer threads: variant 8: 1-4 (0 = 4); the work item's accumulator columns are cut into
                     that many MMA units where the tile width allows (units of at least 16 columns, none across two
                     tiles), so fewer issuers mean wider MMAs;
                     variant 4: 1 or 2 (0 = 1); two threads take alternate pipeline stages of a work item, each into an
                     accumulator of its own that the epilogue adds (the ring then has an even number of stages, and
                     work items of more than 128 channels have one accumulator buffer instead of two) */
    int ksplit;   /* variant 8: ranges the reduction axis is split into, 1-8 (0 = 1); more than one needs scratch */
    int reserved[8];
} nm_plan_t;

/* ---------------------------------------------------------------------------------------------
 * Pruning and the compressed form
 * ------------------------------------------------------------------------------------------- */

/*
 * Column-wise N:M pruning at tile level (Sec. 3.1).
 * Rows of the [c_out, K] filter matrix are cut into tiles of `tile_t` output channels.  Inside a
 * tile a column (its tile_t weights) is one unit scored by its L1 norm; in every group of
 * `m_group` consecutive columns the `n_keep` highest-scoring units are RETAINED (N counts kept
 * columns, N = (1 - sparsity) * M) and all rows of the tile share that kept set.
 * Deterministic rules where the paper is silent: scores are fp64 sums over the tile's rows in
 * ascending row order; a score that is NaN (a NaN weight in the column) ranks as +infinity, like the
 * score of a column holding an infinite weight, so the order of the scores is total for every input
 * and every group keeps exactly N columns; of two equal scores the lower column is kept; a tail group of m' < M
 * columns keeps min(N, m'); a tail tile (c_out % tile_t rows) scores over the rows it has.
 *
 *   w_dense   device, fp32 [c_out][kh][kw][c_in]; read only, may be freed after the stream
 *             has passed this call
 *   out       receives a new handle holding values[c_out][kk] and indices[n_tiles][kk]
 *             (see nm_weights_export) with kk = N*(K / M) + min(N, K % M)
 * Allocates device memory (synchronously); the kernels run on `cuda_stream`.
 * Errors: INVALID_ARG (null, sizes < 1, n_keep > m_group), UNSUPPORTED (K > 65535, kh or kw > 255,
 * tile_t > 256), ALLOC, CUDA.
 */
nm_status_t nm_prune(const float* w_dense, int c_out, int kh, int kw, int c_in, int n_keep,
                     int m_group, int tile_t, void* cuda_stream, nm_weights_t** out);

/*
 * nm_prune for callers that cannot allocate device memory (the paper has no counterpart; this is a
 * deployment aid).  Meant for a plug-in living inside a process whose GPU memory is entirely
 * managed by someone else's pool, where cudaMalloc fails or breaks the host's accounting, and for
 * latency-critical loops that cannot afford the device-wide synchronisation cudaMalloc / cudaFree
 * imply.  It performs the same pruning as nm_prune and produces the same canonical result, but
 *   - writes it straight into caller memory: values  device fp32  [c_out][kk],
 *                                            indices device uint16 [ceil(c_out/tile_t)][kk],
 *     kk = N*(K / M) + min(N, K % M) (no handle is created; feed the pair to nm_weights_import
 *     when a handle is wanted and allocation is possible);
 *   - takes its scratch (fp64 scores and keep flags) from a fixed array compiled into the library,
 *     resident on every GPU that loads it (about 4.5 MiB) until the process ends;
 *   - calls no cudaMalloc, cudaFree or any other allocating routine.
 * Limit: ceil(c_out / tile_t) * K <= NM_NOALLOC_MAX_CELLS and c_out <= 65535; beyond that it returns
 * NM_ERR_UNSUPPORTED and does nothing.  All calls share the one scratch array: calls whose kernels
 * could overlap on the GPU (other streams or threads) race, so issue them one after another on one
 * stream.  The first call on a given device looks up the array's device address (once per device,
 * cached); make that first call outside any stream capture.  With lazy module loading (the CUDA
 * default) that first call is also when the runtime loads the module holding the array: the 4.5 MiB
 * are reserved on the device then, and the load may synchronise it.  So "allocates nothing" holds
 * from the second call on: make one warm-up call per device at start-up, while memory is still to
 * be had.  The cached address does not survive a cudaDeviceReset.  Same limits as nm_prune
 * (kh, kw <= 255, tile_t <= 256), so that the result can be fed to nm_weights_import; `values` and
 * `indices` must hold c_out * kk floats and ceil(c_out / tile_t) * kk uint16 (not checked here; the
 * Python binding checks its tensors).  No column is ever placed outside a group's N slots, whatever
 * the weights hold (NaN and infinities included).  Asynchronous on `cuda_stream`.
 */
#define NM_NOALLOC_MAX_CELLS (1 << 19)
nm_status_t nm_prune_noalloc(const float* w_dense, int c_out, int kh, int kw, int c_in, int n_keep,
                             int m_group, int tile_t, float* values, uint16_t* indices,
                             void* cuda_stream);

/* Dimensions of a handle; any output pointer may be NULL. */
nm_status_t nm_weights_dims(const nm_weights_t* w, int* c_out, int* k, int* kk, int* n_tiles,
                            int* tile_t);

/*
 * L1 mass of the retained weights and of all weights of the layer (sums of |w|, fp64): kept / total is
 * the share of the importance measure of Sec. 3.1 that survived pruning, the accuracy proxy to read
 * next to a tile width (wider tiles share a kept set among more rows and retain less).  Known only
 * for handles made by nm_prune (NM_ERR_UNSUPPORTED for imported ones).  Either pointer may be NULL.
 */
nm_status_t nm_weights_retained_l1(const nm_weights_t* w, double* kept, double* total);

/*
 * Copies the canonical compressed form (the compacted weights plus index array of Sec. 2.1,
 * i.e. Algorithm 1's inputs W[T, N] and Idx[N]) to caller memory on `cuda_stream`:
 *   values   device, fp32 [c_out][kk]: values[o][j] = w[o][indices[o / tile_t][j]], bit-exact
 *   indices  device, uint16 [n_tiles][kk]: absolute column positions k, ascending
 * Either pointer may be NULL to skip it.
 */
nm_status_t nm_weights_export(const nm_weights_t* w, float* values, uint16_t* indices,
                              void* cuda_stream);

/*
 * Builds a handle from an already compressed model (the inverse of nm_weights_export; this is the
 * checkpoint path).  Validates on the device that every index row is strictly ascending, < K, and
 * holds the N:M structure the kernels rely on (retained column j lies in group j / N of M
 * consecutive columns).  Same errors as nm_prune, plus INVALID_ARG for a bad index row (detected
 * synchronously).
 */
nm_status_t nm_weights_import(const float* values, const uint16_t* indices, int c_out, int kh,
                              int kw, int c_in, int n_keep, int m_group, int tile_t,
                              void* cuda_stream, nm_weights_t** out);

/*
 * Scratch memory of a handle.  A plan that splits the reduction axis over several CTAs (variant 4
 * with split > 1) or balances it over the SMs (split = -1: one slot of 128 x bn partial sums and eight
 * flag words per SM) passes partial sums through scratch memory owned by the handle; nm_conv2d never
 * allocates, so the scratch must be there before such a plan is used.  The scratch is cleared when it is
 * reserved (the flag words must start at zero).  In balanced mode CTAs of one launch wait, with a bound,
 * for flags raised by CTAs of lower index of the same launch (all CTAs of the launch fit the GPU at once).  nm_autotune reserves it for the
 * layers it tunes; a caller that brings a plan from elsewhere (a plan cache) asks for the size with
 * nm_plan_scratch_bytes (0 for plans that need none) and reserves it with nm_weights_reserve, which
 * allocates synchronously and keeps the larger of the old and new sizes.  Calls that use the same
 * handle's scratch must not overlap on the GPU.
 */
nm_status_t nm_plan_scratch_bytes(const nm_weights_t* w, int batch, int h, int wd, int stride_h, int stride_w,
                                  int pad_h, int pad_w, int dil_h, int dil_w, const nm_plan_t* plan,
                                  size_t* bytes);
nm_status_t nm_weights_reserve(nm_weights_t* w, size_t bytes);

/* Synchronises `cuda_stream`, then reads the handle's device status word.  Returns NM_OK, or
 * NM_ERR_TIMEOUT if a kernel that used this handle gave up on a bounded wait (the status word is
 * cleared, the context stays usable). */
nm_status_t nm_weights_check(const nm_weights_t* w, void* cuda_stream);

/* Releases the handle and its device memory (synchronises the device first). NULL is accepted. */
nm_status_t nm_weights_free(nm_weights_t* w);

/* ---------------------------------------------------------------------------------------------
 * Convolution
 * ------------------------------------------------------------------------------------------- */

/*
 * y = act(conv(x, W_pruned) + bias): the product of Algorithm 1 taken over the patch matrix of
 * Sec. 2.2, which is never materialised: for each output-channel tile only the retained
 * (kh, kw, c) slices are gathered (Sec. 3.2's fused im2col + packing, done as a gathered load).
 *   y[n][oh][ow][o] = act( bias[o] + sum_j values[o][j] *
 *                          x[n][oh*stride_h - pad_h + kh_j*dil_h][ow*stride_w - pad_w + kw_j*dil_w][c_j] )
 * with (kh_j, kw_j, c_j) decoded from indices[o / tile_t][j] and reads outside the image = 0.
 * Non-finite activations: the kernels that contract over the retained columns only (variants 1, 2, 3, 8) never
 * read a pruned column's activation, as Algorithm 1 does not; the expanded-operand kernels (variants 4-7)
 * multiply it by a zero weight, so an Inf or NaN in a PRUNED column turns the outputs of that pixel into NaN there
 * while the definition above (and variants 1, 2, 3, 8) keep them finite.  Finite inputs give the same results in all.
 * Arithmetic: operands rounded to TF32 (weights once at prune time, round-to-nearest; activations
 * round-to-nearest where they pass through registers (variants 1-3), truncated where the staged
 * slab feeds the tensor core directly (variants 4, 5, 6)), products accumulated in fp32.
 *
 *   x      device fp32 [batch][h][wd][c_in]      bias  device fp32 [c_out] or NULL
 *   y      device fp32 [batch][ho][wo][c_out]    relu  0 = identity, 1 = ReLU
 *   plan   NULL = library default; a plan the shape does not admit gives NM_ERR_UNSUPPORTED
 * Asynchronous on `cuda_stream`; allocates nothing.  Errors: INVALID_ARG (null x / y / w, sizes,
 * no output pixels, misaligned pointers), UNSUPPORTED, CUDA (launch failure).
 */
nm_status_t nm_conv2d(const nm_weights_t* w, const float* x, int batch, int h, int wd,
                      int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                      const float* bias, int relu, float* y, const nm_plan_t* plan,
                      void* cuda_stream);

/*
 * nm_conv2d with the shortcut addition of a residual block fused into the epilogue (the ResNets the
 * paper measures end to end, Sec. 4.5, add the block input to the last convolution's output before
 * the ReLU):   y = act(conv(x, W_pruned) + bias + residual)
 *   residual  device fp32 [batch][ho][wo][c_out] (the output's shape), 16-byte aligned, or NULL
 *             (then this is nm_conv2d); it may not alias y; needs c_out % 4 == 0
 * Everything else as nm_conv2d, including the plans.
 */
nm_status_t nm_conv2d_res(const nm_weights_t* w, const float* x, int batch, int h, int wd,
                          int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                          const float* bias, const float* residual, int relu, float* y,
                          const nm_plan_t* plan, void* cuda_stream);

/*
 * Same operation with HOST buffers: x_host, bias_host and y_host are host pointers (pinned memory
 * makes the copies asynchronous), x_dev / y_dev are caller-owned device staging buffers of the
 * sizes nm_conv2d expects and bias_dev a device buffer of c_out floats (may be NULL iff bias_host
 * is).  Enqueues H2D(x, bias) -> nm_conv2d -> D2H(y) on `cuda_stream`; does not synchronise.
 */
nm_status_t nm_conv2d_host(const nm_weights_t* w, const float* x_host, float* x_dev, int batch,
                           int h, int wd, int stride_h, int stride_w, int pad_h, int pad_w,
                           int dil_h, int dil_w, const float* bias_host, float* bias_dev, int relu,
                           float* y_host, float* y_dev, const nm_plan_t* plan, void* cuda_stream);

/*
 * Max pooling over NHWC fp32 activations (the paper has no counterpart in its method: it is the one
 * layer between the stem and the first residual block of the ResNets of Sec. 4.5, provided so that a
 * whole convolution backbone can run through this library):
 *   y[n][oh][ow][ch] = max over the kh x kw window at (oh*stride_h - pad_h, ow*stride_w - pad_w) of x,
 * window positions outside the image ignored; ho = (h + 2*pad_h - kh) / stride_h + 1 (floor), wo alike.
 *   x  device fp32 [batch][h][w][c]      y  device fp32 [batch][ho][wo][c]      c % 4 == 0, pad < window
 * Asynchronous on `cuda_stream`; allocates nothing.
 */
nm_status_t nm_maxpool2d(const float* x, int batch, int h, int w, int c, int kh, int kw, int stride_h,
                         int stride_w, int pad_h, int pad_w, float* y, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Auto-tuning (Sec. 3.3: profile kernel candidates on the target, keep the fastest)
 * ------------------------------------------------------------------------------------------- */

/*
 * Times every launch plan the library admits for this layer (kernel variant x channels per CTA x
 * ring depth) with CUDA events on `cuda_stream` (a few warm-up launches, then the median of
 * several), writes the fastest to *best and its time to *best_ms (may be NULL).  x and y_scratch
 * are caller buffers of the sizes nm_conv2d expects; y_scratch is overwritten.  Synchronises the
 * stream.  A candidate that fails to launch is skipped; NM_ERR_UNSUPPORTED if none runs.
 * Every timed launch starts with a cold L2: the call allocates a 288 MiB buffer for its own
 * duration and overwrites it before each launch (if that allocation fails the launches run warm), so
 * layers that would fit the cache are tuned for operands that come from HBM.  Candidates are tried
 * most promising first and a later one replaces the best so far only if it is at least 1 % faster.
 * This call allocates (the buffer above, and the split-K scratch described at nm_weights_reserve).
 * The environment variable NM_AUTOTUNE_VARIANTS (a list of variant digits such as "1,2,3,8") restricts the
 * search, e.g. to the kernels that skip the pruned columns.  The handle is not const: the call reserves
 * scratch memory on it.
 * Plan cache: when the environment variable NM_PLAN_CACHE names a file, the call first looks the layer up there
 * (key: nm_plan_key of the layer) and, if the cached plan still runs, returns it without tuning (its time is
 * measured over a few launches); otherwise it tunes and appends the result to the file.
 */
nm_status_t nm_autotune(nm_weights_t* w, const float* x, int batch, int h, int wd,
                        int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                        const float* bias, int relu, float* y_scratch, void* cuda_stream,
                        nm_plan_t* best, float* best_ms);

/*
 * Auto-tuning that also chooses the pruning tile width T (the paper profiles T per layer,
 * Sec. 3.3 / Sec. 4.5): prunes `w_dense` once per entry of tile_candidates, tunes each with
 * nm_autotune and returns the fastest (tile, plan) pair.  *best_tile receives the chosen T.
 * The handles it builds are temporary and freed before returning.
 */
nm_status_t nm_autotune_tile(const float* w_dense, int c_out, int kh, int kw, int c_in, int n_keep,
                             int m_group, const int* tile_candidates, int n_candidates,
                             const float* x, int batch, int h, int wd, int stride_h, int stride_w,
                             int pad_h, int pad_w, int dil_h, int dil_w, const float* bias, int relu,
                             float* y_scratch, void* cuda_stream, int* best_tile, nm_plan_t* best,
                             float* best_ms);

/* ---------------------------------------------------------------------------------------------
 * Diagnostics
 * ------------------------------------------------------------------------------------------- */

/*
 * Self-test of the failure path: launches one small block that waits, with a budget of a few thousand
 * polls, on a barrier nothing will ever complete.  The wait runs out, the block records NM_ERR_TIMEOUT
 * in the handle's status word the way the convolution kernels do and returns normally; the next
 * nm_weights_check(w) reports NM_ERR_TIMEOUT and clears it, and the context stays usable.  Nothing
 * faults, traps or hangs.
 */
nm_status_t nm_selftest_wait_expiry(const nm_weights_t* w, void* cuda_stream);

/*
 * Plan cache: a text file with one line per layer, "<key> variant bn stages split kblk loads issuers ksplit"
 * (the analogue of keeping the profiler's choice per operator, Sec. 3.3; the last line of a key wins).
 *   nm_plan_key           writes the key of a layer (its geometry, pattern and tile width, batch and image size,
 *                         whether it has a bias / ReLU) into `key` (at most key_bytes, NUL-terminated);
 *                         INVALID_ARG if the buffer is too small
 *   nm_plan_cache_store   appends (key, plan) to the file (created if missing); CUDA is not touched
 *   nm_plan_cache_lookup  fills *plan from the file; NM_ERR_UNSUPPORTED if the file or the key is missing
 * A plan taken from a cache is only data: nm_conv2d checks it against the layer like any other plan, and a plan
 * that needs scratch memory still needs nm_plan_scratch_bytes / nm_weights_reserve before its first use.
 */
nm_status_t nm_plan_key(int c_out, int kh, int kw, int c_in, int n_keep, int m_group, int tile_t, int batch, int h,
                        int wd, int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w, int has_bias,
                        int relu, char* key, size_t key_bytes);
nm_status_t nm_plan_cache_store(const char* path, const char* key, const nm_plan_t* plan);
nm_status_t nm_plan_cache_lookup(const char* path, const char* key, nm_plan_t* plan);

const char* nm_status_string(nm_status_t s);
/* Text of the calling thread's most recent failure ("" if none). Valid until its next failure. */
const char* nm_last_error(void);
/* Number of kernel launches this process has enqueued through the library (all threads). */
uint64_t nm_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* NM_H_ */
