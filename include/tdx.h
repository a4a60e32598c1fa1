/*
 * tdx -- dense contractions for B200 (sm_100a): matmul with optionally transposed operands and a
 * fused negate/scale, and zero-padded 2-D convolution with fused bias + ReLU.
 *
 * These are the payload computations that the schedules of "The MLIR Transform Dialect"
 * (arXiv 2409.03864) exist to speed up; each entry point cites the passage that states its operation.
 *
 * Conventions (all entry points)
 *  - Every function returns a tdx_status (int); 0 is success.  Nothing throws, aborts or exits.
 *  - Statuses below 16 are "silenceable" in the sense of the paper's Section 3 error model:
 *    nothing was launched, outputs are untouched, and the caller may try an alternative
 *    (Case Study 4's `alternatives` construct).  Statuses >= 16 are definite errors: the state
 *    of the outputs is unspecified.
 *  - Unless a parameter says "host", every data pointer is DEVICE memory on the current CUDA device,
 *    owned by the caller, and must stay valid until the work enqueued on `stream` has finished.
 *    Inputs are read-only; outputs must not alias inputs.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls enqueue work
 *    and return; device-detected conditions (a bounded wait that ran out) are reported by
 *    tdx_check_device_status.
 *  - All matrices are dense row-major; bf16 values are the upper 16 bits of the fp32 pattern.
 *  - tdx_last_error() returns a thread-local, library-owned description of the last failure.
 *  - Library-owned device scratch (split-K partial sums of the non-_ex calls, the bf16 pieces of the fp32
 *    tensor-core path, staging buffers of the *_host calls, tile tables) is per device, grown on demand with
 *    cudaMalloc and reused from call to call in stream order: calls that use it must all be issued on ONE stream per
 *    device, and from one host thread at a time.  Calls that use none (bf16 GEMM / convolution without split-K, or
 *    with a caller workspace through the _ex entry points) have no such restriction; the caches behind them are locked.
 *  - Environment: TDX_TUNE_CACHE (read by the Python binding: a tuning-cache file to load instead of the shipped one, "0"
 *    for none).  TDX_FORCE_CONFIG="tile_m=128,tile_n=128,split_k=6" (read once by the library): a partial tdx_config
 *    that tdx_gemm, tdx_gemm_batched (bf16) and tdx_conv2d_bias_relu take instead of the automatic choice; an infeasible
 *    one fails those calls with TDX_ERR_CONFIG like an explicit configuration would.  TDX_DEBUG_BOUNDS=1 (read once):
 *    the one-thread-per-output kernels (the last entry of every fallback chain, and the searches' comparator) check each
 *    global index against the extent its operand's shape and strides imply; an index outside is not accessed, the kernel
 *    records it in the device status word and tdx_check_device_status reports TDX_ERR_BOUNDS.  Slower; for debugging.
 */
#ifndef TDX_H_
#define TDX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TDX_OK = 0,
    /* silenceable: nothing launched, outputs untouched */
    TDX_ERR_INVALID_ARG = 1, /* negative size, bad flag, NULL pointer, unknown dtype              */
    TDX_ERR_UNSUPPORTED = 2, /* valid request that no kernel here implements                       */
    TDX_ERR_ALIGNMENT = 3,   /* a pointer or pitch breaks the alignment the chosen kernel needs    */
    TDX_ERR_CONFIG = 4,      /* an explicit tdx_config is infeasible for this problem              */
    TDX_ERR_WORKSPACE = 5,   /* workspace missing or too small                                     */
    /* definite */
    TDX_ERR_CUDA = 16,      /* a CUDA runtime / driver call failed                                 */
    TDX_ERR_TIMEOUT = 17,   /* a kernel gave up on a bounded wait (see tdx_check_device_status)    */
    TDX_ERR_NO_DEVICE = 18, /* no usable sm_100 device / driver                                    */
    TDX_ERR_BOUNDS = 19     /* the bounds-checked debug mode (TDX_DEBUG_BOUNDS=1) caught an index outside its */
                            /* operand; the access was skipped (see tdx_check_device_status)                 */
} tdx_status;

typedef enum {
    TDX_F32 = 0, /* A, B, C fp32; fp32 FMAs on CUDA cores, or bf16 pieces on tensor cores */
    TDX_BF16 = 1 /* A, B bf16; fp32 accumulate (tensor cores); C bf16        */
} tdx_dtype;

typedef enum {
    TDX_KERNEL_AUTO = 0,
    TDX_KERNEL_UMMA = 1,    /* tcgen05 tensor-core pipeline (bf16: needs 16-byte aligned pitches; fp32 GEMM: */
                            /* through three bf16 pieces per operand, any shape)                        */
    TDX_KERNEL_SIMT = 2,    /* tiled fp32 CUDA-core GEMM (fp32 GEMM only)                              */
    TDX_KERNEL_GENERIC = 3  /* one thread per output; any dtype, shape and alignment                   */
} tdx_kernel;

/*
 * Tile configuration: the knobs the paper's Case Study 5 hands to its autotuner (tile sizes per
 * loop, vectorise or not) restated for this hardware.  A zero field means "choose for me".
 */
typedef struct {
    int kernel;     /* tdx_kernel                                                              */
    int tile_m;     /* 128 or 256 (two 128-row halves that share each B slice)                 */
    int tile_n;     /* 32, 64, 96, ..., 256 (multiple of 32; multiple of 64 when transB = 0)    */
    int tile_k;     /* 64                                                                      */
    int stages;     /* depth of the TMA/mbarrier ring, 2..8, bounded by shared memory          */
    int cta_pair;   /* 1 = one CTA per tile; 2 = a cluster of two CTAs per 256-row tile (GEMM only): each  */
                    /*     CTA stages its 128 rows of A and half of the B slice, one thread issues MMAs    */
                    /*     over both, and each CTA keeps a 128 x tile_n accumulator half                  */
    int split_k;    /* >= 1; > 1 needs a workspace and runs a fixed-order reduction afterwards  */
                    /*     (store_mode 3: neither, see there)                                    */
    int store_mode; /* 1 = 16-byte stores from registers; 2 = 32 x 32 blocks staged in shared     */
                    /*     memory and written by TMA store (needs N % 8 == 0, split_k = 1,         */
                    /*     16-byte aligned C; falls back to 1 if C is misaligned)                  */
                    /*     3 = (GEMM, cta_pair = 1, split_k in 2..8, tile_n a multiple of 32 * split_k) the   */
                    /*     split_k CTAs of a tile form a thread-block cluster, exchange column slices of     */
                    /*     their fp32 partial tiles through distributed shared memory and each writes its    */
                    /*     slice of the result, summed over the K slices in ascending order: no workspace,   */
                    /*     no reduction launch.  One CTA per (tile, K slice).                                */
    int raster;     /* width, in tiles along M, of the panels the tile order walks; 0 = all     */
    int patch_w;    /* conv only: output-pixel patch that forms the rows of a tile (w x h,      */
    int patch_h;    /*   w*h a power of two <= 128, w >= 8; tile_m / (w*h) patches per tile); 0 = choose */
    int k_stagger;  /* 1 = each CTA starts its K loop at a different block (rotated order, same terms),  */
                    /*     so that CTAs do not all fetch the same operand lines at the same moment       */
    int halo;       /* conv only: 1 = the input window is fetched again for every filter tap; 2 = it is   */
                    /*     loaded once per 64-channel chunk into shared memory and all taps read it there  */
                    /*     (8 x 16 patches, stride 1, more than one tap); 3 = as 2, but the 16-row patches */
                    /*     are cut from the column formed by all images of the batch, H + pad rows apart, so */
                    /*     that an image height that is no multiple of 16 wastes no rows; 0 = choose        */
    int fit;        /* GEMM (split_k = 1; CTA pairs: transB = 1 only) and convolutions whose filter is streamed, tile_n >= 192: 2 = some row blocks are cut into narrower tiles */
                    /*     (multiples of 64 columns) so that all CTAs finish together when the uniform grid  */
                    /*     would leave the last wave of CTAs partly idle; 1 = uniform grid; 0 = fitted when  */
                    /*     the cost model predicts a gain of at least 3 %.  The first call for a shape on a  */
                    /*     device allocates a small tile table there and copies it synchronously (cudaMalloc */
                    /*     + cudaMemcpy): make that call before any stream capture.                          */
                    /*     3 = (GEMM, few tiles and a long reduction; split_k = 1, store_mode = 1, tile_n a      */
                    /*     multiple of 64) the tiles x K blocks units are dealt evenly to ALL CTAs instead of a  */
                    /*     uniform K split, whose item count rarely fills the SMs; a tile cut by a CTA boundary   */
                    /*     is completed from fp32 partial tiles in ascending K order by a reduction launch.       */
                    /*     Needs the workspace tdx_gemm_workspace_size reports (the library's own when none is   */
                    /*     passed); same first-call table upload as 2.                                           */
} tdx_config;

/*
 * C[M x N] = alpha * op(A)[M x K] . op(B)[K x N]     (C overwritten; no accumulate)
 *
 * The operation is the matmul loop nest of the paper's Case Study 4 (the OpenMP tiling figure),
 * one batch, without the accumulate.  transA / transB are the "matmul that supports transposed
 * operands" of Case Study 3's matmul_of_transpose pattern: the transpose is a property of how the
 * operand is read, never a copy.  The negate of negate_of_transpose commutes with the transpose
 * and the product, so it is alpha = -1.
 *
 *   transA = 0: A stored M x K;  transA = 1: A stored K x M.
 *   transB = 0: B stored K x N;  transB = 1: B stored N x K.
 *   dtype: TDX_F32 (all fp32) or TDX_BF16 (bf16 in, fp32 accumulate, bf16 out, one rounding of alpha*acc).
 *   M or N = 0: no-op.  K = 0: C is zero-filled.
 *   fp32: small problems run fp32 FMAs on the CUDA cores; from about 2^28 multiply-adds on (or with kernel =
 *   TDX_KERNEL_UMMA in an explicit config) each operand is cut into three bf16 pieces that together hold all 24
 *   significand bits, and the tensor cores accumulate the six piece products that matter in fp32 -- same 1e-5
 *   bound, several times faster.  That path keeps its pieces in device scratch owned by the library, grown on
 *   demand by cudaMalloc (make the first call for a size before any stream capture).
 * Errors: INVALID_ARG (negative size, flag not 0/1, NULL pointer with non-empty problem, unknown dtype,
 *         non-finite alpha is allowed), CUDA.  bf16 shapes that miss the tensor-core path's alignment rules
 *         (a row pitch that is no multiple of 16 bytes, a misaligned base) are not rejected: from 2^21
 *         multiply-adds on, the operands are first copied K-major with K padded to a multiple of 64 into device
 *         scratch owned by the library (one more launch; grown by cudaMalloc, so make the first call for a size
 *         before any stream capture) and the tensor cores run on the copies -- the padding adds exact zeros;
 *         smaller ones run on the generic GPU kernel.  There is no CPU fallback.
 */
int tdx_gemm(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, int dtype,
             const void* A, const void* B, void* C, void* stream);

/*
 * Batch-matmul with accumulate: C[b] = beta * C[b] + alpha * op(A[b]) . op(B[b]),  b < batch.
 *
 * With alpha = beta = 1 this is the loop nest of the paper's Case Study 4 exactly as printed
 * (C[b,i,j] += A[b,i,k] * B[b,k,j]; its workload is batch 6, M 196, N 256, K 2305).  Layouts per batch
 * as for tdx_gemm; batch b of an operand starts strideX elements after batch b - 1 (strideA or strideB
 * may be 0: the operand is shared by all batches; strideC >= M * N).  C is read only when beta != 0 and
 * must not alias A or B.  fp32: CUDA cores, or bf16 pieces on the tensor cores from about 2^28 multiply-adds.
 * bf16: ONE tensor-core launch over all batches (3-D tensor maps: contiguous dimension, the other one, batch;
 * rows past M or N of a batch read as zero, never as the next batch), straight from the caller's buffers when
 * every batch's operands meet the 16-byte rules of tdx_gemm (contiguous dims and batch strides multiples of 8
 * elements, 16-byte aligned bases), and otherwise -- K = 2305 is such a case: the paper's treatment of sizes that
 * do not divide is to split and peel, here the remainder is padded with zeros instead -- from K-major copies with
 * K padded to a multiple of 64, made by one more launch into scratch owned by the library.  A K split chosen so
 * that every SM has an item is reduced in a fixed order by one launch for all batches, which also applies beta.
 * Problems under 2^21 multiply-adds in an unaddressable layout run on the generic GPU kernel.
 * batch, M or N = 0: no-op.  K = 0: C = beta * C.  Errors as for tdx_gemm.
 */
int tdx_gemm_batched(int64_t batch, int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, float beta,
                     int dtype, const void* A, int64_t strideA, const void* B, int64_t strideB, void* C, int64_t strideC,
                     void* stream);

/*
 * out = zero_pad(x) + y, computed the way Case Study 3's add_of_zero_pad pattern rewrites it: the padded copy of x is
 * never built and the elements that padding would produce (zeros) are never added.
 *
 *   x:        N x H x W x C  (NHWC, dense)
 *   y, out:   N x (H + pad_top + pad_bottom) x (W + pad_left + pad_right) x C
 *   out[n, h + pad_top, w + pad_left, c] = x[n, h, w, c] + y[n, h + pad_top, w + pad_left, c];  elsewhere out = y.
 *
 * out may be y itself (in place): then only the interior is read and written and the padding ring is not touched at
 * all; otherwise out must not overlap x or y, and the ring is copied.  fp32: one fp32 add; bf16: the fp32 sum of the
 * two values rounded once to bf16.  16-byte accesses when every interior row starts on a 16-byte boundary, scalar
 * otherwise; any shape is accepted.  Empty tensors: no-op.  Errors: INVALID_ARG, ALIGNMENT (element alignment), CUDA.
 */
int tdx_add_zero_pad(int64_t N, int64_t H, int64_t W, int64_t C, int pad_top, int pad_bottom, int pad_left, int pad_right,
                     int dtype, const void* x, const void* y, void* out, void* stream);

/*
 * tdx_gemm with bf16 operands and an fp32 result: C[M x N] (fp32) = alpha * op(A) . op(B), A and B bf16 as for
 * tdx_gemm.  The fp32 accumulator is written as it is (times alpha), without the rounding to bf16 -- for results that
 * feed a reduction or a loss, or that are accumulated further.  Same kernels and layout rules as the bf16 GEMM
 * (tensor cores when the 16-byte rules hold, the generic GPU kernel otherwise); C needs 4-byte alignment.
 */
int tdx_gemm_f32out(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, const void* A, const void* B,
                    void* C, void* stream);

/*
 * Same as tdx_gemm with an explicit configuration and caller-owned split-K workspace.
 * cfg = NULL or cfg->split_k = 0: the library chooses split_k (tuning cache, else the cost model's first-ranked candidate); then
 * `workspace` may be NULL and the library uses an internal, lazily grown buffer.  With an explicit
 * cfg->split_k > 1 the caller must pass at least tdx_gemm_workspace_size bytes (256-byte aligned)
 * -> else WORKSPACE.
 * An infeasible cfg -> CONFIG with C untouched (the paper's `alternatives`: a failed alternative
 * leaves the payload unchanged).
 */
int tdx_gemm_ex(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, int dtype,
                const void* A, const void* B, void* C, void* stream,
                const tdx_config* cfg, void* workspace, size_t workspace_bytes);

/* Bytes of workspace tdx_gemm_ex needs for cfg (0 when cfg->split_k <= 1). */
int tdx_gemm_workspace_size(int64_t M, int64_t N, int64_t K, int dtype, const tdx_config* cfg, size_t* bytes);

/*
 * y[n,p,q,k] = relu?( bias[k] + sum_{r,s,c} X(n, p*stride + r - pad, q*stride + s - pad, c) * w[k,r,s,c] )
 * with X = x inside the image and 0 outside: the zero padding is never materialised and padded
 * elements are never added (the add_of_zero_pad pattern of Case Study 3).  The paper states no
 * convolution formula; this is the standard cross-correlation of the ResNet-50 layers its Case
 * Study 4 draws its loop nest from.
 *
 *   x: N x H x W x Cin (NHWC);  w: Cout x R x S x Cin (KRSC);  bias: fp32 [Cout] or NULL;
 *   y: N x P x Q x Cout with P = floor((H + 2 pad - R) / stride) + 1, Q likewise (0 if negative).
 *   dtype: TDX_BF16 (x, w, y bf16; fp32 accumulate) or TDX_F32 (all fp32).  relu in {0, 1}.
 * Errors: INVALID_ARG (size <= 0 for Cin/R/S, negative N/H/W/Cout/pad, stride < 1, NULL pointers), CUDA.
 * Empty outputs (N, Cout, P or Q = 0) are a no-op.
 */
int tdx_conv2d_bias_relu(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                         int pad, int stride, int dtype, const void* x, const void* w, const float* bias,
                         int relu, void* y, void* stream);

/*
 * The same with a residual term: y = relu?( conv(x, w) + bias + residual ), the closing step of a ResNet block
 * (the network the paper's workload is a layer of).  residual is N x P x Q x Cout in the type of y (NULL: none); it
 * joins the fp32 sum after the bias and before the ReLU, fused into the epilogue.  It must not overlap y.
 * cfg: NULL = choose, else as for tdx_conv2d_bias_relu_ex.
 */
int tdx_conv2d_bias_add_relu(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                             int pad, int stride, int dtype, const void* x, const void* w, const float* bias,
                             const void* residual, int relu, void* y, void* stream, const tdx_config* cfg);

/* As above with an explicit configuration (split_k must be 1).  Infeasible cfg -> CONFIG, y untouched. */
int tdx_conv2d_bias_relu_ex(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                            int pad, int stride, int dtype, const void* x, const void* w, const float* bias,
                            int relu, void* y, void* stream, const tdx_config* cfg);

/*
 * Host-buffer variants: A, B, C (x, w, bias, y) are HOST pointers (pinned memory gives the best
 * copy rate).  The call copies the inputs to device staging buffers owned by the library, runs the
 * same kernels as above, copies the result back and returns after the stream has drained.
 * Large problems move in chunks (tdx_gemm_host with transA == 0: row blocks of A and C;
 * tdx_conv2d_bias_relu_host: groups of images): chunk i goes up on a copy stream owned by the
 * library while chunk i - 1 is computed on `stream` and chunk i - 2 comes down on a second copy
 * stream, ordered by events, so the two directions of the bus and the kernels overlap.  Each
 * output element is the same sum of products as in one call over the whole problem; the tile shape
 * and K split are chosen per chunk, so its fp32 summation order may differ.  The host buffers must stay
 * valid and unmodified until the call returns (it returns only when all three streams are idle).
 */
int tdx_gemm_host(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, int dtype,
                  const void* A_host, const void* B_host, void* C_host, void* stream);
/* tdx_add_zero_pad in place on host buffers: y_host = zero_pad(x_host) + y_host. */
int tdx_add_zero_pad_host(int64_t N, int64_t H, int64_t W, int64_t C, int pad_top, int pad_bottom, int pad_left,
                          int pad_right, int dtype, const void* x_host, void* y_host, void* stream);
/* tdx_gemm_batched on dense host buffers (strides M*K, K*N, M*N); C_host is copied in only when beta != 0. */
int tdx_gemm_batched_host(int64_t batch, int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha,
                          float beta, int dtype, const void* A_host, const void* B_host, void* C_host, void* stream);
int tdx_conv2d_bias_relu_host(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                              int pad, int stride, int dtype, const void* x_host, const void* w_host,
                              const float* bias_host, int relu, void* y_host, void* stream);

/*
 * Tile-configuration search: the stand-in for the autotuner integration of the paper's Case Study 5.
 * Enumerates the configurations that pass the static constraints (the analogue of "tile sizes must
 * divide their dimension, vectorise only if divisible": shared-memory and TMEM budgets, layout
 * divisibility), times each on the device with CUDA events on scratch operands the call allocates,
 * returns the fastest and records it in the in-process tuning cache used by the automatic choice.
 *   iters: timed launches per candidate (>= 1).  best / best_us: outputs (best_us = mean microseconds).
 *   tried / tried_us / cap / n_tried: optional (NULL / 0) list of every candidate with its time.
 * Before a winner is cached its output is checked on the device against the one-thread-per-output kernel's on the
 * same scratch operands (GEMM: up to 16 blocks of 128 rows spread over M; convolution: the whole output), and a
 * candidate whose kernel reported a bounded wait that ran out is dropped; if the fastest candidates all fail that
 * check the call returns UNSUPPORTED and caches nothing.
 */
int tdx_tune_gemm(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, int iters,
                  tdx_config* best, float* best_us, tdx_config* tried, float* tried_us, int cap, int* n_tried,
                  void* stream);
int tdx_tune_conv2d(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                    int pad, int stride, int dtype, int iters, tdx_config* best, float* best_us,
                    tdx_config* tried, float* tried_us, int cap, int* n_tried, void* stream);

/* The statically feasible search space (no device needed).  Writes up to cap configs, *n = total count. */
int tdx_enum_gemm_configs(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype,
                          tdx_config* out, int cap, int* n);
int tdx_enum_conv2d_configs(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                            int pad, int stride, int dtype, tdx_config* out, int cap, int* n);

/*
 * Search on first use (the paper's autotuner integration, Case Study 5, applied lazily).  budget = 0 (the default)
 * switches it off; budget > 0: the first tdx_gemm / tdx_gemm_host call on a bf16 shape that the tuning cache does
 * not know runs the guided search with that budget on scratch operands of the shape (see tdx_tune_gemm_guided:
 * it allocates device memory, launches and synchronises `stream`; typically well under a second) and caches the
 * winner; budget < 0: the same with every candidate timed.  Calls with an explicit configuration, calls inside a
 * stream capture and shapes off the tensor-core path are never searched.  A search that fails does not fail the
 * call.  Process-wide; returns TDX_OK.
 */
int tdx_set_autotune(int budget);

/*
 * Guided search: the candidates of tdx_tune_gemm are ranked by a host-side cost model (MMA time by tile width, L2
 * ingest, epilogue overlap, wave count or fitted plan, split-K traffic, HBM floor) and only the `budget` best-ranked
 * ones, plus the automatic choice, are timed on the device -- the model-guided counterpart of Case Study 5's
 * search under constraints.  n_candidates (may be NULL) receives the size of the full search space.  The cached winners
 * of other shapes with the same operand layouts are tried as well (up to four), so what earlier searches found carries
 * over to a new shape.  bf16 GEMM; other problems are searched exhaustively.  tdx_model_gemm_us evaluates the model for one configuration on
 * `ctas` SMs (host only).
 */
int tdx_tune_gemm_guided(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, int iters, int budget,
                         tdx_config* best, float* best_us, tdx_config* tried, float* tried_us, int cap, int* n_tried,
                         int* n_candidates, void* stream);
int tdx_model_gemm_us(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, const tdx_config* cfg, int ctas,
                      double* us);

/*
 * The same for the convolution: the candidates of tdx_tune_conv2d are ranked by a host-side cost model of the two
 * convolution kernels (wasted patch rows, input-window bytes per filter tap or per channel chunk, resident filter,
 * strided windows, epilogue overlap, wave count) and only `budget` of them, plus the automatic choice, are timed;
 * winner checked and cached as by tdx_tune_conv2d.  tdx_model_conv2d_us evaluates the model (host only).
 */
int tdx_tune_conv2d_guided(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                           int stride, int dtype, int iters, int budget, tdx_config* best, float* best_us, tdx_config* tried,
                           float* tried_us, int cap, int* n_tried, int* n_candidates, void* stream);
int tdx_model_conv2d_us(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad, int stride,
                        int dtype, const tdx_config* cfg, int ctas, double* us);

/*
 * A search space stated by the caller, the way Case Study 5 hands its tuner a list of tuning parameters with ranges
 * and constraints (tile sizes that must divide their dimension; vectorisation only under a divisibility condition):
 *
 *   "tile_m in {128, 256}; tile_n in 64..256 step 64; split_k in {1, 2, 4};
 *    require M % tile_m == 0; require N % tile_n == 0;
 *    store_mode == 2 only if N % 8 == 0 && split_k == 1"
 *
 * Statements are separated by ';'.  `<param> in {a, b, ...}` or `<param> in lo..hi [step s]` gives a parameter its
 * range (parameters: tile_m tile_n tile_k stages cta_pair split_k store_mode raster k_stagger fit; one not mentioned
 * stays "choose for me").  `require <expr>` keeps a candidate only if the expression holds; `<param> == <value> only
 * if <expr>` lets that value through only under the condition.  Expressions are integer expressions over the
 * parameters, the problem (M N K transA transB num_kb = ceil(K / 64)) and literals, with + - * / % == != < <= > >= && ||
 * ! and parentheses.  The cross product of the ranges is filtered by the stated rules, each survivor is completed
 * by the library's rules and checked against the hardware's own constraints (shared memory, tensor memory, layout).
 *
 * tdx_enum_gemm_space lists the survivors (host only; n_product = size of the cross product, n_after_rules = how many
 * pass the stated rules).  tdx_tune_gemm_space searches them -- all of them (budget = 0) or the `budget` the cost model
 * ranks best -- checks the winner's output and caches it like tdx_tune_gemm.  bf16 GEMM with 16-byte aligned pitches.
 * Errors: INVALID_ARG (syntax, unknown name, NULL), UNSUPPORTED (nothing feasible is left; other dtypes / layouts).
 */
int tdx_enum_gemm_space(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, const char* space, tdx_config* out,
                        int cap, int* n, int64_t* n_product, int64_t* n_after_rules);
int tdx_tune_gemm_space(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, const char* space, int iters,
                        int budget, tdx_config* best, float* best_us, tdx_config* tried, float* tried_us, int cap, int* n_tried,
                        int* n_candidates, void* stream);

/* The configuration the automatic choice would use right now: the tuning cache's entry, else (bf16 GEMM on the
 * tensor-core path) the candidate of the search space that the cost model ranks first, else a size heuristic. */
int tdx_default_gemm_config(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, tdx_config* out);
int tdx_default_conv2d_config(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                              int pad, int stride, int dtype, tdx_config* out);

/*
 * The tile plan `fit = 2` would use for a GEMM on `ctas` persistent CTAs (host only, no device needed).
 * It is the counterpart of Case Study 5's divisibility constraints turned around: instead of asking
 * that the tile divide the problem, some row blocks are cut into narrower tiles so that the tile
 * count divides evenly over the CTAs.  table (may be NULL) receives up to cap_tiles triples
 * (row block, first column, width), entry [round * n_ctas + cta]; width 0 = no tile.  n_rounds = 0
 * means the uniform grid is kept.  model_cycles / model_cycles_uniform are the cost model's longest
 * CTA for the plan and for the uniform grid.
 */
int tdx_gemm_tile_plan(int64_t M, int64_t N, int64_t K, int tile_m, int tile_n, int raster, int ctas, int* table,
                       int cap_tiles, int* n_rounds, int* n_ctas, double* model_cycles, double* model_cycles_uniform);

/*
 * The plan `fit = 3` would use on `ctas` persistent CTAs (host only): the tiles x K blocks units of the problem, tile
 * after tile, cut into `ctas` nearly equal runs, so that every SM streams its share of the operands of a problem with
 * few tiles and a long reduction (Case Study 5 tiles the reduction loop too; here the cut points follow the machine,
 * not a divisor of K).  table (may be NULL) receives up to cap_entries groups of six ints, entry [round * n_ctas + cta]
 * = (row block, first column, width, first K block, end K block, partial slot); width 0 = no entry.  max_slots is the
 * largest number of pieces any tile is cut into, i.e. the workspace holds max_slots * M * N floats.
 */
int tdx_gemm_k_balanced_plan(int64_t M, int64_t N, int64_t K, int tile_m, int tile_n, int ctas, int* table, int cap_entries,
                             int* n_rounds, int* n_ctas, int* max_slots);

/* Persist / restore the tuning cache (a small JSON text file). */
int tdx_tune_save(const char* json_path);
int tdx_tune_load(const char* json_path);
int tdx_tune_clear(void);

/*
 * Synchronises `stream`, reads and clears the device status word.  TDX_OK, or TDX_ERR_TIMEOUT if a
 * kernel abandoned a bounded wait since the last check (its outputs are then unspecified), or TDX_ERR_BOUNDS if the
 * bounds-checked debug mode skipped an access.
 */
int tdx_check_device_status(void* stream);

/*
 * Split-K GEMM for callers that must not allocate device memory.  (The paper has no counterpart to
 * this entry point; it exists for integration reasons only.)
 *
 * Who needs it: code that runs where a device allocation is off limits -- a serving loop whose memory
 * was sized and handed out once at start-up, a plug-in living inside another framework's memory pool
 * (a raw cudaMalloc there bypasses the pool's accounting and, like cudaFree, stalls every stream of
 * the device while it runs), or a latency-critical step that cannot afford that stall.  tdx_gemm
 * may grow an internal split-K workspace with cudaMalloc and tdx_gemm_ex wants a workspace from the
 * caller; this call needs neither.
 *
 * It computes exactly what tdx_gemm_ex computes for dtype TDX_BF16 with cfg = {kernel = UMMA,
 * tile_m = 128, tile_n as given (0 = choose), split_k as given}: C = alpha * op(A) . op(B), partial
 * sums of the split_k K-slices reduced in a fixed order.  The partials live in a fixed array of
 * TDX_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads the library holds
 * those bytes until the process exits, whether or not this function is ever called.
 *
 *   split_k >= 1;  split_k * M * N * 4 bytes must not exceed TDX_STATIC_SCRATCH_BYTES, else
 *   TDX_ERR_WORKSPACE (nothing launched, C untouched).  Layout rules are those of the tensor-core
 *   path (16-byte aligned pointers, contiguous dimensions multiples of 8): a shape that misses them
 *   gets TDX_ERR_ALIGNMENT rather than another kernel.
 *   The first call on each device looks up the array's device address (no allocation); make that
 *   first call outside any stream capture.
 *   The call itself performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *   All calls share the one array and it keeps whatever the previous call left there.  Nothing in it
 *   needs to start at zero: each call writes every partial it later reads.  Two calls whose kernels
 *   may overlap on the GPU (different streams, no dependency between them) race on the array --
 *   order them on one stream or with events.
 */
#define TDX_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
int tdx_gemm_splitk_static(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha,
                           const void* A, const void* B, void* C, int tile_n, int split_k, void* stream);

/*
 * Self-test of the bounds-checked debug mode: runs the one-thread-per-output GEMM kernel on a small scratch problem with
 * the extent of one operand understated by four elements.  The kernel must skip exactly those accesses (nothing out of
 * range is touched: the buffers are full size) and record the violation, so the next tdx_check_device_status on that
 * stream reports TDX_ERR_BOUNDS (once).  Allocates and frees a few KB of device memory.
 */
int tdx_selftest_bounds_check(void* stream);

/*
 * Self-test of the failure path: launches a one-warp kernel that waits on a barrier nothing ever signals, with a
 * wait limit of about `limit_us` microseconds (1 .. 100000).  The wait gives up, records its code in the device
 * status word and the kernel returns normally -- nothing traps or hangs, the context stays usable.  The next
 * tdx_check_device_status on that stream therefore reports TDX_ERR_TIMEOUT (once).  This is how the error model
 * of the paper's Section 3 (a definite error is reported, not swallowed) is exercised without faulting a device.
 */
int tdx_selftest_bounded_wait(int limit_us, void* stream);

/* Number of kernels this library has launched in this process (all threads). */
int64_t tdx_kernel_launch_count(void);

const char* tdx_last_error(void);
const char* tdx_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TDX_H_ */
