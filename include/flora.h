/*
 * flora.h — C ABI of the Flora hot path for NVIDIA B200 (sm_100a).
 *
 * Flora (arXiv 2402.03293) keeps, for every 2-D weight W (n x m), an n x r
 * sketch of its gradients instead of an n x m buffer.  The sketch is made with
 * a Gaussian projection A (r x m, i.i.d. N(0, 1/r)) that is never kept: it is
 * regenerated from a 64-bit seed wherever it is needed (Section 2.4, "Memory
 * analysis").  This library provides the device operations of Algorithm 1
 * (gradient accumulation) and Algorithm 2 (momentum):
 *
 *      compress      C <- C + G A^T                     Algorithm 1, "Compression"
 *      decompress    W <- W - lr*scale * (C A)          Algorithm 1, "Decompression"; Algorithm 2, "yield M A'"
 *      momentum      M <- beta M + (1-beta) G A^T       Algorithm 2, update of M
 *      transfer      M <- M A_old A_new^T               Algorithm 2, resampling branch; Section 2.4
 *
 * GENERAL CONVENTIONS
 *  - Every matrix is row-major with a leading dimension `ld` counted in
 *    elements (ld >= cols).  `data` is a DEVICE pointer that the caller owns;
 *    the library never frees, reallocates or keeps it beyond the call (a
 *    flora_set keeps the pointers it was created with until it is destroyed).
 *  - G and W may be FLORA_F32 or FLORA_BF16; the sketches C and M are always
 *    FLORA_F32.  The dtype of G / W also fixes the precision of the projection
 *    as the contraction sees it: fp32 values of A for FLORA_F32, those values
 *    rounded to bf16 (nearest even) for FLORA_BF16.  Products are accumulated
 *    in fp32.
 *  - The rank r is the column count of the sketch, 1 <= r <= 256.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *    Calls are asynchronous: they enqueue work on `stream` and return; they
 *    do not synchronise the device.  One exception: the first single-matrix
 *    call that meets a new (operation, addresses, shape, rank) on the
 *    tensor-core path builds its plan (work split, TMA descriptors, a few KB
 *    of device tables, for ranks above 64 a bf16 copy of the sketch for the
 *    decompression) with a device allocation and a synchronisation of
 *    `stream`; the 32 most recent plans are kept, so a training loop pays
 *    this once per matrix.  flora_set_* calls never do: a set is planned
 *    when it is created.
 *  - Stream capture: the set-level transfers (flora_set_resample_transfer,
 *    flora_set_transfer_axpby, flora_set_momentum_step_resampled),
 *    flora_set_rebind_gradients and a single-matrix call that plans upload
 *    small tables from ordinary host memory that the call does not keep;
 *    do not record these into a CUDA graph.
 *  - Errors are reported by the returned status only; arguments are checked
 *    before anything is launched, and a failed check launches nothing.
 *  - A[j,k] depends on (seed, j, k) only and on r only through the factor
 *    1/sqrt(r): Philox4x32-10 with key = (low, high) half of the seed and
 *    counter (k/4, j, 0, 0) yields four 32-bit words; words (0,1) give columns
 *    4*(k/4)+0 and +1 by the Box-Muller transform (cosine, sine branch), words
 *    (2,3) give columns +2 and +3.  The transform uses fixed polynomials so
 *    that a CPU implementation can reproduce every bit.
 */
#ifndef FLORA_H
#define FLORA_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FLORA_OK = 0,
    FLORA_ERR_NULL = 1,        /* a required pointer is NULL                              */
    FLORA_ERR_SHAPE = 2,       /* negative / inconsistent rows, cols or ld                */
    FLORA_ERR_DTYPE = 3,       /* dtype not allowed for this argument                     */
    FLORA_ERR_ALIGN = 4,       /* pointer or ld not aligned to the element size           */
    FLORA_ERR_RANK = 5,        /* r outside 1..256 or inconsistent between arguments      */
    FLORA_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed                     */
    FLORA_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired (flora_device_status) */
    FLORA_ERR_UNSUPPORTED = 8, /* valid arguments, but no kernel covers them              */
    FLORA_ERR_ALLOC = 9        /* a scratch allocation failed                             */
} flora_status;

typedef enum { FLORA_F32 = 0, FLORA_BF16 = 1 } flora_dtype;

/* A borrowed view of a row-major device matrix. */
typedef struct {
    void*   data;   /* device pointer, aligned to the element size (16 bytes to reach the tensor-core kernels) */
    int64_t rows;
    int64_t cols;
    int64_t ld;     /* elements between consecutive rows, >= cols                                          */
    int32_t dtype;  /* flora_dtype                                                                         */
} flora_mat;

/* ---------------------------------------------------------------------------------------------
 * Single-matrix operations.
 * ------------------------------------------------------------------------------------------- */

/* Algorithm 1, compression step:  C <- C + G A(seed)^T.
 * G: n x m (f32 | bf16), read once.  C: n x r f32, read and written.  `r` must equal C->cols
 * (FLORA_ERR_RANK otherwise).  Empty matrices (n == 0 or m == 0) are accepted and do nothing. */
flora_status flora_compress_accumulate(const flora_mat* G, flora_mat* C, uint64_t seed, int r, void* stream);

/* Algorithm 1, reconstruction, fused with the parameter update:  W <- W - lr*scale*(C A(seed)).
 * The paper returns G~ = scale * C A and hands it to the optimizer; `scale` is 1/tau for an
 * accumulation cycle (the arithmetic mean of Section 2.4) and 1 for Algorithm 2's M A'.
 * W: n x m (f32 | bf16), read and written once.  C: n x r f32, only read: the caller zeroes it
 * and draws a new seed when a cycle ends (Section 2.4). */
flora_status flora_decompress_apply(flora_mat* W, const flora_mat* C, uint64_t seed, float lr, float scale, void* stream);

/* Algorithm 2, momentum update:  M <- beta M + (1-beta) G A(seed)^T.   Shapes as for compression.
 * With beta == 0 the old contents of M are neither read nor blended in (they may be uninitialised, NaN included):
 * M <- G A(seed)^T.  That is also the first compression of an accumulation cycle of Algorithm 1 with its
 * "C <- 0" folded in. */
flora_status flora_momentum_step(const flora_mat* G, flora_mat* M, float beta, uint64_t seed, void* stream);

/* Algorithm 2, resampling branch:  M <- M A(seed_old) A(seed_new)^T, evaluated as M (A_old A_new^T).
 * M: n x r f32, in place.  `m` is the column count of the weight matrix (A is r x m) and
 * `operand` the dtype of the gradients that were compressed into M (it fixes the precision of A).
 * Uses r*r floats of scratch taken from a stream-ordered memory pool that the library owns (one per device,
 * created at the first such call) and returned to it before the call returns; FLORA_ERR_ALLOC if that fails. */
flora_status flora_resample_transfer(flora_mat* M, int64_t m, int32_t operand, uint64_t seed_old, uint64_t seed_new, void* stream);

/* Algorithm 2 at a step where the projection is resampled, as one call:
 *      M <- beta * (M A(seed_old) A(seed_new)^T) + (1 - beta) * G A(seed_new)^T.
 * Equal (up to rounding order) to flora_resample_transfer followed by flora_momentum_step with seed_new, but the
 * factor beta rides on the transfer's last pass over M and the compression then only adds: M is read and written
 * once less.  G: n x m (f32 or bf16), M: n x r f32, in place.  Scratch and errors as for flora_resample_transfer. */
flora_status flora_momentum_step_resampled(const flora_mat* G, flora_mat* M, float beta, uint64_t seed_old, uint64_t seed_new, void* stream);

/* The same operation as flora_resample_transfer for callers that must not allocate.  (The paper has no
 * counterpart to this call: it is a packaging of Algorithm 2's transfer for a constrained caller.)
 *
 * flora_resample_transfer borrows its r x r scratch from a stream-ordered allocation.  That is unusable for code that
 * runs after all device memory has been handed out (an inference or training process whose memory plan is
 * fixed up front and which treats any later allocation as a failure), for code that may not touch the
 * allocator at all at this point (a latency-critical loop, a thread that does not own the memory pool), and
 * wherever an allocation call could block or fail at an inconvenient time.  This variant calls neither
 * cudaMalloc / cudaFree nor their stream-ordered forms, nor any library routine that allocates: its scratch
 * is a fixed array of 256 x 256 floats (256 KB) inside the library image, so every GPU on which the library
 * is used holds those 256 KB until the process exits, whether or not this call is ever made.
 *
 *  - Limit: r = M->cols <= 256 (the scratch size); a larger r returns FLORA_ERR_RANK and launches nothing.
 *  - The first call on each device looks up the device address of the array (cudaGetSymbolAddress, with
 *    that device current); make that first call outside any stream capture.  Later calls only launch.
 *  - All calls on a device share the one array, and it keeps what the last call left in it.  The call clears
 *    it first (a memset on `stream`), so back-to-back calls on one stream are fine; two calls that may run
 *    concurrently on the same GPU (different streams, different threads) race on the array and must be
 *    serialised by the caller.
 * Arguments, result and error codes are otherwise those of flora_resample_transfer. */
flora_status flora_resample_transfer_static(flora_mat* M, int64_t m, int32_t operand, uint64_t seed_old, uint64_t seed_new, void* stream);

/* dst <- b dst + a src A(seed_old) A(seed_new)^T.  With a = (1-beta)/tau, b = beta this feeds the
 * output of Algorithm 1 (G~ = C A_acc / tau) into the update of Algorithm 2 without forming G~.
 * dst, src: n x r f32; they may be the same matrix.  Scratch as for flora_resample_transfer. */
flora_status flora_transfer_axpby(flora_mat* dst, const flora_mat* src, int64_t m, int32_t operand,
                                  uint64_t seed_old, uint64_t seed_new, float a, float b, void* stream);

/* Test hook: writes A(seed) itself, r x m with r = out->rows, as f32 or as bf16 (rounded to
 * nearest even).  Exists so that the generator can be compared bit by bit with a CPU
 * implementation; no operation above ever stores A. */
flora_status flora_materialize_A(flora_mat* out, uint64_t seed, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Weight sets: the same operations over many matrices in one launch each (Algorithms 1 and 2
 * loop "for W in the weight set").  A set records, once, the matrices of a model and the work
 * decomposition and TMA descriptors derived from them; the per-step calls then only launch.
 * ------------------------------------------------------------------------------------------- */
typedef struct flora_set flora_set;

/* count matrices; G[i] and W[i] are n_i x m_i with equal shape and dtype, S[i] (the sketch C or
 * M) is n_i x r f32 with the same r for all i.  W may be NULL if flora_set_decompress_apply is
 * never called, G may be NULL if no compression is.  Allocates a few hundred bytes of device
 * memory per matrix (descriptors and work lists) that flora_set_destroy frees.  The arrays
 * themselves are host memory and are copied. */
flora_status flora_set_create(int count, const flora_mat* G, const flora_mat* W, const flora_mat* S, flora_set** out);
flora_status flora_set_destroy(flora_set* set);

/* Re-point the gradient matrices of a set (same shapes, dtypes and leading dimensions).  The update of
 * the device-side descriptors is enqueued on `stream`: it is ordered after the set's earlier launches on
 * that stream and before its later ones.  */
flora_status flora_set_rebind_gradients(flora_set* set, const flora_mat* G, void* stream);

/* seeds: host array of `count` 64-bit seeds, one per matrix (copied before the call returns). */
flora_status flora_set_compress_accumulate(flora_set* set, const uint64_t* seeds, void* stream);
/* (beta == 0 overwrites the sketches, as for flora_momentum_step) */
flora_status flora_set_momentum_step(flora_set* set, float beta, const uint64_t* seeds, void* stream);
flora_status flora_set_decompress_apply(flora_set* set, const uint64_t* seeds, float lr, float scale, void* stream);
flora_status flora_set_resample_transfer(flora_set* set, const uint64_t* seeds_old, const uint64_t* seeds_new, void* stream);
/* flora_momentum_step_resampled for every matrix of the set (created with gradients). */
flora_status flora_set_momentum_step_resampled(flora_set* set, float beta, const uint64_t* seeds_old, const uint64_t* seeds_new, void* stream);
/* flora_transfer_axpby for every matrix of a set:  dst.S[i] <- b dst.S[i] + a src.S[i] A(seeds_old[i]) A(seeds_new[i])^T.
 * Feeds the accumulated sketches of Algorithm 1 (the set `src`, projections seeds_old) into the momentum of
 * Algorithm 2 (the set `dst`, projections seeds_new) with a = (1-beta)/tau, b = beta, in two launches for the
 * whole model.  Both sets hold the same number of matrices with equal row counts and the same rank
 * (FLORA_ERR_SHAPE otherwise); m_i and the operand dtype are taken from dst's G (or W).  src may be dst. */
flora_status flora_set_transfer_axpby(flora_set* dst, const flora_set* src, const uint64_t* seeds_old, const uint64_t* seeds_new,
                                      float a, float b, void* stream);
/* Sets every sketch of the set to zero (start of an accumulation cycle, Algorithm 1). */
flora_status flora_set_zero_state(flora_set* set, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Host sequencing helpers (Algorithm 1 / 2 bookkeeping; pure host functions).
 * ------------------------------------------------------------------------------------------- */

/* "an independent random seed" (Algorithms 1 and 2): a 64-bit mix of a base seed, the index of the
 * matrix and the resampling epoch (splitmix64 finaliser over base ^ matrix*phi ^ epoch*phi').     */
uint64_t flora_derive_seed(uint64_t base, uint64_t matrix, uint64_t epoch);
/* Algorithm 2: 1 if step t resamples the projection (t = 0 mod kappa), else 0; kappa <= 0 never. */
int flora_resamples_at(int64_t t, int64_t kappa);

/* ---------------------------------------------------------------------------------------------
 * End-to-end step with HOST gradients (what a data loader / offloaded backward pass would hand
 * over): copies G (host, ideally pinned) to the set's device gradient buffers, then compresses.
 * ------------------------------------------------------------------------------------------- */
/* Enqueues on `stream` the host->device copies of host_G[i] (n_i x m_i elements of the set's gradient dtype, densely
 * packed, ideally pinned) into the set's device gradient buffers; the next compression or momentum step of the
 * set on that stream then consumes them. */
flora_status flora_set_upload_gradients(flora_set* set, const void* const* host_G, void* stream);
/* host_G[i]: host pointer to n_i x m_i elements of the set's gradient dtype, densely packed
 * (ld = m_i).  Enqueues the host->device copies and the compression on `stream`.            */
flora_status flora_set_compress_accumulate_from_host(flora_set* set, const void* const* host_G,
                                                     const uint64_t* seeds, void* stream);
/* Enqueues device->host copies of every weight matrix of the set into host_W[i] (dense, ld = m_i). */
flora_status flora_set_read_weights_to_host(flora_set* set, void* const* host_W, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Reproducibility.
 * ------------------------------------------------------------------------------------------- */
/* A is a function of (seed, j, k) alone, so every result is reproducible up to the order of floating-point
 * additions.  By default the work of one matrix may be split over CTAs that add their partial sums in arrival
 * order (compression over column ranges of a wide matrix; the r x r product of the transfer over column ranges),
 * which can change the last bits from run to run.  on != 0: sets created from now on give every row of a sketch a
 * single owner, and every transfer from now on sums its r x r product in one CTA per matrix, so that repeated runs
 * on the same inputs are bit-identical (slower on few, wide matrices).  Process-wide; default off. */
void flora_set_deterministic(int on);

/* ---------------------------------------------------------------------------------------------
 * Diagnostics.
 * ------------------------------------------------------------------------------------------- */
/* Test hook: 0 = choose the kernel automatically (tensor-core kernels when dtype, alignment and
 * rank allow), 1 = always the plain fp32 SIMT kernels.  Process-wide. */
void flora_debug_force_path(int path);

/* Test hook for the host-side work decomposition of the tensor-core kernels (no kernel is launched; works without a
 * GPU, in which case 148 SMs and an unconstrained cluster residency are assumed).  `rows`/`cols`: the shapes of
 * `count` bf16 matrices; `r`: the rank.  which = 0: the compression kernel; items are 6 x int32 {matrix, first row,
 * 128-row tiles, first 64-column step, steps, owns-its-rows flag}; params (8 x int32) = {tiles per CTA T, cluster
 * size S, G stages, A stages, generator warps, teams, launches, shared memory bytes}.  which = 1: the decompression
 * kernel; items are 4 x int32 {matrix, first column, first row, 128-row tiles}; params = {slab width bn, W slots,
 * S chunk stages, slab buffers, generator warps, bf16-sketch flag, launches, shared memory bytes}.  At most
 * `capacity` items are written (host memory, caller-owned); *n_items receives the full count. */
flora_status flora_debug_plan(const int64_t* rows, const int64_t* cols, int64_t count, int32_t r, int32_t which, int32_t* items, int64_t capacity,
                              int64_t* n_items, int32_t* params);
/* Kernels launched by this library since load (your own count of launches). */
uint64_t flora_launch_count(void);
/* Reads (synchronously, with a device->host copy) and clears the device-side error word that
 * bounded waits inside the kernels set when they give up: FLORA_OK or FLORA_ERR_TIMEOUT. */
flora_status flora_device_status(void);
/* Test hook for the bounded device-side waits: launches one small kernel whose only wait (limit 1 ms) can
 * never be satisfied, synchronises `stream` and returns FLORA_ERR_TIMEOUT if the wait gave up as designed
 * (FLORA_OK would mean it did not).  The device error word is raised as by a real timeout, so the next
 * flora_device_status() also reports FLORA_ERR_TIMEOUT, once.  The context stays usable. */
flora_status flora_debug_wait_timeout_selftest(void* stream);
const char* flora_status_string(flora_status s);
int flora_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FLORA_H */
