/*
 * wht_affine.h -- C ABI of the B200 (sm_100a) Walsh-Hadamard head-mixing library.
 *
 * The operation is the paper's replacement for the dense attention output
 * projection (Eq. 1):
 *
 *     y[t, :] = a (.) ( x[t, :] H_d ) / sqrt(d) + b          for every row t < T
 *
 * H_d is the d x d Walsh-Hadamard matrix in Sylvester (natural) order,
 * H[i][j] = (-1)^popcount(i & j) -- the ordering of the 4x4 sign pattern printed
 * in Fig. 1 and of the in-place butterfly of Fig. 2 -- and the 1/sqrt(d) factor
 * makes it orthonormal (the condition H^T H = I stated under Eq. 1).  a and b are
 * the trainable per-channel scale and bias (alpha and beta in Eq. 1).
 *
 * Conventions common to every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller.  x, y, dy, dx
 *     are row-major contiguous [T x d] (row stride = d elements); a, b, da, db
 *     have d elements.  Every pointer must be 16-byte aligned.
 *   - d must be a power of two with 8 <= d <= 32768.  T >= 0; T == 0 is a no-op
 *     for the forward calls, and makes the backward call write zeros to da, db
 *     (the row tensors may then be NULL; a, b, da, db are always required).
 *   - `dtype` selects the storage types (wht_dtype below).  All arithmetic is
 *     fp32 whatever the storage type; bf16 outputs are rounded once, to nearest
 *     even, at the store.  One exception: in the tensor-core kernels (bf16 rows,
 *     512 <= d <= 8192) an fp32 intermediate that feeds a second +-1 product is
 *     narrowed on the way: to a bf16 pair hi + lo (16-17 significant bits instead
 *     of 24) in y of the mma.sync forward (variants 2 and 3) and in dx of the mma.sync
 *     backward, and in dx of the tcgen05 backward either to that pair or, by default,
 *     to one bf16 (see wht_affine_set_bwd_operand_mode).  Sums are fp32 throughout.
 *     The library's tests bound both effects against the 1e-2 * max|row| tolerance
 *     (test_bwd_bf16_operand_mode, test_outputs_are_the_correctly_rounded_values_almost_everywhere).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls are asynchronous: they enqueue work and return without synchronising.
 *   - Exact aliasing y == x and dx == dy is allowed (a row is read completely
 *     before it is written).  Any other overlap is undefined.
 *   - Return value: WHT_OK (0) or a negative wht_status.  On error nothing has
 *     been launched.  No exception crosses this boundary and no kernel traps.
 */
#ifndef WHT_AFFINE_H_
#define WHT_AFFINE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    WHT_F32 = 0,       /* x, y, dy, dx, a, b : float32                              */
    WHT_BF16 = 1,      /* x, y, dy, dx, a, b : bfloat16            (inference)      */
    WHT_BF16_PF32 = 2  /* x, y, dy, dx : bfloat16 ;  a, b : float32 (training)      */
} wht_dtype;           /* da and db are float32 for every dtype                      */

typedef enum {
    WHT_OK = 0,
    WHT_ERR_NULL = -1,        /* a required pointer is NULL                          */
    WHT_ERR_BAD_DIM = -2,     /* d is not a power of two in [8, 32768]               */
    WHT_ERR_BAD_T = -3,       /* T < 0                                               */
    WHT_ERR_BAD_DTYPE = -4,   /* dtype is not a wht_dtype                            */
    WHT_ERR_MISALIGNED = -5,  /* a pointer is not 16-byte aligned                    */
    WHT_ERR_WORKSPACE = -6,   /* workspace missing, too small, or allocation failed  */
    WHT_ERR_CUDA = -7,        /* a CUDA runtime call failed; see wht_affine_last_cuda_error */
    WHT_ERR_BAD_VARIANT = -8, /* unknown kernel variant id                           */
    WHT_ERR_DEVICE_WAIT = -9, /* a kernel's bounded wait (copy, product, hand-over) expired */
    WHT_ERR_GUARD = -10       /* debug build only: a kernel wrote outside an output or scratch buffer */
} wht_status;

/*
 * Forward pass (Eq. 1): y = a (.) (x H_d)/sqrt(d) + b on T rows.
 *   x [T x d] in, a [d] in, b [d] in, y [T x d] out.  Reads x once, writes y once.
 */
int wht_affine_fwd(const void* x, const void* a, const void* b, void* y,
                   int64_t T, int32_t d, int dtype, void* stream);

/*
 * Forward pass fused with the residual connection that follows the attention block
 * (the paper's Sec. 3 motivation: the projection's output feeds that connection):
 *     y[t, :] = resid[t, :] + a (.) (x[t, :] H_d)/sqrt(d) + b
 * resid [T x d] has the layout and storage type of x.  The sum is taken in fp32 and
 * rounded once at the store.  y may alias resid or x exactly.  One kernel: reads x and
 * resid once, writes y once (no separate add pass over HBM).  Its backward is that of
 * wht_affine_fwd plus the identity for resid (d resid = dy), so wht_affine_bwd serves.
 */
int wht_affine_fwd_residual(const void* x, const void* a, const void* b, const void* resid, void* y,
                            int64_t T, int32_t d, int dtype, void* stream);

/*
 * Forward pass tuned for a handful of rows (the decode regime of the paper's
 * inference benchmark: one new token per sequence).  Same arguments, semantics
 * and results as wht_affine_fwd; any T is legal, T <= 256 is what it is shaped
 * for.  Uses no workspace and makes no allocation.
 */
int wht_affine_fwd_decode(const void* x, const void* a, const void* b, void* y,
                          int64_t T, int32_t d, int dtype, void* stream);

/*
 * Backward pass of Eq. 1 (the paper states only its O(d log d) cost in the table
 * comparing the dense and Hadamard projections; the formulas are the chain rule
 * applied to Eq. 1, with z = (x H_d)/sqrt(d) recomputed from x):
 *     dx[t, :] = ( (a (.) dy[t, :]) H_d ) / sqrt(d)         (H is symmetric)
 *     da[j]    = sum_t dy[t, j] * z[t, j]
 *     db[j]    = sum_t dy[t, j]
 *   dy [T x d] in, x [T x d] in, a [d] in, dx [T x d] out, da [d] out, db [d] out.
 * da and db are OVERWRITTEN (not accumulated) and are float32.  The column sums
 * are taken in a fixed order, so results are bit-identical from run to run.
 *
 * This call uses a per-device scratch buffer owned by the library, allocated
 * with cudaMalloc on first use (and grown when a larger problem arrives), so the
 * first call for a given size synchronises and must not happen during stream
 * capture.  Concurrent backward calls on one device through this entry point
 * share that buffer and must be serialised by the caller; use wht_affine_bwd_ws
 * to give each call site its own.
 */
int wht_affine_bwd(const void* dy, const void* x, const void* a,
                   void* dx, float* da, float* db,
                   int64_t T, int32_t d, int dtype, void* stream);

/*
 * Backward pass with caller-owned scratch: identical results to wht_affine_bwd.
 * `workspace` is a 16-byte aligned device buffer of at least
 * wht_affine_bwd_workspace_bytes(T, d, dtype) bytes; its contents on entry are
 * ignored and undefined on exit.  Never allocates.
 */
int wht_affine_bwd_ws(const void* dy, const void* x, const void* a,
                      void* dx, float* da, float* db,
                      int64_t T, int32_t d, int dtype,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass for callers that must not allocate.  (The paper has no counterpart:
 * this entry point exists for the library's users, not for the method.)
 *
 * Some callers cannot let a library call cudaMalloc on their behalf: code running
 * inside a memory-pool or caching-allocator regime where every byte of device
 * memory is already spoken for, real-time or serving loops where an allocation
 * (which synchronises the device) would stall other streams, and set-ups that
 * forbid the call outright once initialisation is over.  wht_affine_bwd allocates
 * its scratch lazily and wht_affine_bwd_ws makes the caller find the memory; this
 * variant needs neither.  Its scratch is a fixed array compiled into the library's
 * device image, WHT_NOALLOC_SCRATCH_BYTES (16 MiB) large, which every GPU that
 * loads the library holds until the process exits.  Same arguments, semantics and
 * bit-identical results as wht_affine_bwd.
 *
 *   - Never calls cudaMalloc, cudaFree or any allocating routine.
 *   - A problem whose scratch need, wht_affine_bwd_workspace_bytes(T, d, dtype),
 *     exceeds WHT_NOALLOC_SCRATCH_BYTES is rejected with WHT_ERR_WORKSPACE and
 *     nothing is launched (on a 148-SM part every d <= 8192 fits for any T).
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress, no allocation) and caches it; make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one array.  The kernels overwrite every
 *     scratch word they later read, so nothing needs clearing between calls and
 *     stale contents from an earlier call are harmless; but two of these calls
 *     that overlap on the GPU (different streams, no ordering) race on it and
 *     give wrong da/db.  Serialise them, or use wht_affine_bwd_ws.
 */
#define WHT_NOALLOC_SCRATCH_BYTES (16u * 1024u * 1024u)
int wht_affine_bwd_noalloc(const void* dy, const void* x, const void* a,
                           void* dx, float* da, float* db,
                           int64_t T, int32_t d, int dtype, void* stream);

/*
 * Grouped (block-diagonal) form for model widths that are not a power of two, d = groups * block
 * with block a power of two in [8, 32768] (d = 768 = 3 * 256 and 1536 = 3 * 512 in the paper's model
 * table):
 *     y[t, g*block + j] = a[g*block + j] * ( x[t, g*block : (g+1)*block] H_block )[j] / sqrt(block)
 *                         + b[g*block + j]
 * i.e. Eq. 1 with H replaced by diag(H_block, ..., H_block); still orthonormal, mixes channels
 * within a group only.  The paper does not say what its implementation does at those widths, so this
 * is an explicit alternative of this library, not a claim about the paper's choice; groups = 1 is
 * exactly wht_affine_fwd / wht_affine_bwd.  Same layouts, storage types, aliasing and error rules as
 * the plain calls; rows are still contiguous [T x d].  One launch of the butterfly kernels, the
 * channel group being the second grid dimension.  The backward takes caller-owned scratch of at
 * least wht_affine_bwd_grouped_workspace_bytes(T, d, block, dtype) bytes and never allocates.
 */
int wht_affine_fwd_grouped(const void* x, const void* a, const void* b, void* y,
                           int64_t T, int32_t d, int32_t block, int dtype, void* stream);
int wht_affine_bwd_grouped(const void* dy, const void* x, const void* a,
                           void* dx, float* da, float* db,
                           int64_t T, int32_t d, int32_t block, int dtype,
                           void* workspace, size_t workspace_bytes, void* stream);
size_t wht_affine_bwd_grouped_workspace_bytes(int64_t T, int32_t d, int32_t block, int dtype);

/*
 * Column-sharded (tensor-parallel) form, for attention whose heads are split over g GPUs: rank s
 * holds channels [s*w, (s+1)*w) of every row, as a contiguous [T x w] tensor of its own, and the
 * model width is d = g * w.  The paper trains data-parallel only and has no such form; it follows
 * from Eq. 1 and the Kronecker structure of the Sylvester matrix, H_d = H_g (x) H_w:
 *     y_r  = a_r (.) ( (sum_s H_g[s][r] x_s) H_w ) / sqrt(d) + b_r,    H_g[s][r] = (-1)^popcount(s & r)
 *     dx_r = ( (sum_s H_g[r][s] (a_s (.) dy_s)) H_w ) / sqrt(d)
 *     da_r = sum_t dy_r (.) z_r,   z_r = ( (sum_s H_g[s][r] x_s) H_w ) / sqrt(d),     db_r = sum_t dy_r
 * which are exactly column block r of wht_affine_fwd / wht_affine_bwd on the concatenated tensors.
 * One kernel per call reads the g blocks (its own and the peers') with plain loads, forms the
 * signed sum of the stored values in fp32 and runs the width-w transform: the exchange of the top
 * log2 g stages and the local stages are fused, no intermediate is written.  Every load is one CTA's own.
 *   x_parts, dy_parts, a_parts  HOST arrays of g DEVICE pointers; entry s is rank s's block
 *                  (x, dy: [T x w] row-major; a: [w]); entry r is this GPU's own memory, the others
 *                  are peer mappings the caller obtained (CUDA IPC, symmetric memory) and keeps valid
 *                  and unchanged until the call has completed on `stream`.  The array itself is
 *                  read before the call returns.
 *   a, b           this rank's parameter blocks [w]; y, dx: this rank's output blocks [T x w];
 *                  da, db [w] fp32, overwritten.
 *   w              power of two in [8, 32768]; g in {1, 2, 4, 8}; 0 <= r < g; g = 1 is the plain call.
 *   Outputs must not alias any input block (other ranks read the inputs at the same time).
 * The call does not synchronise ranks: the caller makes sure every rank's inputs are complete before
 * any rank launches (a barrier across ranks on the host or stream), and that no rank overwrites its
 * inputs before every rank's call has completed.  Gradients of a and b need no reduction across the
 * g ranks (each rank owns its channels); across data-parallel replicas they add as usual.
 * Every storage type.  bf16 rows with 1024 <= w <= 4096: tcgen05 kernels (forward from T*w >= 4 Mi
 * elements, backward from 256 Ki and g >= 2): each source block's tile is bulk-copied into shared memory
 * and multiplied by H_128 into one accumulator, negated where the sign is -1; the backward also adds up
 * +-(a_s/sqrt d) (.) dy_s in registers as the blocks arrive, the rank's own block last.  Otherwise butterfly
 * kernels with multi-source loads.  The backward takes caller-owned scratch of at least
 * wht_affine_bwd_tp_workspace_bytes(T, w, g, dtype) bytes and never allocates; it honours
 * wht_affine_set_bwd_operand_mode.
 * Errors as for the plain calls; g or r out of range -> WHT_ERR_BAD_DIM.
 */
int wht_affine_fwd_tp(const void* const* x_parts, const void* a, const void* b, void* y,
                      int64_t T, int32_t w, int32_t g, int32_t r, int dtype, void* stream);
int wht_affine_bwd_tp(const void* const* dy_parts, const void* const* x_parts, const void* const* a_parts,
                      void* dx, float* da, float* db,
                      int64_t T, int32_t w, int32_t g, int32_t r, int dtype,
                      void* workspace, size_t workspace_bytes, void* stream);
size_t wht_affine_bwd_tp_workspace_bytes(int64_t T, int32_t w, int32_t g, int dtype);

/*
 * Sums the parameter gradients of n backward calls (row chunks of one batch, or micro-batches
 * whose gradients accumulate): da[j] = sum_p parts[p][0][j], db[j] = sum_p parts[p][1][j].
 * da and db of Eq. 1's backward are sums over rows, so the gradients of disjoint row sets add.
 *   parts [n x 2 x d] fp32 in: for each call its da (d values) then its db (d values);
 *   da [d], db [d] fp32 out (overwritten; zeros when n == 0).
 * The order of summation is fixed, so the result is bit-reproducible.  One small kernel.
 */
int wht_affine_reduce_grads(const float* parts, int32_t n, int32_t d, float* da, float* db, void* stream);

/* Scratch bytes wht_affine_bwd_ws needs on the current device (0 on bad arguments). */
size_t wht_affine_bwd_workspace_bytes(int64_t T, int32_t d, int dtype);

/*
 * Kernel family used by the compute calls (for A/B measurements):
 *   0 = automatic (default).  bf16 rows: the tcgen05 kernels when 1024 <= d <= 8192 and there is
 *       enough work for their 32 KiB tiles (forward: T*d >= 4 Mi elements, 8 Mi at d = 8192;
 *       backward: T*d >= 256 Ki); else the mma.sync kernels for 256 <= d <= 8192 (rows loaded
 *       directly when they are few or narrow, streamed through a shared-memory ring otherwise);
 *       butterfly otherwise.  fp32 rows: the streamed mma.sync kernels once T >= 32 rows per SM
 *       (forward: 1024 <= d <= 8192, backward: 256 <= d <= 4096), each
 *       fp32 operand of a pass carried as three bf16 terms, i.e. exactly; butterfly otherwise;
 *   1 = butterfly (registers + warp shuffles + shared memory), every d and dtype;
 *   2 = mma.sync tensor-core assisted with direct row loads (256 <= d <= 8192, every dtype);
 *   3 = mma.sync tensor-core assisted with streamed rows (the same range);
 *   4 = tcgen05: rows copied into shared memory as they are and multiplied by H_128 on the
 *       tensor core (accumulators in tensor memory), the rest in registers;
 *   5 = as 4, the backward with half-size products (H_64, two accumulators side by side in the
 *       lanes of tensor memory, one more register stage) where d <= 4096.
 * A variant that does not support the requested (d, dtype) falls back (5 -> 4 -> 3 -> 1).
 * Process-wide; not meant to be changed while calls are in flight.
 */
int wht_affine_set_variant(int variant);
int wht_affine_get_variant(void);

/*
 * How g = (a/sqrt(d)) (.) dy enters the second +-1 tensor-core product of the tcgen05 backward
 * (bf16 rows, 1024 <= d <= 8192; the other kernels ignore the setting).  The chain rule on Eq. 1
 * fixes dx = ((a (.) dy) H)/sqrt(d); the paper says of precision only "bfloat16 mixed precision"
 * (a framework implementation in that regime rounds a (.) dy, and every butterfly stage after it,
 * to bf16), so both modes are readings of it:
 *   0 = rounded to bf16 once (default): two products per tile.  Every one of the 128 terms of a
 *       product carries a 2^-9 rounding, so dx is off by about 1e-3 of a row's typical magnitude
 *       -- the size of the bf16 rounding of dx itself, and inside the 1e-2 * max|dx_row| bound of
 *       this library's tests even for spike-dominated rows -- but it is not the correctly rounded
 *       fp32 result.  In long runs the backward's speed is set by the board's power limit, i.e. by
 *       energy per row, and this mode needs a third less tensor-core work and less register and
 *       shared-memory work: measured 13 % faster sustained at d = 2048 and 11 % at d = 8192.
 *   1 = as a bf16 pair hi + lo: 16-17 significant bits, three products per tile; dx is then the
 *       fp32-accumulated result rounded once at the store, up to the 2^-17 of the pair.
 * da and db do not pass through g and are bit-identical in both modes.
 * Process-wide; not meant to be changed while calls are in flight.  Unknown mode -> WHT_ERR_BAD_VARIANT.
 */
int wht_affine_set_bwd_operand_mode(int mode);
int wht_affine_get_bwd_operand_mode(void);

/*
 * Bandwidth yardstick with the same access pattern as the forward pass: copies
 * T rows of d elements (element size from dtype) from src to dst.  Used only by
 * the benchmark to report a practical copy ceiling next to the kernels.
 */
int wht_copy_rows(const void* src, void* dst, int64_t T, int32_t d, int dtype, void* stream);

/*
 * The kernels that stream rows through shared memory (the tcgen05 family and the
 * streamed mma.sync family) wait for their async copies, tensor-core products and
 * hand-overs between warps with a bound; a wait that expires does not hang or trap, it sets a flag on the device and the launch's
 * results are invalid.  This call synchronises with the current device's work
 * (it copies the flag back), returns WHT_ERR_DEVICE_WAIT if the flag was set
 * since the last query and clears it, else WHT_OK.  Never expected in normal
 * operation; meant for tests and for debugging after a suspicious result.
 */
int wht_affine_device_status(void);

/*
 * Self-test of that failure path, for test suites (the paper has no counterpart).  Launches one small
 * CTA in which one thread waits, through the kernels' own bounded-wait routine, on a barrier that
 * nothing ever completes, with a limit of about `limit_us` microseconds (1 .. 1000000) instead of the
 * kernels' tenths of a second; a second warp waits on another such barrier with the kernels' long limit
 * and must leave through the CTA's abort flag.  Nothing traps and nothing can hang: every wait is
 * bounded by construction, and the kernel returns by itself after roughly `limit_us`.
 *   out3: DEVICE pointer to three 32-bit words, written by the kernel: [0] = 1 if the short wait ran
 *   out, [1] = 1 if the second warp left through the abort flag, [2] unused.
 * After the launch completes, wht_affine_device_status() returns WHT_ERR_DEVICE_WAIT once and WHT_OK
 * from then on, and the library works as before.
 */
int wht_affine_selftest_wait_expiry(uint32_t limit_us, unsigned int* out3, void* stream);

/*
 * Debug build (the paper has no counterpart).  The library can be compiled with -DWHT_DEBUG
 * (python -m paper_2603_08343_b200.build --debug -> libwht_affine_debug.so): the same kernels, but every
 * compute call then writes its outputs (y; dx, da, db) and its scratch into buffers of the library's own
 * that carry a 4 KiB guard region filled with a canary byte on either side.  After the kernels have run,
 * the call synchronises the stream, checks the guards and only then copies the results into the
 * caller's tensors; a guard that changed makes the call return WHT_ERR_GUARD.  This is the stand-in
 * for a memory checker where none can be run: an out-of-bounds WRITE next to an output is caught (reads
 * are not).  Such a build allocates, synchronises and copies on every call -- wht_affine_bwd_noalloc
 * included -- and is meant for test suites only.
 *   wht_affine_debug_build()            1 in a debug build, 0 in the regular one.
 *   wht_affine_debug_selftest_guard(k)  debug build: sets up a guarded buffer, writes its payload and,
 *                                       for k = 1 / 2, one byte just before / after it (inside the
 *                                       library's own allocation), and returns the verdict of the check:
 *                                       WHT_OK for k = 0, WHT_ERR_GUARD for k = 1, 2.  Regular build:
 *                                       WHT_ERR_BAD_VARIANT.
 */
int wht_affine_debug_build(void);
int wht_affine_debug_selftest_guard(int damage);

/*
 * Failure injection on the host, for test suites (the paper has no counterpart): the next `n`
 * allocations the library would make for itself (the scratch of wht_affine_bwd; the guarded buffers
 * of a debug build) fail as an out-of-memory answer of the allocator would, without the allocator
 * being called.  The failing call returns WHT_ERR_WORKSPACE before anything is
 * launched and leaves the caller's tensors and the library's state as they were; the call after the
 * n-th failure allocates normally.  n = 0 clears the setting; n < 0 -> WHT_ERR_BAD_VARIANT.
 * Returns the number of injected failures still pending before the call.  Process-wide.
 */
int wht_affine_test_fail_allocations(int n);

/* cudaError_t of the most recent failing CUDA call on this thread (0 if none). */
int wht_affine_last_cuda_error(void);

/* Human-readable name of a wht_status. */
const char* wht_affine_status_string(int status);

/* Frees the library-owned scratch buffers of all devices.  Safe to call twice. */
int wht_affine_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* WHT_AFFINE_H_ */
