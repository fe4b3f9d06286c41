/*
 * osdp.h -- C ABI of the operator-split linear layer for NVIDIA B200 (sm_100a).
 *
 * The operation is the paper's "Operator Splitting" (Section 3.3): a large MatMul operator
 * is cut into `slice granularity` slices that are processed one after another, and the
 * partial results are combined.  Here the operator is a linear layer
 *
 *      Y = act(X W^T + b)        X [M,K] tokens x in_features,  W [N,K] row-major,
 *      dX = G W,  dW = G^T X,  db = column sums of G,   G = dY (.) act'(X W^T + b)
 *
 * and k = k_split slices are taken along
 *      OSDP_SPLIT_OUT : the N rows of W (outputs Y, dW, db concatenate; dX is summed), or
 *      OSDP_SPLIT_RED : the K columns of W and X.  This is the split Section 3.3 describes: the
 *                       input is cut along its last dimension, the operator along the matching
 *                       one, and the slice products are added up.  Y is summed; dX, dW concatenate.
 * Slices are visited in ascending order and their products are added in fp32.  Where the sum is kept
 * between two slices depends on who owns the loop over the slices:
 *  - one slice per call (the *_slice entry points, the MLP block, OSDP_FLAG_SLICE_MAJOR): the whole
 *    operator is swept once per slice, and a summed output travels from slice to slice as an fp32
 *    running sum [rows x cols of that output] in the caller's workspace;
 *  - all slices in one call (default): the call walks the output in panels of one tile per CTA pair
 *    (up to 256 x 512 elements each, 148 SMs: about 38 MB of fp32 sums, which is the tensor memory of
 *    the whole GPU) and visits the slices in order inside a panel, so the running sum of a tile stays in
 *    tensor memory from its first slice to its last and never goes through global memory.  Same
 *    products, same ascending order per output element; no carry buffer.
 *
 * Slice rule (the paper gives none for non-divisible extents): slice length
 * L = ceil(D/k) rounded up to a multiple of 8 elements; slice s = [s*L, min(D,(s+1)*L)); a
 * k for which the last slice would be empty is rejected.  k_split 0 means 1 (the paper plots
 * "granularity 0" as no splitting).
 *
 * Conventions for every call
 *  - All tensor pointers are DEVICE pointers unless stated; they stay owned by the caller and
 *    must stay valid until the stream has passed the call.  No device memory is allocated or
 *    freed by any call.  Two things are created once per device at first use and kept until the
 *    process ends: each kernel variant's attributes (shared-memory size), and, by the first
 *    backward call that asks for dX and dW together (or the first osdp_split_mlp_bwd with weight
 *    gradients), two internal non-blocking streams and nine events.  Such a call forks its
 *    weight-gradient launches onto those streams and joins them back into `stream` before it
 *    returns to the caller's ordering; while it enqueues that fork / join section it holds a
 *    host-side lock, so concurrent callers on one device are serialised on the host for the
 *    few microseconds of enqueueing (the GPU work is not serialised).  Make the first call on a
 *    device outside any stream capture.  On the host, every thread that calls the library keeps a
 *    table of its most recent launches' prepared kernel parameters (encoded tensor maps, tile
 *    choice; about 0.4 MB per thread), so that a loop issuing the same calls step after step does
 *    not encode them again; it holds addresses and shapes only and never touches device memory.
 *  - bf16 tensors are row-major, 16-byte aligned; N and K must be multiples of 8.
 *  - W lives inside a flat bf16 parameter buffer `w_flat` at ELEMENT offset `w_offset`
 *    (multiple of 8); it is read in place through TMA descriptors, never copied or unflattened.
 *    dW is written at `dw_offset` of a flat gradient buffer `dw_flat` (bf16 or fp32 elements).
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default
 *    stream) and never synchronise, except osdp_read_device_status.
 *  - `ws` is scratch of at least osdp_split_linear_workspace_bytes(...) bytes, 256-byte
 *    aligned.  Its first word is a device status word (see osdp_read_device_status); the
 *    caller zeroes the first 256 bytes once after allocating it.
 *  - Return value: OSDP_OK or an error code; nothing is launched when an argument check
 *    fails.  Never aborts, never prints.
 */
#ifndef OSDP_H_
#define OSDP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define OSDP_VERSION 111

/* status codes */
#define OSDP_OK 0
#define OSDP_ERR_NULL_POINTER 1
#define OSDP_ERR_BAD_SHAPE 2          /* M, N or K <= 0, or too large for 32-bit tile coordinates */
#define OSDP_ERR_BAD_SPLIT 3          /* k < 0, empty slice, bad split_dim, slice_idx out of range */
#define OSDP_ERR_ALIGNMENT 4          /* pointer / offset not 16-byte aligned, N or K not a multiple of 8 */
#define OSDP_ERR_WORKSPACE_TOO_SMALL 5
#define OSDP_ERR_UNSUPPORTED 6        /* unknown activation, dtype or op */
#define OSDP_ERR_CUDA 7               /* a CUDA call failed; see osdp_last_cuda_error */
#define OSDP_ERR_DEVICE_TIMEOUT 8     /* a bounded device-side wait ran out (status word) */
#define OSDP_ERR_EXCEEDS_STATIC_SCRATCH 9 /* osdp_bias_grad_noalloc: ceil(M/1024) * N too large */
#define OSDP_ERR_SEARCH_LIMIT 10      /* osdp_plan_search: node budget spent; the plan returned is feasible, maybe not optimal */

#define OSDP_SPLIT_OUT 0
#define OSDP_SPLIT_RED 1

#define OSDP_ACT_NONE 0
#define OSDP_ACT_GELU_TANH 1
#define OSDP_ACT_GELU_ERF 2

#define OSDP_DTYPE_BF16 0
#define OSDP_DTYPE_FP32 1

#define OSDP_OP_LINEAR_FWD 0
#define OSDP_OP_LINEAR_BWD 1
#define OSDP_OP_MLP_FWD 2
#define OSDP_OP_MLP_BWD 3

#define OSDP_MAX_SPLIT 1024

/* flags (bitwise or) */
#define OSDP_FLAG_ACCUMULATE_DW 1   /* backward: dW += instead of dW = */
#define OSDP_FLAG_CARRY_BF16 2      /* summed output: keep the running sum in the bf16 output buffer itself
                                     * (slice 0 stores, later slices add in bf16) instead of an fp32 carry in the
                                     * workspace: no carry memory, half the carry traffic, two extra bf16 roundings
                                     * per slice (partial and sum).  Measured relative Frobenius error about
                                     * 1.8e-3 * sqrt(1 + (k+1)/2): within 5e-3 up to k = 8, beyond it for k >= 16.
                                     * Only without activation and without z_save. */
#define OSDP_FLAG_PAIR_SLICES 8     /* summed output, all-slices calls only: a tile accumulates the products of two
                                     * adjacent slices in one pass, so two slices are read at a time (what a
                                     * double-buffered slice gather holds anyway) and the running sum is carried
                                     * half as often.  Exact fp32, but not bit-identical to the unpaired result. */
#define OSDP_FLAG_SLICE_MAJOR 16    /* all-slices calls of a summed output: sweep the whole operator once per slice
                                     * (slice s of every output tile before slice s + 1 of any), the running sum
                                     * carried in fp32 through the workspace, exactly as a sequence of *_slice
                                     * calls does.  In a workspace query: include that carry, i.e. size the
                                     * workspace for the *_slice entry points (which accept and ignore the flag). */
#define OSDP_FLAG_RECOMPUTE 4       /* osdp_split_mlp_bwd: recompute the first layer's pre-activation slice by
                                     * slice instead of reading z1_saved (activation checkpointing). */

int osdp_version(void);
const char *osdp_status_string(int status);
/* The cudaError_t (as int) of the most recent failed CUDA call made by this library on the
 * calling thread, 0 if none. */
int osdp_last_cuda_error(void);

/* Section 3.3 step 1 (partition): [begin,end) of slice s of an extent D cut into k slices by
 * the slice rule above.  Host-only integer arithmetic.  OSDP_ERR_BAD_SPLIT if a slice is empty
 * or s is out of range. */
int osdp_slice_range(int64_t D, int k_split, int slice_idx, int64_t *begin, int64_t *end);

/* Section 3.3 states the memory effect of splitting as size(MatMul) / slice granularity: only one slice of
 * the operator and of its intermediates is live at a time.  This query makes that figure concrete.
 * Exact scratch bytes a call with these arguments uses (the "staging" figure).  For the linear
 * ops (M,N,K) are the layer's; for the MLP ops pass M = tokens, N = ffn, K = hidden.
 * The query assumes every optional output (dx, dbias, ...) is requested.  `flags` as for the call
 * (OSDP_FLAG_SLICE_MAJOR: sized for the *_slice entry points, i.e. with the fp32 carry of a summed
 * output; OSDP_FLAG_CARRY_BF16 removes that carry).  Host-only arithmetic.
 * Errors: NULL bytes, bad shape / split / activation / op / flags as for the call itself. */
int osdp_split_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int k_split, int split_dim,
                                      int act, int op, int flags, size_t *bytes);

/* Slice-granularity suggestion (the paper's Section 5 leaves "how to automatically suggest a
 * desirable slice granularity" as future work; this is the memory half of that question).
 * Returns in *k_split the smallest valid k in [1, max_k] for which the call's workspace
 * (osdp_split_linear_workspace_bytes with the same arguments) is at most budget_bytes: splitting
 * costs time (carry traffic, smaller launches), so the least splitting that fits is preferred.
 * OSDP_ERR_WORKSPACE_TOO_SMALL if no k up to max_k fits (e.g. a k-independent fp32 carry alone
 * exceeds the budget; OSDP_FLAG_CARRY_BF16 removes it).  Host-only arithmetic. */
int osdp_suggest_granularity(int64_t M, int64_t N, int64_t K, int split_dim, int act, int op, int flags,
                             size_t budget_bytes, int max_k, int *k_split);

/* Forward of all k slices (Section 3.3 steps 1-3: partition, process the slices one after another, add
 * the results).
 *   x [M,K] bf16; bias [N] fp32 or NULL; out [M,N] bf16 = act(X W^T + bias);
 *   z_save [M,N] bf16 or NULL: receives the pre-activation (what the backward needs when act != NONE).
 * OUT: slice s writes columns R_s of out.  RED: the slices' products are added in ascending order in fp32
 * (in tensor memory, tile by tile; with OSDP_FLAG_SLICE_MAJOR slice by slice over the whole operator with
 * the running sum in ws, or in `out` itself with OSDP_FLAG_CARRY_BF16); bias and activation are applied once.
 * flags: 0, OSDP_FLAG_SLICE_MAJOR, OSDP_FLAG_CARRY_BF16, OSDP_FLAG_PAIR_SLICES (the last two imply the
 * slice-major order: they are options of its carry). */
int osdp_split_linear_fwd(const void *x, const void *w_flat, int64_t w_offset, const float *bias,
                          int64_t M, int64_t N, int64_t K, int k_split, int split_dim, int act,
                          int flags, void *out, void *z_save, void *ws, size_t ws_bytes, void *stream);

/* One slice of the forward (Section 3.3 step 2: the slices are computed one after another):
 * lets a caller put other work between slices.  Slices must be issued in
 * ascending order on one stream with the same arguments and workspace: under RED slice 0
 * starts the carry and slice k-1 writes `out`.  The workspace must be sized with
 * OSDP_FLAG_SLICE_MAJOR in the query's flags (OSDP_ERR_WORKSPACE_TOO_SMALL otherwise). */
int osdp_split_linear_fwd_slice(const void *x, const void *w_flat, int64_t w_offset, const float *bias,
                                int64_t M, int64_t N, int64_t K, int k_split, int split_dim, int act,
                                int flags, int slice_idx, void *out, void *z_save, void *ws,
                                size_t ws_bytes, void *stream);

/* Backward of all k slices.  The paper states the forward only (Section 3.3) and leaves the backward to
 * automatic differentiation; differentiating  Y = act(sum_s X[:,C_s] W[:,C_s]^T + b)  (RED)  or
 * Y[:,R_s] = act(X W[R_s,:]^T + b[R_s])  (OUT)  slice by slice gives, with G = dY (.) act'(Z):
 *   OUT: dW[R_s,:] = G[:,R_s]^T X, db[R_s] = colsum G[:,R_s], dX = sum_s G[:,R_s] W[R_s,:]
 *   RED: dX[:,C_s] = G W[:,C_s], dW[:,C_s] = G^T X[:,C_s], db = colsum G
 * i.e. the split that concatenates in the forward sums in the backward and vice versa.
 *   dy [M,N] bf16; x [M,K] bf16; z_saved [M,N] bf16 (pre-activation; required iff act != NONE);
 *   dx [M,K] bf16 or NULL; dw_flat + dw_offset: dW [N,K] in dw_dtype (bf16 or fp32), NULL to skip;
 *   flags: OSDP_FLAG_ACCUMULATE_DW (dW += ... instead of dW = ...), OSDP_FLAG_CARRY_BF16 (dX's running
 *   sum in dx itself under OUT split), OSDP_FLAG_PAIR_SLICES (dX under OUT split);
 *   dbias [N] fp32 or NULL (always overwritten).
 *   flags also: OSDP_FLAG_SLICE_MAJOR (dX under OUT split swept slice by slice, fp32 carry in ws).
 * With an activation under OUT split the call stages G_s = dY[:,R_s] (.) act'(Z[:,R_s]) one slice at a
 * time (slice-sized staging) and therefore always runs slice-major with the fp32 carry of dX.
 * When both dx and dw_flat are given, the call runs dW and db on a stream of its own
 * next to dX, forked from and joined back into `stream` (see osdp_split_mlp_bwd for the rules of these
 * internal streams). */
int osdp_split_linear_bwd(const void *dy, const void *x, const void *w_flat, int64_t w_offset,
                          const void *z_saved, int64_t M, int64_t N, int64_t K, int k_split,
                          int split_dim, int act, void *dx, void *dw_flat, int64_t dw_offset,
                          int dw_dtype, int flags, float *dbias, void *ws, size_t ws_bytes,
                          void *stream);

/* One slice of the backward (the per-slice terms of the derivation above; Section 3.3 step 2 applied to
 * the backward); same ordering rule as osdp_split_linear_fwd_slice: under OUT slice 0 starts the carry
 * of dX and slice k-1 writes dx.  Under RED dbias is produced by slice 0.  The workspace must be sized
 * with OSDP_FLAG_SLICE_MAJOR in the query's flags. */
int osdp_split_linear_bwd_slice(const void *dy, const void *x, const void *w_flat, int64_t w_offset,
                                const void *z_saved, int64_t M, int64_t N, int64_t K, int k_split,
                                int split_dim, int act, int slice_idx, void *dx, void *dw_flat,
                                int64_t dw_offset, int dw_dtype, int flags, float *dbias,
                                void *ws, size_t ws_bytes, void *stream);

/* ---- fp8 (e4m3) operands.  The same split linear layer with X, W and dY stored as 8-bit floating point
 * (1 sign, 4 exponent, 3 mantissa bits, no infinities; value = scale * e4m3(byte), one fp32 scale per
 * tensor chosen by the caller).  The tensor cores multiply the e4m3 values exactly and accumulate in fp32;
 * `scale` (= scale_x * scale_w) multiplies the accumulator before bias / activation.  The paper's method is
 * agnostic of the number format; this variant runs the slices on tcgen05.mma.kind::f8f6f4 at twice the
 * bf16 rate.  x8 [M,K], w8_flat (W [N,K] at ELEMENT = byte offset w_offset), out / z_save bf16 as before.
 * N, K, w_offset and, for k > 1, the slice length ceil(D/k) rounded up to 8 must be multiples of 16
 * (OSDP_ERR_ALIGNMENT otherwise).  Workspace: osdp_split_linear_workspace_bytes, same figures.
 * flags as osdp_split_linear_fwd. */
int osdp_split_linear_fwd_f8(const void *x8, const void *w8_flat, int64_t w_offset, float scale,
                             const float *bias, int64_t M, int64_t N, int64_t K, int k_split,
                             int split_dim, int act, int flags, void *out, void *z_save, void *ws,
                             size_t ws_bytes, void *stream);

/* Backward with fp8 operands: dX = scale_dx * (dY8 W8) in bf16, dW = scale_dw * (dY8^T X8) in dw_dtype
 * (scale_dx = scale_dy * scale_w, scale_dw = scale_dy * scale_x).  No activation (dY itself is the fp8
 * operand) and no bias gradient; everything else as osdp_split_linear_bwd. */
int osdp_split_linear_bwd_f8(const void *dy8, const void *x8, const void *w8_flat, int64_t w_offset,
                             float scale_dx, float scale_dw, int64_t M, int64_t N, int64_t K,
                             int k_split, int split_dim, void *dx, void *dw_flat, int64_t dw_offset,
                             int dw_dtype, int flags, void *ws, size_t ws_bytes, void *stream);

/* ---- Slices of a sharded operator (Section 3.3, last part: with zero-redundancy data parallelism
 * only the slice being processed is gathered, so the gathered weights take size(W)/k instead of
 * size(W)).  The caller (one process per GPU) keeps 1/world of every slice, all-gathers slice s
 * into a staging buffer, runs the slice, and reduce-scatters the slice's weight gradient; the
 * three entry points below are the per-GPU part of that loop.  They communicate nothing.
 *
 * Shard layout of slice `slice_idx` (host only, no GPU needed).  A gathered slice is a compact
 * row-major matrix: OUT  W[R_s, :]  as [len(R_s), K], *ld = K;  RED  W[:, C_s]  as [N, len(C_s)],
 * *ld = len(C_s).  *slice_elems = its element count; every rank holds *shard_elems contiguous
 * elements of it (a multiple of 8; world * shard_elems >= slice_elems, the surplus is padding at
 * the end of the gathered buffer); *shard_offset = where the rank's part of this slice starts in the
 * rank's shard buffer (slices stored one after another).  slice_idx == k is allowed and returns
 * the shard buffer's total length in *shard_offset.  Any output pointer may be NULL. */
int osdp_zdp_shard_layout(int64_t N, int64_t K, int k_split, int split_dim, int world, int slice_idx,
                          int64_t *slice_elems, int64_t *shard_elems, int64_t *shard_offset,
                          int64_t *ld);

/* osdp_split_linear_fwd_slice with the slice's weights given as the gathered compact matrix
 * `w_slice` (device, bf16, 16-byte aligned, leading dimension ld_w >= the layout's *ld, a multiple of
 * 8) instead of a window of the flat buffer.  Everything else (x, bias, out, z_save, workspace,
 * ordering of the slices, flags 0 or OSDP_FLAG_CARRY_BF16) as in osdp_split_linear_fwd_slice;
 * outputs are bit-identical to that call's. */
int osdp_zdp_linear_fwd_slice(const void *x, const void *w_slice, int64_t ld_w, const float *bias,
                              int64_t M, int64_t N, int64_t K, int k_split, int split_dim, int act,
                              int flags, int slice_idx, void *out, void *z_save, void *ws,
                              size_t ws_bytes, void *stream);

/* osdp_split_linear_bwd_slice with gathered weights `w_slice` (as above) and the slice's weight
 * gradient written to the compact matrix `dw_slice` (same shape as the gathered slice, leading
 * dimension ld_dw, dtype dw_dtype; NULL to skip), ready to be reduce-scattered.  dx, dbias, z_saved,
 * flags (OSDP_FLAG_ACCUMULATE_DW, OSDP_FLAG_CARRY_BF16) as in osdp_split_linear_bwd_slice. */
int osdp_zdp_linear_bwd_slice(const void *dy, const void *x, const void *w_slice, int64_t ld_w,
                              const void *z_saved, int64_t M, int64_t N, int64_t K, int k_split,
                              int split_dim, int act, int slice_idx, void *dx, void *dw_slice,
                              int64_t ld_dw, int dw_dtype, int flags, float *dbias, void *ws,
                              size_t ws_bytes, void *stream);

/* osdp_zdp_linear_bwd_slice with the reduce-scatter of the slice's weight gradient done by the GEMM's
 * epilogue (compute step and collective in one kernel): instead of writing dW_s to a staging matrix, every
 * 32-row box of it is reduce-added (TMA reduce-add, fp32 or bf16 per dw_dtype) directly into the buffer of the
 * rank that owns those rows.  `dw_peers` is a HOST array of `world` (<= 8) DEVICE pointers; dw_peers[q] is
 * where rank q keeps its part of this slice (shard_elems elements, the layout of osdp_zdp_shard_layout) -- this
 * rank's own memory for q = rank, peer-mapped memory of the other GPUs otherwise (plain peer stores /
 * reductions over NVLink; no multicast).  Every rank's call adds its term, so the buffers hold the sum over
 * ranks once all ranks have finished the slice: every rank zeroes its buffer, the ranks synchronise (nobody
 * may add into a buffer its owner has not zeroed yet), the calls run, the ranks synchronise again, and only
 * then are the buffers read.  Needs the slice's row count (len R_s under OUT, N under RED) to be a multiple of 32 * world,
 * else OSDP_ERR_UNSUPPORTED (use the staging form and a collective for that slice).  OSDP_FLAG_ACCUMULATE_DW
 * is not accepted (the scatter always adds).  Everything else as osdp_zdp_linear_bwd_slice. */
int osdp_zdp_linear_bwd_slice_scatter(const void *dy, const void *x, const void *w_slice, int64_t ld_w,
                                      const void *z_saved, int64_t M, int64_t N, int64_t K, int k_split,
                                      int split_dim, int act, int slice_idx, void *dx,
                                      void *const *dw_peers, int world, int dw_dtype, int flags,
                                      float *dbias, void *ws, size_t ws_bytes, void *stream);

/* One slice of the split MLP block (below) of a sharded operator pair: W1[F_s,:] and W2[:,F_s] are given as
 * the gathered compact matrices w1_slice [len F_s, hidden] (contiguous rows) and w2_slice [hidden, len F_s]
 * (leading dimension ld_w2 >= len F_s, a multiple of 8).  b1 [ffn], z1_save [M,ffn], out, workspace, flags and
 * the ordering of the slices as in osdp_split_mlp_fwd, whose per-slice work this is, bit for bit. */
int osdp_zdp_mlp_fwd_slice(const void *x, const void *w1_slice, const void *w2_slice, int64_t ld_w2,
                           const float *b1, const float *b2, int64_t M, int64_t hidden, int64_t ffn,
                           int k_split, int act, int flags, int slice_idx, void *out, void *z1_save,
                           void *ws, size_t ws_bytes, void *stream);

/* One slice of osdp_split_mlp_bwd with gathered compact weights.  The slice's weight gradients go either
 * to compact matrices dw1_slice [len F_s, hidden] and dw2_slice [hidden, len F_s] (leading dimension
 * ld_dw2), both or neither, ready for a reduce-scatter; or, when dw1_peers / dw2_peers (HOST arrays of `world`
 * DEVICE pointers, both or neither) are given, straight into the owning ranks' shards from the GEMMs'
 * epilogues, as in osdp_zdp_linear_bwd_slice_scatter (row counts len F_s and hidden must both be multiples
 * of 32 * world).  db1 [ffn] receives the slice's part, db2 [hidden] is written by slice 0. */
int osdp_zdp_mlp_bwd_slice(const void *dy, const void *x, const void *w1_slice, const void *w2_slice,
                           int64_t ld_w2, const float *b1, const void *z1_saved, int64_t M, int64_t hidden,
                           int64_t ffn, int k_split, int act, int slice_idx, void *dx, void *dw1_slice,
                           void *dw2_slice, int64_t ld_dw2, void *const *dw1_peers, void *const *dw2_peers,
                           int world, int dw_dtype, int flags, float *db1, float *db2, void *ws,
                           size_t ws_bytes, void *stream);

/* Transformer MLP block split along the ffn dimension (first layer OUT-split + activation,
 * second layer RED-split, Section 3.3 applied to both MatMuls of the block):
 *   out [M,hidden] = sum_s act(X W1[F_s,:]^T + b1[F_s]) W2[:,F_s]^T + b2, slice by slice.
 * W1 [ffn,hidden] at off_w1 and W2 [hidden,ffn] at off_w2 of the same flat buffer; b1 [ffn],
 * b2 [hidden] fp32 or NULL.  Only a slice-sized intermediate A_s [M, ffn/k] lives in ws.
 * z1_save [M,ffn] bf16 or NULL receives the first layer's pre-activation for the backward. */
int osdp_split_mlp_fwd(const void *x, const void *w_flat, int64_t off_w1, const float *b1,
                       int64_t off_w2, const float *b2, int64_t M, int64_t hidden, int64_t ffn,
                       int k_split, int act, int flags, void *out, void *z1_save, void *ws,
                       size_t ws_bytes, void *stream);

/* Backward of the split MLP block, slice by slice, from the saved pre-activation z1_saved
 * [M,ffn] bf16:  dA_s = dY W2[:,F_s]; dZ_s = dA_s (.) act'(Z1_s); dW2[:,F_s] = dY^T act(Z1_s);
 * dW1[F_s,:] = dZ_s^T X; db1[F_s] = colsum dZ_s; dX = sum_s dZ_s W1[F_s,:]; db2 = colsum dY.
 * dW1/dW2 land at dw_off_w1/dw_off_w2 of dw_flat (dw_dtype).  Slice-sized dZ_s and A_s live in ws: one set
 * of them, or two sets used in turn when k > 2 and a slice is small (ceil(M/256) * ceil(L/256) <= 74, L the
 * slice length: each GEMM of a slice is then at most one wave of tiles and the call is bound by the latency of
 * its kernel chain).  With two sets a slice's weight-gradient GEMMs need not finish before the next slice
 * starts, only before the slice after that; the staging is still ~ 1/k, and
 * osdp_split_linear_workspace_bytes reports it.
 * With OSDP_FLAG_RECOMPUTE (the paper's Section 2.3 setting, activation checkpointing) z1_saved is
 * not read (may be NULL): Z1_s = X W1[F_s,:]^T + b1[F_s] is recomputed per slice (one more GEMM,
 * one more slice-sized buffer), so that no [M,ffn] activation exists between forward and backward.
 * dX, dW1, db1 are bit-identical to the saved-activation path; dW2 = dY^T act(Z1_s) uses the
 * activation of the unrounded pre-activation, as the forward did.  b1 [ffn] fp32 or NULL is only
 * read then.
 * When weight gradients are wanted the call runs each slice's two weight-gradient GEMMs
 * on two streams of its own next to the dX GEMM: it forks from `stream` with an event and joins back
 * into `stream` before the next slice (with two sets of slice buffers: before the slice after the next, and
 * at the end of the call), so the caller still sees one ordered call (a stream capture
 * follows the fork).  The two streams and nine events per device are created by the first such call;
 * such calls on one device are serialised on the host while they enqueue. */
int osdp_split_mlp_bwd(const void *dy, const void *x, const void *w_flat, int64_t off_w1, const float *b1,
                       int64_t off_w2, const void *z1_saved, int64_t M, int64_t hidden, int64_t ffn,
                       int k_split, int act, void *dx, void *dw_flat, int64_t dw_off_w1,
                       int64_t dw_off_w2, int dw_dtype, int flags, float *db1, float *db2,
                       void *ws, size_t ws_bytes, void *stream);

/* Failure detection (no counterpart in the paper, which does not discuss faults: the slices of Section
 * 3.3 "executed sequentially" are pipelines of asynchronous copies and tensor-core work whose stages
 * wait on one another, and every such wait here is bounded).  Synchronises `stream`, copies the device
 * status word at the start of `ws` to *status (OSDP_OK, or OSDP_ERR_DEVICE_TIMEOUT if a bounded wait
 * inside a kernel ran out) and clears it.  Every device-side wait in this library is bounded; none can
 * hang the GPU.  This is the one call that synchronises. */
int osdp_read_device_status(void *ws, int *status, void *stream);

/* Diagnostic for the failure-detection path (no counterpart in the paper): launches one warp that
 * waits, with the bounded wait every kernel of this library uses, on a barrier nothing signals.
 * After `limit_us` microseconds (1 .. 1 000 000) the wait gives up, the status word at the start of
 * `ws` is set, and the kernel returns; osdp_read_device_status then reports
 * OSDP_ERR_DEVICE_TIMEOUT.  The GPU context stays usable.  Asynchronous on `stream`. */
int osdp_debug_wait_probe(void *ws, int64_t limit_us, void *stream);

/* Bias gradient for callers that cannot allocate.  (The paper has no counterpart: it is an
 * addition for users of this library.)
 *
 * Computes dbias[n] = sum over m of dy[m,n] -- the same result, bit for bit, as
 * osdp_split_linear_bwd(..., act = OSDP_ACT_NONE, dx = NULL, dw_flat = NULL, dbias) -- without a
 * workspace argument and without calling cudaMalloc, cudaFree or any allocating routine.  It is
 * meant for code that runs where device allocation is forbidden or impossible: inside an
 * allocator or memory-pool callback, in a plug-in whose host application owns all device memory
 * after start-up, in a latency-critical loop that must never wait on the allocator.
 *
 * The partial sums live in a 4 MiB array built into the library image
 * (OSDP_NOALLOC_MAX_PARTIALS floats); every GPU on which the library is loaded holds it until
 * the process exits.  Limit: ceil(M/1024) * N <= OSDP_NOALLOC_MAX_PARTIALS and ceil(M/1024) <= 65535,
 * else OSDP_ERR_EXCEEDS_STATIC_SCRATCH and nothing is launched.
 *
 *   dy [M,N] bf16 device, row-major, 16-byte aligned, N a multiple of 8; dbias [N] fp32 device.
 *   Asynchronous on `stream`; caller keeps the buffers alive until the stream has passed it.
 *
 * The first call on each device looks up the array's device address (with that device
 * current).  With CUDA's lazy module loading that look-up is also what loads the library's device
 * code and reserves the array on that GPU, so the first call is not itself allocation-free: make it
 * once per device at start-up, before the region where allocation is forbidden and before starting
 * any stream capture.  All calls on a device
 * share the one array, which keeps whatever the last call left in it; each call overwrites the
 * part it reads, so no clearing is needed, but two calls that may run at the same time on one
 * GPU (different streams, different threads) race on it: serialise them. */
#define OSDP_NOALLOC_MAX_PARTIALS (1 << 20)
int osdp_bias_grad_noalloc(const void *dy, int64_t M, int64_t N, float *dbias, void *stream);

/* ---- Execution-plan search (host only; Section 3.1: problem formulation and cost model, Algorithm 1).
 * An operator is five doubles {model, act, extra, S, gamma}: bytes of its model states (parameters and
 * optimiser states), activation bytes per sample, other bytes, bytes of its parameters (what the
 * collectives move), computation time per sample.  `ops` holds n of them back to back.  A mode is
 * 0 (DP: states replicated, two collectives per step) or 1 (ZDP: states sharded over the `world` ranks,
 * three collectives).  With N = world:
 *   memory(p, b) = sum_i ( model_i or model_i / N ) + b * act_i + extra_i
 *   time(p, b)   = sum_i ( 2 or 3 ) * (N - 1) * (alpha + S_i / N * beta) + b * gamma_i
 * alpha = latency per communication step, beta = transfer time per byte; all values >= 0 and finite.
 *
 * osdp_plan_cost: memory and time of one given plan at batch size `batch`. */
int osdp_plan_cost(const double *ops, int n, int world, double alpha, double beta, const uint8_t *modes,
                   int batch, double *memory, double *time);

/* osdp_plan_search: for b = 1, 2, ... the feasible plan (memory <= mem_limit) of least time; stops at the
 * first b for which nothing fits or after max_batch (the paper's loop has no such cap; it keeps the loop
 * finite when memory never runs out); returns the candidate with the least time per sample, time / b
 * (the first such b on ties): modes[n], *batch, *time_per_sample.  *batch = 0 and *time_per_sample = +inf
 * if nothing fits at b = 1.  The search is exact (depth-first with the memory and best-so-far prunings
 * and a relaxation bound) unless it visits more than max_nodes nodes in one batch size (<= 0: 2e8), in
 * which case it returns OSDP_ERR_SEARCH_LIMIT with the best feasible plan found.  nodes_visited may be
 * NULL.  n <= 16384. */
int osdp_plan_search(const double *ops, int n, int world, double alpha, double beta, double mem_limit,
                     int max_batch, int64_t max_nodes, uint8_t *modes, int *batch,
                     double *time_per_sample, int64_t *nodes_visited);

/* Section 3.3, last paragraph: an operator cut into k slices is planned slice by slice (some slices DP,
 * the others ZDP).  Writes k operators (5 doubles each) to `slices`: 1/k of every byte count, and
 * gamma * (1 + overhead) / k, `overhead` being the measured relative cost of running the operator
 * split k ways (> -1). */
int osdp_plan_expand_slices(const double *op, int k, double overhead, double *slices);

/* osdp_plan_search with the slice granularity of every operator left free as well (the paper takes it as
 * given and leaves its automatic choice open).  Operator i may be cut into cand_k[a] slices at a measured
 * relative overhead cand_overhead[a] (> -1), a in [cand_begin[i], cand_begin[i+1]); cand_begin has n + 1
 * entries, cand_begin[0] = 0, every operator at least one candidate.  The slices of an operator are priced
 * like osdp_plan_expand_slices prices them and planned one by one; since they are identical only their
 * number in DP matters.  Returns, for the batch size of least time per sample, k_out[i] (the granularity
 * chosen for operator i) and dp_slices[i] (how many of its slices run in DP: the first dp_slices[i], say;
 * the others run in ZDP).
 * surge_factor (>= 0): Section 3.3 names the gathered parameters of a ZDP operator as the memory surge
 * that splitting cuts from size(operator) to size(operator) / granularity.  The sums of Section 3.1 have
 * no term for it, so it is counted here on top of them: a plan fits if
 *     sum_i M_i + surge_factor * max over operators with a ZDP slice of (S_i / k_i)  <=  mem_limit,
 * e.g. 2 for a double-buffered gather, 0 for the paper's memory model as it stands.
 * Batch loop, *batch, *time_per_sample, max_nodes, nodes_visited and the return value as for
 * osdp_plan_search; exact unless OSDP_ERR_SEARCH_LIMIT is returned (a multiple-choice knapsack per value
 * of the largest gathered slice, solved depth first with the memory and best-so-far prunings and a
 * fractional relaxation as bound). */
int osdp_plan_search_granularity(const double *ops, int n, const int *cand_begin, const int *cand_k,
                                 const double *cand_overhead, int world, double alpha, double beta,
                                 double mem_limit, double surge_factor, int max_batch, int64_t max_nodes,
                                 int *k_out, int *dp_slices, int *batch, double *time_per_sample,
                                 int64_t *nodes_visited);

#ifdef __cplusplus
}
#endif
#endif /* OSDP_H_ */
