/* hilberta.h -- C ABI of HilbertA sparse attention (forward and backward) for NVIDIA B200 (sm_100a).
 *
 * The library implements the hot path of Hilbert-curve tiled sparse
 * attention for diffusion transformers: tokens of an H x W image grid are
 * reordered along a Hilbert curve (Sec. 3.1), the reordered sequence is cut
 * into tiles of N_T tokens with dense attention inside each tile, the tile
 * boundaries slide by a per-layer offset with wrap-around (Sec. 3.2), every
 * tile also attends to a static central shared region (Sec. 3.3), and text
 * tokens are treated like the shared region (Appendix A).
 *
 * Conventions
 *   - All functions return an int status: 0 on success, a negative
 *     HILBERTA_ERR_* code otherwise.  Nothing throws or aborts.
 *   - "device pointer" = memory of the CUDA device that was current when the
 *     plan was created; "host pointer" = ordinary host memory.  Calls that launch
 *     kernels return ERR_INVALID if another device is current.
 *   - `stream` arguments are a cudaStream_t passed as void* (NULL = default
 *     stream).
 *   - hilberta_forward, _forward_unpermute, _forward_fused, _forward_lse, _permute and
 *     _unpermute only enqueue kernels on `stream`: no allocation, no synchronisation,
 *     tensor maps passed to the kernels by value.  A sequence of them can be captured
 *     into a CUDA graph and replayed.
 *   - ORIGINAL token order:  [ text 0..n_text ) ++ [ image tokens row-major,
 *     token n_text + r*W + c ].
 *   - PHYSICAL token order (the layout of Appendix A):
 *       [ text | shared-region image tokens by ascending Hilbert index |
 *         remaining image tokens by ascending Hilbert index ].
 *     P = n_text + n_shared is the "global prefix" (the paper's N_s).
 *   - Mask: query i may read key j iff i is in the prefix, or j is in the
 *     prefix, or i and j are image tokens whose slid tile ids
 *     floor(((d + layer_offset) mod NP) / tile) agree, d = Hilbert index.
 *   - General H x W grids (appendix "Hilbert Curve for General Shape"): the
 *     curve is that of the smallest enclosing power-of-two square, side n,
 *     NP = n*n positions; cells outside H x W are padding that no token occupies.
 *     d above is the index on that padded curve (so `tile` must divide NP), while
 *     the exported Hilbert tables and the physical order rank the real cells in
 *     curve order.  For H = W = 2^k nothing is padded and NP = H*W.
 */
#ifndef HILBERTA_H_
#define HILBERTA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HILBERTA_VERSION 100

/* status codes */
#define HILBERTA_OK 0
#define HILBERTA_ERR_INVALID (-1)     /* bad argument value */
#define HILBERTA_ERR_UNSUPPORTED (-2) /* valid in the method, not built (grid or volume too large, head_dim) */
#define HILBERTA_ERR_ARCH (-3)        /* current device is not compute capability 10.x */
#define HILBERTA_ERR_CUDA (-4)        /* a CUDA call failed; see hilberta_last_cuda_error() */
#define HILBERTA_ERR_NOMEM (-5)       /* host or device allocation failed */
#define HILBERTA_ERR_BUFFER (-6)      /* export buffer too small (*needed is set), or problem too large for a fixed scratch array */
#define HILBERTA_ERR_UNBOUND (-7)     /* an attention call before hilberta_plan_bind */
#define HILBERTA_ERR_TIMEOUT (-8)     /* a bounded device-side wait expired (see hilberta_plan_status) */

/* element types */
#define HILBERTA_BF16 0
#define HILBERTA_FP32 1
/* q, k, v are e4m3 bytes (4 exponent bits, 3 mantissa bits, bias 7, no infinities; the "fn"
 * encoding); out is bf16.  Forward only.  The paper's kernel computes in 16-bit types (Sec. 4.1);
 * this is the same Algorithm 1 with 8-bit tensor-core operands: the softmax weights are rounded to
 * e4m3 as well before they multiply V, accumulation and the softmax itself stay fp32.  Any
 * per-tensor quantisation scales are the caller's: fold those of q and k into `scale`, multiply
 * v's into `out`. */
#define HILBERTA_FP8_E4M3 2

/* selectors for hilberta_plan_export */
#define HILBERTA_EXPORT_HIL_D2T 0     /* int32[HW]   Hilbert rank (curve order among the real cells) -> cell r*W+c */
#define HILBERTA_EXPORT_HIL_T2D 1     /* int32[HW]   row-major cell -> Hilbert rank */
#define HILBERTA_EXPORT_PHYS2ORIG 2   /* int32[S]    physical position -> original token */
#define HILBERTA_EXPORT_ORIG2PHYS 3   /* int32[S]    original token -> physical position */
#define HILBERTA_EXPORT_SHARED_RUNS 4 /* int32[n][2] maximal runs (start, length) of shared positions on the padded curve */
#define HILBERTA_EXPORT_WINDOWS 5     /* int32[T][5] per slid tile: lo, seg0_start, seg0_len, seg1_start, seg1_len */
#define HILBERTA_EXPORT_NNZ 6         /* uint64[1]   number of (query, key) pairs the mask keeps */
#define HILBERTA_EXPORT_INFO 7        /* int32[11]   H, W, tile, offset mod NP, shared_region, n_text, n_shared, T, padded side n, frames, shared_frames */
#define HILBERTA_EXPORT_LAUNCH_CLOCK 8 /* int32[2]  SM cycles and nanoseconds that the first CTA of the plan's latest tensor-core forward launch was resident: cycles / ns = the SM clock (GHz) that launch ran at; synchronises the device */

typedef struct hilberta_plan_s hilberta_plan_t;

/* Build the Hilbert permutation and the block-sparsity plan on the current device.
 *
 * Follows Sec. 3.1 (bijection pi between curve index and grid cell), Sec. 3.2
 * (tile[q] = [q N_T, (q+1) N_T) and q_i(l) = floor((i + l Delta)/N_T) mod T with
 * l Delta = layer_offset, wrap-around indexing), Sec. 3.3 (central shared
 * region) and Appendix A (prefix layout).
 *
 *   H, W           image-token grid, 1 <= H, W <= 1024 (larger: HILBERTA_ERR_UNSUPPORTED).
 *   tile           N_T in curve positions; tile >= 1 and NP % tile == 0 (NP = H*W for
 *                  power-of-two squares), else ERR_INVALID.
 *   layer_offset   slide in curve positions, any integer; reduced modulo NP (only
 *                  its value modulo tile changes the mask).
 *   shared_region  side of the centred square shared region in grid cells (rows
 *                  [H/2 - s/2, H/2 + s/2), columns likewise); 0 = none; must be even
 *                  and <= min(H, W), else ERR_INVALID.
 *   n_text         number of text tokens (>= 0) placed before the image tokens.
 *   out            receives the plan.  The library owns it; release with
 *                  hilberta_plan_destroy.  All tables live in device memory.
 *
 * The LUT, the shared-region scan, the permutation and the per-tile key ranges
 * are produced by CUDA kernels.  The call synchronises the device's default
 * stream work it launches and may allocate.  A plan is immutable apart from
 * hilberta_plan_bind and may be reused by any number of forward / permute calls.
 */
int hilberta_plan(int H, int W, int tile, int layer_offset, int shared_region, int n_text,
                  hilberta_plan_t **out);

/* The same plan with the tiles of Appendix A / Algorithm 1 read literally (S = N / G,
 * start = group_id * S): the shared tokens are taken out first, and the remaining
 * R = H*W - shared_region^2 image tokens, in curve order, are cut into `groups` equal
 * groups of R / groups tokens; `layer_offset` slides the group boundaries along that
 * sequence (reduced modulo R).  groups >= 1 and R % groups == 0, else ERR_INVALID.
 * With shared_region = 0 on a power-of-two square this is hilberta_plan with
 * tile = H*W / groups.  The exported window table has `groups` rows whose `lo` is the
 * position in the non-shared sequence.  Everything downstream (bind, forward, permute)
 * is the same.  This is the tiling the paper's Table 1 settings use (16 x 16 shared
 * region at 1024^2: groups of 960 or 240 tokens). */
int hilberta_plan_groups(int H, int W, int groups, int layer_offset, int shared_region, int n_text,
                         hilberta_plan_t **out);

/* The plan for a video volume (Sec. 5, "Extension to Video Diffusion"): `frames` x H x W
 * tokens, original order [text | (f * H + r) * W + c], reordered along a THREE-dimensional
 * Hilbert curve so that a tile is a compact spatio-temporal block; tiles, slide and
 * wrap-around are those of hilberta_plan on that curve.  The paper names the idea and fixes
 * neither the curve nor the shared region; this library's reading: with the frame axis padded
 * to 2^a >= frames and the image axes to 2^b >= max(H, W),
 *   a <  b (a clip shorter than a frame is wide, the usual case): the image plane is cut into
 *          macro cells of 2^a x 2^a pixels visited in the order of the 2-D curve of
 *          hilberta_plan; the cube of 2^a frames above a macro cell is walked by a 3-D
 *          Hilbert curve (Skilling's transpose construction, axes (frame, row, col), starting
 *          at the cube's cell (0, 0, 0)); index = macro index * 8^a + index inside the cube;
 *          the padded curve has 2^(2b + a) positions;
 *   a >= b: the whole volume lies in one cube of side 2^a walked by the 3-D curve.
 * Cells outside the volume are padding, as for general image shapes; `tile` must divide the
 * padded length.  The shared region is a centred BOX of shared_frames x shared_region x
 * shared_region cells (both even, both zero for none).
 * frames >= 2; frames, H, W <= 128.  Everything downstream (export, bind, forward,
 * backward, permute) is unchanged: the kernels only ever see contiguous physical ranges. */
int hilberta_plan_video(int frames, int H, int W, int tile, int layer_offset, int shared_region,
                        int shared_frames, int n_text, hilberta_plan_t **out);

/* Free a plan and every device table it owns.  NULL is accepted. */
int hilberta_plan_destroy(hilberta_plan_t *plan);

/* Copy one canonical table of the plan to HOST memory (for parity checks and
 * callers that want the permutation).  `what` is a HILBERTA_EXPORT_* selector.
 * If `needed` is non-NULL it receives the table's size in bytes.  If host_buf is
 * NULL only the size is reported; if `bytes` is too small: ERR_BUFFER.
 * The definitions are those of Sec. 3.1-3.3 and Appendix A as listed above. */
int hilberta_plan_export(const hilberta_plan_t *plan, int what, void *host_buf, size_t bytes,
                         size_t *needed);

/* Fix the problem shape the plan's forward calls run on (Algorithm 1's
 * configuration line: batch Z, heads, head dim D, softmax scale s, strides).
 *
 *   batch, heads   >= 1.  The same mask serves every (batch, head).
 *   head_dim       bf16: 128 or 64.  fp32: 32, 64 or 128.  e4m3: 128.  Others: ERR_UNSUPPORTED.
 *   dtype          HILBERTA_BF16 (tensor-core kernel), HILBERTA_FP32 (plain FMA kernel) or
 *                  HILBERTA_FP8_E4M3 (tensor-core kernel, 8-bit operands, bf16 output; forward,
 *                  forward only: forward, forward_lse, forward_unpermute, forward_fused and
 *                  forward_host (8-bit q, k, v in, bf16 out) -- hilberta_backward* return
 *                  ERR_UNSUPPORTED).
 *   stride_b, stride_h, stride_s
 *                  element strides of q, k, v and out (all four share them) for
 *                  the batch, head and token axes; the head_dim axis is contiguous.
 *                  0 for all three means the dense [batch, heads, S, head_dim] layout.
 *                  bf16 needs every stride to be a multiple of 8 elements (16 bytes);
 *                  e4m3 a multiple of 16 elements (q, k, v are then 16-byte aligned row
 *                  by row, and so is the bf16 `out`, which uses the same element strides).
 *   scale          softmax scale s; <= 0 selects 1/sqrt(head_dim).
 *
 * Builds the kernel's work list (device memory) and may allocate and synchronise.
 * Rebinding replaces the previous binding. */
int hilberta_plan_bind(hilberta_plan_t *plan, int batch, int heads, int head_dim, int dtype,
                       int64_t stride_b, int64_t stride_h, int64_t stride_s, float scale);

/* Sparse attention forward (Algorithm 1: one launch; for each query block the
 * prefix keys K[0:N_s] and the keys of its own slid tile go through one online
 * softmax; prefix queries read every key).
 *
 *   q, k, v   device pointers, PHYSICAL token order, layout as bound; read only.
 *   out       device pointer, same layout, written; must not share a byte with q, k or v
 *             (ERR_INVALID otherwise).  The test is exact on the bound strides (see
 *             hilberta_check_overlap), so q, k, v and out may be slices of one packed,
 *             interleaved buffer as long as no element of out is an element of an input.
 *             (e4m3 inputs and their bf16 output have different byte strides: there the
 *             address ranges are compared, which also rejects interleaving.)
 *             bf16 and e4m3: all four 16-byte aligned.
 *   values    q, k and v must be finite over the WHOLE tensors: the tensor-core kernels
 *             multiply the rows of a partly masked 128-key block by weights that are
 *             exactly zero, and 0 * Inf or 0 * NaN in a token the mask excludes would
 *             reach rows that must not see it.
 *   plan      a bound plan.
 *   stream    the launch is asynchronous on this stream; no allocation, no
 *             synchronisation.
 *
 * Errors: ERR_INVALID (NULL / misaligned pointers), ERR_UNBOUND, ERR_CUDA. */
int hilberta_forward(const void *q, const void *k, const void *v, void *out,
                     const hilberta_plan_t *plan, void *stream);

/* hilberta_forward that also returns the log-sum-exp of every query row (the
 * max-logits buffer M of Algorithm 1, final step "m + log l"), as a backward pass
 * would need it.  lse: device pointer to [batch * heads, S] fp32, PHYSICAL row
 * order, natural logarithm of the sum over kept keys of exp(scale * <q, k>).
 * Everything else as hilberta_forward.  (Algorithm 1 stores the base-2 value of
 * the scaled logits; multiply by log2(e) to get it.) */
int hilberta_forward_lse(const void *q, const void *k, const void *v, void *out, float *lse,
                         const hilberta_plan_t *plan, void *stream);

/* Backward pass of hilberta_forward: the gradients of  sum(out * dout)  with
 * respect to q, k and v.  The paper fine-tunes through its kernel (Sec. 4.1, LoRA)
 * but does not describe the backward pass; this is the derivative of Algorithm 1's
 * result under the same mask, layout and plan:
 *     P = exp(scale * q k^T - lse) on kept pairs,   dP = dout v^T,
 *     delta_i = sum_d dout[i, d] * out[i, d],       dS = P * (dP - delta),
 *     dq = scale * dS k,    dk = scale * dS^T q,    dv = P^T dout.
 *
 * dout, q, k, v, out : device pointers, PHYSICAL order, the bound dtype, shape and
 *                      strides (bf16: tensor-core kernels; fp32: plain-FMA kernels); `out` and `lse` are what hilberta_forward_lse wrote
 *                      for these q, k, v.
 * lse                : device pointer, [batch * heads, S] fp32 (natural log).
 * dq, dk, dv         : device pointers, written; same shape and strides as q; must
 *                      not alias each other or any input.  Every row is written.
 * All pointers 16-byte aligned (lse: 4).  Asynchronous on `stream`; three kernel
 * launches; no allocation, no synchronisation.  A per-row scratch array
 * (2 * batch * heads * S floats, owned by the plan, allocated by hilberta_plan_bind)
 * carries lse * log2(e) and delta between the launches, so two backward calls on
 * the same plan must not overlap on the device.
 *
 * Errors: ERR_INVALID (NULL or misaligned pointers, an output that shares a byte with
 * another tensor argument -- the exact test of hilberta_check_overlap --, wrong
 * device), ERR_UNBOUND, ERR_CUDA. */
int hilberta_backward(const void *dout, const void *q, const void *k, const void *v, const void *out,
                      const float *lse, void *dq, void *dk, void *dv, const hilberta_plan_t *plan,
                      void *stream);

/* hilberta_backward for callers that must not allocate.  (The paper has no
 * counterpart: this is a deployment variant of the call above.)
 *
 * hilberta_backward keeps its per-row scratch (two floats per batch, head and
 * token) in memory that hilberta_plan_bind obtains from cudaMalloc, once per
 * plan.  Some hosts cannot afford that: a serving process that handed all device
 * memory to its own pool at start-up, so that a later cudaMalloc fails; a
 * latency-bound loop that must avoid the device-wide synchronisation an
 * allocation implies; a process that keeps dozens of bound plans (one per layer
 * offset) and wants them to share one scratch array at call time.  (hilberta_plan_bind
 * itself still allocates: the plan's work lists, schedules and its own per-plan
 * scratch.  Build and bind every plan first, before device memory is handed to the
 * host application's pool; only the calls made afterwards are allocation-free.)
 * This variant puts the
 * scratch in one fixed array of HILBERTA_STATIC_SCRATCH_FLOATS floats (4 MiB)
 * that is part of the library image: every GPU that loads the library holds it
 * until the process exits, and every plan and every call shares it.
 *
 * Arguments, layouts, alignment, results and errors are those of
 * hilberta_backward, and the output is the same.  In addition:
 *   - 2 * batch * heads * S  >  HILBERTA_STATIC_SCRATCH_FLOATS  ->  ERR_BUFFER,
 *     nothing is launched (the Flux shapes at 1024^2 and 2048^2 fit; 4096^2 with 24
 *     heads does not: use hilberta_backward there);
 *   - the call itself performs no cudaMalloc, cudaFree or other allocation;
 *   - the FIRST call on each device looks up the array's device address (with
 *     that device current) and caches it; make that first call before any stream
 *     capture begins;
 *   - the array keeps what the previous call wrote.  Nothing in it has to start at
 *     zero: each call overwrites every entry it later reads, in stream order;
 *   - because the array is shared, two calls that overlap on the GPU (different
 *     streams, different plans, or this call and another thread's) race on it.
 *     Serialise them, or use hilberta_backward, whose scratch is per plan. */
#define HILBERTA_STATIC_SCRATCH_FLOATS (1 << 20)
int hilberta_backward_static(const void *dout, const void *q, const void *k, const void *v, const void *out,
                             const float *lse, void *dq, void *dk, void *dv, const hilberta_plan_t *plan,
                             void *stream);

/* hilberta_forward with the exit gather of Sec. 3.4 fused into its epilogue (the
 * last attention layer of a step): q, k, v are in PHYSICAL order as for
 * hilberta_forward; `out` is written in ORIGINAL token order, i.e. physical row p
 * lands at row phys2orig[p].  Same layout, alignment, error and stream rules as
 * hilberta_forward.  Costs about 2 % more than hilberta_forward (rows that go to
 * scattered positions are stored per lane, rows that keep the physical order leave
 * through bulk tensor stores) and saves the separate hilberta_unpermute pass. */
int hilberta_forward_unpermute(const void *q, const void *k, const void *v, void *out,
                               const hilberta_plan_t *plan, void *stream);

/* Entry gather of Sec. 3.4 (reordering is one row gather through the Hilbert table):
 *   dst[b, p, :] = src[b, phys2orig[p], :]   for b < batch, p < S.
 * src is in ORIGINAL order, dst in PHYSICAL order; both device pointers to
 * [batch, S, row_elems] contiguous arrays of `dtype` (any of the three element
 * types; only the element size matters); rows must be a multiple of
 * 16 bytes and both pointers 16-byte aligned; src and dst must not overlap.
 * Asynchronous on `stream`. */
int hilberta_permute(const void *src, void *dst, const hilberta_plan_t *plan, int batch,
                     int row_elems, int dtype, void *stream);

/* Exit gather of Sec. 3.4 (restores the original layout):
 *   dst[b, t, :] = src[b, orig2phys[t], :]   for b < batch, t < S.
 * Same argument rules as hilberta_permute with the roles of the orders swapped. */
int hilberta_unpermute(const void *src, void *dst, const hilberta_plan_t *plan, int batch,
                       int row_elems, int dtype, void *stream);

/* The attention launch with the entry and / or exit gather of Sec. 3.4 fused in,
 * for the first and last attention layer of a step (or a single layer):
 *   in_original  != 0 : q, k, v are in ORIGINAL token order; every tile row is read
 *                       through the permutation (physical row p from row
 *                       phys2orig[p]) on its way into shared memory, so no permuted
 *                       copy of q, k, v is ever written;
 *   out_original != 0 : `out` is written in ORIGINAL order (as
 *                       hilberta_forward_unpermute does).
 * With both flags zero this is hilberta_forward.  Same shapes, strides, alignment,
 * stream and error rules as hilberta_forward; bf16, e4m3 and fp32 bindings. */
int hilberta_forward_fused(const void *q, const void *k, const void *v, void *out,
                           const hilberta_plan_t *plan, int in_original, int out_original, void *stream);

/* Host-buffer form of the whole path, for callers that hold activations in host
 * memory: copies q, k, v (HOST pointers, ORIGINAL order, dense
 * [batch, heads, S, head_dim]) to the device, runs hilberta_forward_fused with both
 * gathers fused in and copies the result to `out` (HOST pointer, ORIGINAL order).
 * The heads are processed in up to eight slices whose copies (two internal copy
 * streams, one per direction) and launches (`stream`) overlap.
 * Uses a device workspace that the first call on a plan allocates (and
 * hilberta_plan_destroy frees).  Requires a dense binding (strides 0).  The
 * copies are asynchronous if the host buffers are pinned; the call returns
 * after synchronising `stream`. */
int hilberta_forward_host(const void *q, const void *k, const void *v, void *out,
                          hilberta_plan_t *plan, void *stream);

/* After a forward on `stream` has completed: 0, or ERR_TIMEOUT if a bounded wait
 * inside the kernel gave up (the output is then undefined).  Synchronises the
 * device.  Clears the flag. */
int hilberta_plan_status(hilberta_plan_t *plan);

/* Host-side check of a kernel work list (no GPU involved; hilberta_plan_bind runs it on every
 * list it builds and fails with ERR_INVALID rather than upload a bad one).  The attention kernels
 * read the query rows and key ranges of their work items unchecked, so this is what stands
 * between a planning bug and an out-of-range access.  items: n_items records of ten int32:
 * q_start, q_rows, n_seg, seg_start[3], seg_len[3], kv_blocks.  Returns HILBERTA_OK iff every
 * item has 1 <= q_rows <= item_rows and its rows inside [0, S); 1 <= n_seg <= 3 key ranges, each
 * non-empty and inside [0, S), pairwise disjoint; kv_blocks = sum of ceil(seg_len / block); and the
 * items' query ranges cover [0, S) exactly once.  Otherwise ERR_INVALID.  (Sec. 3.2 / 3.3: every
 * query row belongs to the prefix or to exactly one slid tile.) */
int hilberta_check_work_list(const int32_t *items, int n_items, int S, int item_rows, int block);

/* The static schedule of the attention kernels, computed on the host exactly as hilberta_plan_bind
 * computes it (no GPU involved; exposed so that the assignment can be tested and inspected).  Work
 * item i applied to (batch, head) index j is a unit of cost cost[i]; where cost_two_heads is given and
 * cost_two_heads[i] > 0 the item is instead run for two consecutive indices at once (a unit
 * (i, j, j + 1) of that cost; an odd index left over stays single).  Units go, longest first, to the CTA
 * with the smallest load so far (Algorithm 1 runs one query block per program; here a persistent CTA
 * runs a list of them).  units receives three int32 per unit (item, index, second index or -1),
 * grouped by CTA -- at most n_items * bh units; cta_begin receives n_cta + 1 offsets into it (CTAs that
 * get nothing repeat the end offset); largest_load, if not NULL, the largest CTA load.
 * Errors: ERR_INVALID (bad counts, NULL outputs). */
int hilberta_schedule_units(int n_items, const int64_t *cost, const int64_t *cost_two_heads, int bh, int n_cta,
                            int32_t *units, int32_t *cta_begin, int64_t *largest_load);

/* Host-side aliasing test the attention calls run on their pointer arguments (no GPU involved).
 * Two tensors of the layout [batch, heads, S, row] with the same BYTE strides and rows of row_bytes
 * contiguous bytes, at base addresses a and b: returns 1 if they share at least one byte, else 0.
 * Exact (not a comparison of address ranges): they overlap iff b - a equals
 * dx stride_b + dy stride_h + dz stride_s + dc for some |dx| < batch, |dy| < heads, |dz| < S,
 * |dc| < row_bytes.  Algorithm 1 reads K and V blocks of other query blocks' launches in flight, so an
 * output that aliases an input would race; interleaved slices of one buffer are fine. */
int hilberta_check_overlap(uint64_t a, uint64_t b, int batch, int heads, int S, int64_t stride_b_bytes,
                           int64_t stride_h_bytes, int64_t stride_s_bytes, int64_t row_bytes);

/* Failure-detection self-test: launches a one-warp kernel that waits, with a 1 ms
 * deadline, on a barrier nothing arrives on -- the same bounded wait every role of
 * the attention kernel uses -- so that the wait expires, the status words of `plan` are
 * written and the kernel returns normally.  After it, hilberta_plan_status(plan) must
 * return HILBERTA_ERR_TIMEOUT once and the device must stay usable.  Asynchronous on
 * `stream`. */
int hilberta_selftest_timeout(hilberta_plan_t *plan, void *stream);

/* Number of kernels the library has launched in this process (all entry points). */
uint64_t hilberta_launch_count(void);

/* Text for a status code (static storage). */
const char *hilberta_status_string(int status);

/* HILBERTA_VERSION of the loaded library. */
int hilberta_version(void);

/* The cudaError_t of the calling thread's last ERR_CUDA (0 if none). */
int hilberta_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HILBERTA_H_ */
