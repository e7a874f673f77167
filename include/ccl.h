/*
 * ccl.h -- C ABI of the B200 (sm_100a) hot path of Chiplet-Contiguous Layout (CCL).
 *
 * CCL stores a matrix so that the data consumed by one chiplet ("strip") is one
 * contiguous region (paper Sec. 3).  This library provides the four operations on
 * that path: the address map, the row-major <-> CCL repack, a bf16 GEMM whose
 * operands and output are read/written in CCL, and a counter of local/remote HBM
 * bytes that scores a layout against page-granularity placement.
 *
 * Conventions (all entry points)
 *  - A "stored matrix" is rows x cols with cols contiguous in its row-major view.
 *  - P is the chiplet count (the paper's G).  e = elem_bytes.
 *  - Pointers named *_dev are DEVICE pointers on the current CUDA device; everything
 *    else is a host pointer.  The caller owns every buffer; the library never
 *    allocates or frees device memory and keeps no reference after a call returns.
 *  - Device work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *    the legacy default stream) and is asynchronous; no entry point synchronises.
 *  - Input and output buffers of one call must not overlap.
 *  - Every call returns a ccl_status and never aborts, throws or prints.  Arguments
 *    are validated on the host before any launch; on error nothing is launched.
 *    ccl_last_error() gives a thread-local message for the last failing call.
 *  - There is no CPU fallback: without a CUDA device the device entry points return
 *    CCL_ERR_CUDA.
 *
 * Test / diagnostic switches (environment variables, read by the library; none changes a result beyond the
 * rounding order of a split-K sum):
 *   CCL_GEMM_CTAS = 1|2            force one CTA per tile or a cta_group::2 pair
 *   CCL_GEMM_BN = 128|192|256|384|512  force the tile width
 *   CCL_GEMM_SPLITK = n            force the number of K splits
 *   CCL_GEMM_BALANCED = 0|1        never / always (where legal) cut the tiles that do not fill a round into equal shares
 *   CCL_GEMM_CLUSTERK = 0|2|4|8        never / always (where legal) let the CTAs of a cluster of that size share one tile,
 *                                  each over its own part of K (the default picks it for problems of few tiles)
 *   CCL_GEMM_WAVESYNC = 0|n        soft wave barrier off / every n-th round of tiles
 *   CCL_GEMM_PDL = 0               no programmatic dependent launch
 *   CCL_GEMM_RAGGED_DENSE = 0      ragged batches walk the fixed grid of max_rows per problem
 *   CCL_REPACK_PATH = vec|tma      force a repack kernel
 *   CCL_GEMM_VERBOSE = 1           print the chosen plan of every newly planned GEMM to stderr -- the one
 *                                  exception to "never prints"
 */
#ifndef CCL_H_
#define CCL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CCL_OK = 0,
    CCL_ERR_INVALID_ARG = 1, /* NULL pointer, unknown enum value, negative size                  */
    CCL_ERR_SHAPE = 2,       /* split dimension not divisible by P, operand shapes inconsistent */
    CCL_ERR_ALIGN = 3,       /* pointer / stride not aligned as the operation needs             */
    CCL_ERR_UNSUPPORTED = 4, /* valid request this build cannot run (e.g. GEMM with w % 8 != 0) */
    CCL_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed                               */
    CCL_ERR_WORKSPACE = 6,   /* workspace / required output buffer missing or too small        */
    CCL_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired (see ccl_gemm_status)        */
    CCL_ERR_PADDING = 8      /* inverse map: the offset lies in alignment padding               */
} ccl_status;

typedef enum { CCL_ROWMAJOR = 0, CCL_CCL = 1, CCL_CCL_INTERLEAVED = 2 } ccl_layout; /* physical order of a buffer */
typedef enum { CCL_PART_NONE = 0, CCL_PART_ROWS = 1, CCL_PART_COLS = 2, /* stored dim split over chiplets */
               CCL_PART_2D = 3 /* only as the out_part of a GEMM: the output cut into blocks along both dimensions */ } ccl_part;

/*
 * Descriptor of one stored matrix.
 *   layout = CCL_ROWMAJOR : offset(r,c) = r*cols + c                         (Eq. 2)
 *   layout = CCL_CCL, part = CCL_PART_COLS (the paper's case, Eq. 1 + Eq. 3):
 *       w = cols/P, g = c / w, c' = c mod w, offset = g*stride + r*w + c'
 *       stride = rows*w when strip_align_bytes == 0 (packed, Eq. 3 literally), else
 *       rows*w*e rounded up to strip_align_bytes (Sec. 3.2: a strip can be aligned to
 *       the placement granularity).  Padding elements belong to no (r,c).
 *       cols not a multiple of P (the paper assumes it is; this library's reading): w = ceil(cols/P),
 *       Eq. 1 unchanged, the last strip keeps the cols - (P-1)*w >= 1 columns that are left and is a
 *       contiguous rows x (its width) block like the others: offset = g*stride + r*w_g + c' with w_g the
 *       width of strip g.  A packed buffer is still exactly rows*cols elements.  Map, repack and traffic
 *       take such matrices; ccl_gemm returns CCL_ERR_UNSUPPORTED for them.
 *   layout = CCL_CCL, part = CCL_PART_ROWS (split along the non-contiguous dimension,
 *       which Sec. 2.2 calls coarse-grained: already contiguous):
 *       h = rows/P (rounded up, the last strip keeping the rest, as above), offset = (r / h)*stride +
 *       (r mod h)*cols + c, stride = h*cols (rounded up likewise).
 *   layout = CCL_CCL_INTERLEAVED (either part): the page-interleaved form of CCL, under which a plain
 *       address-driven round-robin mapping at the chunk size already puts every strip on its own
 *       chiplet (the setting Sec. 3.3 / 4.1 evaluate).  strip_align_bytes is the chunk size S (> 0).  Element
 *       o of strip g's packed contents (o = r*w + c' resp. (r mod h)*cols + c, as above) sits in that
 *       strip's chunk j = o*e / S, and chunk j of strip g is stored as chunk j*P + g of the buffer:
 *       byte offset = (j*P + g)*S + (o*e mod S).  The buffer holds ceil(strip bytes / S)*P chunks;
 *       the tail of every strip's last chunk is padding.  ccl_strip_stride is not defined for it.
 *       Map, repack and traffic take every such layout; ccl_gemm takes those whose chunks line up with the
 *       strip rows (see ccl_gemm).
 *   A CCL layout with part = CCL_PART_NONE behaves as CCL_ROWMAJOR.
 * Requirements: rows, cols > 0; elem_bytes in {1,2,4}; P >= 1; every strip of the split dimension
 * non-empty, i.e. (P-1)*ceil(dim/P) < dim (else CCL_ERR_SHAPE); strip_align_bytes >= 0 and a multiple of e.
 */
typedef struct ccl_mat {
    int64_t rows, cols;
    int32_t elem_bytes;
    int32_t P;
    int32_t part;   /* ccl_part   */
    int32_t layout; /* ccl_layout */
    int64_t strip_align_bytes;
} ccl_mat;

/* ---- address map (Eq. 1-3; host, pure, O(1)) ------------------------------------------- */

/* Element offset of stored coordinate (r,c). CCL_ERR_INVALID_ARG if (r,c) is out of range. */
ccl_status ccl_map_offset(const ccl_mat* m, int64_t r, int64_t c, int64_t* elem_off);
/* Inverse of the above. CCL_ERR_PADDING if elem_off is a padding element. */
ccl_status ccl_map_inverse(const ccl_mat* m, int64_t elem_off, int64_t* r, int64_t* c);
/* Size in bytes of the buffer the descriptor addresses, padding included (P*stride*e for CCL). */
ccl_status ccl_buffer_bytes(const ccl_mat* m, int64_t* bytes);
/* Elements between the bases of consecutive strips (CCL layouts only). */
ccl_status ccl_strip_stride(const ccl_mat* m, int64_t* elems);

/* ---- repack (Sec. 3.3: operands adopt CCL at load time or are repacked) ---------------- */

/*
 * Permutation copy on the device.
 *   dir = 0: src_dev is row-major [rows x cols]; dst_dev receives the layout `m` describes
 *            (ccl_buffer_bytes(m) bytes); padding bytes are written as zero.
 *   dir = 1: src_dev is in the layout `m` describes; dst_dev receives row-major.
 * Any shape the map accepts is accepted; base pointers must be aligned to elem_bytes.
 * 16-byte aligned bases with (w*e) % 16 == 0 and (stride*e) % 16 == 0 take the fast path.
 */
ccl_status ccl_repack(const ccl_mat* m, const void* src_dev, void* dst_dev, int dir, void* cuda_stream);

/*
 * The same copy for `batch` matrices of one descriptor in one launch (the expert weights of an MoE layer, Sec. 4.1):
 * matrix i is read at src_dev + i * src_stride_bytes and written at dst_dev + i * dst_stride_bytes.
 * batch in [1, 65535]; strides are multiples of elem_bytes (of 16 for the fast path); the destination stride is at
 * least the size of one output (ccl_buffer_bytes(m) for dir = 0, rows*cols*elem_bytes for dir = 1) and the source
 * stride is non-negative (0 repeats one source), else CCL_ERR_INVALID_ARG / CCL_ERR_ALIGN.  Bytes between the
 * outputs are left untouched.
 */
ccl_status ccl_repack_batched(const ccl_mat* m, int32_t batch, const void* src_dev, int64_t src_stride_bytes, void* dst_dev,
                              int64_t dst_stride_bytes, int dir, void* cuda_stream);

/*
 * Transposing repack: src_dev holds the row-major TRANSPOSE [cols x rows] of the matrix `m` describes (a weight
 * kept as [N x K] that a GEMM wants as CCL [K x N], Sec. 3.3 "repacked when profitable"); dst_dev receives the layout
 * `m` describes: element (r, c) of it is src[c * rows + r].  Padding bytes are written as zero.
 * Any descriptor the map accepts; 2-byte elements with rows, cols, strip width, strip stride and chunk size all
 * multiples of 8 elements and 16-byte aligned bases take the fast path (64 x 64 tiles through shared memory).
 */
ccl_status ccl_repack_transpose(const ccl_mat* m, const void* src_dev, void* dst_dev, void* cuda_stream);

/* ---- GEMM on CCL operands (Sec. 2.2 execution model; Sec. 3.3: the layout changes addresses only) */

/*
 * C[M x N] = A[M x K] * B[K x N]; bf16 inputs, fp32 accumulation, bf16 output rounded to
 * nearest-even.  Each operand is described by its own ccl_mat and may be row-major or CCL:
 *   A stored [M x K] (a_trans = 0) or [K x M] (a_trans = 1);
 *   B stored [K x N] (b_trans = 0) or [N x K] (b_trans = 1);   C stored [M x N].
 * out_part / P / grouped_raster describe how C is partitioned over chiplets and whether CTA
 * group g computes only strip g of C (Sec. 3.1: each CTA runs on the chiplet that owns its
 * output tile): out_part = CCL_PART_COLS splits N, CCL_PART_ROWS splits M, CCL_PART_2D cuts C into
 * part_m x (P / part_m) blocks (group qm * (P / part_m) + qn computes block (qm, qn); M divisible by
 * part_m and N by P / part_m -- the output-partition choices Sec. 4.1 sweeps), CCL_PART_NONE (or
 * grouped_raster = 0) uses one plain raster.  The result does not depend on these choices.
 * Requirements (else CCL_ERR_UNSUPPORTED / CCL_ERR_ALIGN, nothing launched): elem_bytes = 2;
 * every contiguous extent a tile row lives in (cols, or w for CCL_PART_COLS) a multiple of 8
 * elements; strip strides multiples of 16 bytes; base pointers 16-byte aligned; where the tile grid follows strips
 * along N (of B, of C, or of out_part with a grouped raster), strips of a multiple of 8 columns -- likewise strips along
 * M when A is stored [K x M].
 * Strips of unequal size (the split dimension not a multiple of P: strips of ceil(. / P), the last one shorter) are
 * taken by ccl_gemm / ccl_gemm_axpby / ccl_gemm_static_ws: not along K, not page-interleaved, a narrower last strip
 * a multiple of 8 columns wide (with the rule above that means P >= 9 for strips along N; strips of rows -- an
 * M-partition with A stored [M x K] -- have no such limit).  K is then never split.
 * A CCL_CCL_INTERLEAVED operand is taken when its chunks line up with its strip rows, so that a tile is an
 * affine box of the buffer: either a chunk holds a power-of-two number of whole strip rows, or a strip row is
 * made of whole chunks of a multiple of 64 elements; the chunk size a multiple of 16 bytes.  (With chunks of
 * whole rows, an operand whose rows run along K must have K a multiple of 64 or rows-per-strip a multiple of
 * the rows per chunk: the padding of a strip's last chunk is not read as zero.)  When neither holds but a strip row
 * and a chunk are both multiples of 64 elements (say rows of 3.5 chunks), every 128-byte piece of a row still lies
 * inside one chunk and the operand is fetched and written row by row in such pieces -- correct, ~10x slower for A or B
 * (store the operand with K along its rows, or pick a chunk size that divides the strip row, where speed matters); it then
 * must not be split along K, an A or B whose rows run along M or N needs K a multiple of 64, and a strip must hold
 * fewer than 2^31 elements.  Other chunkings -> CCL_ERR_UNSUPPORTED.
 */
typedef struct ccl_gemm_desc {
    int64_t M, N, K;
    ccl_mat A, B, C;
    int32_t a_trans, b_trans;
    int32_t out_part; /* ccl_part */
    int32_t P;
    int32_t grouped_raster;
    int32_t part_m;   /* out_part == CCL_PART_2D: blocks along M (a divisor of P); ignored otherwise */
} ccl_gemm_desc;

/*
 * Bytes of device workspace the preferred plan of this problem uses (0 when none): fp32 partial sums of a problem split
 * along K.  (A problem of few tiles is split inside thread-block clusters instead -- the partial sums meet in the
 * cluster's shared memory, in a fixed order -- and needs none.)  Two kinds of plan use it: the classic split (every tile computed by several units over disjoint k ranges,
 * summed by a second kernel) INSISTS on it -- ccl_gemm returns CCL_ERR_WORKSPACE without it --, the balanced split
 * (the tiles that do not fill a round of the machine are cut into equal shares of k blocks, one per unit, and reduced
 * inside the kernel, in the order of k: the same bits on every run) is OPTIONAL: given less than it needs, ccl_gemm
 * falls back to a whole-tile plan.  Calls that can overlap on the GPU must not share a workspace.
 */
ccl_status ccl_gemm_workspace(const ccl_gemm_desc* d, size_t* bytes);
/*
 * Enqueue the GEMM.  ws_dev may be NULL when ccl_gemm_workspace reports 0.
 * Device-side waits are bounded; if one expires the kernel stores a non-zero code in an
 * internal status word and returns early (C is then incomplete): see ccl_gemm_status.
 */
ccl_status ccl_gemm(const ccl_gemm_desc* d, const void* A_dev, const void* B_dev, void* C_dev, void* ws_dev,
                    size_t ws_bytes, void* cuda_stream);
/*
 * A RAGGED batch (the experts of an MoE layer with their routed token counts, Sec. 4.1): `groups` problems share N and
 * K; problem e multiplies rows [row_offsets[e], row_offsets[e+1]) of A [M x K] by its own B (problem e's buffer at
 * B_dev + e * b_stride_bytes, in the layout d->B describes; stride 0 = one shared B) into the same rows of C [M x N].
 * d->M is the total row count of A and C; rows no problem owns are left untouched.
 *   row_offsets_dev  int32[groups + 1] on the DEVICE, non-decreasing, within [0, M]; read by the kernel, so the
 *                    counts can come straight from a router kernel and the call can sit in a CUDA graph.
 *   max_rows         host-known upper bound of the rows of any one problem (1 <= max_rows <= M); the tile grid
 *                    is laid out for it and tiles past a problem's last row cost one loop iteration.
 * A row-major [M x K] (a_trans = 0), not split along M; C row-major or CCL split along N (out_part != CCL_PART_ROWS);
 * B as for ccl_gemm.  Never split along K: no workspace.  A problem whose offsets leave [0, M] or that has more rows
 * than max_rows is not computed and ccl_gemm_status() then returns CCL_ERR_SHAPE (detail 5).
 * Errors: as ccl_gemm; CCL_ERR_UNSUPPORTED for a_trans or operands split along M.
 */
ccl_status ccl_gemm_grouped(const ccl_gemm_desc* d, int32_t groups, int64_t max_rows, const int32_t* row_offsets_dev,
                            const void* A_dev, const void* B_dev, int64_t b_stride_bytes, void* C_dev, void* cuda_stream);
/*
 * The ragged batch with the gated activation of ccl_gemm_swiglu in the epilogue: the first half of an MoE expert FFN
 * in one launch.  d, A, B and C as for ccl_gemm_swiglu (d->N = gate + up columns of every B, C [M x N/2]), the batch
 * arguments as for ccl_gemm_grouped; the conditions and errors of both apply.
 */
ccl_status ccl_gemm_grouped_swiglu(const ccl_gemm_desc* d, int32_t groups, int64_t max_rows, const int32_t* row_offsets_dev,
                                   const void* A_dev, const void* B_dev, int64_t b_stride_bytes, void* C_dev, void* cuda_stream);

/*
 * A batch with RAGGED K: the weight gradients of the experts of an MoE layer (Sec. 4.1; dW_e = X_e^T * dY_e over the
 * tokens routed to expert e).  Problem e contracts rows [k_offsets[e], k_offsets[e+1]) of A, stored [K x M]
 * (a_trans = 1), and of B, stored [K x N] (b_trans = 0) -- K = d->K is the total row count of both -- into its own
 * C [M x N] at C_dev + e * c_stride_bytes (layout d->C).  A problem without rows writes zeros.
 *   k_offsets_dev  int32[groups + 1] on the DEVICE, non-decreasing, within [0, K]; read by the kernel.
 * A and B row-major or CCL split along M / N, not split along K, not page-interleaved; C as for ccl_gemm_batched.
 * The last 64-row block of a problem is cut at the problem's end: only its 16-row steps that hold rows of the problem
 * are multiplied, and the rows of the last step that belong to the next problem are zeroed in shared memory first.
 * Never split along K (no workspace); one CTA per tile.  Offsets outside [0, K] or decreasing: that problem's C is
 * written as zeros and ccl_gemm_status() returns CCL_ERR_SHAPE (detail 5).
 */
ccl_status ccl_gemm_grouped_k(const ccl_gemm_desc* d, int32_t groups, const int32_t* k_offsets_dev, const void* A_dev,
                              const void* B_dev, void* C_dev, int64_t c_stride_bytes, void* cuda_stream);

/*
 * The BLAS form (Sec. 2.2 notes that alpha and beta change nothing for placement: C is read under the partition it
 * is written under):
 *   C <- bf16( alpha * (A*B) + beta * C ),  fp32 arithmetic on the fp32 accumulator, one rounding.
 * C is read (only when beta != 0) and written through the same descriptor d->C; every tile reads its own part
 * of C before it writes it, so C_dev may hold anything when beta = 0.  alpha = 1, beta = 0 is ccl_gemm, bit for
 * bit.  Workspace, requirements, asynchrony and errors as for ccl_gemm; NaN scalars -> CCL_ERR_INVALID_ARG.
 */
ccl_status ccl_gemm_axpby(const ccl_gemm_desc* d, float alpha, float beta, const void* A_dev, const void* B_dev,
                          void* C_dev, void* ws_dev, size_t ws_bytes, void* cuda_stream);
/*
 * `batch` independent GEMMs of one shape and one set of layouts in a single launch, e.g. the expert
 * projections of a mixture-of-experts FFN (Sec. 4.1 evaluates the Qwen expert GEMMs one at a time; the
 * paper has no batched call: the batch only amortises the launch and fills the machine with small problems).
 * Problem e (0 <= e < batch) reads A_dev + e*a_stride_bytes and B_dev + e*b_stride_bytes and writes
 * C_dev + e*c_stride_bytes, each buffer laid out as `d` says; results are those of `batch` ccl_gemm calls
 * (bit for bit unless one of the two plans splits K, which changes the order of the fp32 sum).  A stride of 0 for A or B means every problem shares that operand.  Otherwise a stride must
 * be a multiple of 16 bytes and at least ccl_buffer_bytes of the operand (CCL_ERR_ALIGN / CCL_ERR_INVALID_ARG);
 * 1 <= batch <= 65536.  With batch = 1 the strides are ignored and the call equals ccl_gemm.
 * Workspace: ccl_gemm_batched_workspace bytes (0 when the plan does not split K).  All buffers are the
 * caller's; nothing is allocated.  Errors as for ccl_gemm, nothing launched on error.
 */
ccl_status ccl_gemm_batched_workspace(const ccl_gemm_desc* d, int32_t batch, size_t* bytes);
ccl_status ccl_gemm_batched(const ccl_gemm_desc* d, int32_t batch, const void* A_dev, int64_t a_stride_bytes,
                            const void* B_dev, int64_t b_stride_bytes, void* C_dev, int64_t c_stride_bytes,
                            void* ws_dev, size_t ws_bytes, void* cuda_stream);
/*
 * GEMM on a fused gate/up weight with the gated activation applied in the epilogue, so that the activation the
 * next GEMM consumes is produced directly in its layout (Sec. 3.3 has the kernel upstream of a GEMM write its
 * activations in CCL; Fig. 3 shows the fused up/gate operand and its per-chiplet strips).  The activation
 * itself, silu(x) = x / (1 + exp(-x)), is the standard one of these FFNs; the paper does not define it.
 *   H[M x N] = A * B as in ccl_gemm (fp32 accumulation), N even.  The N columns form S strips of width Wp = N/S,
 *   S = d->P if d->out_part == CCL_PART_COLS and d->P > 1, else S = 1; a strip holds its gate columns in its first
 *   half and its up columns in its second half.
 *   C[m][g*Wp/2 + j] = bf16( silu(H[m][g*Wp + j]) * H[m][g*Wp + Wp/2 + j] ),  0 <= j < Wp/2  (fp32, one rounding).
 * d->A and d->B describe the operands as for ccl_gemm; d->C describes the OUTPUT, [M x N/2].  If B is in CCL split
 * along N its strips must be these S strips (width Wp), if C is in CCL split along its columns, strips of Wp/2;
 * Wp/2 a multiple of 8.  Page-interleaved operands -> CCL_ERR_UNSUPPORTED.  No workspace (K is never split).
 * Other requirements, asynchrony, bounded waits and errors as for ccl_gemm.
 */
ccl_status ccl_gemm_swiglu(const ccl_gemm_desc* d, const void* A_dev, const void* B_dev, void* C_dev, void* cuda_stream);
/*
 * Synchronises `cuda_stream` (the one entry point that does), then reports and clears the status word of the
 * GEMMs and repacks finished on the current device: CCL_OK, or CCL_ERR_TIMEOUT with *detail = the raw device code
 * (1-6: a GEMM wait, 101: a repack wait), or CCL_ERR_SHAPE (detail 5) for bad offsets of a ragged batch.
 * detail may be NULL.  There is ONE status word per device, shared by every stream: with several streams in flight
 * the first caller after an expiry gets the report, whichever stream's kernel it was.
 */
ccl_status ccl_gemm_status(void* cuda_stream, int32_t* detail);

/*
 * Variant of ccl_gemm for callers that must not allocate.  (The paper has no counterpart: this is
 * a convenience of this library, not part of the method.)
 *
 * Who needs it: code that runs where a device allocation is off the table -- a serving loop whose
 * host framework hands out every byte of device memory up front and treats any cudaMalloc as a bug,
 * a plug-in called from inside another allocator, a latency-critical step that cannot afford the
 * device-wide synchronisation and unbounded latency an allocation may bring.  Such a caller can
 * still pass A, B and C (it owns them already) but has nowhere to get the split-K workspace from.
 * This entry point therefore takes no workspace: small problems that ccl_gemm would split along K
 * keep their partial sums in a scratch array of CCL_GEMM_STATIC_WS_BYTES that is compiled into the
 * library image, so every GPU that loads the library carries those bytes until the process exits.
 *
 * Behaviour: identical results to ccl_gemm (same kernels, same plan).  A problem whose plan needs
 * more than CCL_GEMM_STATIC_WS_BYTES is rejected with CCL_ERR_WORKSPACE before anything is
 * launched (ccl_gemm_workspace(d) tells in advance); a problem that needs no workspace runs as
 * usual.  The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 * The first call on each device looks up the scratch array's device address (which may make the
 * runtime load the library's device code), so make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps whatever the previous call left in it;
 * the kernels overwrite every partial sum they later read, so nothing needs clearing, but two
 * calls whose kernels can overlap on the GPU (different streams, no dependency) would race on
 * it: serialise them.
 */
#define CCL_GEMM_STATIC_WS_BYTES (8u * 1024u * 1024u)
ccl_status ccl_gemm_static_ws(const ccl_gemm_desc* d, const void* A_dev, const void* B_dev, void* C_dev,
                              void* cuda_stream);

/* ---- remote-traffic counter (Sec. 4.1 metric, every touched byte counted: no L2 filter) */

typedef enum { CCL_PLACE_RR = 0, CCL_PLACE_BLOCK = 1, CCL_PLACE_BEST = 2 } ccl_place;
typedef enum { CCL_ASSIGN_N_STRIPS = 0, CCL_ASSIGN_M_STRIPS = 1, CCL_ASSIGN_EXPLICIT = 2, CCL_ASSIGN_2D = 3 } ccl_assign;

/*
 * One CTA per BM x BN output tile (Sec. 2.2); it reads its rows of A over all K, its
 * columns of B over all K, and writes its tile of C.  Every operand is an allocation of
 * its own whose base is page 0.  A page of `page_bytes` is owned by one chiplet:
 *   CCL_PLACE_RR    : owner = page mod P            (fixed round-robin interleave, Sec. 4.1)
 *   CCL_PLACE_BLOCK : owner = min(P-1, page*page_bytes*P / buffer_bytes): P equal contiguous
 *                     address blocks (coarse placement, Sec. 4.1); on a CCL buffer whose
 *                     strips are whole pages this is "page -> its strip's chiplet"
 *   CCL_PLACE_BEST  : owner = the chiplet that demands most bytes of the page (ties: lowest
 *                     index; untouched pages: 0): the best any page-granular mapping can do.
 * Tile -> chiplet: CCL_ASSIGN_N_STRIPS: the strip (width N/P, rounded up; the last strip holds the
 * rest) holding the tile's first column; CCL_ASSIGN_M_STRIPS likewise along M; CCL_ASSIGN_2D: the
 * output is cut into part_m x (P / part_m) blocks of ceil(M / part_m) x ceil(N / (P / part_m)) and the
 * tile belongs to chiplet qm * (P / part_m) + qn of the block (qm, qn) holding its first element
 * (Sec. 4.1 sweeps the output partition and reports the best); CCL_ASSIGN_EXPLICIT: cta_chiplet_dev[tile].
 * Every strip / block must be non-empty (else CCL_ERR_SHAPE).
 * strip_tiling = 1 tiles every strip of a partitioned dimension on its own (tiles never
 * straddle strips, the last tile of a strip may be partial); 0 tiles globally.  Tiles are
 * numbered tile_m * tiles_n + tile_n.  Partial tiles touch only valid elements.
 */
typedef struct ccl_traffic_desc {
    int64_t M, N, K;
    int32_t BM, BN;
    ccl_mat A, B, C;
    int32_t a_trans, b_trans;
    int32_t P;
    int64_t page_bytes; /* > 0, multiple of every operand's elem_bytes */
    int32_t place[3];   /* ccl_place for A, B, C */
    int32_t assign;     /* ccl_assign */
    int32_t strip_tiling;
    int32_t part_m;     /* CCL_ASSIGN_2D: blocks along M (a divisor of P); ignored otherwise */
} ccl_traffic_desc;

/* Number of tiles and of pages per operand (sizes of the output arrays below). */
ccl_status ccl_traffic_sizes(const ccl_traffic_desc* d, int64_t* ntiles, int64_t pages[3]);
/*
 * Outputs (device; every one is fully overwritten):
 *   per_cta_dev  uint64 [ntiles][3 (A,B,C)][2 (local, remote)] bytes        (required)
 *   per_page_dev[X] uint64 [pages_X][P] bytes of page demanded per chiplet  (NULL = not wanted;
 *                required for an operand placed with CCL_PLACE_BEST, else CCL_ERR_WORKSPACE)
 *   owner_dev[X] uint8 [pages_X] owning chiplet                              (same rule)
 *   totals_dev   uint64 [3][2]                                               (required)
 * per_page_dev / owner_dev are HOST arrays of three device pointers (or NULL altogether).
 * cta_chiplet_dev: int32 [ntiles], values in [0,P); only read for CCL_ASSIGN_EXPLICIT.
 * Entries outside [0,P) are clamped into the range.
 */
ccl_status ccl_traffic(const ccl_traffic_desc* d, const int32_t* cta_chiplet_dev, uint64_t* per_cta_dev,
                       uint64_t* const per_page_dev[3], uint8_t* const owner_dev[3], uint64_t* totals_dev,
                       void* cuda_stream);

/*
 * The same count behind an IDEAL private L2 per chiplet: a chiplet fetches every byte it needs at most once,
 * however many of its CTAs read it (A is shared by the tiles of a tile row, B by those of a tile column), and
 * every output byte is written once.  This is a step from the every-byte count above towards the metric of
 * Sec. 4.1, which counts only the reads that miss the chiplet's L2 (finite there, unbounded here).
 *   totals_l2_dev uint64 [3 (A,B,C)][2 (local, remote)], summed over chiplets (device, overwritten).
 * Fixed placements only (CCL_PLACE_RR, CCL_PLACE_BLOCK; CCL_PLACE_BEST -> CCL_ERR_UNSUPPORTED).
 */
ccl_status ccl_traffic_l2(const ccl_traffic_desc* d, const int32_t* cta_chiplet_dev, uint64_t* totals_l2_dev,
                          void* cuda_stream);

/*
 * The same count behind a FINITE private L2 per chiplet: the metric of Sec. 4.1 (operand reads from a remote
 * chiplet's memory that miss the L2, plus output writes to one; 8 MB, 128-byte lines, 16 ways per chiplet).  The paper's simulator is not public;
 * this is a tile-level model with everything it leaves open stated here:
 *   - a chiplet's CTAs (its tiles under `assign`) are taken in row-major order of the tile grid (traversal = 0,
 *     n fastest) or column-major (traversal = 1, m fastest); the paper sweeps the traversal and reports the best;
 *   - they run in waves of wave_ctas consecutive CTAs (the CTAs resident on the chiplet at one time) that advance
 *     through K in lockstep, k_slice elements per step (0: all of K at once): in every step each CTA of the wave in
 *     turn touches every line of the k range of its A rectangle in address order, then every line of the k range
 *     of its B rectangle.  wave_ctas = 1, k_slice = 0: one CTA after the other, all of A, then all of B;
 *   - each chiplet's cache has capacity_bytes / (line_bytes * ways) sets, LRU in a set; lines are numbered from the
 *     start of each operand's buffer (assumed line-aligned) and the operand is part of the tag; set index:
 *     hash = 0: line mod sets (the textbook index; power-of-two row pitches then pile up in a few sets),
 *     hash = 1: (line + H(line div sets)) mod sets, H(b) = high 32 bits of b * 0x9E3779B97F4A7C15 -- a skew per
 *     block of `sets` consecutive lines that stands in for the address hashing of a real L2;
 *   - a miss fetches one whole line from the owner of its page: line_bytes local or remote bytes;
 *   - C is written once, past the cache.
 * totals_dev: uint64[3][2] (A, B, C) x (local, remote) bytes.
 * Requirements: capacity a whole number of sets, ways <= 32, wave_ctas in [1, 256], page_bytes a multiple of line_bytes (else
 * CCL_ERR_INVALID_ARG / CCL_ERR_UNSUPPORTED); fixed placements only; any assignment but CCL_ASSIGN_EXPLICIT;
 * A and B row-major or CCL (page-interleaved -> CCL_ERR_UNSUPPORTED).
 * One warp simulates one cache set of one chiplet; cost grows with tiles x K steps x lines per tile / sets.
 */
typedef struct ccl_l2_model {
    int64_t capacity_bytes; /* per chiplet */
    int32_t line_bytes;
    int32_t ways;
    int32_t traversal;      /* 0 row-major over the tile grid, 1 column-major */
    int32_t hash;           /* 0 set = line mod sets, 1 skewed index (see above) */
    int32_t wave_ctas;      /* CTAs of a chiplet in flight together, 1..256 */
    int32_t k_slice;        /* elements of K per lockstep step; 0 = all of K */
} ccl_l2_model;
ccl_status ccl_traffic_lru(const ccl_traffic_desc* d, const ccl_l2_model* m, uint64_t* totals_dev, void* cuda_stream);

/*
 * Experiment support (Sec. 2.1: chiplets with their own L2; a B200 is two dies behind one address space).  Launches
 * `nctas` CTAs that cannot share an SM; CTA i records the SM it ran on in smid_dev[i] and, for each of `nlines` cache
 * lines of a zero-filled device buffer (line j at byte offset j * stride_bytes), the mean round-trip time in SM clock
 * cycles of 64 dependent loads that bypass L1, in lat_dev[i * nlines + j].  SMs of the die whose L2 partition holds
 * a line see it faster than SMs of the other die: the rows of lat_dev cluster by die.
 * zero_buf_dev must hold zeros over [0, (nlines - 1) * stride_bytes + 8); stride_bytes a positive multiple of 4.
 */
ccl_status ccl_probe_l2_latency(const void* zero_buf_dev, int32_t nlines, int64_t stride_bytes, int32_t nctas, float* lat_dev,
                                int32_t* smid_dev, void* cuda_stream);

/*
 * Test support for the bounded device-side waits (no counterpart in the paper).  Launches one small CTA whose wait
 * CANNOT be satisfied, with a limit of limit_us microseconds (1..100000) instead of the library's 2 s, so that the
 * expiry path runs: the wait gives up by itself, the kernel records its code and leaves the way the real kernels do,
 * and the next ccl_gemm_status() returns CCL_ERR_TIMEOUT once.  Nothing is left waiting and the context stays usable.
 *   which = 0: the GEMM's path -- TMEM allocated, an mbarrier nobody arrives at, status code 6, TMEM released;
 *   which = 1: the repack's TMA ring -- four slots, the load of one slot left out, status code 101; the loads still in
 *              flight are drained before the CTA exits.  src_dev: 2048 readable bytes, 16-byte aligned (which = 1 only).
 */
ccl_status ccl_selftest_wait_timeout(int32_t which, uint32_t limit_us, const void* src_dev, void* cuda_stream);

/* Message for the last non-OK status returned on this thread ("" if none). Static storage. */
const char* ccl_last_error(void);
/* Number of CUDA kernels this library has launched in this process (all threads, all streams). */
uint64_t ccl_launch_count(void);
/* Library version, "major.minor". */
const char* ccl_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CCL_H_ */
