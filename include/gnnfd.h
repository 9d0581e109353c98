/*
 * gnnfd — feature-decomposed GNN aggregation on one CUDA device (sm_100a).
 *
 * The library computes the Aggregation phase of message-passing GNN inference
 * (Algorithm 1, the loop over decomposition layers p with its Message,
 * Aggregate and Concat steps): the feature dimension is cut into chunks of
 * `chunk_width` columns, every chunk is aggregated over all vertices, and each
 * chunk's result is written into its own columns of the output.  The
 * Combination (dense) phase comes first (Section III: combination is run ahead
 * of aggregation); its output is the aggregation's input, whether the caller
 * computed it or gnnfd_combine did.
 *
 * Conventions
 *   - Every pointer named d_* is DEVICE memory owned by the caller.  The library
 *     never allocates or frees device memory; it carves what it needs out of
 *     the buffers it is handed.  Host pointers are named without the prefix.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - All entry points return a gnnfd_status_t (0 = success, negative = error);
 *     nothing throws, aborts or traps.  Device-side problems (a vertex id out of
 *     range) are counted on the device and reported as a status.
 *   - Matrices are row-major with a leading dimension in ELEMENTS (ld >= width).
 *     Padding columns are never written and never influence a result.
 *   - Same inputs give bit-identical outputs from run to run: no floating-point
 *     atomics are used anywhere.
 *   - Graph structure is int32 on the device: n and nnz must stay below 2^31.
 */
#ifndef GNNFD_H
#define GNNFD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gnnfd_csr gnnfd_csr_t; /* opaque host-side handle; holds device pointers into caller memory */

typedef enum { GNNFD_F32 = 0, GNNFD_BF16 = 1 } gnnfd_dtype_t;
typedef enum { GNNFD_I32 = 0, GNNFD_I64 = 1 } gnnfd_itype_t;

/* gnnfd_build_csr flags */
enum {
    GNNFD_CSR_ADD_SELF_LOOPS = 1, /* drop every input loop, then add exactly one (v,v) per vertex */
    GNNFD_CSR_DEDUP = 2,          /* keep the first (lowest edge id) of equal (dst, src) pairs */
    GNNFD_CSR_SYMMETRIZE = 4,     /* add the reverse of every non-loop edge, with edge id e + i */
    GNNFD_CSR_INPUT_ORDER = 8     /* light build: sort by destination only; the entries of a row keep the order of
                                     their edge ids instead of ascending source ids (not with DEDUP) */
};

typedef enum {
    GNNFD_OK = 0,
    GNNFD_INVALID_ARG = -1,         /* null pointer, non-positive size, ld < width, heads*dim mismatch */
    GNNFD_BAD_INDEX = -2,           /* a vertex id outside [0, n) was found in the edge list */
    GNNFD_TOO_LARGE = -3,           /* n, e or the resulting nnz does not fit the int32 structure */
    GNNFD_WORKSPACE_TOO_SMALL = -4, /* a caller-provided buffer is smaller than the size query says */
    GNNFD_UNSUPPORTED = -5,         /* unknown dtype / itype enum; an operand layout gnnfd_combine cannot take */
    GNNFD_CUDA_ERROR = -6,          /* a CUDA runtime call failed; see gnnfd_last_cuda_error() */
    GNNFD_STATIC_SCRATCH_EXCEEDED = -7 /* the built-in workspace of a *_static entry point is too small for this call */
} gnnfd_status_t;

/* ------------------------------------------------------------------ graph set-up
 *
 * CSR by destination from a COO edge list (Section II-C: the aggregation's input
 * is the edge set in COO form plus the vertex features).  Edge i goes from
 * src[i] to dst[i]; row v of the CSR lists the sources of the edges that end in
 * v.  Steps, in this order: reject ids outside [0,n); SYMMETRIZE; ADD_SELF_LOOPS;
 * order by (dst, src), ties by ascending edge id; DEDUP.  Besides row_ptr /
 * col_idx the build stores perm (CSR slot -> input edge id; e + i for the
 * reverse of edge i; -1 for an added self-loop), the degree normalisers
 * deg^-1/2 and 1/deg (0 for empty rows, deg = entries in the row), the GCN edge
 * weight deg(src)^-1/2 * deg(dst)^-1/2 per slot, and the launch schedule (rows
 * grouped by degree, rows above GNNFD_HUB_DEGREE cut into segments of at most
 * GNNFD_HUB_SEGMENT edges; see gnnfd_csr_schedule).
 *
 * GNNFD_CSR_INPUT_ORDER is for graphs that are aggregated once or a few times at a narrow width, where the
 * conversion would cost more than the aggregation it serves (Section III, the discussion of format-conversion
 * latency: a conversion can cancel the gain of the format).  The sort then runs over the destination bits only
 * (half the passes), rows list their sources in edge-id order, and everything else (perm, weights, schedule)
 * is as above, so every aggregation entry point takes the handle; results differ from the fully ordered
 * build only in the order of the fp32 additions inside a row.
 */
#define GNNFD_HUB_DEGREE 2048
#define GNNFD_HUB_SEGMENT 1024
#ifndef GNNFD_HUB_RANGE_ROWS
#define GNNFD_HUB_RANGE_ROWS 524288
#endif

/* Sizes (bytes) of the two device buffers gnnfd_build_csr needs for n vertices and e input edges.
 * persistent: must stay alive and untouched while the handle is in use.
 * scratch:    only during the call. */
int gnnfd_csr_workspace_bytes(int64_t n, int64_t e, uint32_t flags, size_t* persistent_bytes,
                              size_t* scratch_bytes);

/* Builds the CSR.  d_src / d_dst: device arrays of e vertex ids of type `itype`, not modified.
 * d_persistent / d_scratch: device buffers, 256-byte aligned, at least as large as the size query
 * says.  Enqueues on `stream` and synchronises it once before returning (the host needs nnz and
 * the bad-index count).  On success *out receives a new handle (release with gnnfd_csr_destroy;
 * the device memory stays the caller's).  On GNNFD_BAD_INDEX no handle is produced. */
int gnnfd_build_csr(int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype,
                    uint32_t flags, void* d_persistent, size_t persistent_bytes, void* d_scratch,
                    size_t scratch_bytes, void* stream, gnnfd_csr_t** out);

/* Reads the handle.  Any output pointer may be NULL.  The d_* results point into d_persistent:
 * row_ptr[n+1], col_idx[nnz], perm[nnz], dinv_sqrt[n], rdeg[n], edge_weight[nnz]. */
int gnnfd_csr_info(const gnnfd_csr_t* csr, int64_t* n, int64_t* nnz, const int32_t** d_row_ptr,
                   const int32_t** d_col_idx, const int32_t** d_perm, const float** d_dinv_sqrt,
                   const float** d_rdeg, const float** d_edge_weight, int32_t* max_degree);

/* The launch schedule.  (The paper has no counterpart: its CPU scatter walks the edge list as it comes.
 * This is how the library balances power-law rows over the GPU; exposed for inspection and tests.)
 * bin_count[5]: rows with degree <= 8, <= 32, <= 128, <= GNNFD_HUB_DEGREE, and
 * hub rows.  d_row_order[n]: row ids sorted by degree class, ascending id inside a class; a class is
 * the exact degree up to 8, then a quarter octave of (degree - 1) up to GNNFD_HUB_DEGREE, then one
 * class for all hub rows, so every bin is a contiguous range and neighbouring rows have near-equal
 * lengths.  Hub rows are cut at the boundaries of source ranges of GNNFD_HUB_RANGE_ROWS vertex ids (doubled
 * until at most 64 ranges cover the graph; one range for a GNNFD_CSR_INPUT_ORDER build) and then into segments of
 * at most GNNFD_HUB_SEGMENT entries.  The segment arrays are in launch order, which goes range by range over all
 * hub rows, so that the hub rows in flight gather from one band of source rows: d_seg_row[n_segments],
 * d_seg_begin / d_seg_end (CSR slots [begin, end) of the segment), d_seg_slot (the segment's number when a row's
 * segments are counted in ascending source order, row after row: partial results are stored by slot).
 * d_hub_seg_ptr[n_hub+1]: the slots of the i-th hub row (i-th row of the last bin) are [ptr[i], ptr[i+1]). */
int gnnfd_csr_schedule(const gnnfd_csr_t* csr, int64_t bin_count[5], const int32_t** d_row_order,
                       int64_t* n_segments, const int32_t** d_seg_row, const int32_t** d_seg_begin,
                       const int32_t** d_seg_end, const int32_t** d_seg_slot, const int32_t** d_hub_seg_ptr);

/* Frees the host-side handle only. */
void gnnfd_csr_destroy(gnnfd_csr_t* csr);

/* ------------------------------------------------------------------ GCN / GraphSAGE aggregation
 *
 * out[v, j] = s_v * sum over the CSR entries k of row v of w_k * x[col_idx[k], j]
 *   GCN : w_k = deg(col_idx[k])^-1/2 * deg(v)^-1/2, s_v = 1   (with the self-loop flag this is
 *         the symmetric normalisation D^-1/2 (A + I) D^-1/2 X of the cited GCN model)
 *   SAGE: w_k = 1, s_v = 1/deg(v)                              (neighbourhood mean)
 * Empty rows give 0.  Products and sums are fp32 (bf16 inputs are widened exactly).
 *
 * chunk_width (>= 1) is the width of one decomposition layer: P = ceil(f / chunk_width) chunks, the
 * last one narrower; chunk_width >= f means no decomposition.  Chunks are swept one after the other
 * over all rows, so the gathered working set of a sweep is n * chunk_width elements.  The result
 * does not depend on chunk_width beyond fp32 rounding (the order of the additions inside a row
 * depends on how many lanes a chunk occupies).
 *
 * d_x: [n, ldx] of xdt.  d_out: [n, ldo] of odt (must not alias d_x).  d_scratch: per-call buffer
 * of gnnfd_aggregate_workspace_bytes(csr, f) bytes (holds the per-segment partial sums of hub rows;
 * 0 bytes when the graph has no hub row, NULL is then accepted).  The call only enqueues work.
 * 16-byte-aligned pointers with ldx*sizeof(x) and chunk offsets multiples of 16 bytes take the
 * 128-bit load path; anything else is still correct through narrower loads. */
int gnnfd_aggregate_workspace_bytes(const gnnfd_csr_t* csr, int32_t f, size_t* scratch_bytes);

int gnnfd_aggregate_gcn(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt,
                        void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t f, int32_t chunk_width,
                        void* d_scratch, size_t scratch_bytes, void* stream);

int gnnfd_aggregate_sage(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt,
                         void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t f, int32_t chunk_width,
                         void* d_scratch, size_t scratch_bytes, void* stream);

/* Choice of the chunk width.  The paper leaves the number of decomposition layers to the user: it
 * depends on the device's memory capacity and on the dataset (Section II-B; the granularity sweep of
 * Section III).  gnnfd_default_chunk_candidates fills `candidates` with f (no decomposition) and the
 * powers of two below f from 256 down to two 16-byte vectors, and returns how many it wrote.
 * gnnfd_tune_chunk_width runs the aggregation (model 0 = GCN, 1 = SAGE) twice per candidate on the
 * caller's own graph and features, times the second call with CUDA events on `stream`, and returns the
 * fastest width in *best_width (its time in *best_ms, may be NULL).  It synchronises the stream;
 * d_out holds the result for the last candidate tried.  Other arguments as for gnnfd_aggregate_gcn. */
int gnnfd_default_chunk_candidates(int32_t f, gnnfd_dtype_t xdt, int32_t* candidates, int capacity);

int gnnfd_tune_chunk_width(const gnnfd_csr_t* csr, int model, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt,
                           void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t f, const int32_t* candidates,
                           int n_candidates, void* d_scratch, size_t scratch_bytes, void* stream,
                           int32_t* best_width, float* best_ms);

/* GCN aggregation without a caller workspace and without any allocation.  (The paper has no
 * counterpart to this entry point; it exists for the library's users.)
 *
 * Who needs it: a host that gave the whole device to its own memory pool at start-up, or that calls
 * from a loop where cudaMalloc's device-wide synchronisation is not acceptable, and that has no spare
 * buffer to hand over.  Such a caller cannot obtain the hub-row workspace gnnfd_aggregate_gcn asks
 * for.  Here that workspace is a fixed array of GNNFD_STATIC_SCRATCH_BYTES inside the library image;
 * every device that loads the library carries it until the process exits.  The call itself performs
 * no cudaMalloc / cudaFree and calls no allocating routine -- with one exception: while the optional
 * per-kernel timing is switched on (gnnfd_kernel_timing_enable(1), a diagnostic that is off by
 * default) every launch of the library creates a pair of CUDA events, this entry point's included;
 * leave the timing off where allocation is not allowed.
 *
 * Same arguments and same results (bit for bit: it runs the same kernels on the same data) as
 * gnnfd_aggregate_gcn, minus the scratch pair.
 * Limits and rules:
 *   - returns GNNFD_STATIC_SCRATCH_EXCEEDED when gnnfd_aggregate_workspace_bytes(csr, f) is larger
 *     than GNNFD_STATIC_SCRATCH_BYTES (hub segments x f rounded up to 4, x 4 bytes); nothing is launched;
 *   - the first call on each device looks up the array's device address (one runtime query, with that
 *     device current); make that first call outside any stream capture;
 *   - all calls on a device share the one array and it keeps whatever the previous call left.  The
 *     kernels overwrite every element before reading it, so nothing needs clearing, but two calls
 *     whose kernels may overlap on the GPU (different streams, no ordering between them) race on it:
 *     serialise them, or use gnnfd_aggregate_gcn with separate buffers. */
#define GNNFD_STATIC_SCRATCH_BYTES (32u << 20)

int gnnfd_aggregate_gcn_static(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt,
                               void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t f, int32_t chunk_width,
                               void* stream);

/* ------------------------------------------------------------------ one-shot aggregation of a COO edge list
 *
 * Edge list in, aggregated features out, for a graph that is used once (or at a narrow width, where a full
 * conversion costs several times the aggregation it serves; Section III of the paper makes that point about
 * conversion latency, its own method taking the COO edge set as it is).  The call does the light build
 * (GNNFD_CSR_INPUT_ORDER: half the sort passes; with GNNFD_CSR_DEDUP in `flags` the fully ordered build instead)
 * and the GCN / SAGE aggregation defined above out of ONE caller buffer, and returns no handle.  Still no
 * atomics: the stable destination sort fixes the order of every row's additions, so results are bit-identical
 * from run to run.  d_scratch: gnnfd_oneshot_workspace_bytes(n, e, flags, f) bytes, 256-byte aligned; it holds the
 * CSR, the sort buffers and the hub-row partial sums (sized for the worst case, because the graph is not known
 * yet).  Other arguments as for gnnfd_build_csr and gnnfd_aggregate_gcn.  Synchronises the stream once (the build
 * reads its counters), then enqueues the aggregation. */
int gnnfd_oneshot_workspace_bytes(int64_t n, int64_t e, uint32_t flags, int32_t f, size_t* scratch_bytes);

int gnnfd_oneshot_gcn(int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype, uint32_t flags,
                      const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                      int32_t f, int32_t chunk_width, void* d_scratch, size_t scratch_bytes, void* stream);

int gnnfd_oneshot_sage(int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype, uint32_t flags,
                       const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                       int32_t f, int32_t chunk_width, void* d_scratch, size_t scratch_bytes, void* stream);

/* The same for the attention aggregator (defined in the GAT section below; arguments as for gnnfd_aggregate_gat). */
int gnnfd_oneshot_gat_workspace_bytes(int64_t n, int64_t e, uint32_t flags, int32_t heads, int32_t dim,
                                      size_t* scratch_bytes);

int gnnfd_oneshot_gat(int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype, uint32_t flags,
                      const void* d_z, int64_t ldz, gnnfd_dtype_t zdt, const float* d_a_src, const float* d_a_dst,
                      int32_t heads, int32_t dim, float negative_slope, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                      int32_t chunk_width, void* d_scratch, size_t scratch_bytes, void* stream);

/* ------------------------------------------------------------------ GAT
 *
 * The attention aggregator is the third model the paper evaluates (Section II-A lists it with GCN and
 * GraphSAGE as the message-passing models under study; Section III runs it with a decomposition
 * granularity of 8 columns, one head, and studies that granularity against the hidden width).  The
 * paper gives no formula; the definition below is the cited GAT model's, evaluated on the
 * destination-indexed edge list as Section II-C describes the framework's chunked `propagate`: the
 * attention coefficients belong to the Message step and depend on whole heads, the weighted sum is the
 * Aggregate step and is what Algorithm 1 decomposes.
 *
 * Scores (full head width, computed once, never per chunk):
 *   s_src[u, h] = sum_d a_src[h, d] * z[u, h*dim + d],   s_dst[v, h] likewise with a_dst.
 * Logit of CSR entry k of row v, head h: LeakyReLU(s_src[col_idx[k], h] + s_dst[v, h]) with the given
 * negative slope.  alpha = softmax of the logits over the entries of the row (multi-edges are
 * separate terms).  out[v, h*dim + d] = sum_k alpha[k, h] * z[col_idx[k], h*dim + d]; empty row -> 0.
 * The fused kernel evaluates logits, a running (max, sum) softmax and the weighted sum in one pass
 * over the row; chunk_width decomposes the flattened heads*dim columns (column j uses head j / dim).
 */

/* The per-vertex halves of the attention logit (the linear part of the cited model's Message step,
 * Section II-A), computed once per layer from the full head width.
 * d_z [n, ldz] of zdt; d_a_src / d_a_dst [heads, dim] fp32; d_s_src / d_s_dst [n, heads] fp32 out. */
int gnnfd_gat_scores(int64_t n, const void* d_z, int64_t ldz, gnnfd_dtype_t zdt, const float* d_a_src,
                     const float* d_a_dst, int32_t heads, int32_t dim, float* d_s_src, float* d_s_dst,
                     void* stream);

/* Scratch for gnnfd_aggregate_gat: the two score arrays plus hub-row partials.
 * gnnfd_aggregate_gat is Algorithm 1's loop over decomposition layers for the attention model: Message
 * (coefficient times source feature) and Aggregate (sum over the row) per chunk of chunk_width columns,
 * Concat by writing each chunk into its own output columns. */
int gnnfd_gat_workspace_bytes(const gnnfd_csr_t* csr, int32_t heads, int32_t dim, size_t* scratch_bytes);

int gnnfd_aggregate_gat(const gnnfd_csr_t* csr, const void* d_z, int64_t ldz, gnnfd_dtype_t zdt,
                        const float* d_a_src, const float* d_a_dst, int32_t heads, int32_t dim,
                        float negative_slope, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                        int32_t chunk_width, void* d_scratch, size_t scratch_bytes, void* stream);

/* Materialised edge softmax (the normalisation inside the cited attention model's Message step,
 * Section II-A, written out instead of fused; Section II-C's gather-scatter framework materialises it
 * the same way): alpha[k, h] for every CSR slot k, [nnz, heads] fp32 in CSR order, from
 * caller-supplied scores d_s_src / d_s_dst [n, heads] fp32 (logit and softmax as defined above).
 * d_scratch: per-call buffer of gnnfd_edge_softmax_workspace_bytes(csr, heads) bytes (the running
 * maximum and sum of every hub-row segment; 0 bytes when the graph has no hub row, NULL is then
 * accepted), 8-byte aligned.  16-byte-aligned pointers with heads a multiple of 4 take the 128-bit
 * path; anything else is still correct through narrower accesses.  The call only enqueues work. */
int gnnfd_edge_softmax_workspace_bytes(const gnnfd_csr_t* csr, int32_t heads, size_t* scratch_bytes);

int gnnfd_edge_softmax(const gnnfd_csr_t* csr, const float* d_s_src, const float* d_s_dst, int32_t heads,
                       float negative_slope, float* d_alpha, void* d_scratch, size_t scratch_bytes, void* stream);

/* ------------------------------------------------------------------ Combination ahead of aggregation
 *
 * z[v, j] = sum_k x[v, k] * w_t[j, k]: the dense transform of a layer, applied to the input features
 * before the aggregation so that the aggregation runs on the f_out transformed columns (Section III of
 * the paper: the Combination phase is executed ahead of Aggregation; Algorithm 1 then decomposes the
 * transformed features).  Not part of the aggregation path proper; offered so that a whole layer stays
 * on the device.
 *
 * d_x [n, ldx] and d_w_t [f_out, ldw] (the weight matrix transposed: one row per output column) both of
 * type xdt; d_z [n, ldz] of type zdt.  The product runs on the tensor cores with fp32 sums:
 *   xdt = GNNFD_F32, mode GNNFD_COMBINE_TF32: both operands are read as tf32 (the low 13 mantissa bits of each
 *                     fp32 value are ignored), products are exact, so |z - exact| <= 2^-9 * sum_k |x[v,k] * w_t[j,k]|
 *                     plus fp32 summation error;
 *   xdt = GNNFD_F32, mode GNNFD_COMBINE_FP32: fp32-faithful.  Each operand is used as a tf32 pair (hi, lo) and
 *                     the three products that matter are accumulated, so the result meets the library's fp32
 *                     bar |z - exact| <= 1e-5 * sum_k |x[v,k] * w_t[j,k]| + 1e-6 (the paper's framework runs
 *                     the Combination in fp32);
 *   xdt = GNNFD_BF16: operands are used as they are, products are exact in fp32 (mode is ignored).
 * zdt = GNNFD_BF16 rounds the fp32 result to nearest even.
 * d_x and d_w_t must be 16-byte aligned with row pitches that are multiples of 16 bytes
 * (GNNFD_UNSUPPORTED otherwise); d_z has no alignment rule.  d_status (may be NULL): one int32 the caller
 * has set to 0; it becomes 1 if a block gave up waiting for its own copies or matrix instructions (each
 * wait is limited to one second), in which case d_z is incomplete.  The calls only enqueue work.
 *
 * gnnfd_combine is the tf32 product alone.  gnnfd_combine_ex adds the mode and, optionally, the GAT scores of
 * the result as part of the same pass (all four of d_a_src, d_a_dst [heads, dim] and d_s_src, d_s_dst
 * [n, heads] given, heads * dim == f_out; all four NULL to leave them out): the scores are formed from the
 * values written to d_z while a thread still holds its output row, so z is not read again.  With more than 256
 * output columns the columns are processed in tiles, which must then hold whole heads (GNNFD_UNSUPPORTED
 * otherwise; use gnnfd_gat_scores on the result instead). */
typedef enum { GNNFD_COMBINE_TF32 = 0, GNNFD_COMBINE_FP32 = 1 } gnnfd_combine_mode_t;

int gnnfd_combine(int64_t n, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t,
                  int64_t ldw, int32_t f_out, void* d_z, int64_t ldz, gnnfd_dtype_t zdt, int32_t* d_status,
                  void* stream);

int gnnfd_combine_ex(int64_t n, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t,
                     int64_t ldw, int32_t f_out, void* d_z, int64_t ldz, gnnfd_dtype_t zdt, int mode,
                     const float* d_a_src, const float* d_a_dst, int32_t heads, int32_t dim, float* d_s_src,
                     float* d_s_dst, int32_t* d_status, void* stream);

/* ------------------------------------------------------------------ a whole layer on a built CSR
 *
 * Combination, then Aggregation of the transformed features (Section III: the Combination phase is run ahead
 * of the Aggregation phase, so that Algorithm 1's decomposed aggregation works on the f_out transformed columns
 * instead of the f_in input columns): out = Aggregate(x * W), with the aggregators defined above.
 *   gnnfd_layer_gcn / gnnfd_layer_sage : gnnfd_combine_ex, then gnnfd_aggregate_gcn / gnnfd_aggregate_sage.
 *   gnnfd_layer_gat : gnnfd_combine_ex with the attention scores formed in its epilogue, then the fused GAT
 *                     aggregation on those scores (no separate scores pass; heads * dim output columns).
 * x, w_t, mode, d_status as for gnnfd_combine_ex; out, chunk_width as for the aggregation calls (chunk_width
 * decomposes the f_out transformed columns).  The transformed features z [n, f_out rounded up to 8] are kept in
 * the scratch buffer in the dtype of x.  d_scratch: gnnfd_layer_workspace_bytes(csr, model, f_out, heads, dim,
 * xdt) bytes, 256-byte aligned (model 0 = GCN, 1 = SAGE, 2 = GAT; heads and dim are ignored for 0 and 1).
 * d_out must not alias d_x.  The calls only enqueue work. */
int gnnfd_layer_workspace_bytes(const gnnfd_csr_t* csr, int model, int32_t f_out, int32_t heads, int32_t dim,
                                gnnfd_dtype_t xdt, size_t* scratch_bytes);

int gnnfd_layer_gcn(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in,
                    const void* d_w_t, int64_t ldw, int32_t f_out, int mode, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                    int32_t chunk_width, void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream);

int gnnfd_layer_sage(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in,
                     const void* d_w_t, int64_t ldw, int32_t f_out, int mode, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                     int32_t chunk_width, void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream);

int gnnfd_layer_gat(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in,
                    const void* d_w_t, int64_t ldw, int32_t heads, int32_t dim, const float* d_a_src,
                    const float* d_a_dst, float negative_slope, int mode, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                    int32_t chunk_width, void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream);

/* ------------------------------------------------------------------ diagnostics */

const char* gnnfd_status_string(int status);

/* cudaError_t of the most recent failed runtime call made by this library on this thread (0 if none). */
int gnnfd_last_cuda_error(void);

/* Kernels launched by this library since it was loaded. */
int64_t gnnfd_launch_count(void);

/* Optional per-kernel timing.  While enabled every launch is bracketed by CUDA events on its stream.
 * gnnfd_kernel_timing_read synchronises the recorded events, clears them, and fills up to `capacity`
 * entries: names[i] (static strings), ms[i] (total milliseconds), launches[i].  Returns the number of
 * distinct kernels seen (may exceed capacity), or a negative status. */
int gnnfd_kernel_timing_enable(int on);
int gnnfd_kernel_timing_read(const char** names, double* ms, int64_t* launches, int capacity);

/* Drill of gnnfd_combine's give-up path, for tests.  (The paper has no counterpart.)  It arms the NEXT
 * gnnfd_combine / gnnfd_combine_ex / gnnfd_layer_* call made by this host thread, and only that one: every
 * barrier wait of that launch is limited to wait_ns nanoseconds (0 keeps the usual second; at most 10^9) and the
 * loads of K block skip_k_block (32 fp32 or 64 bf16 columns of x per block; -1: none) are never issued.
 * Nothing is in flight for the block that was left out, so the waits of the other lanes run out, every thread
 * block sets *d_status to 1, releases its tensor memory and returns; the device stays usable and d_z is
 * incomplete. */
int gnnfd_debug_combine_fault(int64_t wait_ns, int32_t skip_k_block);

#ifdef __cplusplus
}
#endif
#endif /* GNNFD_H */
