/* spws -- sparse-workspace kernels for NVIDIA B200 (sm_100a): C ABI.
 *
 * The library evaluates sparse tensor expressions whose result is scattered into a compressed
 * sparse output through a per-row workspace (arXiv 2404.04541, "Compilation of Modular and
 * General Sparse Workspaces"):
 *
 *   row-wise SpGEMM          C(i,j)   = sum_k A(i,k)   * B(k,j)    A, B, C in CSR
 *   tensor-times-matrix      C(i,j,l) = sum_k A(i,j,k) * B(k,l)    A, C in CSF, B in CSR
 *   outer-product SpGEMM     C(i,j)   = sum_k A(k,i)   * B(k,j)    A, B, C in CSR, A stored by
 *                                                                  its rows k (dims = {K, I})
 *   SpTTM (outer mode)       A(i,j,l) = sum_k B(k,i,j) * C(k,l)    B in CSF, C in CSR, A in COO
 *   SpTTM-I                  A(k,j,l) = sum_i B(k,i,j) * C(i,l)    B in CSF, C in CSR, A in COO
 *   SpMTTKRP                 A(i,j)   = sum_kl B(k,l,i) * C(k,j) * D(l,j)
 *                                                                  B in CSF, C, D in CSR, A in COO
 *
 * following the paper's statement of the problem: an expression over named index variables
 * (Sec. 3), a level format per operand (Sec. 2.1, Fig. 4) and a workspace policy (Sec. 6.1:
 * the workspace tensor's format and policy; Sec. 6.2: dense-workspace optimisation).  The first
 * two expressions are first-order scatters (Sec. 2.2): the loop order i -> k -> j differs from the
 * output order i -> j only by the reduction variable, so every output row (every (i,j) fibre,
 * after hoisting the shared outer loops, Sec. 6.2) owns a first-order workspace along the last
 * index.  The third expression is the paper's running example (Sec. 2.1): the reduction variable is
 * the outermost loop, both output indices scatter, and ONE second-order workspace serves the whole
 * result: sparse (Algorithm 1 on integer labels i*J + j, Sec. 5.2, with the accumulation array
 * and the all array in the scratch buffer) under SPWS_SPARSE_ISM, an I x J value array with
 * flags under SPWS_DENSE (SPWS_WORKSPACE_TOO_LARGE when the scratch given cannot hold it: the
 * paper's dense workspace running out of memory, Sec. 7.2), and under SPWS_AUTO the dense one
 * when it fits and either I*J <= 2^27 or the products number at least I*J/16.  The last three are
 * the higher-order scatters of Sec. 7.3 (sparse output in coordinate form): their workspace is the sparse one on
 * integer labels over all scattered output indices (third order for SpTTM); no dense workspace
 * is offered for them (SPWS_DENSE: SPWS_WORKSPACE_TOO_LARGE at plan creation).
 *
 * Work is split in two device passes (Sec. 5.4: a symbolic phase that precomputes the output
 * structure removes the all array):
 *   spws_symbolic : per-row product count, work binning, exact output size per row through the
 *                   chosen workspace, exclusive scan into C's pos array; returns the sizes.
 *   spws_numeric  : fills C's coordinates and values through the chosen workspace.
 *
 * Memory: every pointer inside a spws_tensor_t and the scratch pointer are DEVICE pointers owned
 * by the caller.  The library never allocates or frees device memory and keeps no pointer after
 * a call returns, except that spws_numeric reads what spws_symbolic left in the same scratch
 * buffer.  All kernels are enqueued on the stream set with spws_set_stream.  Inputs are not
 * modified.  spws_execute_host is the one entry that takes HOST tensors.
 *
 * Errors: every function returns a spws_status_t; nothing aborts, throws or prints.
 */
#ifndef SPWS_H
#define SPWS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int spws_status_t;
enum {
    SPWS_OK = 0,
    SPWS_INVALID_ARGUMENT = 1,       /* null pointer, bad enum, bad option value                    */
    SPWS_UNSUPPORTED_EXPRESSION = 2, /* not one of the two first-order scatters above (any names)   */
    SPWS_DIM_MISMATCH = 3,           /* contracted dimension or output dimensions disagree          */
    SPWS_NONCANONICAL_INPUT = 4,     /* unsorted / duplicate / out-of-range coordinate, bad pos     */
    SPWS_SCRATCH_TOO_SMALL = 5,      /* scratch (or arena) smaller than this call needs             */
    SPWS_WORKSPACE_TOO_LARGE = 6,    /* policy DENSE forced on a row wider than dense_max_span      */
    SPWS_CUDA_ERROR = 7,             /* a CUDA runtime call failed                                  */
    SPWS_INTERNAL_OVERFLOW = 8,      /* a bounded device loop hit its limit                         */
    SPWS_OUTPUT_TOO_SMALL = 9,       /* C's capacity (n[]) is smaller than the result               */
    SPWS_BAD_SEQUENCE = 10           /* numeric without a successful symbolic on this plan          */
};

typedef struct spws_handle_s* spws_handle_t;
typedef struct spws_plan_s* spws_plan_t;

/* Level formats (Sec. 2.1, Fig. 4).  CSR = {Dense, Compressed}; CSF3 = three Compressed levels;
 * COO = coordinate form, the output format of the higher-order scatters (Sec. 7.3): one coordinate
 * array per index (crd[0 .. order-1], each with n[0] entries, sorted lexicographically, no
 * duplicates) and val; pos[] is not used. */
typedef enum { SPWS_CSR = 0, SPWS_CSF3 = 1, SPWS_COO = 2 } spws_format_t;
typedef enum { SPWS_F32 = 0, SPWS_F64 = 1 } spws_dtype_t;
/* Workspace policy.  DENSE: value array + occupancy bitmap along the last index (Gustavson's
 * workspace, Table 2), held in shared memory.  SPARSE_ISM: insert-sort-merge with the
 * coordinate-sort policy (Algorithm 1, Sec. 5.2).  HASH: insert-sort-merge with the reduction at
 * insert time (Sec. 4.3; the Bucket / Hash policies of Sec. 5.2): products are deduplicated into an
 * open-addressing table in shared memory and only the distinct coordinates are sorted; rows with
 * more than 4096 products take the global-memory ISM.  AUTO: chosen per row bin from the product
 * count and the column span.  The policy changes the route, never the result: the structure is
 * identical under every policy; values agree to rounding (routes that add with atomics sum in an
 * order that can differ from run to run). */
typedef enum { SPWS_DENSE = 0, SPWS_SPARSE_ISM = 1, SPWS_AUTO = 2, SPWS_HASH = 3 } spws_policy_t;

/* A tensor stored level by level.  Level l of a CSR matrix: l = 0 is Dense (pos[0], crd[0] unused,
 * n[0] = dims[0]); l = 1 is Compressed: pos[1] has dims[0]+1 entries, crd[1] has n[1] = nnz.
 * CSF3: pos[0] has 2 entries, crd[0] has n[0]; pos[1] has n[0]+1, crd[1] has n[1]; pos[2] has
 * n[1]+1, crd[2] has n[2] = nnz; no level stores an empty fibre.  Coordinates are zero-based and
 * strictly increasing inside a row / fibre.  pos is int64, crd is int32, val is float or double
 * (the plan's value type) with n[order-1] entries.
 * For an OUTPUT tensor n[] holds the CAPACITY of crd[l] (and val) on entry to spws_symbolic /
 * spws_numeric; spws_symbolic overwrites n[] with the sizes of the result. */
typedef struct {
    int32_t order;          /* 2 or 3 */
    int32_t reserved;
    int64_t dims[3];
    int64_t n[3];
    int64_t* pos[3];
    int32_t* crd[3];
    void* val;
} spws_tensor_t;

/* Plan options; zero in a field selects its default.  The thresholds exist so tests can force
 * every route on small inputs. */
typedef struct {
    int32_t validate;         /* 1: check inputs are canonical before any other kernel runs      */
    int32_t ism_warp_cap;     /* rows with <= this many products use the register ISM (<= 32)    */
    int32_t ism_cta_cap;      /* accumulation-array capacity of the shared-memory ISM, power of
                                 two in [64, 4096]; default 4096                                  */
    int32_t dense_unit_outputs;/* outputs of a row the CTA dense workspace accumulates in shared
                                 memory (outputs beyond them accumulate in the row's own value
                                 segment in global memory), power of two in [64, 8192];
                                 default 4096                                                      */
    int32_t dense_max_span;   /* widest column span (jmax - jmin + 1) a dense workspace may cover,
                                 in [32, 2^19]; default 2^19.  Wider rows go to ISM (AUTO) or
                                 fail with SPWS_WORKSPACE_TOO_LARGE (DENSE)                       */
    int32_t fallback_cap;     /* accumulation-array capacity (the paper's `cap`) of the global-
                                 memory ISM, power of two in [2, 2048]; default 2048              */
    float dense_span_words_per_product; /* AUTO prefers DENSE over the shared-memory ISM when
                                 span/32 <= this * products; default 8                            */
    int32_t outer_cap;        /* outer-product form: components the accumulation array of the
                                 second-order sparse workspace holds (the paper's `cap`); when
                                 full it is sorted, reduced and united with the all array.
                                 0 (default): all products in one round                           */
    int32_t reserved[4];
} spws_options_t;

typedef struct {
    int64_t rows;             /* output rows (SpGEMM) / input fibres (TTM)                        */
    int64_t products;         /* intermediate products = sum of the per-row upper bounds          */
    int64_t nnz;              /* stored entries of C                                              */
    int64_t max_row_products;
    int64_t rows_per_class[10];/* empty, ISM-register, ISM-shared(small), ISM-shared, dense-warp,
                                 dense-CTA(hub), dense-CTA, ISM-global, hash(small), hash         */
    int64_t dense_units;      /* CTA work units (row, share of its A entries) of the dense numeric
                                 pass                                                               */
    int32_t device_status;    /* last status word read back from the device                      */
    int32_t reserved;
    int64_t products_per_class[10];
    int64_t nnz_per_class[10];
    int32_t launches_symbolic; /* kernels enqueued by the last spws_symbolic / spws_numeric       */
    int32_t launches_numeric;
    int64_t dense_warp_rows;  /* dense rows the warp-per-row numeric kernel takes ...             */
    int64_t dense_warp_products; /* ... and their products and outputs                            */
    int64_t dense_warp_nnz;
    int64_t bitmap_bytes;     /* bytes of the bitmap arena in use                                 */
} spws_stats_t;

/* Kernel groups timed by spws_set_profiling (index into the array spws_get_timings fills). */
enum {
    SPWS_T_SYM_BOUNDS = 0,    /* per-row upper bound, span and class; word lists of long B rows    */
    SPWS_T_SYM_BIN = 1,       /* binning + dense work units                                        */
    SPWS_T_SYM_ISM_REG = 2,
    SPWS_T_SYM_ISM_SMEM_S = 3,
    SPWS_T_SYM_ISM_SMEM = 4,
    SPWS_T_SYM_DENSE_WARP = 5,
    SPWS_T_SYM_DENSE_CTA = 6,
    SPWS_T_SYM_ISM_GLOBAL = 7,
    SPWS_T_SYM_HASH = 8,
    SPWS_T_SYM_SCAN = 9,      /* exclusive scan, numeric routing of dense rows (+ CSF level
                                 rebuild for the 3-tensor form)                                    */
    SPWS_T_NUM_ISM_REG = 10,
    SPWS_T_NUM_ISM_SMEM_S = 11,
    SPWS_T_NUM_ISM_SMEM = 12,
    SPWS_T_NUM_DENSE_WARP = 13,
    SPWS_T_NUM_DENSE_EMIT = 14, /* coordinates of the CTA dense rows; clears the value segments
                                 that several work units add into                                  */
    SPWS_T_NUM_DENSE_CTA = 15,
    SPWS_T_NUM_ISM_GLOBAL = 16,
    SPWS_T_NUM_HASH = 17,
    SPWS_T_CEIL_DENSE_WARP = 18, /* spws_gather_ceiling: the warp-per-row dense rows ...             */
    SPWS_T_CEIL_DENSE_CTA = 19,  /* ... and the CTA-unit dense rows                                   */
    SPWS_T_COUNT = 20
};

spws_status_t spws_create(spws_handle_t* handle);
spws_status_t spws_destroy(spws_handle_t handle);
/* `cuda_stream` is a cudaStream_t (NULL = the default stream). */
spws_status_t spws_set_stream(spws_handle_t handle, void* cuda_stream);

/* Parses `expr` -- "C(i,j)=A(i,k)*B(k,j)", "C(i,j,l)=A(i,j,k)*B(k,l)", "C(i,j)=A(k,i)*B(k,j)",
 * "A(i,j,l)=B(k,i,j)*C(k,l)" or "A(k,j,l)=B(k,i,j)*C(i,l)" with any tensor and index names and
 * optional blanks -- and checks it against the formats: fmts[0] is the result's,
 * fmts[1], fmts[2] the operands' in the order written.  The expression is accepted when it has
 * exactly one reduction variable, the second operand is a CSR matrix indexed (reduction, last
 * output index), and the first operand's and result's level orders match the loop order
 * (Sec. 2.2 classification: first-order scatter), or when both operands are CSR matrices whose
 * first index is the shared reduction variable (second-order scatter).  Anything else:
 * SPWS_UNSUPPORTED_EXPRESSION. */
spws_status_t spws_plan_create(spws_handle_t handle, const char* expr, const spws_format_t fmts[3],
                               spws_dtype_t value_type, spws_policy_t policy,
                               const spws_options_t* options /* may be NULL */, spws_plan_t* plan);
spws_status_t spws_plan_destroy(spws_plan_t plan);

/* Three operands: "A(i,j) = B(k,l,i) * C(k,j) * D(l,j)" (SpMTTKRP with a sparse result, Sec. 7.3);
 * fmts[0] is the result's format (SPWS_COO), fmts[1..3] the operands' (SPWS_CSF3, SPWS_CSR,
 * SPWS_CSR).  Plans made here run through spws_workspace_size3 / spws_symbolic3 / spws_numeric3,
 * which are the two-operand calls with the third operand added. */
spws_status_t spws_plan_create3(spws_handle_t handle, const char* expr, const spws_format_t fmts[4],
                                spws_dtype_t value_type, spws_policy_t policy,
                                const spws_options_t* options /* may be NULL */, spws_plan_t* plan);
spws_status_t spws_workspace_size3(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                                   const spws_tensor_t* D, size_t* bytes);
spws_status_t spws_symbolic3(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                             const spws_tensor_t* D, spws_tensor_t* C, void* scratch, size_t scratch_bytes,
                             int64_t* sizes_out);
spws_status_t spws_numeric3(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                            const spws_tensor_t* D, spws_tensor_t* C, void* scratch, size_t scratch_bytes);

/* The expression check of spws_plan_create on its own (host only, needs no device): the
 * classification of Sec. 2.2 applied to `expr` and `fmts`.  `kind` (may be NULL) receives 0 for
 * the matrix form, 1 for the 3-tensor form, 2 for the outer-product form. */
spws_status_t spws_check_expression(const char* expr, const spws_format_t fmts[3], int* kind);

/* Upper bound of the scratch bytes spws_symbolic + spws_numeric need for these operands (reads
 * only dims and n[] of A and B; host-side, launches nothing; spws_workspace_size_exact gives the
 * size actually used -- except for the outer-product form,
 * whose workspace is sized by the number of products: there the call needs A's and B's pos arrays
 * on the device, counts the products with one kernel on the plan's stream and synchronises).  It always suffices; the largest
 * part is room for one occupancy bitmap per row (rows x min(columns, dense_max_span) / 8 bytes),
 * of which only the rows routed to the dense workspace use their exact span, so a smaller buffer
 * works for narrow rows and spws_symbolic reports SPWS_SCRATCH_TOO_SMALL when it does not.
 * 256-byte alignment is required of the scratch pointer. */
spws_status_t spws_workspace_size(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                                  size_t* bytes);

/* The scratch bytes spws_symbolic + spws_numeric really use for these operands, found by running
 * the first two steps of the symbolic pass (per-row product bound and span, binning; Sec. 5.4's
 * "balance workloads" needs them anyway): the fixed tables, the occupancy bitmaps of exactly the
 * rows routed to the dense workspace over exactly their spans, and the all-array slots of the
 * global-memory ISM (one per CTA it keeps busy, sized for its largest row, 2 GiB at most).  Two steps: with scratch = NULL the call writes to *bytes the size of the
 * buffer it needs itself (host only, no launch); with such a buffer (DEVICE, 256-byte aligned) it
 * runs the two kernels on the plan's stream, synchronises and writes the exact size.
 * `row_products` (DEVICE, int64, one entry per output row / input fibre; may be NULL) receives the
 * per-row product counts, which a caller that shards rows over devices balances on.  A buffer of
 * the returned size suffices for both passes; the call overwrites what an earlier symbolic pass
 * left in `scratch`. */
spws_status_t spws_workspace_size_exact(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                                        void* scratch, size_t scratch_bytes, size_t* bytes,
                                        int64_t* row_products);

/* Symbolic pass.  (For a COO result nothing needs to be allocated yet: sizes_out[0] / C->n[0]
 * receive the number of entries; like the outer-product form, these forms size their workspace
 * from the product count, which spws_workspace_size counts on the device.)
 * C->pos[] must be allocated by the caller: CSR: pos[1] with dims[0]+1 entries;
 * CSF3: pos[0] (2), crd[0] (A->n[0]), pos[1] (A->n[0]+1), crd[1] (A->n[1]), pos[2] (A->n[1]+1),
 * i.e. the sizes of A's upper levels, which bound C's.  On return C->n[] holds the result sizes
 * and `sizes_out` (host, 3 entries, may be NULL) a copy.  Synchronises the stream twice: after
 * binning, to learn which workspaces have rows (only those are launched), and at the end, to read
 * the sizes back. */
spws_status_t spws_symbolic(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                            spws_tensor_t* C, void* scratch, size_t scratch_bytes,
                            int64_t* sizes_out);

/* Numeric pass.  C->crd[last] and C->val must now hold C->n[last] entries.  Asynchronous: returns
 * after enqueueing; a device-side failure is reported by the next spws_get_stats.  (The sparse
 * workspace of the outer-product form synchronises once per round of its accumulation array.) */
spws_status_t spws_numeric(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                           spws_tensor_t* C, void* scratch, size_t scratch_bytes);

/* Synchronises the plan's stream and reports the last symbolic pass's statistics. */
spws_status_t spws_get_stats(spws_plan_t plan, spws_stats_t* stats);

/* Per-kernel timing for measurement (Sec. 7.1 reports kernel runtimes; the split by kernel is
 * this library's).  With profiling on, both passes record a CUDA event on the plan's stream after
 * every kernel group; spws_get_timings synchronises the stream and writes the milliseconds of
 * each group of the last symbolic and numeric pass into ms[0 .. SPWS_T_COUNT) (0 for a group that
 * did not run).  `n` is the capacity of `ms` and must be at least SPWS_T_COUNT. */
spws_status_t spws_set_profiling(spws_plan_t plan, int enabled);
spws_status_t spws_get_timings(spws_plan_t plan, float* ms, int n);

/* Iteration-only lower bound of the dense-workspace numeric kernels (Sec. 7.2 measures, as a
 * lower bound for any workspace, the generated code with the workspace stripped and only the
 * sparse iteration kept).  Runs, on the rows the last spws_symbolic routed to the dense workspace,
 * the same traversal as spws_numeric's two dense kernels -- same work units, same launch shape,
 * same gathers of A's entries and of the B rows they pick -- without bitmap, rank or
 * accumulation: every gathered column index is added into *index_sum and every product a*b into
 * *value_sum (both DEVICE pointers, cleared by the call; the value sum is taken in an order that
 * varies from run to run).  C is not written.  Call after spws_symbolic, with the same operands
 * and scratch; asynchronous.  With profiling on, spws_get_timings reports the two kernels in
 * SPWS_T_CEIL_DENSE_WARP / SPWS_T_CEIL_DENSE_CTA. */
spws_status_t spws_gather_ceiling(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                                  const spws_tensor_t* C, void* scratch, size_t scratch_bytes,
                                  uint64_t* index_sum, double* value_sum);

/* Whole path with HOST tensors: copies A and B to the device, runs both passes, copies C back.
 * A, B, C hold host pointers; C's arrays must be allocated with capacities n[] (crd/val of the
 * last level sized for the expected nnz; SPWS_OUTPUT_TOO_SMALL if the result is larger, with
 * C->n[] set to the needed sizes).  `arena` is DEVICE memory of `arena_bytes` supplied by the
 * caller, from which the call carves the device copies, C and the scratch.  `arena_needed`
 * (may be NULL) receives the bytes this call needed.  Synchronous. */
spws_status_t spws_execute_host(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B,
                                spws_tensor_t* C, void* arena, size_t arena_bytes,
                                size_t* arena_needed);

/* Row pointer from per-row counts, without any scratch argument (the paper has no counterpart:
 * this entry exists for the sake of callers, not of the method).
 *
 * Some code that wants the symbolic pass's last step -- pos[0] = 0, pos[i+1] = pos[i] + counts[i]
 * -- is not in a position to obtain device memory: a plug-in running inside a host whose
 * allocator already owns the whole GPU, a component that must not trigger the device-wide
 * synchronisation cudaMalloc / cudaFree imply, or a context (a host callback, a start-up path
 * before any pool exists) where allocation calls are simply off limits.  spws_symbolic needs a
 * caller-supplied scratch buffer for its scan; this variant keeps the scan's partial sums in a
 * fixed 64 KiB array that is part of the library image and therefore sits on every GPU that
 * loads the library until the process exits.  It calls no allocation routine of any kind.
 *
 * counts : DEVICE, int32, n entries (row i's number of stored outputs), each >= 0; all sums are
 *          carried in 64 bits, so any non-negative int32 counts are admissible.
 * pos    : DEVICE, int64, n+1 entries, written by the call; pos[n] is the total.
 * n      : 0 <= n <= SPWS_STATIC_MAX_ROWS; a larger n is refused with SPWS_SCRATCH_TOO_SMALL and
 *          nothing is launched.
 * Work is enqueued on `cuda_stream` (a cudaStream_t, NULL = default stream); the call does not
 * synchronise.  The first call on each device looks up the array's address on that device
 * (with that device current) and caches it, so make that first call outside any stream capture.
 * All calls on one GPU share the one array: two calls whose kernels can overlap on that GPU
 * (different streams, no ordering between them) race on it; order them.  The array keeps
 * whatever the last call left there, which is harmless because each call writes every partial
 * sum before reading it. */
#define SPWS_STATIC_MAX_ROWS 16777216
spws_status_t spws_row_pointer_static(const int32_t* counts, int64_t n, int64_t* pos, void* cuda_stream);

const char* spws_status_string(spws_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* SPWS_H */
