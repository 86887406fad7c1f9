/*
 * const_b200 -- execution of fused sparse tensor-network contraction trees on one B200 GPU.
 *
 * The library runs the computation that the CoNST code generator emits (arXiv 2401.04836): a tree
 * of binary contractions over CSF sparse tensors and dense factors, executed as one fused loop
 * nest in which every intermediate keeps only the modes below the fused loops (Sec. 2.2, Fig. 4(b),
 * Fig. 5).  The schedule -- contraction order, loop order of every contraction, CSF mode order of
 * every sparse tensor (the ap / lp / dp values of Sec. 3.2) -- is an input; finding it is not part
 * of this library.
 *
 * Conventions for every entry point
 *   - C ABI, no exceptions, nothing is printed, nothing calls exit().
 *   - "dev" pointers are CUDA device pointers on the current device; everything else is host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - The caller owns COO inputs, dense factors and outputs.  The library owns CSF arrays, work lists
 *     and scratch (stream-ordered allocations on the given stream) until const_destroy.
 *   - Dense operands and outputs are row-major in the index order written in the expression, and their
 *     base addresses are 16-byte aligned (rows are read and written with 128-bit accesses).
 *   - Every function returns a const_status_t; on error no output handle is produced.
 */
#ifndef CONST_B200_H
#define CONST_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CONST_OK = 0,
    CONST_ERR_INVALID_ARG = 1,      /* null pointer, bad order, malformed expression ...               */
    CONST_ERR_UNSUPPORTED = 2,      /* beyond a capacity: schedule too large for any executor, nnz >= 2^31 ... */
    CONST_ERR_ILLEGAL_SCHEDULE = 3, /* violates a constraint of Sec. 3.2                               */
    CONST_ERR_DUPLICATE_COORD = 4,  /* the same coordinate tuple appears twice in a COO input          */
    CONST_ERR_COORD_RANGE = 5,      /* a coordinate is negative or >= its extent                       */
    CONST_ERR_WORKSPACE = 6,        /* a size exceeds a fixed internal capacity                        */
    CONST_ERR_CUDA = 7,             /* a CUDA runtime call failed                                      */
    CONST_ERR_TIMEOUT = 8           /* a bounded device-side wait gave up                              */
} const_status_t;

typedef enum { CONST_F32 = 0, CONST_F64 = 1 } const_dtype_t;

typedef struct const_csf const_csf_t;     /* opaque: a sparse tensor in CSF form, on the device */
typedef struct const_plan const_plan_t;   /* opaque: a checked schedule bound to a kernel family */

typedef struct { char index; int64_t extent; } const_extent_t;   /* one per iteration index */

/* One operand of const_execute: exactly one of `csf` / `dense_dev` is non-NULL. */
typedef struct { const char *name; const const_csf_t *csf; const void *dense_dev; } const_operand_t;

/*
 * COO -> CSF (Sec. 2.1, "CSF representation").
 *
 * The tensor has `order` modes (2..4) with extents dims[0..order).  coords_dev[m] is a device array
 * of nnz int32 coordinates of mode m; vals_dev holds nnz values of `dtype`.  The inputs are read,
 * never modified, and may be released once the stream has passed this call.
 * mode_order[l] is the mode stored at CSF level l (outermost first): the layout <d1,d2,d0> of the
 * paper's example is mode_order = {1,2,0}.
 *
 * Result arrays (all int32, all levels compressed, nodes in lexicographic order):
 *   crd[l][n]  coordinate of node n of level l;
 *   pos[l][p]  first child (index into level l) of node p of level l-1, pos[l][n_{l-1}] = n_l;
 *              pos[0] = {0, n_0};
 *   vals[n]    value of leaf n (bit pattern untouched; explicit zeros are kept).
 * The coordinate tuple is packed into one 64-bit key (sum of ceil(log2 extent) over modes must be
 * <= 64), radix-sorted with its value, then each level is compressed with a flag/scan/scatter pass.
 * Per-slice nonzero counts and the light / heavy / giant work lists used by const_execute are built
 * here as well (on the device; the host does not wait for them).
 *
 * Errors: CONST_ERR_COORD_RANGE, CONST_ERR_DUPLICATE_COORD (both detected on the device; the call
 * waits for the stream once, after the sort, to read the level sizes and the status),
 * CONST_ERR_UNSUPPORTED for nnz >= 2^31 - 1 or a key wider than 64 bits, CONST_ERR_TIMEOUT when a
 * bounded device-side wait of the sort gave up (nothing is stored then), CONST_ERR_INVALID_ARG,
 * CONST_ERR_CUDA.  Safe to call from several host threads at once.
 */
const_status_t const_csf_build(int order, const int64_t *dims, int64_t nnz,
                               const int32_t *const *coords_dev, const void *vals_dev, const_dtype_t dtype,
                               const int *mode_order, void *stream, const_csf_t **out);

/*
 * COO -> CSF without any allocation.  (The paper has no counterpart: this exists for deployment.)
 *
 * Who needs it: code that is not allowed to obtain device memory at the point where it must build a
 * CSF tensor -- a plug-in running inside a host application that hands out a fixed arena and
 * forbids cudaMalloc, a real-time loop where the driver's allocation lock and its unbounded latency
 * are unacceptable, or a process already so close to the memory limit that a temporary allocation
 * could fail.  const_csf_build cannot serve them, because it obtains its sort buffers, scan
 * buffers and result arrays from the stream-ordered allocator.
 *
 * Same arguments and same result arrays as const_csf_build, except that the caller supplies the
 * outputs and no handle is created (so there are no work lists: the arrays are the product):
 *   pos_out_dev[l]  device buffer of at least nnz + 1 int32 (2 for l = 0);
 *   crd_out_dev[l]  device buffer of at least nnz int32;
 *   vals_out_dev    device buffer of nnz values of `dtype`; also used as a sort buffer during the call;
 *   level_sizes     host array of `order` entries (may be NULL): number of nodes of each level.
 * Every temporary lives in one array that the library holds in static device memory, about 6.4 MB
 * on every GPU that loads the library, for as long as the process runs.  Limit: nnz <= 262 144;
 * a larger nnz returns CONST_ERR_WORKSPACE and touches nothing.  The call issues no cudaMalloc,
 * cudaFree, stream-ordered allocation or allocating library routine.
 *
 * The first call on each device looks up the device address of that array (one
 * cudaGetSymbolAddress with that device current); make that first call outside any stream capture.
 * With CUDA's lazy module loading that first call is also the moment the driver loads the kernels and
 * places the array on the device, so "obtains no device memory" holds from the second call on: make
 * one warm-up call per device at start-up, while allocating is still allowed.
 * All calls share the array and it keeps whatever the previous call left in it; the call clears the
 * parts that must start at zero.  Two calls whose GPU work overlaps (different streams, or different
 * host threads) race on it: serialise them.  Like const_csf_build, the call synchronises the stream
 * once to read the level sizes and the error word, and returns the same error codes.
 */
const_status_t const_csf_build_noalloc(int order, const int64_t *dims, int64_t nnz,
                                       const int32_t *const *coords_dev, const void *vals_dev, const_dtype_t dtype,
                                       const int *mode_order, void *stream,
                                       int32_t *const *pos_out_dev, int32_t *const *crd_out_dev, void *vals_out_dev,
                                       int64_t *level_sizes);

/*
 * Dense array -> CSF (Sec. 2.1: the nonzeros of a result are the entries that are not zero).  dense_dev is a
 * row-major device array with extents dims[0..order) of `dtype`; every entry that compares unequal to zero
 * becomes a stored nonzero (so -0.0 is dropped and NaN is kept), the rest as for const_csf_build.  This is how
 * the dense result of one network becomes a sparse operand of the next, e.g. the 3-index integrals E of
 * Sec. 5.1 Eq. 1 as the two CSF operands of the 4-index contraction of Eq. 3, and how a result is handed out
 * in CSF form.  The call waits for the stream twice (the number of nonzeros, then the level sizes).
 * CONST_ERR_UNSUPPORTED for more than 2^40 cells or 2^31 - 2 nonzeros.
 */
const_status_t const_csf_from_dense(int order, const int64_t *dims, const void *dense_dev, const_dtype_t dtype,
                                    const int *mode_order, void *stream, const_csf_t **out);

/* Borrowed device pointers of one level (valid until const_destroy).  *pos has n_{level-1}+1 entries
 * (2 for level 0), *crd has *n entries.  Any output pointer may be NULL. */
const_status_t const_csf_level(const const_csf_t *csf, int level, const int32_t **pos, const int32_t **crd,
                               int64_t *n);
/* Borrowed device pointer of the leaf values, in leaf order. */
const_status_t const_csf_values(const const_csf_t *csf, const void **vals, int64_t *nnz);

/*
 * Load balancing over slices of the root level (work lists consumed by const_execute).
 * A slice with at most light_max_nnz nonzeros is processed by one warp; up to heavy_max_nnz by one
 * thread block; a larger ("giant") slice is split into blocks of about chunk_nnz nonzeros whose
 * partial results are added atomically.  const_csf_build applies defaults; this call replaces them
 * (used to force each bin in tests and to tune).  Values <= 0 keep the current setting.
 */
const_status_t const_csf_set_bins(const_csf_t *csf, int64_t light_max_nnz, int64_t heavy_max_nnz,
                                  int64_t chunk_nnz, void *stream);
/* Number of slices in each bin and of thread-block work items; any pointer may be NULL.  The counts live on
 * the device; the first request after a (re)binning waits for the stream that did it. */
const_status_t const_csf_bin_counts(const const_csf_t *csf, int64_t *n_light, int64_t *n_heavy,
                                    int64_t *n_giant, int64_t *n_items);
/*
 * Borrowed device pointers of the work lists, for checking the load balancer (valid until the next
 * const_csf_set_bins or const_destroy; any pointer may be NULL):
 *   slice_ptr[n_0 + 1]   leaf offset of every root-level slice (slice s holds leaves [slice_ptr[s], slice_ptr[s+1]));
 *   light_list[n_light]  the light slices, by falling size class floor(log2(nonzeros));
 *   items[n_items][4]    one record {slice, f0, f1, kind} of four int32 per thread block:
 *                          kind 1: heavy slice `slice`, all its level-1 nodes [f0, f1);
 *                          kind 2: level-1 nodes [f0, f1) of giant slice `slice` (its chunks tile the slice);
 *                          kind 0: entries [slice, slice + f0) of light_list, one slice per warp.
 */
const_status_t const_csf_work_lists(const const_csf_t *csf, const int32_t **slice_ptr, const int32_t **light_list,
                                    int64_t *n_light, const int32_t **items, int64_t *n_items);

/*
 * Check a schedule and bind it to a kernel family (Sec. 3.1 input/output; Sec. 3.2 constraints;
 * Sec. 4.2 the sequence of <assignment, loop permutation> pairs).
 *
 *   expression      the whole network, e.g. "Y[i,a,b] = X[i,j,k] * U[j,a] * V[k,b]".  Index names are
 *                   single letters; tensor names are identifiers.
 *   tree            n_contractions binary contractions in execution order (the ap order), e.g.
 *                   "T[i,j,b] = X[i,j,k] * V[k,b]", "Y[i,a,b] = T[i,j,b] * U[j,a]".  The last one
 *                   produces the result of `expression`.
 *   sparse_names / mode_orders
 *                   the n_sparse input tensors held in CSF and, for each, mode_orders[t][l] = mode at
 *                   level l (dp).  Every other input is a dense row-major array.
 *   loop_orders     one string per contraction: its indices, outermost loop first (lp).
 *   extents         extent of every index that occurs.
 *
 * Checks (-> CONST_ERR_ILLEGAL_SCHEDULE): each contraction's operands are inputs or results of
 * earlier contractions and every intermediate is consumed exactly once, later (Sec. 3.2.1); mode
 * orders and loop orders are permutations (3.2.2, 3.2.3); each CSF operand's level order agrees with
 * the loop order of the contraction that reads it, dense operands and dense-workspace intermediates
 * being exempt (3.2.4); for each intermediate the loops shared as a common prefix by its producer,
 * its consumer and every contraction between them are indices of the intermediate -- they are the
 * modes fusion removes (3.2.5).  The tree must also compute `expression` (same inputs, same result
 * indices, an index is summed in exactly one contraction).
 *
 * Kernel families (hand-written fused kernels; a schedule that matches none of them runs on the generic
 * executor described below, and CONST_ERR_UNSUPPORTED remains for schedules beyond its fixed capacities:
 * more than 12 contractions, 16 indices, 6 CSF operands, a dense tensor of 2^31 elements or more):
 *   chain   one CSF tensor of order 3 or 4 contracted leaf level first with one dense factor per
 *           non-root level; the result is indexed by the root level followed by the rank indices in
 *           level order (TTMc), or by one rank index shared by all factors (MTTKRP).  Ranks must be
 *           8, 16 or 32 (order-4 TTMc: 8).  The loops above each contracted level must be fused, so
 *           intermediates reduce to order 1 (order 2 for the middle one of order-4 TTMc).  CONST_F32.
 *   network T[i,k,l] = U[i,j,k] * V[j,l]; Z[i,m] = T[i,k,l] * W[k,l,m] with V dense, U in CSF with
 *           levels (i,k,j) and W in CSF with levels (l,m,k), loop orders i,k,j,l and i,l,m,k: both
 *           contractions then gather along a fibre; fused over i only (T reduced to order 2).  CONST_F64.
 *   tree    the generic executor (Sec. 4.2: it walks the loop tree that Algorithm 1 prints as forall / where
 *           constructs).  Any checked schedule, any number of CSF operands, fp32 or fp64: e.g. the running
 *           example R_ijk = A_ipq B_jpr C_kqr D_jkr with X and Y as 2-D workspaces inside the fused r, j
 *           loops (Fig. 5), order-4 MTTKRP, TTMc at other ranks, the network with U stored (i,j,k) and W
 *           (k,l,m), or a network multiplied by a sparse 0/1 map (Sec. 5.1, Eq. 2).  The outermost loop is
 *           spread over the grid (the two outermost fused loops together when both walk the same CSF
 *           operand), one iteration per thread block, or per warp when its workspaces are small; a forall
 *           walks the nodes of a CSF operand where skipping the other
 *           coordinates cannot change the result, else the dense range of its index, and looks the other CSF
 *           operands up; intermediates are dense workspaces over the indices fusion left them (Sec. 2.2),
 *           cleared at every iteration of the innermost forall shared by producer and consumer.  A producer
 *           and its consumer are fused under a forall only if the intermediate carries that index.  Slower
 *           than the families above; results are accumulated with atomic adds.
 */
const_status_t const_plan_create(const char *expression, const char *const *tree, int n_contractions,
                                 const char *const *sparse_names, const int *const *mode_orders, int n_sparse,
                                 const char *const *loop_orders, const const_extent_t *extents, int n_indices,
                                 const_dtype_t dtype, const_plan_t **out);

/*
 * The legality check of const_plan_create alone (Sec. 3.2), for any contraction tree, whether or not
 * a kernel family exists for it.  On CONST_OK reduced_orders[c] (may be NULL) receives the order of
 * the intermediate produced by contraction c after fusion (0 for the last contraction): its order
 * minus the number of fused loops, the quantity the paper's parameter l bounds.  Host only.
 */
const_status_t const_schedule_check(const char *expression, const char *const *tree, int n_contractions,
                                    const char *const *sparse_names, const int *const *mode_orders, int n_sparse,
                                    const char *const *loop_orders, const const_extent_t *extents, int n_indices,
                                    int *reduced_orders);

/* Facts about a checked plan, for tests: reduced order of the intermediate produced by contraction
 * c (0 for the last contraction), and the family ("ttmc3", "ttmc4", "mttkrp3", "network", "tree"). */
const_status_t const_plan_reduced_order(const const_plan_t *plan, int contraction, int *order);
const char *const_plan_family(const const_plan_t *plan);

/*
 * Run the fused contraction tree (Fig. 4(b) / Fig. 5 structure).  `operands` binds every input name
 * of the expression to a CSF handle or a dense device array; CSF handles must have been built with
 * the mode order and dtype the plan was created with.  out_dev is overwritten (it is zeroed first:
 * "R[*] = 0" precedes the nest).  Asynchronous on `stream`; no host synchronisation, the first call
 * included (the plan's status word is allocated and cleared in stream order then).  A plan stays on
 * the device of its first execute.  Every dense operand and out_dev must be 16-byte aligned
 * (CONST_ERR_INVALID_ARG otherwise, before anything is launched).
 * Partial results of split slices are combined with floating-point atomics, so results can differ
 * in the last bits between runs.
 */
const_status_t const_execute(const_plan_t *plan, const const_operand_t *operands, int n_operands,
                             void *out_dev, void *stream);

/*
 * Concrete index notation of a schedule (Sec. 4.2, Algorithm 1 `generate` with its helper `remove`):
 * the contractions, each with its loop permutation, become a nest of forall(index, ...) and
 * where(consumer, producer) constructs, e.g. for the running example of Sec. 4.1
 *   forall(r, forall(j, where(forall(k, forall(i, R(j, k, i) = Y(k, i) * D(r, j, k))), where(...))))
 * References are printed in stored order (a CSF input by its mode order, an intermediate by the loop
 * order of its producer) and an intermediate loses every index whose forall encloses both its
 * producer and its consumer.  Arguments as for const_plan_create; validate != 0 runs the Sec. 3.2
 * checks first (CONST_ERR_ILLEGAL_SCHEDULE), validate == 0 accepts any parsable sequence, such as one
 * whose fused loops were already removed.  The zero-terminated text goes to buf (host memory, buf_len
 * bytes, may be NULL); *needed receives its length including the terminator; CONST_ERR_WORKSPACE when
 * the buffer was too small (the text is truncated).  Host only, no device work.
 */
const_status_t const_schedule_cin(const char *expression, const char *const *tree, int n_contractions,
                                  const char *const *sparse_names, const int *const *mode_orders, int n_sparse,
                                  const char *const *loop_orders, const const_extent_t *extents, int n_indices,
                                  int validate, char *buf, int64_t buf_len, int64_t *needed);

/*
 * Choose where the dense per-slice stage of a plan runs.  The last contraction of a TTMc, summed over
 * the fibres of a slice, is the contraction Y_i = U_J^T * T_J (K = fibres of the slice; the consumer
 * statement of the Fig. 4(b) structure regrouped).  enable != 0: const_execute runs it on the tensor
 * cores (tcgen05, tf32 operands split into two terms each, fp32 accumulation in tensor memory:
 * per-term relative error below 2^-19, so the fp32 tolerance holds); enable == 0: on the fp32 FMA pipes.
 * Plans that have the stage: order-4 TTMc at rank 8 (const_plan_create switches it on: it is the faster
 * path) and order-3 TTMc at rank 16 x 16 (off unless asked for: the FMA path is faster there).
 * CONST_ERR_UNSUPPORTED for enable != 0 on any other plan.  Host-only call; takes effect at the next
 * const_execute.  A device-side wait that runs out is reported through const_last_device_status.
 */
const_status_t const_plan_set_tensor_stage(const_plan_t *plan, int enable);

/*
 * enable != 0: const_execute runs this plan on the generic executor (family "tree" of const_plan_create)
 * although a hand-written family matches it; enable == 0: back to the family.  CONST_ERR_UNSUPPORTED when
 * the schedule exceeds the generic executor's capacities (enable != 0) or when the plan has no other
 * kernel (enable == 0).  Host-only call.
 */
const_status_t const_plan_set_generic_executor(const_plan_t *plan, int enable);

/*
 * What the generic executor will do for this plan (Sec. 4.2 loop structure, as compiled): one line per loop and
 * per assignment -- which loop is spread over thread blocks, which CSF operand a loop walks ("walks B level 1"),
 * which operands it looks up ("locates D level 1") or that it runs over a dense range, where a workspace is
 * cleared and how many elements it has, and the private loops of every assignment.  Text protocol as for
 * const_schedule_cin (buf may be NULL, *needed receives the length including the terminator, CONST_ERR_WORKSPACE
 * when truncated).  CONST_ERR_UNSUPPORTED for a plan the generic executor cannot run.  Host only.
 */
const_status_t const_plan_describe(const const_plan_t *plan, char *buf, int64_t buf_len, int64_t *needed);

/* Synchronise `stream` and return the device-side status word of the plan's last executions
 * (CONST_OK, or the first error a kernel recorded, e.g. CONST_ERR_TIMEOUT). */
const_status_t const_last_device_status(const_plan_t *plan, void *stream);

/* Release a CSF handle or a plan (NULL is a no-op).  Device memory is freed in stream order on the
 * stream the handle was built on. */
void const_destroy(void *handle);

const char *const_status_string(const_status_t status);

/*
 * Test hook for the bounded device-side waits (the look-back of the radix sort, the mbarrier wait of the
 * tensor-core stage).  what = 0: number of polls after which a wait gives up (0 restores the defaults);
 * what = 1: value != 0 withholds the signal those waits wait for -- sort tiles do not publish their
 * counts, the tensor-core stage issues and commits nothing -- so that every such wait runs out, the
 * kernel records CONST_ERR_TIMEOUT, skips its stores and returns normally;
 * what = 2: which of the tile shapes a launcher keeps for measurement is launched (0: the default; the
 * two-contraction network has variants 1..5, every one of them computes the same result).  Process-wide; not
 * for production use.  CONST_ERR_INVALID_ARG for an unknown `what` or a value outside [0, 2^31).
 */
const_status_t const_debug_set(int what, int64_t value);

/*
 * Per-kernel timing (off by default).  While enabled, every kernel the library launches is
 * bracketed by two CUDA events recorded on the launch stream.  const_profile_enable(1) also clears
 * earlier records; const_profile_enable(0) stops recording and clears them.
 * const_profile_read waits for the recorded events and returns, per kernel name in first-launch
 * order, the number of launches and the summed duration in milliseconds.  `names` (host, may be
 * NULL) receives the names separated by '\n'.  *n_kernels is the number of distinct names; at
 * most max_kernels entries of `launches` / `total_ms` (host arrays, may be NULL) are written.
 * Not thread-safe with respect to concurrent library calls on other threads beyond a mutex
 * around the record list; meant for benchmarking, not for production paths.
 */
const_status_t const_profile_enable(int on);
const_status_t const_profile_read(char *names, int64_t names_bytes, int64_t *launches, double *total_ms,
                                  int max_kernels, int *n_kernels);

/*
 * Micro-benchmarks of the machine limits the fused kernels are rated against (the paper has no counterpart;
 * its measurements are single-threaded CPU times).  Each kind launches one warm-up and then `repeats`
 * back-to-back launches on `stream`, timed with two CUDA events, waits for them, and returns the mean
 * milliseconds per launch and the work one launch does:
 *   CONST_BENCH_FP32_FMA / CONST_BENCH_FP64_FMA   register-only fused multiply-adds on every SM; work in flop;
 *   CONST_BENCH_TF32_MMA     tcgen05.mma kind::tf32, M 128 x N 256 x K 8, operands in shared memory, accumulator
 *                            in tensor memory, one block per SM; work in flop;
 *   CONST_BENCH_FP64_MMA     mma.sync m8n8k4 in fp64 from registers on every SM (the fp64 matrix path); work in flop;
 *   CONST_BENCH_ROW_GATHER   rows_dev[n] (device, int32 row numbers, e.g. a leaf-level crd array) are gathered
 *                            from a table of table_rows x rank floats (rank 8, 16 or 32) with 128-bit loads, rank / 4
 *                            lanes per row, four rows in flight per lane; work in bytes of rows read.
 * rows_dev, n, table_rows and rank are ignored by every kind but the row gather.  The call allocates its table and a
 * status word stream-ordered and frees them before it returns.  CONST_ERR_TIMEOUT if the bounded wait for the
 * tensor pipe gave up.
 */
typedef enum { CONST_BENCH_FP32_FMA = 0, CONST_BENCH_FP64_FMA = 1, CONST_BENCH_TF32_MMA = 2,
               CONST_BENCH_ROW_GATHER = 3, CONST_BENCH_FP64_MMA = 4 } const_microbench_kind_t;
const_status_t const_microbench(int kind, const int32_t *rows_dev, int64_t n, int64_t table_rows, int rank, int repeats,
                                void *stream, double *ms_per_launch, double *work_per_launch);

#ifdef __cplusplus
}
#endif
#endif /* CONST_B200_H */
