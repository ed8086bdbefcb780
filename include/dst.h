/*
 * dst -- densify assumed-sparse (IndexedSlices) gradients on one NVIDIA B200.
 *
 * The operation is the one the paper "Densifying Assumed-sparse Tensors"
 * (arXiv 1905.04035) introduces in Section 4 / Listing 1: a gradient held as
 * IndexedSlices (row indices + [n_rows, d] value rows, Section 3) is converted
 * to a dense [vocab, d] tensor so that gradients are accumulated by reduction
 * (Algorithm 1, "reduce" branch) instead of by concatenation ("gather" branch).
 * For the tied embedding / pre-softmax projection weight of Section 3 the
 * dense partner is the projection gradient, added in the same pass:
 *
 *     out[v, c] = (dense_in ? dense_in[v, c] : 0)
 *               + sum over slices r and rows i with indices_r[i] == v of values_r[i, c]
 *
 * Conventions for every entry point
 *   - All tensor arguments are DEVICE pointers unless a comment says "host".
 *     Buffers are owned by the caller; the library never allocates, frees or
 *     synchronises.  All work is enqueued on `stream`.
 *   - values_r is row-major contiguous [n_rows_r, d]; dense_in and out are
 *     row-major contiguous [vocab, d] in `out_type`; inputs are read-only.
 *   - `out` may alias `dense_in` (in-place accumulate).  It must not overlap
 *     indices, values or the workspace.
 *   - Duplicate indices are summed.  Rows whose index lies outside [0, vocab)
 *     are skipped and counted (result->n_out_of_range, result->status =
 *     DST_ERR_INDEX_OUT_OF_RANGE); they never fault.
 *   - The summation order is fixed by the shapes alone (ascending input
 *     position inside fixed-size chunks, a fixed combine tree, dense_in last),
 *     so two calls on the same inputs give bit-identical results, and
 *     dst_densify_concat equals dst_densify on the physical concatenation.
 *   - Return value: DST_OK when everything was enqueued.  Problems found on
 *     the host (bad argument, workspace too small, unsupported type) return an
 *     error and enqueue nothing.  Problems found on the device are reported in
 *     `result` once the stream has run.
 *   - The fast kernels need 16-byte aligned base pointers and row sizes that
 *     are multiples of 16 bytes; other shapes take a slow scalar kernel.
 */
#ifndef DST_H_
#define DST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DST_OK = 0,
    DST_ERR_INVALID_ARG = 1,
    DST_ERR_UNSUPPORTED = 2,
    DST_ERR_WORKSPACE_TOO_SMALL = 3,
    DST_ERR_INDEX_OUT_OF_RANGE = 4, /* device-side: some rows were skipped */
    DST_ERR_TIMEOUT = 5,            /* device-side: a bounded wait gave up; output invalid */
    DST_ERR_CUDA = 6
} dst_status_t;

typedef enum { DST_I32 = 0, DST_I64 = 1 } dst_index_t;
typedef enum { DST_F32 = 0, DST_BF16 = 1 } dst_dtype_t;

/* Element types.  Accumulation is always fp32.  flags must be 0. */
typedef struct {
    int32_t index_type; /* dst_index_t: type of indices and of unique_rows */
    int32_t value_type; /* dst_dtype_t: type of the value rows */
    int32_t out_type;   /* dst_dtype_t: type of dense_in and out */
    uint32_t flags;
} dst_opts_t;

/* One IndexedSlices object (Section 3): device pointers. */
typedef struct {
    const void* indices; /* [n_rows] */
    const void* values;  /* [n_rows, d] */
    int64_t n_rows;
} dst_slice_t;

/* Written by the device when the enqueued work runs (device or pinned host memory). */
typedef struct {
    int32_t status;         /* dst_status_t */
    int32_t n_unique;       /* number of distinct valid rows */
    int64_t n_out_of_range; /* input rows skipped */
    int64_t max_segment;    /* largest number of input rows naming one output row */
} dst_result_t;

/* Footprints in bytes (Section 4, Fig. 5a: gather of slices vs one dense tensor). */
typedef struct {
    int64_t n_rows_total;
    int64_t sparse_value_bytes;     /* sum_r n_rows_r * d * sizeof(value) */
    int64_t sparse_index_bytes;     /* sum_r n_rows_r * sizeof(index) */
    int64_t sparse_bytes;           /* the two above */
    int64_t dense_bytes;            /* vocab * d * sizeof(out) */
    int64_t gather_all_value_bytes; /* sum_r (vocab + n_rows_r) * d * sizeof(value): Algorithm 1's
                                       gather branch also turns the dense partner into vocab slices */
    double sparse_over_dense;
    double gather_all_over_dense;
} dst_bytes_report_t;

typedef struct CUstream_st* dst_stream_t; /* a cudaStream_t */

int dst_version(void);
const char* dst_status_string(int status);

/* Bytes of device workspace dst_densify / dst_densify_concat need for inputs of
 * at most n_rows_total rows in R slices.  Returns 0 for invalid arguments. */
size_t dst_workspace_bytes(int64_t n_rows_total, int32_t R, int64_t d, int64_t vocab, const dst_opts_t* opts);

/*
 * Densify one IndexedSlices gradient and add the dense partner
 * (Section 4, Listing 1: convert_to_tensor of an IndexedSlices; Algorithm 1 line 4: sum).
 *   indices [n_rows], values [n_rows, d], dense_in [vocab, d] or NULL, out [vocab, d].
 *   workspace: >= dst_workspace_bytes(n_rows, 1, d, vocab, opts) bytes, 256-byte aligned.
 *   unique_rows (index_type) / counts (int32): optional outputs with room for
 *   min(n_rows, vocab) entries -- the distinct valid rows in ascending order and
 *   how many input rows named each.  result: optional.
 * n_rows == 0 gives out = dense_in (or zeros).  vocab == 0 or d == 0 is a no-op.
 */
int dst_densify(const void* indices, const void* values, int64_t n_rows, int64_t d, int64_t vocab,
                const void* dense_in, void* out, dst_stream_t stream, const dst_opts_t* opts,
                void* workspace, size_t workspace_bytes,
                void* unique_rows, int32_t* counts, dst_result_t* result);

/*
 * Same, for the R slices a sparse gather would have concatenated (Algorithm 1
 * line 6; the cross-rank gather of Section 3).  `slices` is a HOST array of R
 * descriptors holding device pointers; it is read during the call only.  No
 * concatenated copy is made; the result is bit-identical to dst_densify on the
 * physical concatenation in slice order.  Empty slices are allowed.  R == 0
 * behaves like n_rows == 0.
 */
int dst_densify_concat(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab,
                       const void* dense_in, void* out, dst_stream_t stream, const dst_opts_t* opts,
                       void* workspace, size_t workspace_bytes,
                       void* unique_rows, int32_t* counts, dst_result_t* result);

/*
 * The whole "after" pipeline of the paper in one pass (Section 4, Fig. 3b: every rank converts its own
 * IndexedSlices, then everything is reduced; Fig. 5 for the sizes): the gradients R ranks hold for the
 * tied weight -- per rank one dense [vocab, d] tensor (the projection gradient, may be NULL) and any
 * number of IndexedSlices (the embedding lookups) -- accumulated into one dense tensor,
 *
 *     out[v, c] = sum over ranks r of ( dense_r[v, c] + sum of rank r's value rows that name v )
 *
 * Every dense tensor and every value row is read once, on the way to its output row, and `out` is
 * written once; no per-rank dense gradient and no running sum is ever materialised.  `ranks` is a
 * HOST array of R descriptors (device pointers inside; `slices` a HOST array of n_slices entries),
 * read during the call only.  At most 64 ranks may bring a dense tensor (DST_ERR_UNSUPPORTED beyond;
 * dst_accumulate takes longer lists).  A row's value rows are summed first, in rank and slice order as
 * dst_densify_concat would take the concatenation of all slices, then the dense rows in rank order.
 * `out` may be one of the dense tensors.  Workspace: dst_workspace_bytes(all slice rows, all slices,
 * d, vocab, opts).  Everything else as dst_densify_concat.
 */
typedef struct {
    const void* dense;         /* [vocab, d] in opts->out_type, or NULL */
    const dst_slice_t* slices; /* host array */
    int32_t n_slices;
    int32_t reserved;
} dst_rank_grads_t;

int dst_densify_batch(const dst_rank_grads_t* ranks, int32_t R, int64_t d, int64_t vocab, void* out,
                      dst_stream_t stream, const dst_opts_t* opts, void* workspace, size_t workspace_bytes,
                      void* unique_rows, int32_t* counts, dst_result_t* result);

/*
 * dst_densify_concat fused with the step that follows accumulation in the training loop (Section 4:
 * the optimizer the accumulated gradient is handed to), for plain SGD on the tied weight:
 *
 *     weight[v, c] <- weight[v, c] - lr * (dense_in[v, c] + sum of the value rows that name v)
 *
 * The dense gradient is never written: every weight row is read once and written once, next to the
 * one read of dense_in and of the value rows.  fp32 only (value_type and out_type DST_F32, otherwise
 * DST_ERR_UNSUPPORTED); `weight` is [vocab, d], updated in place, and must not be dense_in.  The
 * gradient of a row is summed in the order dst_densify_concat uses, dense_in last, then one fused
 * multiply-add takes the step.  All other arguments, the optional outputs and the error behaviour are
 * those of dst_densify_concat; rows with an out-of-range index are skipped and reported.
 */
int dst_densify_apply_sgd(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab,
                          const void* dense_in, void* weight, float lr, dst_stream_t stream,
                          const dst_opts_t* opts, void* workspace, size_t workspace_bytes,
                          void* unique_rows, int32_t* counts, dst_result_t* result);

/*
 * The same fusion for the optimizers that keep state (Section 4: whatever optimizer the distributed
 * wrapper is handed; Section 1 for training in reduced precision).  With g the dense gradient
 *
 *     g[v, c] = grad_scale * (dense_in[v, c] + sum of the value rows that name v)
 *
 *   DST_OPT_SGD       weight <- weight - lr * g
 *   DST_OPT_MOMENTUM  state1 <- momentum * state1 + g;   weight <- weight - lr * state1
 *   DST_OPT_ADAM      state1 <- beta1 * state1 + (1 - beta1) * g;   state2 <- beta2 * state2 + (1 - beta2) * g * g
 *                     weight <- weight - lr * (state1 / (1 - beta1^step)) / (sqrt(state2 / (1 - beta2^step)) + eps)
 *
 * g is never written.  weight, state1 and state2 are [vocab, d] fp32 device tensors, updated in
 * place; every row takes the step, named or not (with momentum or Adam a zero gradient still
 * moves the state), and every row of each tensor is read once and written once.  value rows and
 * dense_in have one type, fp32 or bf16 (opts->value_type == opts->out_type, otherwise
 * DST_ERR_UNSUPPORTED): bf16 is the reduced-precision gradient, grad_scale the reciprocal of its
 * loss scale (1 for unscaled gradients), applied to the fp32 sum.  All arithmetic is fp32; the
 * gradient of a row is summed in the order dst_densify_concat uses, dense_in last.  weight must
 * not be dense_in or a state tensor; state tensors a kind does not use may be NULL.  `optimizer`
 * is a HOST struct read during the call.  All other arguments, the optional outputs and the
 * error behaviour are those of dst_densify_concat.
 */
typedef enum { DST_OPT_SGD = 0, DST_OPT_MOMENTUM = 1, DST_OPT_ADAM = 2 } dst_optimizer_kind_t;
typedef struct {
    int32_t kind;     /* dst_optimizer_kind_t */
    int32_t step;     /* DST_OPT_ADAM: the number t of this step, starting at 1 */
    float lr;
    float momentum;   /* DST_OPT_MOMENTUM */
    float beta1;      /* DST_OPT_ADAM */
    float beta2;
    float eps;
    float grad_scale; /* multiplies the summed gradient */
    void* state1;     /* DST_OPT_MOMENTUM: the momentum buffer; DST_OPT_ADAM: the first moment */
    void* state2;     /* DST_OPT_ADAM: the second moment */
} dst_optimizer_t;

int dst_densify_apply(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab,
                      const void* dense_in, void* weight, const dst_optimizer_t* optimizer, dst_stream_t stream,
                      const dst_opts_t* opts, void* workspace, size_t workspace_bytes,
                      void* unique_rows, int32_t* counts, dst_result_t* result);

/*
 * dst_densify without a caller-supplied workspace.  (The paper has no counterpart:
 * this entry point exists for the sake of callers, not of the method.)
 *
 * Who needs it: code that must not, or cannot, obtain device memory at the time it
 * calls -- a plugin running inside a framework whose allocator it may not re-enter,
 * a callback on a path where cudaMalloc's implicit device synchronisation is not
 * acceptable, a process whose memory pool was sized up front and is full.  For those
 * callers the scratch memory lives inside the library: one array of
 * DST_STATIC_WORKSPACE_BYTES in device global memory, reserved on every GPU that
 * loads the library for as long as the process lives.  This call allocates and frees
 * nothing, on the host side through CUDA or otherwise.
 *
 * Arguments, results and summation order are those of dst_densify; the output is
 * bit-identical to dst_densify on the same inputs.  Differences:
 *   - Shapes whose workspace need, dst_workspace_bytes(n_rows, 1, d, vocab, opts),
 *     exceeds DST_STATIC_WORKSPACE_BYTES are refused with
 *     DST_ERR_WORKSPACE_TOO_SMALL before anything is enqueued.
 *   - The first call on each device looks up the array's device address (with that
 *     device current) and keeps it; make that first call outside any stream capture.
 *     A failure of the look-up is reported as DST_ERR_CUDA.
 *   - All calls on one device share the one array, and it keeps what the last call
 *     left in it (each call clears the part that has to start at zero, on `stream`).
 *     Two calls whose work can overlap on the GPU -- different streams without an
 *     ordering between them -- race on it and give wrong results: order them.
 */
#define DST_STATIC_WORKSPACE_BYTES (4u << 20)
int dst_densify_static(const void* indices, const void* values, int64_t n_rows, int64_t d, int64_t vocab,
                       const void* dense_in, void* out, dst_stream_t stream, const dst_opts_t* opts,
                       void* unique_rows, int32_t* counts, dst_result_t* result);

/* Bytes of device staging memory dst_densify_concat_host needs. */
size_t dst_host_staging_bytes(int64_t n_rows_total, int64_t d, int64_t vocab, const dst_opts_t* opts);

/*
 * End-to-end variant for callers whose gradients live in HOST memory: `slices`
 * holds HOST pointers, host_dense_in (nullable) and host_out are HOST buffers
 * (pinned memory makes the copies asynchronous).  Enqueues host-to-device
 * copies of every slice and of dense_in into `staging`, the densify itself,
 * and the device-to-host copy of the result; host_result (nullable, host)
 * receives the dst_result_t.  Nothing is synchronised: host_out is valid once
 * `stream` has drained.  staging: >= dst_host_staging_bytes(...) device bytes.
 */
int dst_densify_concat_host(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab,
                            const void* host_dense_in, void* host_out, dst_stream_t stream,
                            const dst_opts_t* opts, void* staging, size_t staging_bytes,
                            void* workspace, size_t workspace_bytes, dst_result_t* host_result);

/*
 * Accumulating a list of gradients of one variable: the strategies of the paper.
 *
 * A gradient is either a dense [vocab, d] tensor (DST_GRAD_DENSE: `values` holds it, in
 * opts->out_type; `indices` and `n_rows` are ignored) or IndexedSlices (DST_GRAD_SLICES:
 * `indices` [n_rows] in opts->index_type, `values` [n_rows, d] in opts->value_type).
 *
 *   DST_ACC_STOCK            Algorithm 1 (Section 3): fewer than two gradients pass through; if all
 *                            are dense they are summed ("reduce"); otherwise every gradient is
 *                            treated as IndexedSlices -- a dense one becomes vocab slices, row v
 *                            with index v -- and they are concatenated in the order given ("gather").
 *   DST_ACC_PROPOSED         Algorithm 2 (Section 6): as above, but if at least one gradient is dense
 *                            every gradient is converted to a dense tensor and they are summed.
 *   DST_ACC_SPARSE_AS_DENSE  Listing 1 (Section 4): every IndexedSlices gradient is converted to a
 *                            dense tensor first, then Algorithm 1 runs (and can only reduce).
 *
 * dst_accumulate_plan (host only, touches no device memory) says which branch a list takes, what
 * the output is and how large: call it to size the output buffers and the workspace
 * (dst_workspace_bytes(plan.n_slice_rows, plan.n_slices, d, vocab, opts) when plan.converts != 0).
 *
 * dst_accumulate enqueues the work on `stream`:
 *   - dense output  -> out_dense [vocab, d] in opts->out_type, summed in fp32.  With IndexedSlices
 *     among the gradients (or more than eight dense ones and a workspace) everything is accumulated
 *     in one pass, as dst_densify_batch does: a row's value rows first, then the dense gradients in
 *     the order given, except that a gradient that is out_dense itself is taken first; every tensor
 *     crosses the memory bus once.  More than 64 dense gradients: the first ones are summed into
 *     out_dense beforehand (eight per pass, the running sum in opts->out_type between passes).
 *     Dense gradients only, at most eight or without a workspace: those passes alone.
 *     `result` (optional) is written only when slices were converted (plan.converts != 0).
 *   - slices output -> out_indices [out_rows], out_values [out_rows, d]: the concatenation.  Needs
 *     out_capacity_rows >= plan.out_rows, and value_type == out_type when a dense gradient is
 *     among them (its rows are copied, not converted); otherwise DST_ERR_UNSUPPORTED.
 *   - an empty list enqueues nothing (plan.out_kind == -1).
 * A pass-through copies the one gradient into the output buffers of its kind.  `grads` is a HOST
 * array read during the call only.  Outputs must not overlap inputs, except that out_dense may be
 * one of the dense gradients.  `plan` (optional, host) receives what dst_accumulate_plan returns.
 */
typedef enum { DST_GRAD_DENSE = 0, DST_GRAD_SLICES = 1 } dst_grad_kind_t;
typedef struct {
    int32_t kind; /* dst_grad_kind_t */
    int32_t reserved;
    const void* indices;
    const void* values;
    int64_t n_rows;
} dst_grad_t;
typedef enum { DST_ACC_STOCK = 0, DST_ACC_PROPOSED = 1, DST_ACC_SPARSE_AS_DENSE = 2 } dst_strategy_t;
typedef enum {
    DST_BRANCH_EMPTY = 0,
    DST_BRANCH_PASS_THROUGH = 1,
    DST_BRANCH_REDUCE = 2,
    DST_BRANCH_CONVERT_AND_REDUCE = 3,
    DST_BRANCH_GATHER = 4
} dst_branch_t;
typedef struct {
    int32_t branch;       /* dst_branch_t: the line of the algorithm that applies */
    int32_t out_kind;     /* dst_grad_kind_t of the output, -1 for an empty list */
    int64_t out_rows;     /* rows of the output: vocab if dense, the concatenated row count if slices */
    int64_t out_bytes;    /* bytes the output occupies (values, plus indices if slices) */
    int32_t n_dense;      /* dense gradients in the list */
    int32_t n_slices;     /* IndexedSlices gradients in the list */
    int64_t n_slice_rows; /* their rows in total */
    int32_t converts;     /* 1 when IndexedSlices are converted to dense (a workspace is needed) */
    int32_t reserved;
} dst_accum_plan_t;

int dst_accumulate_plan(const dst_grad_t* grads, int32_t n, int64_t d, int64_t vocab, int32_t strategy,
                        const dst_opts_t* opts, dst_accum_plan_t* plan);

int dst_accumulate(const dst_grad_t* grads, int32_t n, int64_t d, int64_t vocab, int32_t strategy,
                   void* out_dense, void* out_indices, void* out_values, int64_t out_capacity_rows,
                   dst_stream_t stream, const dst_opts_t* opts, void* workspace, size_t workspace_bytes,
                   dst_result_t* result, dst_accum_plan_t* plan);

/*
 * Footprint report (Section 4: 11.4 GB gathered vs 139 MB dense at 64 processes).
 * n_rows_per_slice: HOST array of R row counts.  report: HOST.  Pure host arithmetic.
 */
int dst_bytes_report(const int64_t* n_rows_per_slice, int32_t R, int64_t d, int64_t vocab,
                     const dst_opts_t* opts, dst_bytes_report_t* report);

/*
 * Measurement hooks (the paper instruments its runs with Horovod timelines, Section 3
 * Fig. 3; these are the equivalent for this library).
 *
 * dst_profile_events: give two cudaEvent_t handles; every later densify call made by
 * this host thread records `before` right before and `after` right after the
 * row-reduction kernel (the kernel that moves the value, dense_in and out rows) on
 * the call's stream.  Pass NULL, NULL to switch it off (the default).
 * dst_kernel_launches: number of kernels this library has launched in this process.
 * dst_profile_ranges: 1 switches on NVTX ranges on the calling host thread around a call and its
 * phases (index work, row reduction), as a timeline tool shows them; 0 (the default) switches
 * them off.  Process-wide; no environment variable is read.
 */
void dst_profile_events(void* before, void* after);
int64_t dst_kernel_launches(void);
void dst_profile_ranges(int on);

/*
 * Diagnostic of the library's bounded device-side waits (the paper has no counterpart: its
 * failure mode is a host that runs out of memory, Section 3).  Every wait a kernel of this
 * library makes -- on a copy's completion barrier, on a flag another CTA sets -- gives up after
 * a limit, raises DST_ERR_TIMEOUT in the workspace header, and the kernel returns; nothing
 * hangs and nothing traps.  This call runs that give-up path by itself: one CTA waits, with the
 * routine the row-reduction kernel uses, on a barrier that nobody ever arrives on, for at most
 * limit_cycles SM clock cycles (0 < limit_cycles <= 2^31).  When the stream has run,
 * result->status (device or pinned memory, optional) holds DST_ERR_TIMEOUT, and so does the
 * first word of `workspace` (>= 256 bytes, 256-byte aligned, cleared by the call).  The context
 * stays usable; a densify call that follows behaves as usual.
 */
int dst_selftest_wait_limit(int64_t limit_cycles, void* workspace, size_t workspace_bytes, dst_stream_t stream,
                            dst_result_t* result);

#ifdef __cplusplus
}
#endif
#endif /* DST_H_ */
