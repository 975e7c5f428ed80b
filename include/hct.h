/*
 * hct — fused operator-chain execution on one NVIDIA B200 (sm_100a).
 *
 * A computation graph is a DAG whose nodes are computations and whose edges
 * are data flow (paper §3.2).  The operators are the classes of the paper's
 * Table 1 that dominate fused deep-learning chains: elementwise and
 * activation, broadcast, row reductions (softmax, layer normalisation, sums),
 * GEMM and conv2d.  hct_graph_create() reads a text description of such a
 * graph, checks it (acyclic, operand shapes and dtypes consistent, nothing
 * dangling — the validity rules of §3.2), partitions it into fused kernels,
 * generates and compiles them for sm_100a, and returns a handle;
 * hct_graph_run() launches those kernels on caller-owned device memory.
 *
 * There is no CPU execution path: if the device is not compute capability
 * 10.x, or a kernel cannot be built, the call fails with an error code.
 *
 * Spec text (line oriented, '#' starts a comment):
 *
 *     hct 1
 *     input  NAME DTYPE [d0,d1,...] [nhwc]    DTYPE: f32 | bf16, rank 1..4; `nhwc` after a bf16 [N,C,H,W] shape says
 *                                             the buffer is channels-last, x[n][h][w][c] (only as conv2d's first
 *                                             operand: such a convolution needs no layout pass over its activations)
 *     node   NAME = OP(arg, ..., key=value)   args: earlier names or (binary ops) a number
 *     output NAME [DTYPE [nhwc]]              stored dtype, default f32; `nhwc` after the dtype of a rank-4 value says the
 *                                             output buffer is channels-last, y[n][h][w][c] (extents stay [N,C,H,W]); only
 *                                             for values stored by a convolution kernel (the convolution or the elementwise
 *                                             nodes fused behind it), otherwise HCT_ERR_UNSUPPORTED.  With an nhwc input
 *                                             and an nhwc output a chain of graphs stays channels-last with no layout pass
 *
 *   unary   relu gelu_tanh gelu_erf sigmoid exp tanh sqrt sin cos neg abs log rsqrt square reciprocal
 *           cast_bf16(x)   rounds to bfloat16 (nearest even); the result may be the first operand of a bf16
 *           gemm / conv2d and is kept as bf16 where it is materialised between kernels
 *           dropout(x, p=0.5, seed=0)   inverted dropout with the counter-based mask of the
 *           paper's first case study (Section 5.3, "Detailed Case Study"): with i the element's row-major offset,
 *           h = i + seed; h ^= h >> 17; h ^= h << 31; h ^= h >> 8 (unsigned 64 bit); the
 *           element is kept and scaled by 1/(1-p) when h mod 1000 >= round(1000 p), else 0
 *   binary  add sub mul div max min   operands broadcast like numpy; supported
 *           patterns: equal shapes, [C] against [..,C], [..,1] against [..,C],
 *           [K,1,1] against [N,K,H,W], a number
 *   row     row_softmax(x)  row_sum(x)  row_mean(x)  row_max(x)  row_min(x)   x: [R,C]; reductions give [R,1]
 *           row_argmax(x)  row_argmin(x)   column of the extreme element, the first among equals, as an fp32 value
 *           (row_softmax also accepts a single column, where it is identically one)
 *           row_layernorm(x, gamma, beta, eps=1e-5)   biased variance, eps inside the root
 *   row_argsort(x, descending=0)  row_topk_indices(x, k=K)   the columns the values of row_sort / row_topk came
 *                         from, as fp32 values; among equal values (-0 and +0 are equal) the smaller column first
 *   transpose(x)          y[j,i] = x[i,j] for x[R,C]; elementwise consumers are applied at the store
 *   permute(x, axes=DIGITS)  the axes of x (rank 2..4) in another order: output axis d is input axis DIGITS[d]
 *                         (axes=0231 turns [N,C,H,W] into [N,H,W,C]); a bf16 value stays bf16; one pass, elementwise
 *                         consumers applied at the store
 *   reshape(x, rows=R, cols=C)   the elements of x (any rank) in row-major order as [R,C], R*C = numel(x);
 *                         a bf16 value stays bf16; one copy pass, elementwise consumers applied at the store
 *   row_sort(x, descending=0)   the values of every row of x[R,C] in non-decreasing (descending=1:
 *                         non-increasing) order; row_topk(x, k=K) the K largest values of every row,
 *                         largest first, as [R,K].  C <= 8192.  Values are moved, never changed;
 *                         elementwise consumers are applied at the store
 *   gemm(a, b)            a[M,K] · b[K,N], both row-major, both f32 or both bf16 inputs;
 *                         bf16 multiplies on tensor cores with fp32 accumulation, f32
 *                         uses error-compensated TF32 products (or fp32 FMA for shapes
 *                         the tensor-core path does not take)
 *   conv2d(x, w, stride=1, pad=0, dilation=1, groups=1)   x[N,C,H,W], w[K,C/groups,R,S]; cross-correlation,
 *                         zero padding; y[n,k,h,w] = sum x[n,c,h*stride-pad+r*dilation, w*stride-pad+s*dilation] * w[k,c',r,s]
 *                         over the C/groups channels c of filter k's group (groups = C: depthwise).
 *                         bf16 operands run on tensor cores (strides up to 8): 1x1 at stride 1 on NCHW data as one
 *                         GEMM per image with no layout pass at all; groups between 1 and C by contracting, per
 *                         block of 128 filters, the dense window of input channels its groups span against weights
 *                         that are zero outside each filter's own group (so a non-finite activation in one group
 *                         makes NaN in the results of the other groups of its window, where the definition gives a
 *                         finite value).  Depthwise convolutions, fp32 operands and grouped shapes whose windows do
 *                         not start on 16-byte boundaries run on fp32 FMA kernels
 *
 * Every computed value is fp32; bf16 inputs are widened exactly; an output
 * stored as bf16 is rounded to nearest-even once, at the store.
 *
 * All tensors are dense, contiguous and row-major (conv2d: NCHW / KCRS).
 * Pointers passed to hct_graph_run are DEVICE pointers, 16-byte aligned.
 * Functions return HCT_OK or an error code; the text of the last error on the
 * calling thread is available from hct_last_error().  No exception crosses
 * this boundary.
 */
#ifndef HCT_H_
#define HCT_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define HCT_API __attribute__((visibility("default")))
#else
#define HCT_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hct_graph hct_graph_t; /* opaque; owned by the library until hct_graph_destroy */

typedef enum {
  HCT_OK = 0,
  HCT_ERR_INVALID_ARG = 1, /* null pointer, wrong count, misaligned pointer, workspace too small */
  HCT_ERR_PARSE = 2,       /* spec syntax; message carries the line                         */
  HCT_ERR_GRAPH = 3,       /* undefined or forward operand (cycle / dangling node), node that
                              reaches no output, dtype or shape mismatch (paper §3.2)       */
  HCT_ERR_UNSUPPORTED = 4, /* valid graph outside the supported set; never a CPU fallback   */
  HCT_ERR_COMPILE = 5,     /* kernel compilation or module load failed                      */
  HCT_ERR_CUDA = 6,        /* driver error at launch or query; code in the message          */
  HCT_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired (read by hct_graph_status) */
  HCT_ERR_ARCH = 8,        /* device is not compute capability 10.x                         */
  HCT_ERR_OOM = 9
} hct_status_t;

enum { HCT_F32 = 0, HCT_BF16 = 1 };

/* Device id that asks for planning and kernel compilation only (no CUDA driver
 * needed); the handle can be queried but not run. */
#define HCT_DEVICE_NONE (-1)

/*
 * Build a graph handle from spec text (host memory, spec_len bytes, need not
 * be NUL-terminated).  Parses and validates the DAG (§3.2), infers shapes,
 * plans the fused kernels, compiles them for sm_100a and, unless device is
 * HCT_DEVICE_NONE, loads them on CUDA device `device` (its primary context).
 * On success *out owns the handle; on failure *out is NULL.
 * Host-only work plus module loading; no kernel is launched.
 */
HCT_API hct_status_t hct_graph_create(const char* spec, size_t spec_len, int device, hct_graph_t** out);

/*
 * Launch the graph's kernels, in dependency order, on `cuda_stream`
 * (a cudaStream_t / CUstream; NULL is the default stream).  This is the step
 * the paper's pipeline repeats for every candidate (Section 3.5: compile, then
 * execute on the device and time).  Does not synchronise.
 *   inputs[i]   device pointer to the i-th `input` line's tensor (read only)
 *   outputs[i]  device pointer to the i-th `output` line's tensor (written)
 *   workspace   device scratch of at least hct_graph_workspace_bytes() bytes,
 *               256-byte aligned, caller-owned; may be NULL when that is 0
 * Outputs must not alias inputs or the workspace.  A handle is used by one
 * thread at a time.  Errors: HCT_ERR_INVALID_ARG (counts, NULL or misaligned
 * pointers, small workspace), HCT_ERR_CUDA (launch failure).
 */
HCT_API hct_status_t hct_graph_run(hct_graph_t* g, const void* const* inputs, int n_inputs, void* const* outputs,
                           int n_outputs, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * hct_graph_create with a schedule: `schedule` is NULL (defaults) or text of the form
 * "knob=integer;knob=integer" that overrides launch-shape knobs of the generated kernels
 * (threads per row, vectors per thread, CTAs per SM, ring sizes, which convolution schedule;
 * the knob names are those printed by hct_graph_schedule after a tuning run).  Results do not
 * depend on the schedule beyond rounding order.  An unknown knob gives HCT_ERR_INVALID_ARG.
 */
HCT_API hct_status_t hct_graph_create_scheduled(const char* spec, size_t spec_len, int device, const char* schedule,
                                                hct_graph_t** out);

/*
 * Measure-and-pick: builds the graph under up to max_trials candidate schedules, runs each on
 * the caller's buffers (same arguments as hct_graph_run; all DEVICE pointers, caller-owned,
 * outputs are overwritten), times it with events on `cuda_stream`, and returns the fastest
 * handle in *out.  Trials run with a cold L2 when the workspace has at least 160 MiB to spare
 * beyond what the candidates need (that part is overwritten before every run; nothing is
 * allocated), otherwise warm; a trial is the smallest of three batches of ten runs, and a
 * candidate replaces the incumbent only when it is at least 2 % faster.  This is the role the measurement trials of the auto-scheduler play in the
 * paper's pipeline (Section 3.5: every candidate is compiled and executed on the device, the
 * best one is kept), restricted to this library's own knobs.  The call SYNCHRONISES the stream
 * repeatedly and is meant for set-up time.  Candidates that need more workspace than
 * workspace_bytes, do not apply to the graph or fail to build are skipped; the default
 * schedule is always measured, so a handle is returned whenever hct_graph_create would succeed
 * and the buffers fit.  Errors as for hct_graph_create / hct_graph_run.
 */
HCT_API hct_status_t hct_graph_autotune(const char* spec, size_t spec_len, int device, const void* const* inputs, int n_inputs,
                                        void* const* outputs, int n_outputs, void* workspace, size_t workspace_bytes,
                                        void* cuda_stream, int max_trials, hct_graph_t** out);

/* The schedule text a handle was built with ("" for the defaults); owned by the handle. */
HCT_API const char* hct_graph_schedule(const hct_graph_t* g);

/*
 * The "execute" phase's error report (paper Section 3.6: a candidate that loads and compiles may
 * still fail when it runs).  After the caller has synchronised the stream: reads the handle's device
 * status word.  HCT_OK, or HCT_ERR_TIMEOUT if a kernel gave up on a bounded
 * wait (its outputs are then undefined).  Clears the word.
 */
HCT_API hct_status_t hct_graph_status(hct_graph_t* g);

/* Release the handle and everything it owns: modules, the status word, host state (Section 3.5: a compiled
 * candidate is discarded after its measurement).  NULL is accepted. */
HCT_API hct_status_t hct_graph_destroy(hct_graph_t* g);

/* ---- queries (host only): what shape and type inference (Section 3.2: operator types must agree with the
 * shapes and dtypes of their operands) and the fusion plan (Section 3.5: one schedule per fused graph) decided ---- */
HCT_API int hct_graph_num_inputs(const hct_graph_t* g);
HCT_API int hct_graph_num_outputs(const hct_graph_t* g);
/* Name (owned by g), dtype (HCT_F32/HCT_BF16), rank and extents of an input (is_output = 0)
 * or output (is_output = 1) tensor, as inferred from the spec. */
HCT_API hct_status_t hct_graph_tensor_info(const hct_graph_t* g, int is_output, int idx, const char** name, int* dtype,
                                   int* rank, int64_t shape[4]);
HCT_API size_t hct_graph_workspace_bytes(const hct_graph_t* g);
/* Number of kernel launches one hct_graph_run issues. */
HCT_API int hct_graph_num_kernels(const hct_graph_t* g);
/* Memory layout of input `idx`: 0 = row-major in the declared order of extents (NCHW for rank 4),
 * 1 = declared `nhwc`: extents are still reported as [N,C,H,W], the buffer holds x[n][h][w][c].  -1: bad index. */
HCT_API int hct_graph_input_layout(const hct_graph_t* g, int idx);
/* Memory layout of output `idx`, same codes: 1 = declared `output NAME DTYPE nhwc`. */
HCT_API int hct_graph_output_layout(const hct_graph_t* g, int idx);
/*
 * Work accounting for roofline figures.  algorithmic_bytes: every graph input
 * read once and every output written once, plus one write and one read for
 * each intermediate that no single pass can keep on chip: a value that
 * depends on a reduction (row reduction or contraction) and feeds a
 * contraction or transposition, and a contraction's result that feeds a row
 * reduction over rows wider than 512 columns.  Elementwise producers of a
 * contraction, sorts and reshapes are free.
 * flops: 2·M·N·K summed over the contractions.
 */
HCT_API hct_status_t hct_graph_cost(const hct_graph_t* g, double* algorithmic_bytes, double* flops);
/* Human-readable fusion plan: one line per kernel with its nodes.  Owned by g. */
HCT_API const char* hct_graph_plan_text(const hct_graph_t* g);
/* Generated CUDA source / entry-point name of kernel `idx` (0 <= idx < num_kernels).  Owned by g. */
HCT_API const char* hct_graph_kernel_source(const hct_graph_t* g, int idx);
HCT_API const char* hct_graph_kernel_name(const hct_graph_t* g, int idx);

/*
 * relu(A*B + bias) in fp32 without any device allocation, for callers that must not or cannot
 * allocate: code that runs inside another framework's memory pool with a fixed budget, real-time
 * loops where an allocation would be a stall or a failure point, and start-up paths that run
 * before an allocator exists.  (The paper has no counterpart; this is a convenience of this
 * library.)  hct_graph_run needs caller-provided workspace for the split operands of an fp32
 * GEMM; here that scratch is a fixed array of HCT_STATIC_SCRATCH_BYTES inside the library image,
 * present on every GPU that loads the library until the process exits.
 *   a[m,k], b[k,n], out[m,n] row-major fp32 DEVICE pointers on `device`; bias[n] or NULL;
 *   apply_relu != 0 applies max(.,0).  Operands are split into TF32 head and tail and multiplied
 *   as three products per term with fp32 FMA accumulation; results agree with hct_graph_run's
 *   fp32 GEMM to the library's fp32 tolerance, not bit for bit.
 * Limit: m*k + k*n <= HCT_STATIC_SCRATCH_BYTES/8 elements, else HCT_ERR_UNSUPPORTED.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with that
 * device made current for the duration of the call); make that first call before starting any
 * stream capture.  The call launches on `cuda_stream` and does not synchronise.  It calls no
 * allocating routine.  All calls share the one array: nothing in it needs to start at zero (each
 * call overwrites the part it reads), but two calls whose kernels overlap on the GPU (different
 * streams, or several host threads) race on it; keep them on one stream or order them yourself.
 * A CUDA error already pending on the calling thread is reported by this call (HCT_ERR_CUDA) and
 * left pending.  The looked-up address is cached per device for the life of the process: after
 * cudaDeviceReset on that device it is stale and this entry point must not be used again.
 */
#define HCT_STATIC_SCRATCH_BYTES (8u << 20)
HCT_API hct_status_t hct_gemm_bias_relu_f32_static(const float* a, const float* b, const float* bias, float* out, int64_t m,
                                                   int64_t k, int64_t n, int apply_relu, int device, void* cuda_stream);

/* Message of the last failing call on this thread ("" if none). */
HCT_API const char* hct_last_error(void);
HCT_API const char* hct_version(void);

#ifdef __cplusplus
}
#endif
#endif /* HCT_H_ */
