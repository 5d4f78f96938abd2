/*
 * xenos.h - C ABI of the linked-chain CNN inference library for NVIDIA B200 (sm_100a).
 *
 * The calls follow the paper's statement of the problem (Xenos, arXiv 2302.00282): the user
 * hands over the model as a graph of Table 3 operators together with a description of the
 * hardware (Section 6); the library fuses
 * Conv+Bn+Bias+Relu (Section 4.3), links adjacent operators so a producer hands its tile to
 * the consumer in the order the consumer reads it (Section 4.1, Table 1), splits operators
 * across the parallel units (Section 4.2, Eq. 1), and runs the optimised model, which is
 * equivalent to the original one (Section 3).
 *
 * Conventions
 *  - Plain C, no exceptions cross the boundary.  Every call returns xenos_status_t
 *    (0 = XENOS_OK, negative = error); xenos_last_error() gives a message for the last
 *    failing call on that graph.
 *  - HOST pointers: every pointer inside xenos_op_desc_t, xenos_hw_info_t, id arrays, the
 *    JSON buffer.  They are read during the call only; the caller keeps ownership.
 *  - DEVICE pointers: the workspace given to xenos_graph_bind and the input / output
 *    arrays given to xenos_graph_run.  The library never allocates or frees device memory;
 *    the caller (typically PyTorch) owns all of it and owns the stream.
 *  - There is no CPU fallback: xenos_graph_bind / xenos_graph_run fail with XENOS_E_CUDA
 *    when no sm_100 device is usable.
 *  - State machine: create -> add_input / add_op / mark_output -> (link)* -> (split)* ->
 *    compile -> bind -> run* -> destroy.  A call made in the wrong state returns
 *    XENOS_E_STATE and changes nothing.
 */
#ifndef XENOS_H_
#define XENOS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define XENOS_API __attribute__((visibility("default")))
#else
#define XENOS_API
#endif

typedef struct xenos_graph xenos_graph_t;   /* opaque; owned by the library */
typedef int32_t xenos_status_t;
typedef int32_t xenos_id_t;                 /* tensor id; an operator is named by its output tensor */

enum {
    XENOS_OK = 0,
    XENOS_E_INVALID = -1,       /* null pointer, unknown enum value, bad id                     */
    XENOS_E_SHAPE = -2,         /* operand shapes do not fit the operator                        */
    XENOS_E_UNSUPPORTED = -3,   /* valid request the library has no kernel for                   */
    XENOS_E_NOT_LINKABLE = -4,  /* explicit link request that matches no Table 1 pattern         */
    XENOS_E_BAD_SPLIT = -5,     /* split request that does not divide the operator               */
    XENOS_E_STATE = -6,         /* call out of order                                             */
    XENOS_E_WORKSPACE = -7,     /* workspace missing, too small or misaligned                    */
    XENOS_E_CUDA = -8,          /* CUDA runtime / driver error, or no usable device              */
    XENOS_E_TIMEOUT = -9,       /* a bounded device-side wait expired (status word set)          */
    XENOS_E_BOUNDS = -10        /* a device-side index check failed (status word set)            */
};

/* Operator kinds: the operators of Table 3.  A matrix is a feature map of width 1: h rows of c columns per
 * image (in memory [batch][h][c], the NHWC layout of such a map).  x.matmul takes a constant right operand; a
 * product of two run-time tensors is not implemented (XENOS_E_UNSUPPORTED). */
enum {
    XENOS_OP_CONV = 1,            /* x.conv; groups == 1 dense, groups == Cin == Cout depthwise      */
    XENOS_OP_FC = 2,              /* x.matmul as y = W x + B (Eq. 1); input is a [C] vector per image */
    XENOS_OP_POOL_MAX = 3,        /* x.gampool                                                        */
    XENOS_OP_POOL_AVG = 4,        /* x.gampool, unpadded windows only                                 */
    XENOS_OP_POOL_GLOBAL_AVG = 5, /* x.gampool; output is a [C] vector per image                      */
    XENOS_OP_ADD = 6,             /* x.add, two inputs of equal shape                                 */
    XENOS_OP_CONCAT = 7,          /* x.concat along channels, inputs in argument order               */
    XENOS_OP_RELU = 8,
    XENOS_OP_RELU6 = 9,
    XENOS_OP_BATCHNORM = 10,      /* inference form: gamma * (x - mean) / sqrt(var + eps) + beta      */
    XENOS_OP_MUL = 11,            /* x.mul: element-wise product of two inputs of equal shape          */
    XENOS_OP_MAC = 12,            /* x.mac: three inputs of equal shape, a * b + c element-wise (product rounded, then sum) */
    XENOS_OP_TRANSPOSE = 13,      /* x.transpose of a matrix: (c, h, 1) -> (h, c, 1), y[r][q] = x[q][r] */
    XENOS_OP_SPLIT = 14,          /* x.split, one part per call: channels [pad, pad + cout) of the input */
    XENOS_OP_MATMUL = 15          /* x.matmul: A (h rows x c columns, or a vector) times the constant matrix
                                     `weight` = B [c][cout] row-major, plus `bias` [cout] if given; the
                                     result has cout columns.  MatmulX -> MatmulY (Table 1): two such products
                                     with no activation between them are linked by multiplying the constants
                                     when that does not add work */
};

enum { XENOS_ACT_NONE = 0, XENOS_ACT_RELU = 1, XENOS_ACT_RELU6 = 2 };
enum { XENOS_DTYPE_F32 = 0, XENOS_DTYPE_BF16 = 1 };
enum { XENOS_LAYOUT_NCHW = 0, XENOS_LAYOUT_NHWC = 1 };

/* Arithmetic of a compiled graph.
 *  FP32_CUDA_CORE: fp32 storage and fp32 FMA on CUDA cores, NCHW tensors.
 *  BF16_TENSOR:    bf16 storage (round to nearest even), fp32 accumulation; dense and
 *                  pointwise convolutions and FC run as implicit GEMM on tcgen05 tensor
 *                  cores; tensors between kernels are NHWC bf16. */
enum { XENOS_PRECISION_FP32_CUDA_CORE = 0, XENOS_PRECISION_BF16_TENSOR = 1 };

/* The hardware description the optimiser needs - sizes of the memory levels and the number
 * of parallel units (Section 6) - in this device's terms.  Pass NULL to xenos_graph_create for the B200 defaults
 * (148 SMs, 227 KB shared memory per block, 512 tensor-memory columns, 126 MB L2). */
typedef struct {
    int32_t sm_count;             /* parallel units the split pass deals tiles to       */
    int32_t smem_bytes_per_cta;   /* private memory of one unit                         */
    int32_t tmem_columns;         /* accumulator columns of one unit (fp32, 128 lanes)  */
    int64_t l2_bytes;             /* memory shared by all units                         */
} xenos_hw_info_t;

/* One operator (Table 3).  Unused fields are zero / NULL.
 * weight: CONV: [cout][cin/groups][kh][kw] fp32;  FC: [cout][cin] fp32.
 * bias:   [cout] fp32 or NULL.
 * bn_*:   CONV / FC may carry an inference BatchNorm directly (all four non-NULL), and an
 *         activation, i.e. the already fused CBR form; alternatively BATCHNORM, RELU and
 *         RELU6 are added as operators of their own and fused by xenos_graph_compile.
 *         For XENOS_OP_BATCHNORM the four bn_* arrays are [C] of the input.
 * kh must equal kw.  POOL_*: kh = window, stride, pad; POOL_AVG requires pad == 0. */
typedef struct {
    int32_t kind;
    int32_t cout, kh, kw, stride, pad, groups;
    int32_t act;
    const float *weight;
    const float *bias;
    const float *bn_gamma, *bn_beta, *bn_mean, *bn_var;
    float bn_eps;
} xenos_op_desc_t;

/* Create an empty graph.  hw may be NULL.  *out is owned by the library until
 * xenos_graph_destroy.  Section 6 (user supplies graph + hardware information). */
XENOS_API xenos_status_t xenos_graph_create(const xenos_hw_info_t *hw, xenos_graph_t **out);

/* Declare a graph input of c x h x w per image (batch is given at compile / run).
 * dtype / layout describe the caller's device buffer handed to xenos_graph_run:
 * FP32_CUDA_CORE graphs take F32 NCHW; BF16_TENSOR graphs take F32 or BF16 NCHW when the
 * input feeds a convolution with fewer than 8 input channels (an image), BF16 NHWC with a
 * channel count that is a multiple of 8 otherwise. */
XENOS_API xenos_status_t xenos_graph_add_input(xenos_graph_t *g, int32_t dtype, int32_t layout,
                                               int32_t c, int32_t h, int32_t w, xenos_id_t *tensor);

/* Append one operator reading `inputs` (tensor ids) and producing *out_tensor.  Shapes are
 * inferred here: out = floor((in + 2 pad - k) / stride) + 1.  Weights are copied. */
XENOS_API xenos_status_t xenos_graph_add_op(xenos_graph_t *g, const xenos_op_desc_t *desc,
                                            const xenos_id_t *inputs, int32_t n_inputs,
                                            xenos_id_t *out_tensor);

/* Mark a tensor as a graph output.  The caller's buffer is dense: feature maps
 * [batch][C][H][W] (NCHW) or [batch][H][W][C] (NHWC), vectors [batch][C].
 * FP32 graphs: F32 NCHW.  BF16 graphs: vectors F32; feature maps BF16 NHWC. */
XENOS_API xenos_status_t xenos_graph_mark_output(xenos_graph_t *g, xenos_id_t tensor,
                                                 int32_t dtype, int32_t layout);

/* Operator linking (Section 4.1, Table 1).
 *  n_ops == 0: automatic scan of the whole graph for every linkable pattern.
 *  n_ops  > 0: link exactly this producer->consumer sequence (ids of the operators' output
 *              tensors, in execution order; BatchNorm / activation records belong to their
 *              convolution and are not listed).  XENOS_E_NOT_LINKABLE if the sequence is
 *              not adjacent (checked here) or matches no pattern with a kernel (checked by
 *              xenos_graph_compile).
 * Never called: every operator runs as its own kernel (the unlinked baseline; the
 * Conv-Bn-Relu pre-fusion still applies, as in the paper's Section 3). */
XENOS_API xenos_status_t xenos_graph_link(xenos_graph_t *g, const xenos_id_t *ops, int32_t n_ops);

/* Operator split (Section 4.2, Eq. 1).  op == -1: automatic for every chain (output
 * channels first, then rows / columns of the feature map; the reduction is cut only when
 * the tiles would leave most units idle and the reduction is long: fc, late convolutions
 * at small batch).  Otherwise fix the split of the chain that produces tensor `op`:
 * parts_outc x parts_h x parts_w pieces (0 = automatic for that dimension); parts_k > 1
 * requests the reduction (C / R / S) split of Section 4.2.2: the reduction index, in the
 * kernel's (tap, channel) order and in blocks of 64 elements, is cut into parts_k chunks
 * of equal size (the last may be shorter); each chunk's partial sums are fp32 and are
 * added in ascending chunk order, so results do not vary from run to run, but they are not
 * bit-equal to the unsplit plan.  parts_k applies to tensor-core convolutions (a linked
 * shortcut convolution is cut with its block: the chunks are blocks of the concatenated
 * reduction), depthwise -> pointwise chains and fc that store their tile; not to an image
 * stem or a pooling / global-average epilogue (XENOS_E_UNSUPPORTED, from compile).
 * XENOS_E_BAD_SPLIT (from this call or from compile) if a count exceeds the extent it
 * divides, leaves a chunk empty or breaks a kernel limit. */
XENOS_API xenos_status_t xenos_graph_split(xenos_graph_t *g, xenos_id_t op, int32_t parts_outc,
                                           int32_t parts_h, int32_t parts_w, int32_t parts_k);

/* Profiling-driven split search (Algorithm 1, "Enumerating Partition Schemes", Section 5, restated for one
 * GPU): for every chain the library enumerates split schemes (output-channel parts and reduction parts of a
 * tensor-core chain; output-channel / row / column parts of the fp32 chain), compiles trial plans, runs each
 * `repeats` times at batch = max_batch on the caller's buffers and keeps, per chain, the fastest scheme, which
 * it records as if xenos_graph_split had been called; chains whose split the caller fixed are left alone.
 * Call it after the link requests and before xenos_graph_compile, with the same max_batch and precision.
 * workspace_dev: DEVICE, 256-byte aligned, large enough for every trial plan (a little more than the plain
 * plan: XENOS_E_WORKSPACE names the size when it is not); inputs_dev / outputs_dev as for xenos_graph_run, with
 * valid images in the inputs (outputs are overwritten).  The call synchronises the stream.  report_json
 * (HOST, may be NULL) receives {"trials", "chains":[{"id","tensor","chosen","candidates":[{"label",
 * "parts_outc","parts_h","parts_w","parts_k","us"}]}]}; *needed (HOST) the bytes it takes.
 * Errors: XENOS_E_STATE after compile, XENOS_E_CUDA without an sm_100 device, otherwise those of compile / run. */
XENOS_API xenos_status_t xenos_graph_search_split(xenos_graph_t *g, int32_t max_batch, int32_t precision,
                                                  void *workspace_dev, size_t workspace_bytes,
                                                  const void *const *inputs_dev, void *const *outputs_dev,
                                                  void *cuda_stream, int32_t max_trials, int32_t repeats,
                                                  char *report_json, size_t cap, size_t *needed);

/* Host only: pre-fusion, BatchNorm folding, link + split plans, weight packing, workspace
 * layout.  *workspace_bytes receives the device bytes xenos_graph_bind needs. */
XENOS_API xenos_status_t xenos_graph_compile(xenos_graph_t *g, int32_t max_batch, int32_t precision,
                                             size_t *workspace_bytes);

/* Attach a caller-owned DEVICE workspace (256-byte aligned, >= workspace_bytes) and upload
 * the packed weights into it on `cuda_stream` (a cudaStream_t; NULL = default stream).
 * The workspace must stay valid and unshared until destroy or the next bind. */
XENOS_API xenos_status_t xenos_graph_bind(xenos_graph_t *g, void *workspace_dev, size_t bytes,
                                          void *cuda_stream);

/* Enqueue one inference of `batch` (<= max_batch) images on `cuda_stream`.
 * inputs_dev / outputs_dev: HOST arrays of DEVICE pointers in declaration order; every
 * pointer must be 16-byte aligned (XENOS_E_INVALID otherwise: the kernels use 16-byte
 * vector accesses and TMA).  Asynchronous; does not synchronise.  Launch errors are returned, device-side status is
 * read with xenos_graph_status. */
XENOS_API xenos_status_t xenos_graph_run(xenos_graph_t *g, int32_t batch,
                                         const void *const *inputs_dev, void *const *outputs_dev,
                                         void *cuda_stream);

/* Like xenos_graph_run, but brackets every kernel launch with CUDA events on `cuda_stream`,
 * synchronises, and writes the device time of launch i (milliseconds) to ms_per_launch[i]
 * (HOST array of n_launches = xenos_graph_launch_count entries).  This is the PROFILING step
 * of the paper's Algorithm 1 ("Enumerating Partition Schemes") for one fixed scheme; it
 * creates and destroys CUDA events, allocates no device memory, and is not for hot loops. */
XENOS_API xenos_status_t xenos_graph_profile(xenos_graph_t *g, int32_t batch,
                                             const void *const *inputs_dev, void *const *outputs_dev,
                                             void *cuda_stream, float *ms_per_launch, int32_t n_launches);

/* Run one inference WITHOUT a caller-provided workspace.  (The paper has no counterpart: this
 * entry point exists for deployment settings, not for the method.)
 *
 * Who needs it: code that runs where device allocation is forbidden or unavailable - a plugin
 * inside a host application that owns and has already carved up all device memory, a
 * real-time loop that is not allowed to call the allocator, a process whose memory pool is
 * exhausted.  Such a caller cannot obtain the workspace xenos_graph_bind expects.  Here the
 * workspace is a fixed 16 MiB array that is part of the library image (every device that
 * loads the library holds it until the process exits); the caller passes only its input and
 * output buffers, exactly as for xenos_graph_run.
 *
 *  - Valid on a compiled graph, bound or not; an existing xenos_graph_bind binding is left
 *    untouched.  Graphs whose workspace_bytes exceed 16 MiB are refused with
 *    XENOS_E_WORKSPACE and a message giving both sizes.
 *  - Calls no cudaMalloc / cudaFree and no allocating library routine.
 *  - The first call on a device looks up the array's device address and uploads the graph's
 *    parameters into it; make that first call outside any stream capture.  Parameters are
 *    uploaded again whenever another graph has used the array in between.
 *  - All graphs and all calls share the one array, and it keeps the previous call's contents
 *    (the library clears the words that must start at zero).  Two calls that overlap on the
 *    device - different streams or different host threads - race; serialise them.
 *  - Synchronous: it waits for `cuda_stream` and returns the device status like
 *    xenos_graph_status. */
XENOS_API xenos_status_t xenos_graph_run_builtin_scratch(xenos_graph_t *g, int32_t batch,
                                                         const void *const *inputs_dev,
                                                         void *const *outputs_dev, void *cuda_stream);

/* Synchronise `cuda_stream` and return the device status word: XENOS_OK, or
 * XENOS_E_TIMEOUT / XENOS_E_BOUNDS if a kernel gave up a bounded wait or failed an index
 * check since the last call (the word is then cleared). */
XENOS_API xenos_status_t xenos_graph_status(xenos_graph_t *g, void *cuda_stream);

/* Diagnostic.  Every device-side wait of the chain kernels is bounded; when one runs out the
 * kernel records XENOS_E_TIMEOUT in the graph's status word and returns.  This call enqueues
 * a one-thread kernel on `cuda_stream` that waits for four short polls on a barrier nothing
 * signals and then reports exactly that way, so that the report path can be checked on a
 * healthy device: the next xenos_graph_status returns XENOS_E_TIMEOUT once, later runs are
 * unaffected.  Valid on a bound graph.  (No counterpart in the paper.) */
XENOS_API xenos_status_t xenos_graph_selftest_wait_expiry(xenos_graph_t *g, void *cuda_stream);

/* Write the compiled plan as JSON into `json` (capacity `cap`, always NUL-terminated when
 * cap > 0); *needed receives the length including the NUL.  Contents: fused operators,
 * chains with their Table 1 pattern, tiles, halos, grid, CTA -> tile rule, workspace
 * offsets, and modelled bytes / FLOPs per chain.  Deterministic: equal graphs and options
 * give byte-identical plans. */
XENOS_API xenos_status_t xenos_graph_get_plan(const xenos_graph_t *g, char *json, size_t cap,
                                              size_t *needed);

/* Graph image (Section 6: the optimiser's output is an executable of the optimised model that is stored and later
 * handed to the runtime; Section 3: it takes the place of the original model file).
 * xenos_graph_save writes g as one self-contained byte string into host_buf (host memory, capacity cap bytes) and
 * sets *needed to its length; with host_buf == NULL it only reports the length.  The image holds the hardware
 * description, every tensor and operator with its parameters, the link and split requests and, if g has been
 * compiled, the compile options.  It holds no pointer and no device address.  g is not changed and may be in any
 * state.  Errors: XENOS_E_INVALID (needed is NULL, buffer too small).
 * xenos_graph_load builds a new graph (owned by the library, release with xenos_graph_destroy) from the bytes bytes
 * at host_buf.  If the saved graph was compiled, the new one is compiled with the same options (planning is
 * deterministic: its plan equals the saved graph's byte for byte) and *workspace_bytes, when not NULL, receives the
 * workspace it needs; otherwise the graph is returned in build state and *workspace_bytes is 0.  The caller binds a
 * workspace as usual.  Errors: XENOS_E_INVALID for anything that is not an intact image of this library version
 * (bad magic, version, checksum, counts or indices), or the status of the failing compile; *out is NULL then and
 * xenos_last_error(NULL) holds the message. */
XENOS_API xenos_status_t xenos_graph_save(const xenos_graph_t *g, void *host_buf, size_t cap, size_t *needed);
XENOS_API xenos_status_t xenos_graph_load(const void *host_buf, size_t bytes, xenos_graph_t **out,
                                          size_t *workspace_bytes);

/* Number of kernel launches one xenos_graph_run enqueues (valid after compile). */
XENOS_API xenos_status_t xenos_graph_launch_count(const xenos_graph_t *g, int32_t *launches);

XENOS_API xenos_status_t xenos_graph_destroy(xenos_graph_t *g);

/* Message of the last failing call on g (never NULL; valid until the next call on g).
 * With g == NULL: message of the last failing xenos_graph_create on this thread. */
XENOS_API const char *xenos_last_error(const xenos_graph_t *g);

#ifdef __cplusplus
}
#endif
#endif /* XENOS_H_ */
