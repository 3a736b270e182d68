/*
 * gi - graph inference of fused convolutional networks on one NVIDIA B200 (sm_100a).
 *
 * The library implements the GPU inference path of "On-Device Neural Net Inference with
 * Mobile GPUs" (arXiv 1907.01989): a sub-graph of supported operators is handed over once,
 * initialised once, then run many times (Section 3, "General Architecture").
 *
 *   build    gi_graph_create / gi_graph_input / gi_add_op / gi_graph_output
 *   compile  gi_compile   - topological order, fusion of element-wise operators into the
 *                           convolution before them (Section 3.2), tensor lifetimes and the
 *                           memory plan for intermediate tensors (Section 5), weight packing
 *   run      gi_exec_bind, gi_run - enqueue every kernel on the caller's stream, no
 *                           synchronisation with the CPU (Section 3.2, "Running Inference")
 *
 * All functions return a gi_status; none throws, aborts or prints.  A textual description
 * of the last failure on the calling thread is available from gi_last_error().
 *
 * Memory.  The library owns only host memory.  Every device buffer - graph inputs and
 * outputs, the arena that holds intermediate tensors, the packed-weight blob - is allocated
 * and freed by the caller; the library never allocates or frees device memory.  Device
 * pointers passed in must be 256-byte aligned.
 *
 * Layout.  Activations live in a channel-sliced layout (PHWC4, Section 4 "Data Layout"):
 * a [H,W,C] tensor is cut into S = ceil(C/4) slices of 4 channels, missing channels are
 * zero.  For a batch of B images the B planes of one slice are adjacent and the slices
 * follow one another: element (b,h,w,c) is at element index
 *     ((c/4 * B + b) * plane + h*W + w) * 4 + c%4,      plane = H*W rounded up to even.
 * The extra pixel of an odd plane must hold finite values (the library writes zeros or
 * finite values there).  Caller-visible tensors can instead be plain NHWC, in which case
 * the executable starts / ends with a layout conversion kernel (Section 3, "Running
 * Inference").
 */
#ifndef GI_H_
#define GI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define GI_API __attribute__((visibility("default")))
#else
#define GI_API
#endif

typedef int32_t gi_status;
typedef int32_t gi_tensor; /* tensor id within one graph, >= 0 */
typedef struct gi_graph gi_graph;
typedef struct gi_exec gi_exec;

enum {
  GI_OK = 0,
  GI_E_INVALID = -1,     /* bad argument: null pointer, unknown id or kind, shape mismatch */
  GI_E_UNSUPPORTED = -2, /* a well-formed request this library has no kernel for */
  GI_E_NOMEM = -3,       /* host allocation failed */
  GI_E_CUDA = -4,        /* a CUDA call failed; gi_last_error() holds the CUDA error string */
  GI_E_STATE = -5,       /* call out of order (e.g. gi_run before gi_exec_bind) */
  GI_E_ARENA = -6        /* arena / weight buffer too small or misaligned */
};

enum { GI_F16 = 1, GI_F32 = 2 };   /* storage type of activations (and of NHWC inputs/outputs) */
enum { GI_NHWC = 0, GI_PHWC4 = 1 }; /* layout of a caller-visible tensor */

enum {
  GI_OP_CONV2D = 1,           /* full convolution, square kernel 1x1, 2x2 or 3x3, stride 1 to 3 (the sizes and
                                 strides of the search space in Section 4, "Work Group: Choosing the Right Size") */
  GI_OP_DEPTHWISE_CONV2D = 2, /* depthwise 3x3, stride 1 or 2, depth multiplier 1 */
  GI_OP_ADD = 3,              /* element-wise sum of two tensors of the same shape; with inputs[1] = -1 the identity */
  GI_OP_ACTIVATION = 4,       /* ReLU or ReLU6 */
  GI_OP_GLOBAL_AVG_POOL = 5,  /* mean over H*W */
  GI_OP_RESIZE_BILINEAR = 6,  /* bilinear up/down-sampling */
  GI_OP_CONCAT = 7            /* channel concatenation of two tensors of the same height and width: channels of
                                 inputs[0], then those of inputs[1]; with inputs[1] = -1 the identity */
};

enum { GI_ACT_NONE = 0, GI_ACT_RELU = 1, GI_ACT_RELU6 = 2 };

/* Memory planners for intermediate tensors (Section 5, "Memory Manager for Intermediate Tensors"). */
enum {
  GI_PLAN_GREEDY_BY_SIZE = 0,        /* offsets into one buffer, largest tensor first, best-fit gap (default) */
  GI_PLAN_GREEDY_SHARED_OBJECTS = 1, /* Algorithm 1 of the paper, objects laid out in creation order */
  GI_PLAN_NAIVE = 2,                 /* every tensor its own memory (the paper's baseline) */
  GI_PLAN_MIN_COST_FLOW = 3          /* the paper's minimum-cost flow strategy (successive shortest paths, SPFA); shared
                                        objects laid out in creation order; O(N^4) in the number of tensors */
};

/* Kernel choice for full convolutions. */
enum {
  GI_PW_AUTO = 0,      /* tensor-core kernels for fp16 storage (which one: the measured launch table, else a rule), CUDA-core
                          kernel for fp32 storage */
  GI_PW_SIMT = 1,      /* force the plain CUDA-core kernel for every full convolution (validation) */
  GI_PW_TC_PAIR = 2,   /* 1x1: always the pixel-pair tensor-core kernel (operands by TMA) */
  GI_PW_TC_LANE = 3,   /* 1x1: always the lane-per-pixel tensor-core kernel (activations through tensor memory) */
  GI_PW_TC_WIDE = 4,   /* 1x1: always the wide-tile tensor-core kernel built for tensor-bound shapes (256 pixels x up to
                          256 output channels per CTA, both operands streamed) */
  GI_PW_RULE = 5       /* like GI_PW_AUTO, but by the selection rule alone: the table of measured choices (the counterpart of
                          the paper's work-group table, Section 4) is not consulted */
};

/* Cross-operator kernels (fp16 storage).  The "Shader Program Optimization" paragraph of Section 3.2 folds element-wise
 * operators into their producer; these fold whole operators, so that the tensors between them never reach memory:
 *   (1) an inverted-residual block - 1x1 expansion, depthwise 3x3 (stride 1 or 2), 1x1 projection, optional residual
 *       add - on planes of at most 256 pixels with a multiple of 16 input channels runs as ONE kernel;
 *   (2) a depthwise 3x3 convolution whose only consumer is a 1x1 convolution runs with it as one kernel;
 *   (3) two consecutive 1x1 convolutions - a block's projection and the next block's expansion - run as one kernel
 *       that stores both outputs and never reads the tensor between them back.
 * Results are those of the operators run one after the other: the tensors in between are still rounded to fp16.  The
 * memory plan is not affected: those tensors keep their place in the arena, unused; operators whose input and output the
 * planner placed on the same bytes (legal for separate kernels, not for one that reads while it writes) stay separate. */
enum {
  GI_XOP_AUTO = 0,  /* the library's choice, from whole-network measurements (default): (3) for seams on planes of 65 to 256
                       pixels with at most 64 channels between the two convolutions, at least 192 into the first and two
                       pixel tiles per SM; never (1) or (2), which have not measured faster than separate kernels inside
                       the benchmark networks */
  GI_XOP_OFF = 1,   /* one kernel per fused op */
  GI_XOP_ON = 2,    /* (1) wherever the block kernel supports the three ops, else (2) wherever the pair kernel does */
  GI_XOP_CHAIN = 3  /* (3) wherever that kernel supports the two ops; neither (1) nor (2) */
};

/*
 * One operator (Section 3.1: the operators of the delegated sub-graph).
 * Convolutions compute, with out-of-range input reading as zero,
 *   out[b,oy,ox,co] = bias[co] + sum_{ky,kx,ci} in[b, oy*stride_h - pad_t + ky*dilation_h,
 *                                                ox*stride_w - pad_l + kx*dilation_w, ci] * w[co,ky,kx,ci]
 * (Section 4, "For a 2D Convolution"); depthwise is the same sum with co = ci.
 * Output extent: (in + pad_before + pad_after - ((k-1)*dilation + 1)) / stride + 1.
 *
 * weights: host pointer, [cout][kh][kw][cin] for CONV2D, [1][kh][kw][c] for DEPTHWISE_CONV2D,
 * of type weight_dtype (GI_F32 or GI_F16); bias: host pointer to cout floats or NULL.  Both
 * are copied by gi_add_op; the caller may free them as soon as it returns.
 * Unused fields must be zero.  inputs[1] is used by GI_OP_ADD and GI_OP_CONCAT only (elsewhere -1 or 0); there -1
 * means "no second input": the operator is then an identity, which gi_compile removes (Section 3.1).
 */
typedef struct gi_op_desc {
  int32_t kind;
  gi_tensor inputs[2];
  int32_t kh, kw;
  int32_t stride_h, stride_w;
  int32_t dilation_h, dilation_w;
  int32_t pad_t, pad_l, pad_b, pad_r;
  int32_t cout;          /* CONV2D only */
  int32_t act;           /* ACTIVATION only: GI_ACT_RELU | GI_ACT_RELU6 */
  int32_t out_h, out_w;  /* RESIZE_BILINEAR only */
  int32_t align_corners; /* RESIZE_BILINEAR only: 1 -> src = o*(in-1)/(out-1), 0 -> src = o*in/out */
  int32_t weight_dtype;
  const void* weights;
  const float* bias;
} gi_op_desc;

typedef struct gi_compile_options {
  int32_t planner;   /* GI_PLAN_* */
  int32_t fuse;      /* 1: fold element-wise ops into convolutions (default), 0: one kernel per op */
  int32_t align;     /* arena offset / tensor size granularity in bytes, power of two >= 256; 0 -> 256 */
  int32_t pointwise; /* GI_PW_* */
  int32_t cross_op;  /* GI_XOP_* */
} gi_compile_options;

typedef struct gi_exec_info {
  int32_t n_ops;           /* executed ops: layout conversions + fused ops = kernel launches per gi_run */
  int32_t n_fused_ops;     /* fused ops only */
  int32_t n_tensors;       /* tensors of the graph (ids 0 .. n_tensors-1) */
  int32_t batch, storage;
  uint64_t arena_bytes;    /* bytes gi_run needs in dev_arena under the chosen planner */
  uint64_t naive_bytes;    /* sum of all intermediate tensor sizes */
  uint64_t lower_bound_bytes; /* max over ops of bytes alive at that op */
  uint64_t weight_bytes;   /* bytes gi_exec_bind needs in dev_weights */
} gi_exec_info;

typedef struct gi_tensor_info {
  int32_t h, w, c;
  int32_t alive;        /* 0 if fusion removed the tensor */
  int32_t intermediate; /* 1 if it lives in the arena; 2 if it lives inside another arena tensor (an input of a CONCAT
                           that needs no copy: `offset` then points into that tensor) */
  int32_t first_op, last_op; /* executed-op indices, inclusive; -1 if not alive */
  uint64_t bytes;       /* physical size under the size formula */
  uint64_t offset;      /* arena offset (intermediate tensors only) */
} gi_tensor_info;

typedef struct gi_op_info {
  int32_t kind;         /* GI_OP_* of the leading op; GI_EXEC_PACK / GI_EXEC_UNPACK for layout conversions */
  int32_t graph_op;     /* index of the leading op in gi_add_op order; -1 for conversions */
  gi_tensor inputs[2];  /* tensors the leading op reads (-1 = unused / caller buffer) */
  gi_tensor residual;   /* tensor added in the epilogue, or -1 */
  gi_tensor output;     /* tensor written (-1 = caller buffer) */
  int32_t act_pre;      /* activation applied before the residual add */
  int32_t act_post;     /* activation applied after the residual add */
  int32_t kernel;       /* GI_KERNEL_* that runs this op */
  uint64_t bytes;       /* algorithmic bytes: inputs + residual + output once, weights once */
  uint64_t flops;       /* algorithmic flops (2 per multiply-add) */
} gi_op_info;

enum { GI_EXEC_PACK = 100, GI_EXEC_UNPACK = 101 };
enum {
  GI_KERNEL_PACK = 1, GI_KERNEL_UNPACK = 2, GI_KERNEL_CONV_SIMT = 3, GI_KERNEL_POINTWISE_TC = 4,
  GI_KERNEL_DEPTHWISE = 5, GI_KERNEL_ELTWISE = 6, GI_KERNEL_POOL = 7, GI_KERNEL_RESIZE = 8, GI_KERNEL_CONV3X3_TC = 9, GI_KERNEL_POINTWISE_TS = 10,
  GI_KERNEL_DEPTHWISE_POINTWISE = 11, /* this op and the next one, as one kernel */
  GI_KERNEL_NONE = 12,                /* no launch: the op ran inside the previous op's kernel */
  GI_KERNEL_CONCAT = 13,
  GI_KERNEL_CONV_TC = 14,             /* k x k convolution, any number of input channels, on the tensor cores */
  GI_KERNEL_INVERTED_RESIDUAL = 15,   /* this op (1x1 expansion) and the next two (depthwise 3x3, 1x1 projection) as one kernel */
  GI_KERNEL_POINTWISE_MM = 16,        /* 1x1 convolution, wide tiles for tensor-bound shapes */
  GI_KERNEL_POINTWISE_CHAIN = 17      /* this op (1x1) and the next one (1x1) as one kernel; both outputs are stored */
};

/* ---- graph construction (Section 3.1, "Initialization": the sub-graph given to the GPU backend) ---- */

/* Create an empty graph for `batch` images whose activations are stored as `storage`
 * (GI_F16: fp16 storage with fp32 accumulation; GI_F32: fp32 everywhere, for validation).
 * *out is owned by the caller: release with gi_graph_destroy. */
GI_API gi_status gi_graph_create(gi_graph** out, int32_t batch, int32_t storage);

/* Declare a graph input of logical shape [batch,H,W,C]; `layout` says how the caller's device
 * buffer handed to gi_run is laid out (GI_NHWC: batch*H*W*C storage elements; GI_PHWC4: the
 * layout above).  Inputs are numbered in declaration order. */
GI_API gi_status gi_graph_input(gi_graph* g, int32_t H, int32_t W, int32_t C, int32_t layout, gi_tensor* out);

/* Append an operator; its inputs must already exist, so insertion order is a topological
 * order (Section 5 sorts topologically; here the order is given and verified).  *out
 * receives the id of its single output tensor.  GI_E_UNSUPPORTED for kernels other than square
 * 1x1, 2x2 or 3x3 (full convolution, strides 1 to 3) or 3x3 (depthwise, strides 1 or 2), GI_E_INVALID
 * for shape or id errors, GI_E_NOMEM if the copies of weights and bias cannot be allocated (the graph is
 * then unchanged). */
GI_API gi_status gi_add_op(gi_graph* g, const gi_op_desc* desc, gi_tensor* out);

/* Mark a tensor as graph output, delivered to the caller's buffer in `layout`.  Outputs are
 * numbered in the order of these calls.  A graph input cannot be an output. */
GI_API gi_status gi_graph_output(gi_graph* g, gi_tensor t, int32_t layout);

GI_API void gi_graph_destroy(gi_graph* g);

/* ---- compile (Sections 3.2 and 5) ---- */

/* Build an executable: verify the order, clean the graph (Section 3.1: an identity operator - a RESIZE to its
 * input's own size, an ADD or CONCAT with one input - is dropped and its readers read its input, unless its
 * output is a graph output; the dropped op's output tensor is then not alive), fuse, compute lifetimes, plan
 * memory, pack weights, choose a kernel and launch shape per fused op.  With `fuse` set, a CONCAT whose first
 * input has a multiple of 4 channels, and whose inputs and output are neither graph inputs nor outputs, needs
 * no copy: its inputs are placed inside its output (the slices of a tensor follow one another in memory,
 * Section 4), their producers write there, and the CONCAT launches nothing (GI_KERNEL_NONE).
 * Host work only; no CUDA call is made.
 * `opt` may be NULL for defaults.  The graph stays valid and may be compiled again.
 * Two tables generated from measurements on the device (the counterpart of the paper's table of optimal work-group sizes,
 * Section 4) are consulted: which 1x1 kernel runs a shape, and how much the depthwise stencil stages at a time.  The
 * environment variables GI_DW_BUF_KB and GI_DW_CTA_KB, read here, override the second table for every depthwise operator of
 * the graph (largest staging buffer and shared memory of one CTA, in KB); they exist for the tuner that generates it. */
GI_API gi_status gi_compile(const gi_graph* g, const gi_compile_options* opt, gi_exec** out);

GI_API gi_status gi_exec_query(const gi_exec* e, gi_exec_info* info);
GI_API gi_status gi_exec_tensor(const gi_exec* e, gi_tensor t, gi_tensor_info* info);
GI_API gi_status gi_exec_op(const gi_exec* e, int32_t index, gi_op_info* info);

/* Copy the packed weights (info.weight_bytes) into the caller's device buffer, asynchronously
 * on `stream` (a cudaStream_t, NULL for the default stream).  Must precede gi_run; the buffer
 * must stay alive and unmodified as long as the executable is used.  The host staging copy is
 * kept, so binding again (another buffer or device) is allowed. */
GI_API gi_status gi_exec_bind(gi_exec* e, void* dev_weights, size_t weight_bytes, void* stream);

/* Enqueue one inference on `stream` and return without synchronising (Section 3.2: the GPU
 * executes the queued programs without synchronisation with the CPU).  dev_inputs[i] /
 * dev_outputs[i] are device pointers for input / output i in their declared layouts;
 * dev_arena holds the intermediates (>= info.arena_bytes).  Nothing is launched if an
 * argument check fails (GI_E_INVALID, GI_E_ARENA, GI_E_STATE).  Two runs of one executable
 * may overlap on the GPU only if they use different arenas and outputs; several host threads may then
 * call gi_run on that executable at the same time (the per-executable cache of tensor maps is guarded,
 * and keeps the maps of the last four distinct input addresses per launch, so alternating between a
 * few arenas or input buffers re-encodes nothing).  gi_exec_bind and gi_exec_destroy must not run
 * concurrently with gi_run on the same executable.  Results are deterministic: the same inputs give
 * bit-identical outputs. */
GI_API gi_status gi_run(gi_exec* e, const void* const* dev_inputs, void* const* dev_outputs, void* dev_arena,
                 size_t arena_bytes, void* stream);

/* gi_run for callers that cannot allocate device memory.  (The paper has no counterpart: its
 * engine always allocates the buffers its memory manager planned.)
 *
 * Some hosts of this library have no way to hand over an arena: a plug-in whose embedding
 * application owns every device allocation and exposes none to it, a process started with a
 * fixed device-memory budget that is already spent, a service loop that must not call
 * cudaMalloc because that call synchronises the whole device and can fail under fragmentation.
 * For them the intermediates live in a fixed array that is part of the library image itself:
 * GI_STATIC_ARENA_BYTES of device memory on every GPU that loads the library, held until the
 * process exits.  The caller still passes the input and output buffers and must have called
 * gi_exec_bind with a weight buffer it obtained by whatever means it has.
 *
 * The call allocates nothing: no cudaMalloc, cudaFree or allocating library routine.  The
 * first call on a device looks up the array's device address (once per device, with that
 * device current); make that first call outside any stream capture.  An executable whose
 * info.arena_bytes exceeds GI_STATIC_ARENA_BYTES is refused with GI_E_ARENA before anything is
 * launched.  All calls on a device share the one array and it keeps the previous call's
 * contents; nothing in it has to start at zero, because every kernel writes each byte of its
 * output that a later kernel reads (padding lanes and pixels included).  Two calls that overlap
 * on the GPU (different streams, or another thread) race on the array: serialise them. */
#define GI_STATIC_ARENA_BYTES (16u << 20)
GI_API gi_status gi_run_static(gi_exec* e, const void* const* dev_inputs, void* const* dev_outputs, void* stream);

/* Profiling aid: the same launches as gi_run, with a CUDA event recorded before each executed op
 * and after the last one; synchronises `stream` before returning and writes the device time of
 * op i, in milliseconds, to op_ms[i] (n_op_ms must be >= info.n_ops).  The paper's own protocol
 * times whole inferences (Section 6); per-op times are what the per-kernel roofline needs.
 * Creates and destroys CUDA events; not capturable; not for the production path. */
GI_API gi_status gi_run_timed(gi_exec* e, const void* const* dev_inputs, void* const* dev_outputs, void* dev_arena,
                              size_t arena_bytes, void* stream, float* op_ms, int32_t n_op_ms);

/* Health word of the device-side waits.  The tensor-core kernel waits on copy and MMA
 * completion with a limit of about one second per wait; a wait that runs out sets a bit here
 * (1 producer, 2 MMA issuer, 4 epilogue, 8 drain; 0x10000 depthwise staging copy;
 * 0x100000 / 0x200000 / 0x400000 gather / MMA issuer / epilogue of the k x k tensor-core kernels; 0x1000000..0x8000000
 * producer / MMA issuer / data warps / drain of the lane-per-pixel 1x1 kernel; 0x10000000..
 * 0x80000000 copy warp / MMA issuer / compute warps / drain of the depthwise + pointwise kernel), lets the
 * kernel finish without its results
 * and leaves the CUDA context usable.  Sticky until the process exits.  Synchronous: copies
 * the word from the current device. */
GI_API gi_status gi_device_status(uint32_t* flags);

/* Self-test of the give-up path of the device-side waits.  Launches one warp that waits, with the library's own
 * bounded-wait routine and a limit of `limit_us` microseconds (1 .. 100000), on a barrier that nothing ever
 * completes; the wait must run out, raise the kernel's abort flag and error bit, and the kernel must return
 * normally.  Synchronises `stream`.  *waited_us receives how long the wait lasted on the device, *gave_up 1 if it
 * ended by running out (0 would mean the barrier completed, which cannot happen).  The error bit it sets lives in a
 * word of its own: gi_device_status() is not affected and the CUDA context stays usable.  (The paper has no
 * counterpart; its engine has no device-side waits.) */
GI_API gi_status gi_selftest_bounded_wait(uint32_t limit_us, uint32_t* waited_us, int32_t* gave_up, void* stream);


/* Layout experiment (not on the inference path): a 1x1 convolution + bias + activation on tensors stored in slices of
 * EIGHT channels instead of four - [ceil(C/8)][batch][plane][8] fp16, plane = H*W rounded up to even, channels beyond
 * C and the padding pixel zero.  Section 4, "Data Layout", fixes 4 channels per slice because a texel is 4 values; at
 * fp16 a 4-channel pixel-slice is 8 bytes, half of the 16 bytes the tensor core reads as one operand row, so the
 * library's 1x1 kernels either pair pixels or rearrange slices in shared memory.  With 8 channels a pixel-slice IS an
 * operand row and a tiled copy lands a tile where the MMA reads it.  These three calls run the wide-tile 1x1 kernel
 * that way, so that the two layouts can be compared on the same layer (bench.py --sweep slice8):
 *   gi_slice8_pointwise_blob_bytes  bytes of the packed weights + bias of a layer
 *   gi_slice8_pointwise_pack        packs w[cout][cin] and bias[cout] (host, fp32; weights are rounded to fp16 as in
 *                                   gi_add_op) into `host_blob`, which the caller copies to the device (256-byte aligned)
 *   gi_slice8_pointwise_run         enqueues out = act(conv1x1(in) + bias) on `stream`; `dev_in` / `dev_out` are device
 *                                   tensors in the layout above (16-byte aligned, gi_slice8_tensor_bytes each), `act`
 *                                   a GI_ACT_* value.  Needs the wide-tile kernel's support for (cin, cout).
 * The library allocates nothing; errors as everywhere else (GI_E_INVALID, GI_E_UNSUPPORTED, GI_E_CUDA). */
GI_API uint64_t gi_slice8_tensor_bytes(int32_t batch, int32_t H, int32_t W, int32_t C);
GI_API gi_status gi_slice8_pointwise_blob_bytes(int32_t cin, int32_t cout, uint64_t* bytes);
GI_API gi_status gi_slice8_pointwise_pack(const float* w, const float* bias, int32_t cin, int32_t cout, void* host_blob,
                                          uint64_t blob_bytes);
GI_API gi_status gi_slice8_pointwise_run(const void* dev_in, void* dev_out, const void* dev_blob, int32_t batch, int32_t H,
                                         int32_t W, int32_t cin, int32_t cout, int32_t act, void* stream);

GI_API void gi_exec_destroy(gi_exec* e);

/* ---- helpers ---- */
GI_API const char* gi_status_str(gi_status s);
GI_API const char* gi_last_error(void); /* thread-local, valid until the next failing call on this thread */

/* Physical bytes of a [batch,H,W,C] tensor in the library's PHWC4 layout, rounded up to
 * `align` (Section 4; C = 5 costs as much as C = 8). */
GI_API uint64_t gi_tensor_bytes(int32_t batch, int32_t H, int32_t W, int32_t C, int32_t storage, int32_t align);

/* Round n floats to fp16 bit patterns (round to nearest even) exactly as weight packing does. */
GI_API void gi_f32_to_f16(const float* src, uint16_t* dst, size_t n);

#ifdef __cplusplus
}
#endif
#endif /* GI_H_ */
