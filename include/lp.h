/*
 * lp.h - C ABI of the layer-parallel training step (single B200, sm_100a).
 *
 * One step of the method (paper Algorithm 1, penalty / augmented-Lagrangian form of
 * Sections 3-4):
 *   1. lp_auxnet_forward      x_{k+1} = AuxNet_k(x_k), k = 0..K-2          (Eq. AV-Net-FP-lambda)
 *   2. lp_module_fwd_bwd(k)   out_k = F_k(x_k)                             (Eq. Parallel-ResNet-Feature-Flow)
 *                             local loss + terminal adjoint                (Eq. Parallel-ResNet-Gradient-Propagation-Equation)
 *                             parameter and input gradients                (Eq. Parallel-ResNet-Backpropagation)
 *      lp_modules_fwd_bwd_all the same for all K modules concurrently      (Algorithm 1, "par for")
 *   3. lp_step                theta <- theta - lr*g ; kappa <- kappa + c*r  (Eq. Parallel-ResNet-Multiplier-Update)
 *
 * Conventions
 *   - Every function returns an lp_status (0 = LP_OK, negative = error).  Bad arguments are
 *     reported on the host before anything is launched; nothing here aborts or throws.
 *   - "device" pointers are CUDA device addresses, 16-byte aligned, owned by the caller and not
 *     retained after the call returns unless stated.  "host" pointers are ordinary memory.
 *   - Activations are NHWC in the descriptor's dtype (LP_F32: float, LP_BF16: bfloat16).
 *     Convolution weights are [C_out][R][S][C_in] fp32 masters; labels are int32.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls are
 *     asynchronous on it; lp_last_device_status synchronises and reports device-side errors.
 *   - The library allocates no device memory for activations or parameters: the caller passes
 *     one workspace of lp_workspace_bytes() bytes to lp_create, 256-byte aligned, and keeps it
 *     alive until lp_destroy.
 *   - Penalty coefficient: the paper's beta*||.||^2 is (rho/2)*||.||^2 here, rho = 2*beta.
 *     `lambda_k` is the multiplier of the constraint F_k(x_k) = x_{k+1} (the paper's kappa_{k+1}).
 */
#ifndef LP_H_
#define LP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lp_status {
  LP_OK = 0,
  LP_ERR_NULL = -1,           /* a required pointer is NULL */
  LP_ERR_BAD_DESC = -2,       /* inconsistent or unsupported network descriptor */
  LP_ERR_BAD_INDEX = -3,      /* module / AuxNet index out of range */
  LP_ERR_ALIGN = -4,          /* a device pointer is not 16-byte aligned */
  LP_ERR_WORKSPACE = -5,      /* workspace too small or misaligned */
  LP_ERR_ORDER = -6,          /* call sequence violated (e.g. lp_step before any fwd_bwd) */
  LP_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait ran out */
  LP_ERR_CUDA = -8,           /* a CUDA runtime / driver call failed */
  LP_ERR_SIZE = -9,           /* a size argument does not match the network */
  LP_ERR_UNSUPPORTED = -10    /* valid request that this build does not implement */
} lp_status;

enum { LP_F32 = 0, LP_BF16 = 1 };
enum { LP_STEM_CONV3X3 = 0, LP_STEM_CONV7X7S2_MAXPOOL = 1 };
enum { LP_POSTBN = 0, LP_PREACT = 1, LP_BOTTLENECK = 2 };
/* `which` argument of the parameter calls: module k is k, AuxNet k is LP_AUX(k). */
#define LP_AUX(k) (256 + (k))
/* Recursive auxiliary-variable networks (aux_recursive = 1; Section 4.3, Eq. ReAuxNet-FP): x_k, k = 1..K-1,
 * is generated from the images alone by a stack of k units with parameters of its own, unit j having
 * the architecture of AuxNet_j.  LP_REAUX(k, j) names unit j (0 <= j < k) of stack k; the K-1 stacks
 * do not depend on one another, so the AuxNet chain's serial dependency is gone. */
#define LP_REAUX(k, j) LP_AUX((k) * ((k) - 1) / 2 + (j))
enum { LP_KIND_CONV_W = 0, LP_KIND_BN_GAMMA = 1, LP_KIND_BN_BETA = 2, LP_KIND_FC_W = 3, LP_KIND_FC_B = 4 };
enum { LP_CONV_IMPL_AUTO = 0, LP_CONV_IMPL_SIMT = 1, LP_CONV_IMPL_TENSOR = 2 };
/* May be OR-ed into conv_impl: keep one kind of convolution on the CUDA cores (diagnostics). */
enum { LP_CONV_NO_TENSOR_FWD = 16, LP_CONV_NO_TENSOR_DGRAD = 32, LP_CONV_NO_TENSOR_WGRAD = 64 };
/* May be OR-ed into conv_impl: pre-activation networks take the local loss of an interior module
 * (residual against x_{k+1}, its two sums and the terminal adjoint of
 * Eq. Parallel-ResNet-Gradient-Propagation-Equation) inside the epilogue of the module's last
 * tensor-core convolution instead of in a pass of its own over the stored module output.  Same
 * arithmetic, same results; with the present row-per-thread epilogue it is the slower of the two
 * (the extra operands are read and written in 16-byte pieces), hence off by default. */
enum { LP_CONV_LOSS_IN_EPILOGUE = 128 };
/* The tensor-core forward / input-gradient kernel has two epilogues with the same results: "direct" (bf16
 * stores from registers) and "staged" (the tile goes through shared memory and leaves by TMA tile stores;
 * a residual operand arrives by TMA loads a tile ahead and is added in place).  By default a convolution
 * with a residual operand takes the staged one where it applies (measured faster there: the residual is no
 * longer read in 16-byte pieces 2*C_out bytes apart) and every other convolution the direct one.  These
 * flags, OR-ed into conv_impl, force one or the other wherever it applies (comparisons, tests). */
enum { LP_CONV_DIRECT_EPILOGUE = 256, LP_CONV_STAGED_EPILOGUE = 512 };
/* May be OR-ed into conv_impl: 3x3 stride-1 tensor-core convolutions (forward and input gradient) with
 * 64-channel K chunks run on pairs of CTAs (tcgen05 cta_group::2: two pixel tiles per instruction, each CTA
 * fetching half of every weight stage).  Same results as the one-CTA kernel. */
enum { LP_CONV_TWO_CTA = 1024 };
/* May be OR-ed into conv_impl: a tensor-core input-gradient convolution whose output is the dy of a batch norm
 * takes the reduction pass of that batch norm's backward (sum dy_m, sum dy_m * xhat) in its epilogue, and only the
 * apply pass is left to run (Eq. Parallel-ResNet-Backpropagation: a module's backward pass is the chain
 * conv^T -> BN' -> conv^T ...; the sums are taken where dy is produced).  Same gradients up to the order of fp32
 * additions.  Not the default: the epilogue's extra shared-memory traffic costs the convolution more than the
 * separate kernel takes. */
enum { LP_CONV_BN_REDUCE_IN_EPILOGUE = 2048 };
/* May be OR-ed into conv_impl: the weight gradients of a module stay in its stream, in the order of the
 * backward pass.  By default each module has a second stream for them (they feed nothing but the update), so
 * that the chain of input gradients and batch-norm backward passes does not wait for them. */
enum { LP_CONV_WGRAD_IN_CHAIN = 4096 };
enum { LP_CONV_FWD = 0, LP_CONV_DGRAD = 1, LP_CONV_WGRAD = 2 };

#define LP_MAX_STAGES 8
#define LP_MAX_MODULES 16

/*
 * Network and split.  A residual network: stem S, num_stages stages of residual blocks
 * X + F(X, W) (Eq. ResNet-Training-Task), head T, cut into K modules of consecutive blocks
 * (every n-th block, Section 4.1); the stem belongs to module 0 and the head to module K-1.
 *   LP_POSTBN block: conv3x3-BN-ReLU-conv3x3-BN + shortcut (no ReLU after the sum)
 *   LP_PREACT block: BN-ReLU-conv3x3-BN-ReLU-conv3x3 + shortcut
 *   LP_BOTTLENECK block: conv1x1-BN-ReLU-conv3x3-BN-ReLU-conv1x1-BN + shortcut, inner width C_out/4, the
 *             block's stride in the 3x3 convolution (the block of the paper's ResNet-50 workload);
 *             stem, head and shortcut as in LP_POSTBN
 *   shortcut: identity, or a 1x1 convolution with the block's stride where shape changes
 *             (followed by BN in LP_POSTBN; applied to the pre-activated tensor in LP_PREACT)
 *   stem: LP_POSTBN conv-BN-ReLU (7x7/2 variant adds a 3x3/2 max-pool); LP_PREACT conv only
 *   head: [BN-ReLU in LP_PREACT] global average pool, linear layer with bias, softmax CE
 *   AuxNet_k: conv3x3(s1)-BN[-ReLU-conv3x3(s2)-BN] from x_k to the shape of x_{k+1}; hidden
 *             width C_out/aux_width_div; strides chosen to reach the boundary's spatial size.
 * Batch statistics everywhere (training mode), biased variance, eps = bn_eps.
 */
typedef struct lp_net_desc {
  uint32_t struct_size;               /* sizeof(lp_net_desc) */
  int32_t dtype;                      /* LP_F32 | LP_BF16 */
  int32_t N, H, W, C_in, num_classes; /* input batch NHWC, classes */
  int32_t stem_kind, stem_channels;
  int32_t block_kind;
  int32_t post_add_relu;              /* must be 0 */
  int32_t num_stages;
  int32_t stage_channels[LP_MAX_STAGES], stage_blocks[LP_MAX_STAGES], stage_stride[LP_MAX_STAGES];
  int32_t K;                          /* number of modules, 1..LP_MAX_MODULES */
  int32_t module_block_end[LP_MAX_MODULES]; /* cumulative block index ending each module */
  int32_t aux_convs_per_boundary;     /* 1 or 2 */
  int32_t aux_width_div;              /* >= 1 */
  float bn_eps;
  int32_t conv_impl;                  /* LP_CONV_IMPL_*: AUTO picks tensor cores where shapes allow */
  int32_t aux_recursive;              /* 0: serial AuxNet chain; 1: recursive AuxNets (see LP_REAUX) */
} lp_net_desc;

typedef struct lp_param_entry {
  char name[48];
  int32_t kind;                       /* LP_KIND_* */
  int32_t shape[4];                   /* unused trailing dims are 0 */
  uint64_t offset;                    /* element offset in the flat fp32 blob */
} lp_param_entry;

typedef struct lp_handle lp_handle;

const char* lp_status_string(int status);

/* Host-only queries (no GPU needed). */
size_t lp_workspace_bytes(const lp_net_desc* desc);     /* 0 on an invalid descriptor */
int lp_validate_desc(const lp_net_desc* desc);
/* Parameter layout of module `which` or AuxNet LP_AUX(k), in blob order.  `entries` may be NULL
 * to query the count; at most `max_entries` are written; *n_entries receives the total. */
int lp_param_layout(const lp_net_desc* desc, int which, lp_param_entry* entries, int max_entries,
                    int* n_entries);
/* Shape (NHWC) of x_k, k = 0..K-1 (x_0 is the image batch), from the descriptor alone. */
int lp_boundary_shape_desc(const lp_net_desc* desc, int k, int shape_nhwc[4]);

/* Create a handle over the caller's device workspace.  The call zero-fills the workspace with a
 * synchronous cudaMemset (it returns after the fill; work of the caller still running on other
 * streams must not touch the workspace meanwhile); parameters start at zero until lp_set_params.
 * The handle owns host memory, streams and events only. */
int lp_create(const lp_net_desc* desc, void* dev_workspace, size_t bytes, lp_handle** out);
int lp_destroy(lp_handle* h);

int lp_param_count(lp_handle* h, int which, size_t* n);
int lp_set_params(lp_handle* h, int which, const float* host, size_t n); /* synchronous */
int lp_get_params(lp_handle* h, int which, float* host, size_t n);       /* synchronous */
int lp_get_grads(lp_handle* h, int which, float* host, size_t n);        /* synchronous */
int lp_boundary_shape(lp_handle* h, int k, int shape_nhwc[4]);

/* Step 1.  images: device [N,H,W,C_in]; x_out: host array of K-1 device pointers, x_out[k-1]
 * receives x_k (shape lp_boundary_shape(k)). */
int lp_auxnet_forward(lp_handle* h, const void* images, void* const* x_out, void* stream);

/* Step 2 for one module.  x_k: device input of module k (images for k = 0).
 * x_next_or_labels: k < K-1: x_{k+1} (device, shape of boundary k+1); k == K-1: int32 labels[N].
 * lambda_k: multiplier, same shape as x_{k+1}, or NULL for the penalty method (ignored for K-1).
 * loss_out: device float[2] = { local loss, ||F_k(x_k) - x_{k+1}||^2 (0 for the last module) }.
 * dx_k: device output, gradient of the local loss with respect to x_k (the paper's P^k_{kn});
 *       may be NULL; ignored for k = 0.
 * Parameter gradients stay in the workspace (lp_get_grads) until the next call for module k. */
int lp_module_fwd_bwd(lp_handle* h, int k, const void* x_k, const void* x_next_or_labels,
                      const void* lambda_k, float rho, float* loss_out, void* dx_k, void* stream);

/* Step 2 for all modules at once: x[k] = x_k (K device pointers, x[0] = images), labels,
 * lambdas[k] for k < K-1 (array or entries may be NULL), loss_out device float[K][2], dx[k]
 * (array or entries may be NULL).  The K modules run on K internal streams forked from and
 * joined back into `stream`. */
int lp_modules_fwd_bwd_all(lp_handle* h, const void* const* x, const int32_t* labels,
                           const void* const* lambdas, float rho, float* loss_out,
                           void* const* dx, void* stream);

/* Step 3.  SGD on every module whose gradients are fresh; kappa <- kappa + kappa_step * r for
 * every interior module with a non-NULL lambdas_inout[k] (r = F_k(x_k) - x_{k+1} kept from the
 * last fwd_bwd).  momentum = weight_decay = 0 is the paper's plain SGD. */
int lp_step(lp_handle* h, float lr, float momentum, float weight_decay, float kappa_step,
            void* const* lambdas_inout, void* stream);

/* Steps 1-3 in one call with every dependency of Algorithm 1 and no more: the AuxNet chain runs
 * on its own stream; module k starts as soon as x_k exists, takes its local loss as soon as
 * x_{k+1} exists, and updates its own parameters (and multiplier) right after its own backward
 * pass ("update unlocking", Section 4.1) without waiting for the other modules.  Arguments as in
 * lp_auxnet_forward (x_out[k-1] receives x_k), lp_modules_fwd_bwd_all (loss_out float[K][2];
 * dx[k] for k >= 1, array or entries may be NULL) and lp_step.  Everything is joined back into
 * `stream` before the call's work is complete in stream order. */
int lp_layer_parallel_step(lp_handle* h, const void* images, void* const* x_out, const int32_t* labels,
                           void* const* lambdas_inout, float rho, float* loss_out, void* const* dx, float lr,
                           float momentum, float weight_decay, float kappa_step, void* stream);

/* Second parallel loop of Algorithm 1, for every boundary k = 1..K-1: the correction direction of
 * the auxiliary variable, g_k = dx_k - seed_{k-1} (Eq. Parallel-ResNet-Slack-Variables-Update: the
 * input gradient of module k plus the gradient of module k-1's penalty/AL term with respect to
 * x_k, which is minus its terminal adjoint), the corrected variable x_k_new = x_k - lr_lambda*g_k,
 * and ONE SGD step (rate lr_aux) of AuxNet_{k-1} on ||x_k_new - AuxNet_{k-1}(x_{k-1})||^2 with
 * x_{k-1} and x_k_new held constant (Eq. AV-Net-lambda, local knowledge distillation).
 * Call after lp_auxnet_forward and the module passes of the same batch (the AuxNet activations and
 * the terminal adjoints are taken from the workspace).
 *   x[k-1] = x_k as produced by lp_auxnet_forward (K-1 device pointers); dx[k] = dx_k (K entries,
 *   entry 0 unused); x_new[k-1] (array or entries may be NULL) receives x_k_new;
 *   loss_out: device float[K-1], the distillation losses before the update (= lr_lambda^2 ||g_k||^2). */
int lp_auxnet_distill(lp_handle* h, const void* images, void* const* x, const void* const* dx, float lr_lambda,
                      float lr_aux, void* const* x_new, float* loss_out, void* stream);

/* Stored-auxiliary-variable mode (Section 4.1, Eq. Parallel-ResNet-Slack-Variables-Update, without
 * an AuxNet): the caller keeps x_1..x_{K-1} for the batch, runs lp_modules_fwd_bwd_all and lp_step
 * on them, and this call applies the correction in place,
 *     x_k <- x_k - lr_lambda * (dx_k - seed_{k-1}),   k = 1..K-1,
 * where seed_{k-1} is module k-1's terminal adjoint of the same batch (taken from the workspace).
 *   x_inout[k-1] = x_k (device, K-1 pointers, updated in place); dx[k] = dx_k (K entries, entry 0
 *   unused); norm_out: device float[K-1] or NULL, receives lr_lambda^2 ||dx_k - seed_{k-1}||^2.
 * LP_ERR_ORDER if module k-1 has not run. */
int lp_aux_correct(lp_handle* h, void* const* x_inout, const void* const* dx, float lr_lambda, float* norm_out,
                   void* stream);

/* Layer-serial comparator (K = 1 in the paper's notation): forward through all modules with
 * x_{k+1} := F_k(x_k); logits: device float[N][num_classes]. */
int lp_forward_serial(lp_handle* h, const void* images, float* logits, void* stream);
/* Layer-serial training pass with the same kernels: forward through all modules, cross-entropy,
 * back-propagation through all modules in reverse; loss_out: device float[2]. */
int lp_serial_fwd_bwd(lp_handle* h, const void* images, const int32_t* labels, float* loss_out,
                      void* stream);

/* Output of module k's last forward, F_k(x_k) - x_{k+1} residual and terminal adjoint, copied to
 * host-visible device buffers for tests: dst device buffers of the boundary k+1 shape (NULL to
 * skip).  Valid after lp_module_fwd_bwd(k) for k < K-1. */
int lp_get_residual(lp_handle* h, int k, void* r_dst, void* seed_dst, void* stream);

/* Synchronise `stream` and return LP_OK, LP_ERR_DEVICE_TIMEOUT or LP_ERR_CUDA. */
int lp_last_device_status(lp_handle* h, void* stream);
/* Self-test of the device-side bounded wait (the mechanism behind LP_ERR_DEVICE_TIMEOUT): launches one
 * small kernel in which a thread waits, for at most limit_ms (0 < limit_ms <= 100), on a barrier that
 * nothing ever signals.  The wait runs out, the kernel records it the way the convolution kernels do and
 * returns; the next lp_last_device_status reports LP_ERR_DEVICE_TIMEOUT and clears it, and the handle
 * stays usable.  waited_ms (nullable; makes the call synchronous) receives the time the thread waited. */
int lp_selftest_bounded_wait(lp_handle* h, double limit_ms, double* waited_ms, void* stream);
/* Number of kernels the library launched since the counter was last reset. */
int64_t lp_launch_count(lp_handle* h, int reset);
/* Time (ms, CUDA events on the launching stream) spent in tensor-core convolution kernels and
 * their count since the last reset; only collected while profiling is enabled (serialises). */
int lp_conv_profile(lp_handle* h, int enable, double* ms, double* flops, int64_t* launches);

/* Per-operation time line of everything the library launches while it is enabled: one record per
 * operation of a module or AuxNet plan (a convolution, a batch-norm pass, the local loss, the
 * update, ...), timed with CUDA events on the stream the operation runs on, so that the phases of
 * the paper's cost model (Section 4.3: T_f, T_b per module, t_psi, the AuxNet pass and the AuxNet
 * distillation) can be measured per module while the modules overlap.  Events cannot be recorded
 * into a graph: lp_graph_begin returns LP_ERR_ORDER while the time line is enabled.
 *   enable       0/1: state after the call (records collected so far are dropped either way)
 *   records      host array of max_records entries, or NULL; when given (or n_records is), the
 *                device is synchronised and the records collected so far are written, times in ms
 *                relative to the earliest recorded start
 *   n_records    receives the number of records collected (may exceed max_records) */
#define LP_PHASE_AUX_FORWARD 0
#define LP_PHASE_FORWARD 1
#define LP_PHASE_BACKWARD 2
#define LP_PHASE_UPDATE 3
#define LP_PHASE_DISTILL 4
/* operation kinds in lp_timeline_record.op */
#define LP_OP_CONV_FWD 0
#define LP_OP_CONV_DGRAD 1
#define LP_OP_CONV_WGRAD 2
#define LP_OP_BN_STATS 3
#define LP_OP_BN_APPLY 4
#define LP_OP_OUT_LOSS 5
#define LP_OP_BN_BWD 6
#define LP_OP_MAXPOOL_FWD 7
#define LP_OP_MAXPOOL_BWD 8
#define LP_OP_HEAD_FWD 9
#define LP_OP_HEAD_BWD 10
#define LP_OP_COPY 11
#define LP_OP_UPDATE 12
typedef struct lp_timeline_record {
  int32_t plan;   /* module k, or LP_AUX(k) */
  int32_t op;     /* LP_OP_* */
  int32_t phase;  /* LP_PHASE_* */
  float start_ms, end_ms;
  double bytes;   /* algorithmic global-memory bytes of the operation: every operand read once, every result
                     written once (batch-norm backward: its two passes; update: parameters, gradients, copies) */
} lp_timeline_record;
int lp_timeline(lp_handle* h, int enable, int max_records, lp_timeline_record* records, int* n_records);

/* CUDA-graph helpers: record every launch the library makes on `stream` between begin and end
 * (the internal module streams are forked from and joined into it), then replay the recording.
 * Pointer arguments of the recorded calls are baked into the graph.  Up to 8 graphs per handle;
 * *graph_id receives the slot.  The first call of every kind must have run once outside a capture
 * (kernel attributes are set on first use). */
int lp_graph_begin(lp_handle* h, void* stream);
int lp_graph_end(lp_handle* h, void* stream, int* graph_id);
int lp_graph_launch(lp_handle* h, int graph_id, void* stream);

/* Stand-alone convolution on caller buffers (tests and kernel benchmarks).
 * op = LP_CONV_FWD:   a = x [N,H,W,Cin],   b = w fp32 [Cout,R,R,Cin], out = y  [N,OH,OW,Cout]
 * op = LP_CONV_DGRAD: a = dy [N,OH,OW,Cout], b = w fp32,               out = dx [N,H,W,Cin]
 * op = LP_CONV_WGRAD: a = x,               b = dy (activation dtype),  out = dw fp32 [Cout,R,R,Cin]
 * scratch: device buffer of lp_conv2d_scratch_bytes() (packed bf16 weights, statistics).
 * stats (nullable, FWD only): device double[2*Cout] receives per-channel sum and sum of squares
 * of y.  Returns LP_ERR_UNSUPPORTED if `impl` cannot run this shape. */
size_t lp_conv2d_scratch_bytes(int Cin, int Cout, int R);
int lp_conv2d(int op, int dtype, int impl, int N, int H, int W, int Cin, int Cout, int R,
              int stride, int pad, const void* a, const void* b, void* out, double* stats,
              void* scratch, size_t scratch_bytes, float* elapsed_ms, void* stream);

/*
 * Forward convolution for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of lp_conv2d(LP_CONV_FWD, LP_BF16, tensor cores).)
 *
 * Some callers may not call cudaMalloc at all: code that runs inside a memory pool it does not
 * own, plug-ins whose host forbids driver allocations after start-up, or a latency-critical loop
 * in which an allocation would synchronise the device.  lp_conv2d needs a scratch buffer from
 * its caller (bf16 operand copy of the weights, an error word, a small table); this entry point
 * keeps that scratch in a fixed array inside the library instead, LP_NOALLOC_SCRATCH_BYTES long,
 * which every GPU that loads the library holds until the process exits.  It calls no cudaMalloc,
 * cudaFree or allocating library routine; the caller passes only inputs and outputs.
 *
 *   x: device bf16 [N,H,W,Cin]; w: device fp32 [Cout,R,R,Cin]; y: device bf16 [N,OH,OW,Cout].
 *   Same shape rules as the tensor-core path of lp_conv2d (Cin, Cout multiples of 8, R in {1,3},
 *   stride in {1,2}); LP_ERR_UNSUPPORTED otherwise.  The call is synchronous on `stream`.
 *   LP_ERR_SIZE ("size mismatch") if the scratch does not fit the array: the call needs
 *   512 + 2*Cout*R*R*Cin bytes, the middle term rounded up to a multiple of 256 (an error word, the
 *   bf16 weights, a one-entry table), e.g. up to 640 -> 640 channels with a 3x3 kernel.
 *
 * The first call on a device looks up the array's device address (once per device, with that
 * device current) and sets kernel attributes: make it before any stream capture.  All calls share
 * the one array, which keeps the previous call's contents; the words that must start at zero are
 * cleared by each call.  Two calls that overlap on the GPU (different streams or threads) race on
 * the array: serialise them.
 */
#define LP_NOALLOC_SCRATCH_BYTES (8u << 20)
int lp_conv2d_fwd_noalloc(int N, int H, int W, int Cin, int Cout, int R, int stride, int pad, const void* x,
                          const float* w, void* y, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LP_H_ */
