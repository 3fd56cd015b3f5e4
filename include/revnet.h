/*
 * revnet.h -- C ABI of the reversible residual network library for NVIDIA B200 (sm_100a).
 *
 * The calls follow the paper's statement of the problem (arXiv 1707.04585):
 *   - a reversible block maps (x1, x2) to (y1, y2) with y1 = x1 + F(x2), y2 = x2 + G(y1)
 *     (Section 3.1), F and G being chains of BN -> ReLU -> conv layers (Section 2.2, Eq. 2);
 *   - its backward is given only (y1, y2) and (dy1, dy2) and returns (x1, x2), (dx1, dx2) and
 *     the parameter gradients (Section 3.2, Algorithm 1);
 *   - a stack of such blocks keeps only the inputs of its non-reversible layers (Section 3.2).
 *
 * Conventions that hold for every call
 *   - All tensor pointers are DEVICE pointers unless a parameter is marked "host".
 *   - Activations are NHWC float32.  x1 and x2 (and y1, y2, their gradients) are two separate
 *     contiguous tensors [N,H,W,c]; x1 holds channels [0,c) of the block input, x2 channels [c,2c).
 *   - Convolution weights are float32 [Cout][kh][kw][Cin], cross-correlation, zero padding k/2,
 *     no bias.  BN is train-mode (batch statistics over N,H,W, biased variance); no running
 *     statistics are kept.
 *   - The caller owns every buffer.  The library allocates no device memory in any call
 *     below; scratch comes from the workspace the caller passes.
 *   - Work is enqueued on the caller's stream (a cudaStream_t passed as void*); calls do not
 *     synchronise unless stated.  A backward call may fork part of its work onto streams the
 *     context owns (weight gradients beside the data-gradient chain; in a train step the
 *     recomputation of F beside the gradient steps of G) and joins them again before it returns:
 *     to the caller everything is ordered as if it ran on the stream passed in.  Device pointers
 *     must be 16-byte aligned, channel counts multiples of 4.
 *   - Aliasing y1==x1, y2==x2 in revnet_block_fwd and x1==y1, x2==y2, dx1==dy1, dx2==dy2 in
 *     revnet_block_bwd is legal: that is how a stack runs in place.
 *   - Gradient outputs are overwritten, not accumulated.
 *   - Every call returns 0 (REVNET_OK) or a negative revnet_status; the text of the last error
 *     of a context is available from revnet_last_error.  No exception crosses the ABI.
 *   - Coupling state.  With state_frac_bits = 0 the tensors x1, x2, y1, y2 (and a stack's stage
 *     buffers) hold float32 and reconstruction is exact only up to rounding, which low-precision
 *     residual functions amplify.  With state_frac_bits = k > 0 they hold int32 fixed-point
 *     numbers (value = i * 2^-k): the residual function's float result is rounded to that grid
 *     before the add, y = x + round(F * 2^k) is undone exactly by x = y - round(F * 2^k), and the
 *     reversal returns the forward pass's inputs bit for bit (Section 3.2, "Numerical error":
 *     fixed point on the x's and y's, floating point inside F and G).  Range |value| < 2^(31-k).
 *     Gradients are float32 in either format.
 *   - mode 0: convolution operands rounded to bf16, products accumulated in fp32 on the tensor
 *     cores where the shape allows; mode 1: strict fp32 arithmetic throughout (verification).
 *     The coupling state (x, y and their gradients) is fp32 in both modes.
 */
#ifndef REVNET_H_
#define REVNET_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    REVNET_OK = 0,
    REVNET_E_INVALID_ARG = -1,
    REVNET_E_UNSUPPORTED_SHAPE = -2,
    REVNET_E_WORKSPACE_TOO_SMALL = -3,
    REVNET_E_MISALIGNED = -4,
    REVNET_E_CUDA = -5,
    REVNET_E_TIMEOUT = -6,
    REVNET_E_INTERNAL = -7
} revnet_status;

typedef struct revnet_ctx revnet_ctx;
typedef struct revnet_plan revnet_plan;

/* Create / destroy a context bound to one CUDA device.  Creation allocates a few hundred
 * bytes of device memory for status words; nothing else is ever allocated by the library. */
int revnet_create(revnet_ctx **out, int device);
int revnet_destroy(revnet_ctx *ctx);
/* Text of the last error recorded on ctx (never NULL; valid until the next failing call on the same
 * context: a context is meant to be used from one thread at a time). */
const char *revnet_last_error(const revnet_ctx *ctx);

/* A residual function: n_layers (1..3) layers, each BN -> ReLU -> conv k x k, stride 1
 * (Section 2.2, Eq. 2: Basic = c3(c3(x)), Bottleneck = c1(c3(c1(x)))).
 * cin[0] and cout[n_layers-1] must equal the block's half-channel count c. */
typedef struct {
    int n_layers;
    int k[3];
    int cin[3];
    int cout[3];
} revnet_fn_desc;

typedef struct {
    int N, H, W, c;          /* x1, x2: [N,H,W,c] each */
    revnet_fn_desc F, G;
    float eps;               /* BN epsilon */
    int mode;                /* 0 = bf16 tensor-core operands, 1 = strict fp32 */
    int state_frac_bits;     /* 0: x, y are float32.  k in 1..24: x, y are int32 fixed point with k
                                fractional bits (value = i * 2^-k); see "coupling state" above */
} revnet_block_desc;

/* Parameters of one residual function (device pointers): W[l] is [cout][k][k][cin],
 * gamma[l], beta[l] are [cin[l]] (the BN in front of conv l).
 * Wpack_fprop / Wpack_dgrad: optional bf16 copies of W[l] in the layout the tensor-core kernels read
 * (forward: [cout][tap][cin]; data gradient: [cin][mirrored tap][cout]; both padded), written by
 * revnet_pack_weights.  NULL: the block call that needs one builds it from W[l] into its workspace,
 * every time.  A pack is valid until W[l] changes.  Ignored in mode 1. */
typedef struct {
    const float *W[3];
    const float *gamma[3];
    const float *beta[3];
    const void *Wpack_fprop[3];
    const void *Wpack_dgrad[3];
} revnet_fn_params;

/* Gradient outputs of one residual function, same shapes as the parameters. */
typedef struct {
    float *dW[3];
    float *dgamma[3];
    float *dbeta[3];
} revnet_fn_grads;

/* Workspace (bytes) that revnet_block_fwd / revnet_block_bwd need for this shape. */
int revnet_block_workspace_bytes(revnet_ctx *ctx, const revnet_block_desc *desc,
                                 size_t *fwd_bytes, size_t *bwd_bytes);

/* bf16 weight packs of a block, built once and reused by any number of forward / backward calls
 * (Appendix 6.3 hands each layer its weights as they are; a pack is the same weights rounded to the
 * operand precision of Eq. 2's convolutions in the layout the kernels read).  revnet_block_pack_bytes
 * gives the size of the caller-owned device buffer; revnet_pack_weights enqueues the pack kernels on
 * `stream` and stores the pack pointers into F and G (host structs), NULL for layers whose shape the
 * tensor-core kernels do not take and in mode 1 (0 bytes).  The buffer must be 256-byte aligned.
 * Errors: REVNET_E_INVALID_ARG (null), REVNET_E_MISALIGNED, REVNET_E_WORKSPACE_TOO_SMALL. */
int revnet_block_pack_bytes(revnet_ctx *ctx, const revnet_block_desc *desc, size_t *bytes);
int revnet_pack_weights(revnet_ctx *ctx, const revnet_block_desc *desc,
                        revnet_fn_params *F, revnet_fn_params *G,
                        void *pack_buffer, size_t pack_bytes, void *stream);

/* Block forward (Section 3.1): y1 = x1 + F(x2); y2 = x2 + G(y1). */
int revnet_block_fwd(revnet_ctx *ctx, const revnet_block_desc *desc,
                     const void *x1, const void *x2,
                     const revnet_fn_params *F, const revnet_fn_params *G,
                     void *y1, void *y2,
                     void *workspace, size_t workspace_bytes, void *stream);

/* Block forward for callers that cannot allocate device memory (the paper has no counterpart; this
 * is an integration aid).  Who: code running under a memory pool or a capture / real-time section
 * where cudaMalloc and friends are forbidden or would stall, and plugins that receive tensors but
 * no allocator.  Same computation and same results as revnet_block_fwd, but the scratch comes from
 * a 16 MiB array built into the library (held on every GPU that loads the library until the
 * process exits) instead of a caller workspace.  The call itself calls no allocating CUDA routine;
 * the array is part of the library image, which the CUDA runtime places on a device when the library
 * is first used there -- that can be inside this entry point's first call on that device.  Shapes whose forward scratch (revnet_block_workspace_bytes) exceeds
 * 16 MiB are rejected with REVNET_E_WORKSPACE_TOO_SMALL and a message naming both sizes.
 * The first call on a device looks up the array's device address (with that device current, as it
 * must be for every call); make that first call before starting any stream capture.  All calls
 * share the one array, which keeps whatever the previous call left in it: calls that overlap on the
 * GPU (different streams, or threads) race on it, so serialise them.  Nothing needs clearing
 * between calls: each call writes every scratch region before reading it. */
int revnet_block_fwd_noalloc(revnet_ctx *ctx, const revnet_block_desc *desc,
                             const void *x1, const void *x2,
                             const revnet_fn_params *F, const revnet_fn_params *G,
                             void *y1, void *y2, void *stream);

/* Block backward without stored activations (Algorithm 1): from (y1,y2) and (dy1,dy2) compute
 * x2 = y2 - G(y1), x1 = y1 - F(x2), dx1 = dy1 + (dG/dz1)^T dy2, dx2 = dy2 + (dF/dx2)^T dx1,
 * and the gradients of the parameters of F and G.  The activations computed while
 * reconstructing are reused for the gradient steps (four convolution passes per layer in all,
 * counting the forward: Section 3.2 "Computational overhead", Section 5.1). */
int revnet_block_bwd(revnet_ctx *ctx, const revnet_block_desc *desc,
                     const void *y1, const void *y2, const float *dy1, const float *dy2,
                     const revnet_fn_params *F, const revnet_fn_params *G,
                     void *x1, void *x2, float *dx1, float *dx2,
                     const revnet_fn_grads *gF, const revnet_fn_grads *gG,
                     void *workspace, size_t workspace_bytes, void *stream);

/* ---- stored (non-reversible) layer: BN -> ReLU -> conv k x k with stride 1 or 2 (Section 3.1: a
 * reversible block must have stride 1; Section 3.2: such layers keep their input).  The input is
 * either one float32 tensor [N,H,W,cin] (in_split = 0, in2 unused) or the two halves of a
 * coupling state, cin/2 channels each, in the state format (in_split = 1).  The output
 * [N,H/stride,W/stride,cout] is written as two halves (out1: channels [0,cout/2), out2: the rest)
 * in the state format: it is the (x1,x2) the next stage starts from. */
typedef struct {
    int N, H, W;             /* input geometry */
    int cin, cout, k, stride;
    int in_split;
    float eps;
    int mode;
    int state_frac_bits;
} revnet_transition_desc;

int revnet_transition_workspace_bytes(revnet_ctx *ctx, const revnet_transition_desc *desc,
                                      size_t *fwd_bytes, size_t *bwd_bytes);
int revnet_transition_fwd(revnet_ctx *ctx, const revnet_transition_desc *desc,
                          const void *in1, const void *in2,
                          const float *W, const float *gamma, const float *beta,
                          void *out1, void *out2,
                          void *workspace, size_t workspace_bytes, void *stream);
/* Backward from the stored input: din (float32, same split as the input), dW, dgamma, dbeta. */
int revnet_transition_bwd(revnet_ctx *ctx, const revnet_transition_desc *desc,
                          const void *in1, const void *in2,
                          const float *dout1, const float *dout2,
                          const float *W, const float *gamma, const float *beta,
                          float *din1, float *din2, float *dW, float *dgamma, float *dbeta,
                          void *workspace, size_t workspace_bytes, void *stream);

/* ---- classification stack (Section 3.2: only non-reversible layers keep their inputs) ---- */

typedef struct {
    int units;         /* reversible units in the stage */
    int c;             /* channels per half */
    int w;             /* bottleneck width (kind 2), else 0 */
    int kind;          /* 0: F,G = one conv3x3; 1: basic (3x3,3x3); 2: bottleneck (1x1,3x3,1x1) */
    int trans_k;       /* stored BN-ReLU-conv transition in front of the stage (0 = none) */
    int trans_stride;  /* 1 or 2 */
    int down;          /* 1: paper-shaped stage (Table "Architectural details" counts the down-sampling inside the
                          first unit of a stage): no transition (trans_k = 0); the first of the `units` units is a
                          stored, non-invertible coupling unit  y1 = S(x1) + F(x2), y2 = S(x2) + G(y1)  on the
                          previous stage's output, S = 2x2 average pooling (stride 2) followed by zero channels up to
                          c, F with one stride-2 layer (the first 3x3 of a basic function, the 3x3 of a bottleneck);
                          the other units - 1 units are reversible.  Its parameters come first in the stage: F layers
                          (gamma, beta, W each), then G layers.  Not for stage 0. */
} revnet_stage_desc;

#define REVNET_MAX_STAGES 8

typedef struct {
    int N, img, in_ch, n_classes;
    int stem_k, stem_stride, stem_cout, maxpool;    /* bare conv stem (+ 3x3/2 max-pool) */
    int n_stages;
    revnet_stage_desc stage[REVNET_MAX_STAGES];
    float eps;
    int mode;
    int state_frac_bits;                            /* format of the stage buffers, as in revnet_block_desc */
    float lr, momentum, weight_decay;               /* SGD (Appendix 6.1); decay on conv/FC weights only */
    int verify_reconstruction;                      /* debug: keep a copy of each stage input and report
                                                       max |reconstructed - original| per stage */
    int use_cuda_graph;                             /* 1: the first revnet_train_step with a given set of buffer
                                                       addresses records the step as a CUDA graph (on a private
                                                       stream) and launches it on the caller's stream; later
                                                       calls with the same addresses only replay it.  Ignored
                                                       with verify_reconstruction or while profiling. */
    int store_activations;                          /* 1: ordinary backprop for comparison (Section 3.2: the cost
                                                       the method trades storage for).  Every unit keeps its inputs,
                                                       its outputs and the internals of F and G from the forward
                                                       pass in the workspace; the backward pass recomputes nothing
                                                       (3N convolution cost instead of 4N) and storage grows with
                                                       the number of units.  Same gradients as the reversible step.
                                                       verify_reconstruction is ignored. */
} revnet_stack_desc;

typedef struct {
    uint64_t stored_activation_bytes;  /* activations kept between forward and backward */
    uint64_t workspace_peak_bytes;     /* high-water mark of scratch use during the step */
    uint64_t flops_fwd, flops_bwd;     /* dense conv + FC flops issued (2 per multiply-add) */
    uint64_t kernel_launches;          /* kernels enqueued by the step */
    float recon_max_abs[REVNET_MAX_STAGES]; /* filled only with verify_reconstruction */
    int device_status;                 /* what the step's kernels recorded on the device (0, REVNET_E_TIMEOUT, REVNET_E_INVALID_ARG).
                                          Filled only by calls that synchronise the stream anyway (revnet_train_step with
                                          verify_reconstruction, revnet_train_step_host); otherwise 0: an asynchronous call
                                          cannot know yet, ask revnet_check_device */
} revnet_step_stats;

/* Plan a stack: validates the description and sizes the caller's buffers.
 * param_count: floats in each of params / grads / momentum.  Parameter order is forward order:
 * stem W; per stage: [transition gamma, beta, W]; per unit: F layers (gamma, beta, W each) then
 * G layers; FC W [n_classes][C], FC b.  The activation buffer holds the stored tensors (stem /
 * max-pool output where a transition follows, one (x1,x2) pair per stage); its size does not
 * depend on the number of units per stage. */
int revnet_stack_plan(revnet_ctx *ctx, const revnet_stack_desc *desc, revnet_plan **plan,
                      size_t *param_count, size_t *activation_bytes, size_t *workspace_bytes);
int revnet_plan_destroy(revnet_plan *plan);
/* Optional: declare how large the activation and workspace buffers passed to revnet_train_step are.
 * Once declared, a step whose buffers are smaller than the plan needs returns
 * REVNET_E_WORKSPACE_TOO_SMALL instead of writing past them (the step takes pointers only). */
int revnet_plan_set_buffer_sizes(revnet_plan *plan, size_t activation_bytes, size_t workspace_bytes);
/* How the planned workspace divides: the part that holds per-parameter data (bf16 weight packs,
 * the SGD segment table) grows with depth like the parameters do; the rest is activation scratch
 * (gradient pair, one block's recomputed internals, reduction partials) and does not depend on the
 * number of units per stage (Section 3.2: storage independent of depth). */
int revnet_plan_scratch_split(const revnet_plan *plan, size_t *param_scratch_bytes, size_t *activation_scratch_bytes);

/* One SGD training step: forward, loss, reconstructing backward through every stage
 * (Algorithm 1 applied block by block from the stage outputs), SGD-with-momentum update.
 * images: [N,img,img,in_ch] float32; labels: [N] int32 in [0,n_classes).
 * loss: 1 float (mean softmax cross-entropy); pred: [N] int32 arg-max (lowest index on ties);
 * logits: [N][n_classes] or NULL.  params/momentum are updated in place, grads overwritten.
 * stats (host, may be NULL) is filled from host-side accounting; with verify_reconstruction the
 * call synchronises the stream to read the per-stage error back. */
int revnet_train_step(revnet_ctx *ctx, revnet_plan *plan,
                      const float *images, const int32_t *labels,
                      float *params, float *grads, float *momentum,
                      void *activations, void *workspace,
                      float *loss, int32_t *pred, float *logits,
                      revnet_step_stats *stats, void *stream);

/* Same step fed from HOST memory: copies images_host / labels_host (pinned memory recommended)
 * into the device staging buffers images_dev / labels_dev, runs revnet_train_step, copies loss
 * and pred back to loss_host / pred_host and synchronises the stream.  Being synchronous it also
 * returns the status its kernels recorded on the device, if any (see revnet_check_device). */
int revnet_train_step_host(revnet_ctx *ctx, revnet_plan *plan,
                           const float *images_host, const int32_t *labels_host,
                           float *images_dev, int32_t *labels_dev,
                           float *params, float *grads, float *momentum,
                           void *activations, void *workspace,
                           float *loss_dev, int32_t *pred_dev,
                           float *loss_host, int32_t *pred_host,
                           revnet_step_stats *stats, void *stream);

/* Waits inside the library's kernels (on shared-memory barriers) are bounded; a kernel whose wait
 * runs out stops its work, records a status word on the device and exits normally.  The loss kernel
 * records REVNET_E_INVALID_ARG the same way when a label lies outside [0, n_classes) (it reads
 * nothing at that label and the step's loss becomes NaN).
 * revnet_check_device synchronises the stream, returns REVNET_OK or the recorded status and clears it
 * together with the counters of the kernels' grid-wide reductions, so the context stays usable.
 * No counterpart in the paper: failure reporting. */
int revnet_check_device(revnet_ctx *ctx, void *stream);

/* Self-test of that path (no counterpart in the paper): enqueues one small kernel whose single wait,
 * on a barrier nothing ever arrives on, is limited to limit_ns (at most 100 ms).  The wait runs out,
 * the kernel records REVNET_E_TIMEOUT and returns normally; the next revnet_check_device reports it. */
int revnet_selftest_bounded_wait(revnet_ctx *ctx, uint64_t limit_ns, void *stream);

/* ---- per-kernel timing (no counterpart in the paper: measurement support) ----
 * While enabled, every kernel the library launches on behalf of this context is followed by a
 * CUDA event on the caller's stream.  revnet_profile_summary waits for the last event and writes
 * one text line per kernel name: "name<TAB>launches<TAB>total_ms<TAB>algorithmic_bytes<TAB>flops".
 * The time of a launch is the span between the previous event and its own, so the first record
 * after enabling is only a boundary.  buf may be NULL with buflen 0 to query `needed`.
 * Enabling (or disabling) clears earlier records.  on = 2 enables with one line per kernel name AND
 * launch shape: the name then reads "name|algorithmic_bytes|flops" of one launch.  A profiled train
 * step first holds the stream for 5 ms, so that its launches are queued by the time they run and
 * the spans hold device time only; that hold is the record "step_begin".
 * on = 3 is the timeline mode, for train steps only: no events; instead the convolution, weight-
 * gradient and BN-ReLU apply kernels write the GPU's nanosecond timer when their first CTA starts
 * and their last CTA ends (one slot per launch, reset at the start of every step, also inside the
 * replayed graph).  The summary then describes the LAST step that ran, as it ran (overlapping
 * streams, no events in between): one line per kernel name and launch shape with the sum of its
 * launches' start-to-end times, a line "stamped_busy" (time during which at least one stamped kernel
 * was running; launches = stamped launches) and a line "stamped_span" (first start to last end).
 * Kernels that overlap each count their own time, so the lines can add up to more than the span. */
int revnet_profile_enable(revnet_ctx *ctx, int on);
int revnet_profile_summary(revnet_ctx *ctx, char *buf, size_t buflen, size_t *needed);

#ifdef __cplusplus
}
#endif
#endif /* REVNET_H_ */
