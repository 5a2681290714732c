/*
 * ffint8.h — C ABI of libffint8: the FF-INT8 per-layer Forward-Forward train step on one
 * NVIDIA B200 (sm_100a).
 *
 * The library implements the single-layer dataflow of the FF-INT8 paper (Sec. IV-B, Fig. 4):
 * symmetric uniform quantisation (Sec. IV) of the layer input A (stochastic rounding) and of
 * the weights W, an INT8 x INT8 -> INT32 MAC (dense or 3x3 convolution), goodness
 * G = ||y||^2 (Sec. III; Alg. 1, goodness step), the negative-log-likelihood losses of Eq. 1 / Eq. 2
 * with the look-ahead term of Eq. 3 / Eq. 4, the output gradient g^Y quantised to INT8, the
 * weight gradient g^W as a second INT8 MAC, and the weight update (Alg. 1, update step).  No input
 * gradient g^A is ever formed (Sec. IV-B).
 *
 * Conventions
 *  - Every pointer inside ff_layer_bufs is a DEVICE pointer owned by the caller, 16-byte
 *    aligned, valid on the device the context was created for.  Pointers to ff_layer_desc /
 *    ff_layer_bufs structs and all by-value scalars are HOST data.
 *  - Batch layout: B positive samples followed by B negative samples ("positive and negative
 *    sets", Alg. 1, sample generation).  M = 2B.  R = rows per sample: 1 for a linear layer, Ho*Wo for a
 *    convolution (one row per output position, NHWC); the input of a convolution has H*Wd rows.
 *  - Calls are asynchronous on the given CUDA stream (a cudaStream_t passed as void*; NULL =
 *    the legacy default stream) and never synchronise.  Host-detectable errors are returned
 *    before anything is launched.  Device-detected conditions (non-finite input, a bounded wait
 *    that ran out) are OR-ed into a status word that ff_poll_status reads.
 *  - The library never allocates device memory after ff_create; scratch space is the caller's
 *    workspace (ff_set_workspace).
 *  - Arithmetic contract: all INT8 tensors, INT32 accumulators, absmax values, S, rowmax, coef
 *    and the updated weights have exactly one correct bit pattern (each FP32/FP64 operation is
 *    a single IEEE round-to-nearest operation in a fixed order, no fused multiply-add); only the
 *    scalar `loss` depends on summation order.
 */
#ifndef FFINT8_H
#define FFINT8_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ff_ctx ff_ctx; /* opaque; holds device id, workspace pointer, last error text */

typedef enum {
  FF_OK = 0,
  FF_ERR_ARG = -1,             /* NULL pointer, non-positive size, unknown enum value          */
  FF_ERR_ALIGN = -2,           /* a device pointer is not 16-byte aligned                      */
  FF_ERR_WORKSPACE = -3,       /* workspace missing or smaller than ff_workspace_bytes says    */
  FF_ERR_NONFINITE = -4,       /* an input tensor held Inf/NaN (device-detected)               */
  FF_ERR_RANGE = -5,           /* worst-case INT32 accumulator or 32-bit index range exceeded  */
  FF_ERR_DEVICE_TIMEOUT = -6,  /* a bounded in-kernel wait ran out (device-detected)           */
  FF_ERR_CUDA = -7,            /* a CUDA runtime / driver call failed                          */
  FF_ERR_UNSUPPORTED_ARCH = -8 /* the device is not compute capability 10.x                    */
} ff_status;

enum { FF_OPT_SGD = 0, FF_OPT_ADAM = 1 };  /* ff_layer_desc.optimizer */
enum { FF_LINEAR = 0, FF_CONV3X3 = 1, FF_CONV1X1 = 2, FF_DWCONV3X3 = 3 };  /* ff_layer_desc.kind */
enum { FF_ROUND_NEAREST_EVEN = 0, FF_ROUND_STOCHASTIC = 1 }; /* rounding modes (Sec. IV-B) */
enum { FF_GEMM_AUTO = 0, FF_GEMM_SIMT = 1, FF_GEMM_TENSOR = 2 }; /* ff_set_gemm_path       */

/* indices into ff_layer_bufs.absmax (per-tensor SUQ ranges a = max|x|, Sec. IV; s = a/127) */
enum {
  FF_A_X_POS = 0, FF_A_X_NEG = 1, /* layer input, positive / negative set                    */
  FF_A_W = 2,                     /* weights                                                 */
  FF_A_DH_POS = 3, FF_A_DH_NEG = 4, /* output gradient g^Y                                   */
  FF_A_XNEXT_POS = 5, FF_A_XNEXT_NEG = 6, /* the normalised output (next layer's input)      */
  FF_ABSMAX_LEN = 8
};

/* One FF layer (host struct).  linear: X[M,K] -> Y[M,N], W[N,K].
 * conv3x3 (stride 1 or 2, zero padding 1, NHWC): X[M,H,Wd,Cin] -> Y[M,Ho,Wo,N], W[N,3,3,Cin] stored
 * as [N,K] with K = 9*Cin and k = (r*3+s)*Cin + ci; Ho = H, Wo = Wd at stride 1.
 * conv1x1 (pointwise, NHWC): X[M,H,Wd,Cin] -> Y[M,H,Wd,N], W[N,Cin], K = Cin: the dense MAC applied
 * at every position; goodness and normalisation over all H*Wd*N values of a sample.
 * dwconv3x3 (depthwise: one 3x3 filter per channel, no sum over channels; stride 1 or 2, zero padding 1,
 * NHWC): X[M,H,Wd,C] -> Y[M,Ho,Wo,C] with N = Cin = C, K = 9, W[C,3,3] stored as [C,9] (k = r*3+s). */
typedef struct {
  int32_t kind;
  int32_t K, N;
  int32_t H, Wd, Cin;   /* conv3x3 / conv1x1 only; 1,1,0 for linear                           */
  int32_t index;        /* position of the layer in the network (keys the rounding hash)      */
  int32_t round_x, round_w, round_dh; /* rounding of A, W, g^Y (paper: stochastic for A)      */
  float theta;          /* threshold of Eq. 1 / Eq. 2                                         */
  float lr;             /* SGD step size of the update (Alg. 1, update step)                        */
  float tau, eps;       /* length normalisation of the output: x = y*tau/(sqrt(G)+eps), eps>0 */
  uint64_t seed;        /* keys the stochastic-rounding hash                                  */
  int32_t stride;       /* conv3x3 / dwconv3x3 only: 0 or 1 = every position, 2 = every second row and column; */
                        /* the output then has Ho = (H-1)/2 + 1 rows of Wo = (Wd-1)/2 + 1 positions */
  float momentum;       /* update rule: 0 = plain SGD (W -= lr*g); mu > 0 = heavy-ball SGD on the   */
                        /* buffer Mom: m = mu*m + g, W -= lr*m (the paper names no optimiser)       */
  int32_t optimizer;    /* FF_OPT_SGD (the two forms above) or FF_OPT_ADAM: m = b1*m + (1-b1)*g,    */
                        /* v = b2*v + (1-b2)*g*g, W -= lr*(m*c1)/(sqrt(v*c2) + adam_eps) with       */
                        /* b1 = momentum, b2 = beta2, c_i = 1/(1 - b_i^t), t = step + 1; buffers   */
                        /* Mom and Var; the weight-gradient sums pass through accW_dump if given,  */
                        /* else through the workspace                                              */
  float beta2;          /* Adam only, in [0, 1)                                                    */
  float adam_eps;       /* Adam only, >= 0                                                         */
  int32_t pool;         /* 0 or 1: none; 2: the normalised output (Xnext and the next layer's input) */
                        /* is max-pooled 2x2 with stride 2 over the positions, [M,Ho/2,Wo/2,N]      */
                        /* (spatial layers with even Ho, Wo; goodness, loss and g^Y stay at full    */
                        /* resolution - no gradient passes through the pooling, Sec. IV-B)          */
  float skip_scale;     /* weight of the skip path: with ff_layer_bufs.Skip given, the layer hands         */
                        /* z = y*tau/(sqrt(G)+eps) + skip_scale*Skip to the next layer (a residual block,   */
                        /* Sec. IV-C / Table II; each operation rounded once).  The layer's own goodness,   */
                        /* loss and gradient are untouched: only what the next layer sees changes.          */
} ff_layer_desc;

/* Device buffers of one layer (host struct of device pointers; caller-owned). */
typedef struct {
  float* W;          /* [N,K] FP32 master weights; ff_layer_update rewrites them in place      */
  const float* X;    /* [M*Rin,Kin] FP32 input, already length-normalised (Kin = K, conv: Cin;  */
                     /* Rin = input rows per sample: 1, conv: H*Wd).                            */
                     /* In ff_train_step it may be NULL for layers > 0: the layer then takes   */
                     /* the previous layer's normalised output without materialising it.      */
  float* Y;          /* [M*R,N] FP32 out: max(0, float(acc)*s_x*s_w)                           */
  float* G;          /* [M] FP32 out: goodness per sample                                      */
  float* Xnext;      /* [M*R,N] FP32 out, nullable: Y*tau/(sqrt(G)+eps); [M*R/4,N] with pool = 2 */
  int8_t* Xq;        /* [M*Rin,Kin] INT8 out                                                   */
  int8_t* Wq;        /* [N,K] INT8 out                                                         */
  int8_t* dHq;       /* [M*R,N] INT8 out (ff_layer_loss_grad)                                  */
  float* absmax;     /* [FF_ABSMAX_LEN] FP32 out, see FF_A_*                                   */
  uint64_t* S;       /* [M] out: exact integer sum over the sample of relu(acc)^2              */
  int32_t* rowmax;   /* [M] out: max over the sample of relu(acc)                              */
  float* coef;       /* [M] out: per-sample dL_new/dG / M  (g^Y = 2*coef*Y)                    */
  float* loss;       /* [1] out: L_new averaged over the M samples (Eq. 3)                     */
  int32_t* acc_dump; /* [M*R,N] INT32 out, nullable: the forward accumulators                  */
  int32_t* accW_dump;/* [2,N,K] INT32 out, nullable: g^W accumulators of the two sets          */
  float* Mom;        /* [N,K] FP32 in/out momentum buffer; needed (and touched) only if momentum != 0 */
                     /* or the optimiser is Adam (first moment)                                */
  float* Var;        /* [N,K] FP32 in/out second-moment buffer; Adam only                      */
  const float* Skip; /* [M*R,N] FP32 in, nullable: skip path of a residual block, added (times skip_scale) to the */
                     /* normalised output - typically the X of the block's first layer or the Xnext of the layer  */
                     /* before it.  Needs Xnext (the sum is written there, then quantised for the next layer) and */
                     /* no pooling.  Must not alias Xnext.                                                       */
  int32_t ld_xq;     /* linear layers only: row pitch of Xq in bytes, 0 = K (dense).  A pitch that is a */
  int32_t ld_dhq;    /* multiple of 128 keeps every TMA box row of the contractions aligned when K (N  */
                     /* for dHq) is not: >= the row length, a multiple of 16.  All rows x pitch bytes  */
                     /* belong to the buffer; the padding bytes are never written, and whatever they  */
                     /* hold reaches no result (copies may fetch them)                                */
} ff_layer_bufs;

/* Create / destroy a context for CUDA device `device` (must be compute capability 10.x).
 * ff_create makes the device current and allocates nothing on it.  A context holds host state only
 * (route choices, the last error text, captured launch sequences) and is not thread-safe: calls on one
 * context must not overlap in time; its kernels share the workspace, so they belong on one stream (or on
 * streams the caller orders).  Several contexts, each with its own workspace, are independent. */
ff_status ff_create(ff_ctx** out, int device);
ff_status ff_destroy(ff_ctx* ctx);

/* Scratch bytes needed for n_layers layers at batch B (host computation only). */
ff_status ff_workspace_bytes(const ff_layer_desc* layers, int n_layers, int B, size_t* out_bytes);
/* Hand the context a caller-owned device buffer (256-byte aligned) of at least that size.  The
 * first call on a stream after this zeroes the status word. */
ff_status ff_set_workspace(ff_ctx* ctx, void* dev_ptr, size_t bytes);

/* Choose the contraction kernels: AUTO picks the tcgen05 tensor-core kernels whenever the shape
 * allows and the SIMT kernels otherwise; SIMT / TENSOR force one (TENSOR fails with FF_ERR_ARG on
 * shapes it cannot take).  Both produce identical bits. */
ff_status ff_set_gemm_path(ff_ctx* ctx, int path);

/* The tensor-core kernels run either one CTA per 128 x 256 output tile or a pair of CTAs (tcgen05
 * cta_group::2) per 256 x 256 tile.  ctas_per_tile = 0 chooses by problem size (pairs once the
 * output has more than 128 rows), 1 / 2 force one form.  Identical bits. */
ff_status ff_set_tensor_form(ff_ctx* ctx, int ctas_per_tile);

/* Positive / negative / candidate batches by label embedding (Sec. III: the true label makes a
 * positive sample, a wrong one a negative; Alg. 1, sample generation).  x [B, n] FP32 raw samples (device),
 * labels [sets, B] INT32 (device; the wrong labels of a negative set are drawn by the caller).
 * out [sets*B, n] FP32 (device): row s*B + b = sample b with labels[s, b] written one-hot over its
 * label places - flat positions 0, label_stride, ..., (n_classes-1)*label_stride hold on_value at the
 * label and zero elsewhere (label_stride = 1 for a vector, = channels for a channels-last image whose
 * first pixels of channel 0 carry the label).  tau0 > 0: every row is then scaled to length tau0,
 * r = tau0 / (float(sqrt(sum of squares, FP64)) + eps), one FP32 multiply per element (the sum's
 * order is free, so rows agree with a reference to FP32 rounding, not always bit for bit); tau0 <= 0:
 * no scaling.  sets = 2 with (true, wrong) labels gives a training batch for ff_train_step, sets =
 * n_classes with labels[c, b] = c the candidate batch for ff_predict.  x and out must not overlap.
 * A label outside [0, n_classes) leaves its row without a hot place and makes the next ff_poll_status
 * return FF_ERR_RANGE.  Asynchronous on the stream; nothing is allocated. */
ff_status ff_embed_labels(ff_ctx* ctx, const float* x, const int32_t* labels, int B, int n, int sets, int n_classes,
                          int label_stride, float on_value, float tau0, float eps, float* out, void* cuda_stream);

/* ---- data-parallel train step --------------------------------------------------------------
 * The batch of one step split by rows over several devices, each holding a replica of the weights:
 * forward, goodness, loss coefficient and output gradient are per sample (Sec. III, Sec. IV-B), so a
 * shard computes them alone; what couples the shards are (1) the per-tensor ranges of the symmetric
 * quantiser (a maximum over the whole batch), (2) the batch mean of the loss, (3) the INT32
 * weight-gradient sums g^W = g^Y^T A (Sec. IV-B), which add exactly in integers.  With those
 * three combined over the shards every replica applies the same update, bit-identical to
 * ff_train_step on the whole batch on one device (the stochastic-rounding counters are the element
 * indices of the unsplit tensors).  The paper trains on one device and describes no such split.
 *
 * The step is cut at the points where shards must exchange data.  The caller runs phases
 * 0 .. ff_dp_phase_count(n_layers)-1 in order, on every shard; after each phase it combines, in place
 * and over all shards, the n_reduce device arrays listed in `reduce` (element type and operation given
 * per entry; any all-reduce will do, e.g. NCCL's, ordered after the phase on the stream).  Every entry
 * names the first phase that reads the combined array (needed_by_phase): the reduction must have
 * finished when that phase starts, and the library touches the array in none of the phases between.
 * The library itself performs no communication.  With n = n_layers:
 *   phase 0: ranges of the network input              -> MAX of 2 floats                 (needed by 1)
 *   phase 1+l: forward of layer l                     -> MAX of the output / next-input ranges (next phase)
 *   phase n+1: losses and coefficients, all layers    -> MAX of the dH ranges, SUM of the loss shares (n+2)
 *   phase n+2+l: INT8 dH and local g^W sums of layer l -> SUM of INT32 accW_dump [2][N][K] (needed by 2n+2+l)
 *   phase 2n+2+l: update of layer l from the combined sums
 * so the large INT32 reduction of layer l can run (on a stream of its own, after an event recorded behind
 * phase n+2+l) while the weight-gradient contractions of the layers after it still compute, and a layer's
 * update waits for its own sums only.
 * B_local rows per set are rows [row_offset, row_offset + B_local) of the B_total rows per set of the
 * whole batch.  Layers must be chained (X of layers > 0 NULL), accW_dump of every layer non-NULL (it
 * carries the sums), and every shard must pass the same descriptors (seed included), lambda and step.
 * A spatial layer whose whole-batch contraction could leave INT32 in the worst case is held to a share of
 * the INT32 range per shard in proportion to its rows (FF_ERR_RANGE otherwise), so that the 32-bit sums of
 * the shards cannot wrap.  `reduce` has room for FF_DP_MAX_REDUCE entries.  Errors as ff_train_step. */
#define FF_DP_MAX_REDUCE 96
enum { FF_DP_F32 = 0, FF_DP_I32 = 1 };
enum { FF_DP_MAX = 0, FF_DP_SUM = 1 };
typedef struct ff_dp_reduce {
  void* dev_ptr;   /* device array to combine in place over the shards */
  uint64_t count;  /* elements */
  int32_t dtype;   /* FF_DP_F32 / FF_DP_I32 */
  int32_t op;      /* FF_DP_MAX / FF_DP_SUM */
  int32_t needed_by_phase;  /* first phase that reads the combined array */
  int32_t reserved;
} ff_dp_reduce;
int ff_dp_phase_count(int n_layers);
ff_status ff_dp_train_phase(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B_local,
                            int B_total, int row_offset, int phase, float lambda, uint64_t step, void* cuda_stream,
                            ff_dp_reduce* reduce, int* n_reduce);

/* Launch-sequence replay for ff_train_step and ff_predict (the paper's edge setting, batch 32 in Sec. V, makes a step a
 * chain of short kernels whose cost is launch overhead; it states no counterpart of this switch).
 * on = 1: the first ff_train_step (or ff_predict) call of a call shape runs its kernels one by one, the second is
 * captured into a CUDA graph, and every later one is a single graph launch; the step counter and
 * lambda are read from device memory, so they may change from call to call.  A call shape is the byte
 * content of the layer and buffer arrays (zero any padding), n_layers, B, the workspace and the
 * contraction route (the stream may change, the legacy default stream included); another shape gets a graph of its own (16 are kept, least recently used
 * dropped), so a value inside a descriptor that changes every step (lr, theta) defeats the replay.
 * Results are bit-identical to on = 0.  Replay is bypassed while ff_profile_start is active or the stream
 * is already being captured by the caller.  on = 0 (default) drops the graphs.  Host state only: no
 * device memory is allocated by the library beyond what graph instantiation itself takes. */
ff_status ff_set_graph_mode(ff_ctx* ctx, int on);
/* ff_train_step / ff_predict calls served by a graph launch so far (0 while the mode is off).  A call shape whose
 * capture fails keeps running kernel by kernel and says why through ff_last_error. */
uint64_t ff_graph_replay_count(const ff_ctx* ctx);

/* Forward of one layer (Sec. IV-B: quantise A and W, INT8 MAC with INT32 accumulation; Sec. III /
 * Alg. 1, goodness step: goodness).  Reads X, W.  Writes Xq, Wq, absmax[X,W,XNEXT], Y, S, rowmax, G,
 * Xnext (if non-NULL), acc_dump (if non-NULL).  `step` keys the stochastic rounding. */
ff_status ff_layer_forward(ff_ctx* ctx, const ff_layer_desc* layer, const ff_layer_bufs* bufs,
                           int B, uint64_t step, void* cuda_stream);

/* Loss and output gradient of one layer (Eq. 1, Eq. 2; look-ahead Eq. 3, Eq. 4; Sec. IV-B: g^Y is formed and
 * quantised to INT8 before the weight gradient).  G_later[j] (device, [M] each) and
 * theta_later[j] (host) are the goodness and thresholds of the n_later subsequent layers; with
 * n_later = 0 or lambda = 0 this is the vanilla FF loss.  Reads G, Y, rowmax, absmax[X,W].
 * Writes loss, coef, absmax[DH], dHq. */
ff_status ff_layer_loss_grad(ff_ctx* ctx, const ff_layer_desc* layer, const ff_layer_bufs* bufs,
                             int B, const float* const* G_later, const float* theta_later,
                             int n_later, float lambda, uint64_t step, void* cuda_stream);

/* Weight gradient and update of one layer (Sec. IV-B: g^W is a second INT8 MAC and is the only
 * gradient formed and applied; Alg. 1, update step).  Reads dHq, Xq, absmax, W.  Writes W
 * (W - lr*(float(accP)*cP + float(accN)*cN)) and accW_dump (if non-NULL); with momentum != 0 or
 * optimizer = FF_OPT_ADAM the step follows that rule and Mom (and Var) are rewritten.  `step` is the
 * step counter of the update (Adam's update number is t = step + 1; the other rules do not read it). */
ff_status ff_layer_update(ff_ctx* ctx, const ff_layer_desc* layer, const ff_layer_bufs* bufs,
                          int B, uint64_t step, void* cuda_stream);

/* Body of Algorithm 1's epoch loop for n_layers layers: one INT8 forward through all layers with
 * the pre-update weights, goodness of every layer, then per layer the loss with look-ahead
 * weight `lambda` (Eq. 3) and the INT8 gradient + update.  Layer 0
 * reads bufs[0].X; layer l > 0 reads bufs[l].X if non-NULL, else layer l-1's normalised output.
 * With n_layers = 1 and lambda = 0 it equals forward -> loss_grad -> update. */
ff_status ff_train_step(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs,
                        int n_layers, int B, float lambda, uint64_t step, void* cuda_stream);

/* One step of layer-by-layer training (Sec. III: a layer is trained to the end before its successor
 * is; Sec. IV-B trains every layer this way when the look-ahead of Sec. IV-C is off).  As
 * ff_train_step, but the layers [0, first_trained) are frozen: they run the INT8 forward with their
 * current weights and hand their normalised output on; no loss, g^Y, g^W or update is computed for
 * them and their coef, loss, dHq, absmax[DH] and W stay untouched.  Layers first_trained .. n_layers-1
 * are trained as in ff_train_step (each looks ahead at the layers after it).  first_trained = 0 is
 * ff_train_step itself; first_trained = n_layers-1 with lambda = 0 is one step of the greedy schedule.
 * Replayed like ff_train_step when ff_set_graph_mode is on (one captured sequence per first_trained). */
ff_status ff_train_step_from(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers,
                             int first_trained, int B, float lambda, uint64_t step, void* cuda_stream);

/* Classification of B samples by goodness with the current weights.  The paper reports accuracy but
 * does not describe the procedure; this is the Forward-Forward one its Sec. III builds on (layers are
 * trained to respond strongly to positive samples): every sample is presented once per candidate label,
 * label written one-hot into the input exactly as for the positive set; each candidate runs through
 * the same INT8 forward as training (Sec. IV-B; Alg. 1, forward pass); the goodness of the layers
 * first_counted_layer .. n_layers-1 is added per candidate (FP32, in layer order) and the label with
 * the largest total wins (lowest label on ties).
 * Layout: the caller builds the candidate batch [n_classes*B, ...] in bufs[0].X, row c*B + b = sample
 * b with candidate label c, already length-normalised.  Every layer input of the candidate batch is
 * quantised with one per-tensor range (all candidates of a sample under the same quantisation step;
 * both entries of absmax[X] / absmax[XNEXT] hold it).  The rows are processed as two halves, so
 * n_classes*B must be even and every buffer of `bufs` must be sized for n_classes*B rows (i.e. as for
 * a batch of n_classes*B/2 positives + negatives).  Writes scores [n_classes*B] (row c*B + b) and pred [B] (device, 16-byte
 * aligned) and, as a side effect, the forward outputs of every layer.  No weights change. */
ff_status ff_predict(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B,
                     int n_classes, int first_counted_layer, float* scores, int32_t* pred, uint64_t step,
                     void* cuda_stream);

/* Synchronises `cuda_stream`, reads the device status word and clears it.  Returns FF_OK,
 * FF_ERR_DEVICE_TIMEOUT (a bounded wait inside a kernel ran out), FF_ERR_NONFINITE (a tensor to be quantised
 * held Inf / NaN), FF_ERR_RANGE (a label outside its range, or a weight-gradient sum outside INT32: convolution
 * weight gradients sum over every position of a set, are accumulated in parts that cannot wrap and added in
 * 64 bits; a weight whose sum leaves INT32 keeps its value) or FF_ERR_CUDA. */
ff_status ff_poll_status(ff_ctx* ctx, void* cuda_stream);

/* Self-test of the library's failure reporting (the paper has no counterpart).  Every wait inside the
 * contraction kernels is bounded: when one runs out, the kernel raises a status bit and returns instead of
 * hanging, and ff_poll_status turns the bit into FF_ERR_DEVICE_TIMEOUT.  This call launches a one-thread kernel
 * that runs that same wait, with a limit of limit_ns nanoseconds (1 .. 1e9), on a barrier nothing ever arrives
 * on; the next ff_poll_status must therefore return FF_ERR_DEVICE_TIMEOUT, and the context stays usable.
 * Nothing else is touched. */
ff_status ff_selftest_bounded_wait(ff_ctx* ctx, uint64_t limit_ns, void* cuda_stream);

/* How the library would cut a layer's weight gradient so that no INT32 sum can wrap (Sec. IV-B: INT8 operands,
 * INT32 accumulation; a sum over more than 133144 = floor((2^31 - 1) / 127^2) products could).  Host arithmetic
 * only - no context, no device: the planning functions the launches themselves call, for tests and for inspection.
 * route: FF_PLAN_TENSOR_SLABS (tcgen05 split contraction of 3x3 / pointwise convolutions), FF_PLAN_FIRST_LAYER
 * (3x3 layers with at most four input channels), FF_PLAN_DP4A_SLABS (the fallback kernels; workspace_bytes limits
 * its slabs).  On FF_OK: `splits` work items along the contraction, `parts` INT32 arrays left for the 64-bit reduce +
 * update kernel, `longest_register_sum` / `longest_part_sum` the most products any accumulator / any array element
 * sums (contraction elements of one set).  FF_ERR_ARG: the route does not take this layer; FF_ERR_WORKSPACE: the
 * workspace cannot hold as many slabs as safety needs. */
enum { FF_PLAN_TENSOR_SLABS = 0, FF_PLAN_FIRST_LAYER = 1, FF_PLAN_DP4A_SLABS = 2 };
typedef struct ff_wgrad_plan {
  int32_t splits;
  int32_t parts;
  int64_t longest_register_sum;
  int64_t longest_part_sum;
} ff_wgrad_plan;
ff_status ff_plan_wgrad(const ff_layer_desc* layer, int32_t B, int32_t sm_count, int32_t route, uint64_t workspace_bytes,
                        ff_wgrad_plan* out);

/* Text of the last error returned for this context (host string, valid until the next call). */
const char* ff_last_error(const ff_ctx* ctx);

/* Number of kernels the library has launched through this context so far (host counter). */
uint64_t ff_launch_count(const ff_ctx* ctx);

/* Per-kernel device timing.  Between ff_profile_start and ff_profile_stop every kernel the library
 * launches through this context is bracketed by a pair of CUDA events on its stream.
 * ff_profile_stop synchronises `cuda_stream` and returns, per kernel kind (FF_K_*), the summed
 * device time in milliseconds and the number of launches (host arrays of FF_K_COUNT entries). */
enum {
  FF_K_ABSMAX = 0,   /* per-tensor max|x| (Sec. IV, SUQ range)                                   */
  FF_K_QUANTIZE,     /* SUQ of A or W to INT8 (the W call also clears S and rowmax)              */
  FF_K_FWD_GEMM,     /* forward INT8 MAC + dequantise/ReLU/goodness epilogue                     */
  FF_K_FINALIZE,     /* G from S, range of the normalised output                                 */
  FF_K_NORMALIZE,    /* length normalisation (+ next layer's SUQ)                                */
  FF_K_LOSS,         /* Eq. 1-4: loss and per-sample coefficient                                 */
  FF_K_DH_QUANTIZE,  /* g^Y to INT8                                                              */
  FF_K_UPD_GEMM,     /* g^W INT8 MAC + SGD update epilogue                                       */
  FF_K_RAW_GEMM,     /* ff_int8_gemm                                                             */
  FF_K_CLASSIFY,     /* ff_predict: per-candidate goodness totals and their argmax               */
  FF_K_DW_FWD,       /* depthwise 3x3 forward MAC + dequantise/ReLU/goodness                     */
  FF_K_DW_UPD,       /* depthwise 3x3 g^W sums + update                                          */
  FF_K_COUNT
};
ff_status ff_profile_start(ff_ctx* ctx);
ff_status ff_profile_stop(ff_ctx* ctx, void* cuda_stream, float* ms_per_kernel, uint32_t* launches_per_kernel);

/* Stand-alone INT8 contraction used by the unit tests and the kernel benchmark (Sec. IV-B,
 * "integer matrix multiplication with INT8 inputs and INT32 accumulation"):
 *   trans = 0: C[m,n] = sum_k A[m,k]*B[n,k]   A [M,K], B [N,K]  (forward orientation)
 *   trans = 1: C[m,n] = sum_k A[k,m]*B[k,n]   A [K,M], B [K,N]  (weight-gradient orientation)
 * A, B device INT8 row-major; C device INT32 [M,N] row-major. */
ff_status ff_int8_gemm(ff_ctx* ctx, const int8_t* A, const int8_t* B, int32_t* C, int M, int N,
                       int K, int trans, void* cuda_stream);

/* Loss, per-sample coefficient and g^Y range of one layer without any caller-provided scratch.
 * (The paper has no counterpart: this is a packaging variant of the loss step of
 * ff_layer_loss_grad, not a different computation.)
 *
 * Who it is for: code that runs where device memory cannot be allocated -- a plug-in called inside
 * another framework's stream callback or memory-pool critical section, a process whose memory was
 * handed out in full at start-up, a caller that holds no ff_ctx and no workspace.  Everything else
 * in this library keeps its partial sums in the workspace the caller allocates; here they live in a
 * small array (about 16 KiB) built into the library image, which every GPU that loads the library
 * keeps until the process ends.  The call allocates nothing: no cudaMalloc, no cudaFree, no
 * workspace, no context.
 *
 * Same arithmetic and same outputs as the loss kernel behind ff_layer_loss_grad: reads G [2B],
 * rowmax [2B] and absmax[FF_A_X_POS..FF_A_W]; writes coef [2B], loss [1] and
 * absmax[FF_A_DH_POS..FF_A_DH_NEG].  It does not quantise g^Y.  All pointers are device pointers
 * on the CURRENT device; G_later / theta_later are host arrays as in ff_layer_loss_grad.
 *
 * Limits and rules:
 *  - 2*B <= FF_STATIC_LOSS_MAX_SAMPLES (the array is laid out for that many samples); larger
 *    batches are refused with FF_ERR_RANGE.
 *  - The first call on each device looks up the array's device address (a synchronous runtime
 *    query); make that first call before starting any stream capture on that device.
 *  - All calls share the one array per device.  It keeps the previous call's contents; the call
 *    clears the one word that must start at zero.  Two calls whose kernels can run at the same time
 *    on one device (different streams) race on it: keep calls on a device in stream order.
 *  - `err` (nullable) receives a short text when the return value is not FF_OK. */
#define FF_STATIC_LOSS_MAX_SAMPLES 65536
ff_status ff_loss_coef_static(const float* G, float theta, const float* const* G_later, const float* theta_later,
                              int n_later, float lambda, int B, const int32_t* rowmax, float* absmax, float* coef,
                              float* loss, void* cuda_stream, char* err, size_t err_len);

#ifdef __cplusplus
}
#endif
#endif /* FFINT8_H */
