/*
 * pb.h - C interface of the B200 Pipelined Backpropagation engine.
 *
 * One handle simulates fine-grained Pipelined Backpropagation (PB) at batch
 * size one on a single GPU: the network is cut into S stages; at every tick
 * each stage runs a forward on the sample that has reached it and a backward
 * on the sample whose gradient has come back to it, then updates its own
 * weights with SGD-momentum, Spike Compensation (SC) and Linear Weight
 * Prediction (LWP), each with that stage's delay D_s = 2 (S - 1 - s)
 * (paper: Appendix "Pipelined Backpropagation", Eqs. W_i / F_i; Section
 * "Methods", SC_D coefficients, LWP velocity form, "Combined Mitigation").
 *
 * Conventions
 *   - Every function returns PB_OK (0) or a negative pb_status; nothing throws
 *     or aborts across this boundary.  pb_last_error() gives the text of the
 *     last failure on a handle (or of pb_create when given NULL).
 *   - "host" pointers are ordinary CPU memory, "dev" pointers are CUDA device
 *     memory on the device that was current at pb_create.  The caller owns
 *     every buffer it passes; the library owns all state behind the handle.
 *   - All work is issued on the stream given to pb_create (a cudaStream_t cast
 *     to void*, NULL = the default stream).  Calls taking host output
 *     pointers synchronise that stream; the others do not.
 *   - Tensors of one sample are [C, H, W], float32.  Parameters are one flat
 *     float32 vector in layer-list order: FC -> weight [out, in] then bias
 *     [out]; CONV2D -> weight [c_out, c_in, k, k]; GROUPNORM -> scale [c] then
 *     shift [c].
 */
#ifndef PB_B200_H
#define PB_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pb_handle pb_handle; /* opaque */

typedef enum {
    PB_OK = 0,
    PB_E_ARG = -1,      /* NULL pointer, bad size, bad flag                     */
    PB_E_SHAPE = -2,    /* layer list does not chain (channel/size mismatch)    */
    PB_E_ALLOC = -3,    /* device or host allocation failed                     */
    PB_E_CUDA = -4,     /* a CUDA call or kernel launch reported an error       */
    PB_E_DEVICE = -5,   /* a kernel set the device error word (index check)     */
    PB_E_UNSUPPORTED = -6
} pb_status;

/* Layer kinds.  A stage begins with PB_FC or PB_CONV2D (the layer that owns
 * the weights); the others ride in the stage of the layer before them, in the
 * order conv -> groupnorm -> add_skip -> relu -> maxpool | avgpool_global,
 * or fc -> relu, or fc -> softmax_ce (last stage only).  Grouping convolution,
 * normalisation and activation into one stage follows Section 2.1. */
typedef enum {
    PB_FC = 0, PB_CONV2D = 1, PB_GROUPNORM = 2, PB_RELU = 3, PB_MAXPOOL = 4,
    PB_AVGPOOL_GLOBAL = 5, PB_ADD_SKIP = 6, PB_SOFTMAX_CE = 7
} pb_op;

typedef struct {
    int32_t op;        /* pb_op                                                  */
    int32_t c_in;      /* FC: flattened input size; CONV2D/GROUPNORM: channels   */
    int32_t c_out;     /* FC: outputs; CONV2D: output channels                   */
    int32_t k;         /* CONV2D / MAXPOOL window                                */
    int32_t stride;    /* CONV2D / MAXPOOL                                       */
    int32_t pad;       /* CONV2D / MAXPOOL                                       */
    int32_t groups;    /* GROUPNORM                                              */
    int32_t src;       /* FC/CONV2D: stage whose output is read (-1: the stage
                          before, or the network input for stage 0);
                          ADD_SKIP: stage whose output is added                  */
    int32_t skip_mode; /* ADD_SKIP: 0 identity, 1 every second pixel + zero
                          channels appended up to c_out.  + 2 (pre-activation
                          residual networks, Section "Experiments" / Experiment
                          Details): the input joins the convolution output
                          BEFORE the normalisation, and it is the source
                          stage's own convolution output after ITS such
                          addition (the running residual sum) instead of that
                          stage's output; such an ADD_SKIP is listed before the
                          stage's GROUPNORM, joins two CONV2D stages and runs on
                          the float32 convolution path only (with PB_CONV_BF16:
                          PB_E_UNSUPPORTED)                                      */
} pb_layer;

/* Mitigation switches (Section "Methods").  PB_SC: a = m^D, b = (1-m^D)/(1-m),
 * else a = 1, b = 0.  PB_LWP: forward weights w_hat = w - lr*T*v with T = D,
 * else T = 0.  PB_LWP_WFORM (with PB_LWP): predict with the weight-difference
 * form w_hat = w + T (w - w_previous) instead of the velocity form; the two
 * differ once SC is on (Section "Combined Mitigation").  PB_CONV_BF16:
 * convolutions multiply bf16 operands with fp32 accumulation; master weights,
 * velocity and everything else stay fp32.
 * PB_WEIGHT_STASH: the comparison mode of Appendix "Pipelined Backpropagation"
 * (Eq. W_{i+1} = W_i - eta grad L(x_i; F_i), PipeDream's weight stashing):
 * every stage keeps, per sample in flight, the weights its forward pass used
 * (D_s + 1 versions) and takes that sample's backward pass with them instead
 * of the current weights; the update still moves the current weights.  It
 * costs (D_s + 1) copies of every stage's weights in device memory and one more
 * read and write of the weights per tick, and can be combined with the other
 * flags.  pb_create returns PB_E_UNSUPPORTED when the copies would need more
 * than 16 GiB. */
enum { PB_SC = 1, PB_LWP = 2, PB_LWP_WFORM = 4, PB_CONV_BF16 = 8, PB_WEIGHT_STASH = 16 };

/* Builds the engine.  layers/stage_of_layer: host arrays of n_layers entries,
 * stage indices non-decreasing from 0.  (in_c, in_h, in_w): shape of one
 * sample.  The last stage must end in PB_SOFTMAX_CE over n_classes outputs.
 * stream: cudaStream_t as void*.  All device memory is allocated here, once
 * (weights, velocity, activation rings of D_s + 1 slots per stage, gradient
 * hand-off buffers); ticks allocate nothing.  Weights start at zero: call
 * pb_set_weights.  On failure *out is NULL. */
int pb_create(const pb_layer* layers, int n_layers, const int32_t* stage_of_layer,
              int in_c, int in_h, int in_w, int n_classes,
              float lr, float momentum, unsigned flags, void* stream,
              pb_handle** out);

/* Copies n = pb_num_params() floats from host memory into the master weights,
 * zeroes the velocity and restarts the pipeline at tick 0. */
int pb_set_weights(pb_handle* h, const float* host_w, size_t n);

/* Over- or under-compensation (paper: generalized Spike Compensation with
 * other a, b, e.g. SC_2D; Appendix "Extended Weight Prediction Horizons",
 * T = alpha D).  Stage s then uses a = m^(sc_delay_scale * D_s),
 * b = (1 - a)/(1 - m) and T = horizon_scale * D_s; (1, 1) is the default
 * SC_D + LWP_D.  Takes effect for ticks issued after the call, for every
 * stage alike: the next forward of each stage already predicts with the new T
 * (stored predicted weights are re-made from the current w and v), and its
 * next update uses the new a, b.  With PB_LWP_WFORM the prediction is made from
 * the previous weights, which are not kept, so there the call is only accepted
 * before the first tick (PB_E_UNSUPPORTED afterwards).  Synchronises the
 * stream.  Scales must be >= 0. */
int pb_set_mitigation(pb_handle* h, float sc_delay_scale, float horizon_scale);

/* Fill-and-drain training (Section 1; Appendix "Pipelined Backpropagation":
 * mini-batch SGD on a pipeline).  With n_samples = N > 0 the engine stops
 * being asynchronous: time is cut into cycles of N + 2 (S - 1) ticks; a
 * sample enters at each of the first N ticks of a cycle, nothing enters while
 * the pipeline drains (the dev_x / dev_xs entry and label of such a tick must
 * still be valid memory, but their values are not used, and the tick's loss is
 * NaN when no sample reaches the last stage), and each stage takes ONE plain
 * SGD-with-momentum step per cycle with the mean of the N gradients,
 * v <- m v + mean g, w <- w - lr v, once its last backward of the cycle is
 * done.  Forward and backward of every sample then use the same weights, so
 * SC and LWP have nothing to compensate and are off in this mode whatever the
 * flags say; weights and velocities are those of ordinary mini-batch SGD at
 * every cycle boundary.  N = 0 returns to pipelined backpropagation.  Call it
 * while the tick count is zero (after pb_create or pb_set_weights), else
 * PB_E_ARG.  Synchronises the stream. */
int pb_set_update_size(pb_handle* h, int n_samples);

/* One tick.  dev_x: the new sample (in_c*in_h*in_w floats, device memory; it
 * is copied into the engine's input ring, so it may be reused after the call
 * returns in stream order).  label in [0, n_classes).  If host_loss is not
 * NULL the stream is synchronised and *host_loss receives the loss the last
 * stage computed in this tick, which belongs to the sample fed S-1 ticks
 * earlier (a sample needs 2S-1 steps, Appendix "Pipelined Backpropagation");
 * it is NaN during the first S-1 ticks.
 * Alignment: dev_x (and dev_xs of pb_run / pb_mlp_run_static) must be 16-byte
 * aligned when the network is fully connected and the sample length is a
 * multiple of 4 (the first stage then reads the sample 16 bytes at a time);
 * otherwise PB_E_ARG is returned before anything is launched.  In every other
 * case 4-byte alignment is enough. */
int pb_tick(pb_handle* h, const float* dev_x, int label, float* host_loss);

/* n_ticks ticks without host synchronisation.  dev_xs: [n_ticks, sample]
 * floats, dev_labels: [n_ticks] int32, both device memory that must stay
 * valid and unchanged until the stream has run the ticks (each sample and label
 * is copied into the engine's rings at its tick, because stage 0 reads the
 * sample again at its backward 2(S-1) ticks later); dev_losses: [n_ticks]
 * floats (device) or NULL, entry k receiving what pb_tick would have returned
 * at the k-th tick of this call.  Continues from the current tick, so
 * consecutive calls feed one continuous stream of samples.  n_ticks == 0 is a
 * no-op (the pointers are not examined); a negative count is PB_E_ARG. */
int pb_run(pb_handle* h, const float* dev_xs, const int32_t* dev_labels,
           int n_ticks, float* dev_losses);

/* Same as pb_run but every pointer is host memory: the call copies the inputs
 * to the device, runs the ticks, copies the losses back and synchronises. */
int pb_run_host(pb_handle* h, const float* host_xs, const int32_t* host_labels,
                int n_ticks, float* host_losses);

/* Master weights / velocities to host memory (n must equal pb_num_params);
 * synchronises the stream. */
int pb_get_weights(pb_handle* h, float* host_w, size_t n);
int pb_get_velocity(pb_handle* h, float* host_v, size_t n);

/* Waits for the stream and reports a set device error word as PB_E_DEVICE. */
int pb_sync(pb_handle* h);

size_t pb_num_params(const pb_handle* h);
int pb_num_stages(const pb_handle* h);
/* D_s = 2 (S - 1 - s); negative status for a bad stage index. */
int pb_stage_delay(const pb_handle* h, int s);
/* Ticks run since the last pb_set_weights. */
long long pb_tick_count(const pb_handle* h);
/* Kernel launches issued by the last pb_tick/pb_run/pb_run_host call. */
long long pb_last_launch_count(const pb_handle* h);
/* Bytes of device memory the handle holds. */
size_t pb_device_bytes(const pb_handle* h);

/* Timing hooks for benchmarks: device time in milliseconds that the kernel
 * class `which` (0 = FC tick kernel, 1 = last-stage loss/backward kernel,
 * 2 = update kernel, 3 = float32 conv GEMMs, 4 = tensor-core fprop, 5 = conv
 * normalise/activate/pool forward, 6 = its backward, 7 = tensor-core wgrad,
 * 8 = tensor-core dgrad) took over the last pb_run, measured
 * with CUDA events on the engine's stream when enabled (enable != 0 costs a
 * pair of event records per launch).  Returns a negative value when disabled
 * or never run; *launches receives the number of launches timed. */
int pb_profile_enable(pb_handle* h, int enable);
double pb_profile_ms(pb_handle* h, int which, long long* launches);

/* ---- Stage split over several GPUs (Section 2.1: stages split over GPUs, one
 * host thread per GPU; Appendix "Batch Parallel vs Pipeline Parallel
 * Computation": neighbours exchange one activation forward and one gradient
 * backward per tick, nothing else).  Fully connected networks only.
 *
 * pb_split_plan: contiguous stage ranges [lo[r], hi[r]) for n_ranks ranks that
 * minimise the largest per-tick weight traffic (16 bytes per parameter) of any
 * rank.  Host arithmetic only (no device is touched).  lo / hi: n_ranks ints.
 *
 * pb_create_split: as pb_create, but the handle runs only the stages of `rank`
 * in that plan, on the device current at the call.  Every rank is fed the same
 * tick stream: pb_tick / pb_run use dev_x only on the rank that owns stage 0
 * (elsewhere it may be NULL) and the label only on the rank that owns the last
 * stage, whose loss is the tick's loss (other ranks return NaN).
 * pb_set_weights takes the whole network's vector on every rank and keeps its
 * own stages' part; pb_get_weights / pb_get_velocity return the own stages'
 * values and zeros elsewhere (the caller adds the ranks' vectors up).
 *
 * Hand-off: pb_split_ports gives the device addresses where THIS rank receives
 * (its copy of the previous rank's boundary activation ring, of the next
 * rank's boundary gradient buffer, and their tick stamps); pb_split_connect is
 * given the neighbours' ports (NULL where there is no neighbour).  At the end
 * of every tick a rank writes its boundary tensors and the stamp t + 1 into
 * its neighbours' ports with plain stores (the ranks' devices must have peer
 * access to each other when they differ; nothing else is required), and at the
 * start of tick t it waits, for at most one second, until both of its own
 * stamps have reached t; an expired wait is reported as PB_E_DEVICE by the next
 * synchronising call.  Ranks may therefore run at most one tick apart.  On ONE
 * device (testing), tick the ranks in turn with pb_tick, rank 0 first: then
 * every stamp is already in place when it is looked at and nothing waits. */
typedef struct {
    void* act;          /* boundary activation ring [slots][dim] floats          */
    void* act_stamp;    /* int64 tick stamp                                      */
    void* grad;         /* boundary gradient buffer [2][dim] floats              */
    void* grad_stamp;   /* int64 tick stamp                                      */
} pb_split_port;

int pb_split_plan(const pb_layer* layers, int n_layers, const int32_t* stage_of_layer,
                  int in_c, int in_h, int in_w, int n_classes, int n_ranks, int32_t* lo, int32_t* hi);
int pb_create_split(const pb_layer* layers, int n_layers, const int32_t* stage_of_layer,
                    int in_c, int in_h, int in_w, int n_classes,
                    float lr, float momentum, unsigned flags, void* stream,
                    int rank, int n_ranks, pb_handle** out);
int pb_split_range(const pb_handle* h, int32_t* lo, int32_t* hi);
int pb_split_ports(pb_handle* h, pb_split_port* mine);
int pb_split_connect(pb_handle* h, const pb_split_port* prev_rank, const pb_split_port* next_rank);

/* Least device-memory traffic, in bytes per steady-state tick, of kernel class
 * `which` as the engine is configured: 0 = the FC tick kernel (one read and one
 * write of w and v per FC parameter: the optimizer's full-model pass that
 * Appendix "GPU Bottlenecks for Fine-Grained Pipelined Training" names, fused
 * with forward and backward), 2 = the update kernel of conv stages (w, v and
 * every weight-gradient slice read, w, v and the predicted weights written).
 * Negative for other classes.  Benchmarks divide it by the measured duration. */
double pb_kernel_min_bytes(const pb_handle* h, int which);

/* Roofline denominators that a plain HBM copy does not give (measurement aids,
 * no counterpart in the paper).  pb_bench_l2_bandwidth: read + write GB/s of an
 * in-place sweep over `bytes` of device memory repeated `iters` times; with
 * `bytes` well under the L2 capacity this is the L2 bandwidth that bounds the
 * update of networks whose weights and velocities stay cached.
 * pb_bench_fp32_fma: float32 fused-multiply-add rate of the CUDA cores in
 * TFLOP/s (2 flops per FMA), the bound of the float32 convolutions.  Both
 * allocate and free their own scratch and synchronise `stream`. */
int pb_bench_l2_bandwidth(size_t bytes, int iters, void* stream, double* gbs);
int pb_bench_fp32_fma(int iters, void* stream, double* tflops);

/* Allocation-free variant of pb_create + pb_set_weights + pb_run for small fully
 * connected pipelines.  (The paper has no counterpart: this exists for callers
 * that must not allocate device memory - code running inside a pre-sized memory
 * budget, under another framework's caching allocator whose pool must not be
 * disturbed, or in a phase where cudaMalloc's implicit device synchronisation
 * is not acceptable.)
 *
 * Runs n_ticks ticks of PB + SC + LWP on the MLP sizes[0] -> ... ->
 * sizes[n_sizes-1] (ReLU between, softmax cross-entropy last; one stage per FC
 * layer, 1..16 stages), starting from an empty pipeline.  The caller passes
 * every input and output as device memory: dev_w / dev_v are the master
 * weights and velocities (flat, layer-list order, pb_num_params layout; read
 * and updated in place; zero dev_v for a fresh start), dev_xs [n_ticks,
 * sizes[0]], dev_labels [n_ticks], dev_losses [n_ticks] or NULL.  Everything
 * else the tick kernels need (tick state, stage tables, activation rings,
 * gradient hand-off rows) lives in one static 4 MiB device array inside the
 * library, which every GPU that loads the library holds until the process
 * exits.  A network whose scratch exceeds 4 MiB is rejected with PB_E_ARG and a
 * message giving the size.  No cudaMalloc, cudaFree or other allocating device
 * call is made; host-side bookkeeping uses ordinary heap memory.
 *
 * The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress) and should therefore come before any stream capture.
 * That look-up fills a per-device cache without a lock: two threads making the
 * first call on one device at the same moment both store the same address,
 * which is harmless, but the calls themselves must not overlap anyway (below).
 * All calls share the array and it keeps the previous call's contents: each
 * call clears the part it uses, and two calls that overlap on the GPU (other
 * streams, other threads) race on it.  The call waits for `stream` before it
 * returns.  Errors: status code, text via pb_last_error(NULL). */
int pb_mlp_run_static(const int32_t* sizes, int n_sizes, float lr, float momentum, unsigned flags,
                      float* dev_w, float* dev_v, const float* dev_xs, const int32_t* dev_labels,
                      int n_ticks, float* dev_losses, void* stream);

const char* pb_last_error(const pb_handle* h);
void pb_destroy(pb_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* PB_B200_H */
