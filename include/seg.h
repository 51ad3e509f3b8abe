/*
 * seg.h - C ABI of the segment trainer: one independently trained, fully connected
 * network segment with synthetic intermediate labels (SIL), on one NVIDIA B200 (sm_100a).
 *
 * Method: "Partitioned Neural Network Training via Synthetic Intermediate Labels".
 * A network is cut into consecutive segments.  Each cut gets one random target vector
 * per class (Eq. 1); a non-final segment is trained to map its input to the target
 * vector of the sample's class, the final segment is trained on the class labels
 * (Section 2).  Segments never exchange activations or gradients while training
 * (Section 1), so one handle holds everything a segment needs.
 *
 * Conventions
 *   - All tensor arguments are DEVICE pointers unless a comment says "host".
 *   - Matrices are row-major and dense (pitch = number of columns) at this boundary.
 *   - A Linear layer l computes Z = A_prev * W^T + b with W stored [out][in].
 *   - Every call enqueues its work on the stream given at seg_create and returns
 *     without synchronising.  The caller keeps argument buffers alive and unchanged
 *     until the stream has consumed them.
 *   - Argument errors are reported synchronously through the return code and enqueue
 *     nothing.  Device-side problems (a bounded wait that ran out) are recorded in a
 *     status word that seg_poll_status reads.
 *   - Nothing is thrown across this boundary and nothing aborts the process.
 *   - A handle is not thread-safe; different handles may be created and used from
 *     different threads and on different streams concurrently (the library's one-time
 *     set-up and its per-device caches are synchronised).
 *   - A handle lives on the device that was current when seg_create ran.  Later calls may
 *     come with any device current: every call switches to the handle's device for its own
 *     duration and restores the caller's.
 *
 * Diagnostic environment switches, read when a handle is created (first handle of the
 * process for the kernel-selection ones); all default to off / automatic:
 *   SEG_NO_GRAPH=1        launch every kernel eagerly instead of replaying a captured step
 *   SEG_NO_FORK=1         run every branch of a step on one stream
 *   SEG_NO_PDL=1          ordinary launches instead of programmatic dependent launches
 *   SEG_NO_FUSED_LOSS=1   always run the intermediate-label loss as a launch of its own (default: inside
 *                         the last forward product's epilogue where the tensor-core path can take it)
 *   SEG_FUSED_UPDATE=1    apply the optimizer update inside the weight-gradient product where a persistent
 *                         tensor-core kernel runs it (default: a launch of its own, which measured faster)
 *   SEG_NO_SMALL_FUSED=1  run a small fp32 segment (at most 4 layers of at most 128 units, 1024 inputs) launch by launch
 *                         (default: its whole step in two launches, see small_step.cu)
 *   SEG_NO_SPLITK=1       never use the cluster split-K product kernel
 *   SEG_NO_PAIRS=1        never use the CTA-pair product kernel
 *   SEG_NO_STAGED_EPILOGUE=1  persistent product kernels store their output with per-lane stores (default: through
 *                         shared memory and bulk tensor stores)
 *   SEG_PAIR_MIN_TILES=n  use CTA pairs exactly when a product has n or more tiles of 256 x 256
 *                         (default: a cost model of the main loop chooses)
 *   SEG_DEBUG=1           report on stderr when a step could not be captured into a graph
 */
#ifndef SEG_H_
#define SEG_H_

#include <stdint.h>

#if defined(__GNUC__)
#define SEG_API __attribute__((visibility("default")))
#else
#define SEG_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct seg_handle seg_handle; /* opaque, owned by the library */

typedef enum {
  SEG_OK = 0,
  SEG_ERR_INVALID_ARG = 1,    /* null pointer, value out of range                      */
  SEG_ERR_SHAPE = 2,          /* batch > max_batch, layer index out of range, ...      */
  SEG_ERR_UNSUPPORTED = 3,    /* combination the library does not implement            */
  SEG_ERR_ALLOC = 4,          /* device allocation failed                              */
  SEG_ERR_CUDA = 5,           /* a CUDA runtime or driver call failed                  */
  SEG_ERR_STATE = 6,          /* call order: e.g. training on labels never generated   */
  SEG_ERR_DEVICE_TIMEOUT = 7, /* a kernel gave up a bounded wait and returned early    */
  SEG_ERR_NO_DEVICE = 8,      /* no CUDA device / not an sm_100 device                 */
  SEG_ERR_CLASS_RANGE = 9     /* a step met a class index outside [0, M) (clamped there) */
} seg_status;

/* Arithmetic of the matrix products.  Accumulation is always fp32.
 *   SEG_FP32: fp32 operands (FFMA).               x, y are float.
 *   SEG_TF32: fp32 storage, operands rounded to TF32 (nearest even) where they are
 *             stored: weights in a rounded copy, activations and dZ on store.  x, y float.
 *   SEG_BF16: fp32 master weights with a bf16 copy, bf16 activations and dZ.
 *             x and the y of a non-final segment are bf16 (raw 16-bit patterns);
 *             the logits of a final segment are float.                                    */
typedef enum { SEG_FP32 = 0, SEG_TF32 = 1, SEG_BF16 = 2 } seg_precision;

/* Section 3 uses SGD with momentum 0.9; plain SGD and Adam serve the synthetic workloads.
 *   SEG_SGD:          p -= lr * g
 *   SEG_SGD_MOMENTUM: buf = momentum * buf + g;  p -= lr * buf        (buf starts at 0)
 *   SEG_ADAM:         m = b1 m + (1-b1) g;  v = b2 v + (1-b2) g^2;
 *                     p -= lr * (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps),  t = 1, 2, ... */
typedef enum { SEG_SGD = 0, SEG_SGD_MOMENTUM = 1, SEG_ADAM = 2 } seg_optimizer;

/* Distribution of the intermediate labels.
 *   SEG_LABEL_UNIFORM_KAPPA: Eq. 1, SIL_ij ~ kappa * U(0,1) (Section 3 uses kappa = 10).
 *   SEG_LABEL_NORMAL:        N(0,1) targets (the synthetic workloads); kappa is ignored.  */
typedef enum { SEG_LABEL_UNIFORM_KAPPA = 0, SEG_LABEL_NORMAL = 1 } seg_label_dist;

/* Which matrix-product kernels a handle uses. */
typedef enum {
  SEG_GEMM_AUTO = 0,   /* tensor cores for SEG_TF32 / SEG_BF16, FFMA for SEG_FP32 */
  SEG_GEMM_SIMT = 1,   /* FFMA kernels for every precision (same rounding points)  */
  SEG_GEMM_TCGEN05 = 2 /* tensor-core kernels only: SEG_ERR_UNSUPPORTED with SEG_FP32, and from any call
                          whose product the tensor-core path cannot take (no FFMA stand-in) */
} seg_gemm_backend;

typedef struct {
  int32_t n_layers;        /* Linear layers in this segment, 1..16 (Section 3: 2 and 3)   */
  const int32_t* widths;   /* host; n_layers+1 entries: input width, then every layer's
                              output width.  Copied by seg_create.                         */
  int32_t n_classes;       /* M, the number of classes (Section 2)                         */
  int32_t is_final;        /* 0: trained against SIL[class] with mean squared error;
                              1: last segment, softmax cross-entropy on the class labels   */
  int32_t last_relu;       /* ReLU on this segment's last layer: 1 / 0, or -1 for the
                              default (1 if !is_final, 0 if is_final: Section 3 exempts
                              only the network's final layer from ReLU)                    */
  int32_t segment_id;      /* index of the segment / its cut; enters the random streams     */
  int32_t precision;       /* seg_precision                                                */
  int32_t optimizer;       /* seg_optimizer                                                */
  float lr, momentum, beta1, beta2, eps;
  int32_t max_batch;       /* workspaces are sized for this batch                          */
  int32_t gemm_backend;    /* seg_gemm_backend                                             */
  uint64_t init_seed;      /* seed of the weight-initialisation streams                    */
  void* stream;            /* cudaStream_t every call of this handle enqueues on           */
} seg_config;

/* Creates a segment on the current device: allocates parameters, optimizer state,
 * gradient, activation and dZ workspaces (all owned by the handle, freed by
 * seg_destroy) and initialises W, b ~ U(-1/sqrt(fan_in), 1/sqrt(fan_in)) from Philox
 * streams keyed by init_seed (Section 2 refers to the framework's default Linear
 * initialisation).  cfg and out are host pointers.  On failure *out is NULL.             */
SEG_API seg_status seg_create(const seg_config* cfg, seg_handle** out);

/* Generates this segment's intermediate labels on the device (Eq. 1): an [M][N_P] fp32
 * matrix, row j = target vector of class j (the paper's N_P x M matrix stored by
 * columns), N_P = last width.  Element (j, i), flat index e = j*N_P+i, is word e mod 4 of
 * the Philox4x32-10 block with key = (seed lo, seed hi) and counter
 * (e/4 lo, e/4 hi, segment_id, 0); values are bit-reproducible on any device.  Valid for non-final segments only
 * (SEG_ERR_STATE otherwise).                                                              */
SEG_API seg_status seg_gen_labels(seg_handle* h, uint64_t seed, int32_t dist, float kappa);

/* One training step on one batch (Section 2: forward, loss against the intermediate
 * target of each sample's class - or against the class label on the final segment -,
 * backprop inside the segment, optimizer update).
 *   x        [batch][widths[0]]  float (FP32/TF32) or bf16 (BF16)
 *   cls      [batch] int32 class index in [0, M).  An index outside that range is clamped to
 *            it by the step's staging kernel (nothing is read out of bounds) and recorded:
 *            the next seg_poll_status returns SEG_ERR_CLASS_RANGE.
 *   batch    1..max_batch
 *   loss_out device float, receives the batch loss before the update; may be NULL
 *   y_out    optional [batch][widths[n_layers]] copy of this step's forward output
 *            (dtype as for seg_forward); may be NULL
 * No gradient with respect to x is formed.                                                */
SEG_API seg_status seg_train_step(seg_handle* h, const void* x, const int32_t* cls, int32_t batch,
                          float* loss_out, void* y_out);

/* The step of the fully separate variant (Section 2, the flowchart in which middle
 * partitions are trained with intermediate labels both as input and as target): the input
 * of sample b is row cls[b] of sil_in, the [M][widths[0]] fp32 label matrix of the PREVIOUS
 * cut (as seg_get_labels of the previous segment returns it); it is gathered on the device,
 * no per-sample input tensor is materialised.  Everything else as seg_train_step.          */
SEG_API seg_status seg_train_step_label_input(seg_handle* h, const float* sil_in, const int32_t* cls,
                                              int32_t batch, float* loss_out);

/* The same step for callers whose batch lives in HOST memory (x_host, cls_host: host pointers).
 * Page-locked (pinned, mapped) buffers are read by the step's staging kernel directly over the bus;
 * pageable ones are first copied to device buffers the handle owns (allocated at the first such
 * call).  The loss is written by the kernel into a page-locked float of the handle and returned in
 * *loss_host (host float, may be NULL); the call synchronises the stream before returning.       */
SEG_API seg_status seg_train_step_host(seg_handle* h, const void* x_host, const int32_t* cls_host,
                                       int32_t batch, float* loss_host);

/* The host-buffer step without the wait, for training loops that keep the GPU fed: x_host, cls_host
 * and loss_host (may be NULL) must all be page-locked, mapped host memory (SEG_ERR_INVALID_ARG
 * otherwise).  The call enqueues a copy of the batch on a copy stream of the handle (into one of two
 * device buffers, allocated at the first such call, so that the transfer overlaps the steps enqueued
 * before it), enqueues the step behind that copy and returns; the loss kernel writes *loss_host when
 * the step is done.  The caller leaves the batch unchanged, and does not read the loss, until the
 * stream has passed that step (seg_poll_status, or a synchronisation of the handle's stream).      */
SEG_API seg_status seg_train_step_host_async(seg_handle* h, const void* x_host, const int32_t* cls_host,
                                             int32_t batch, float* loss_host);

/* Forward pass only (the response handed to the next segment, Section 2):
 *   y [batch][widths[n_layers]]: float for FP32/TF32 and for the logits of a final
 *   segment, bf16 for a non-final BF16 segment.                                           */
SEG_API seg_status seg_forward(seg_handle* h, const void* x, int32_t batch, void* y);

/* Epoch driver (Section 2, both phases): trains the segment for `epochs` passes over a
 * device-resident data set, in the stored order - the method does not shuffle -, in steps
 * of `batch` samples; a last partial batch is a smaller step (its means run over its own
 * size).  x [n][widths[0]] and cls [n] as for seg_train_step; losses, if not NULL, is a
 * device array that receives the loss of every step, epochs * ceil(n / batch) floats.
 * Equivalent to calling seg_train_step in that order; nothing synchronises.               */
SEG_API seg_status seg_train_epochs(seg_handle* h, const void* x, const int32_t* cls, int64_t n,
                                    int32_t batch, int32_t epochs, float* losses);

/* The stored response of a trained segment over a whole data set (Section 2: the left
 * partition's final response, which is the next partition's input): seg_forward over
 * consecutive chunks of `batch` rows.  y [n][widths[n_layers]], dtype as for seg_forward. */
SEG_API seg_status seg_forward_dataset(seg_handle* h, const void* x, int64_t n, int32_t batch, void* y);

/* Recovery step (Section 5, "recovery epochs"): after both partitions are trained, the
 * left one is trained some more THROUGH the right one, whose weights stay frozen.  Runs
 * left forward, right forward on the left output, softmax cross-entropy on the class
 * labels, backprop through the right segment down to its input (no weight gradient, no
 * update there), then the usual backward pass and optimizer update of the left segment.
 * left must be non-final and right final, widths must chain, precision and stream must be
 * the same (SEG_ERR_STATE / SEG_ERR_SHAPE / SEG_ERR_UNSUPPORTED otherwise).  x, cls, batch,
 * loss_out as for seg_train_step; the loss is the joined network's.  The left segment's
 * intermediate labels are not used.                                                        */
SEG_API seg_status seg_recovery_step(seg_handle* left, seg_handle* right, const void* x,
                                     const int32_t* cls, int32_t batch, float* loss_out);

/* Frees everything the handle owns.  Synchronises the handle's stream first.             */
SEG_API seg_status seg_destroy(seg_handle* h);

/* ---- auxiliary calls: inspection, injection, accounting ------------------------------ */

/* Copies the [M][N_P] fp32 label matrix to / from a device buffer. */
SEG_API seg_status seg_get_labels(seg_handle* h, float* dst);
SEG_API seg_status seg_set_labels(seg_handle* h, const float* src);

/* fp32 master parameters of layer `layer` (0-based): W [out][in], b [out]; either
 * pointer may be NULL.  seg_set_params also refreshes the reduced-precision copy.        */
SEG_API seg_status seg_get_params(seg_handle* h, int32_t layer, float* W, float* b);
SEG_API seg_status seg_set_params(seg_handle* h, int32_t layer, const float* W, const float* b);

/* Gradients of the last seg_train_step: dW [out][in], db [out], fp32. */
SEG_API seg_status seg_get_grads(seg_handle* h, int32_t layer, float* dW, float* db);

/* Optimizer state of layer `layer`: which = 0 momentum buffer / Adam first moment,
 * which = 1 Adam second moment; shapes as the parameters.                                */
SEG_API seg_status seg_get_opt_state(seg_handle* h, int32_t layer, int32_t which, float* sW, float* sb);
SEG_API seg_status seg_set_opt_state(seg_handle* h, int32_t layer, int32_t which, const float* sW,
                                     const float* sb);

/* Number of optimizer steps taken (the t of Adam's bias correction); host pointer.  Setting it
 * together with parameters and optimizer state resumes a saved segment.                     */
SEG_API seg_status seg_get_step(const seg_handle* h, uint64_t* step);
SEG_API seg_status seg_set_step(seg_handle* h, uint64_t step);

/* Stored output A_layer of the last step, layer = 1..n_layers, converted to fp32
 * [batch][widths[layer]] for the batch size of that step.                                */
SEG_API seg_status seg_get_activation(seg_handle* h, int32_t layer, float* dst);

/* Bytes of device memory the handle holds now and at its peak. host pointers. */
SEG_API seg_status seg_mem_bytes(const seg_handle* h, uint64_t* current, uint64_t* peak);

/* Number of kernels the handle has launched so far (host counter). */
SEG_API seg_status seg_launch_count(const seg_handle* h, uint64_t* launches);

/* Matrix-product launches of this handle so far, by kernel family (host counters; counts[5], host):
 *   [0] tensor-core, one CTA per tile      [1] tensor-core, K split over a cluster
 *   [2] tensor-core, CTA pair per tile     [3] FFMA
 *   [4] of [0] and [2]: weight-gradient products that also applied the optimizer update
 * The two launches of a small fp32 segment's step (kinds 7 and 4 of seg_profile_get) count as two FFMA
 * launches and one of [4].  Tests use it to show which kernels actually ran.                                           */
SEG_API seg_status seg_product_launches(const seg_handle* h, uint64_t* counts);

/* Synchronises the handle's stream and returns SEG_ERR_DEVICE_TIMEOUT if any kernel of
 * this handle gave up a bounded wait since the last poll, SEG_ERR_CLASS_RANGE if a step met
 * a class index outside [0, M), SEG_ERR_CUDA on a CUDA error.  The record is cleared.       */
SEG_API seg_status seg_poll_status(seg_handle* h);

/* Self-test of the bounded wait every product kernel uses: launches one small block that waits,
 * with the product kernels' own wait routine, on a barrier nothing ever arrives at, for at most
 * limit_ns nanoseconds (1,000 .. 1,000,000,000; SEG_ERR_INVALID_ARG otherwise).  The wait runs
 * out, the block records it in the handle's status word and returns; the next seg_poll_status
 * reports SEG_ERR_DEVICE_TIMEOUT and the handle stays usable.  Nothing faults or hangs.        */
SEG_API seg_status seg_selftest_bounded_wait(seg_handle* h, uint64_t limit_ns);

/* Hand-off between segments that live on different devices (Section 2.1: each partition trains on
 * its own GPU and the only transfer is the previous partition's stored response, once).  Copies
 * `bytes` bytes from src, device memory on the producer's device (typically the y of
 * seg_forward_dataset), into dst, device memory on the consumer's device, as one peer copy
 * enqueued on the producer's stream; the consumer's stream then waits for it, so that a following
 * seg_train_epochs(consumer, dst, ...) reads the data from its own GPU's memory.  No kernel of
 * either handle ever reads the other device's memory.  Both handles on one device: an ordinary
 * device-to-device copy.                                                                         */
SEG_API seg_status seg_handoff_copy(seg_handle* producer, const void* src, seg_handle* consumer,
                                    void* dst, uint64_t bytes);

/* Index of the device the handle lives on (host int out). */
SEG_API seg_status seg_device(const seg_handle* h, int32_t* device);

/* Timing hooks: seg_timer_start / seg_timer_stop record CUDA events on the handle's
 * stream; seg_timer_elapsed_ms synchronises on the stop event (host float out).          */
SEG_API seg_status seg_timer_start(seg_handle* h);
SEG_API seg_status seg_timer_stop(seg_handle* h);
SEG_API seg_status seg_timer_elapsed_ms(seg_handle* h, float* ms);

/* Per-kernel timing (off by default).  While enabled, every launch of this handle is
 * bracketed by CUDA events on the handle's stream.  seg_profile_get synchronises and
 * returns, for one kernel kind, the number of launches and their summed device time
 * since profiling was enabled; kinds: 0 forward product, 1 dgrad product, 2 wgrad
 * product, 3 loss, 4 wgrad product that also applies the optimizer update to the weights,
 * 5 optimizer update as a launch of its own (forms the bias gradient too; after a kind-4
 * product it has only the bias left), 6 copies / staging, 7 the first launch of a small
 * fp32 segment's two-launch step (staging, forward, loss and dgrad chain; its second launch,
 * all weight and bias gradients with the update, counts as kind 4).  count and
 * total_ms are host pointers.                                                            */
SEG_API seg_status seg_profile_enable(seg_handle* h, int32_t on);
SEG_API seg_status seg_profile_get(seg_handle* h, int32_t kind, uint64_t* count, float* total_ms);

/* The intermediate-label loss without any allocation (the paper has no counterpart: this
 * entry point exists for the callers described below, not for the method).
 *
 * Some callers cannot allocate device memory: a plug-in running inside another program's
 * fixed memory budget, a latency-bound loop where the device synchronisation that
 * cudaMalloc implies is not acceptable, code that is given a stream and buffers but no
 * allocator.  For them this call computes what a non-final segment's loss kernel computes -
 *     loss = mean_{b,i} (out[b][i] - sil[cls[b]][i])^2,
 *     dz[b][i] = 2 (out[b][i] - sil[cls[b]][i]) / (batch * n_p) * (relu_mask ? out[b][i] > 0 : 1)
 * - without a handle and without calling cudaMalloc, cudaFree or any allocating routine.
 * The reduction scratch is a static device array of 8 KiB inside the library, present on
 * every GPU that loads the library until the process exits.
 *   out [batch][n_p] float, cls [batch] int32 in [0, n_classes) (an index outside that range is
 *   clamped to it; nothing is read out of bounds), sil [n_classes][n_p] float,
 *   dz [batch][n_p] float (written), loss_out device float (written; may be NULL),
 *   stream: cudaStream_t.  All device pointers, dense row-major, caller-owned.
 * Limits: n_p <= SEG_NOALLOC_MAX_WIDTH, batch <= SEG_NOALLOC_MAX_BATCH; anything larger
 * returns SEG_ERR_SHAPE and enqueues nothing.
 * The first call on a device looks up the array's device address (once per device, with
 * that device current); make that first call before starting any stream capture.
 * Every call on a device shares the one array: calls whose kernels may overlap on the GPU
 * (different streams, no dependency between them) race on it and give wrong losses; order
 * them on one stream or with events.  Nothing needs clearing by the caller.               */
#define SEG_NOALLOC_MAX_WIDTH 65536
#define SEG_NOALLOC_MAX_BATCH 65536
SEG_API seg_status seg_label_loss_noalloc(const float* out, const int32_t* cls, const float* sil,
                                          int32_t n_classes, int32_t n_p, int32_t batch,
                                          int32_t relu_mask, float* dz, float* loss_out, void* stream);

SEG_API const char* seg_status_string(int32_t s);

/* Text of the last CUDA error seen by this handle ("" if none); valid until the next call. */
SEG_API const char* seg_last_error(const seg_handle* h);

/* Static description of the build: "sm_100a ..." */
SEG_API const char* seg_build_info(void);

#ifdef __cplusplus
}
#endif
#endif /* SEG_H_ */
