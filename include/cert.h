/*
 * cert.h - C ABI of the B200 DeepPoly back-substitution library.
 *
 * The calls follow the paper's problem statement (Section 2, "DNN
 * Certification"): a ReLU network, a set of input regions given as concrete
 * per-neuron bounds, and an abstract shape (here the concrete bounds l, u)
 * out for every neuron, computed by the DeepPoly certifier (Appendix C,
 * DeepPoly listing): polyhedral back-substitution at every affine layer
 * (traverse + replace_lower/upper), concretisation against the input box
 * (map(simplify_lower/upper)), and the ReLU relaxation chosen from the
 * resulting bounds (Relu transformer: relu_n, compute_upper).
 *
 * All compute runs in CUDA kernels for sm_100a on the current device; there
 * is no CPU fallback.  No function throws, aborts or traps: every failure is
 * a return code.
 */
#ifndef CERT_H_
#define CERT_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cert_net cert_net_t; /* opaque; owns device copies of the weights and a workspace */

typedef enum {
    CERT_OK = 0,
    CERT_ERR_INVALID_ARG = 1,     /* null pointer, bad size, non-finite eps, layer chain mismatch */
    CERT_ERR_UNSUPPORTED = 2,     /* a geometry the kernels do not cover                         */
    CERT_ERR_OOM = 3,             /* device or host allocation failed                            */
    CERT_ERR_BATCH_TOO_LARGE = 4, /* batch > max_batch given at create                           */
    CERT_ERR_CUDA = 5,            /* a CUDA runtime or driver call failed                        */
    CERT_ERR_TIMEOUT = 6,         /* a bounded device-side wait ran out (see cert_net_last_status) */
    CERT_ERR_RANGE = 7,           /* a coefficient left the fp16 range of CERT_CONTRACTION_TC3XFP16  */
    CERT_ERR_BOUNDS = 8           /* checking build only: a kernel tried to store outside every buffer */
} cert_status_t;

enum { CERT_LAYER_FC = 0, CERT_LAYER_CONV2D = 1 };

/*
 * One affine layer of the network, optionally followed by a ReLU layer
 * (the paper treats Affine and Relu as separate layers; relu_after = 1 means
 * a Relu layer sits on top of this affine layer).
 *   FC:     z = W a + b, weight[out_features][in_features] row-major.
 *   CONV2D: cross-correlation with zero padding on an input of shape
 *           (c_in, h_in, w_in), weight[c_out][c_in][kh][kw], one bias per
 *           output channel, output size floor((in + 2*pad - k)/stride) + 1;
 *           neurons are flattened (channel, row, column) row-major.
 * weight and bias are HOST pointers to float32; they are copied during
 * cert_net_create and may be freed afterwards.
 */
typedef struct {
    int kind;       /* CERT_LAYER_FC or CERT_LAYER_CONV2D */
    int relu_after; /* 0 or 1 */
    int in_features, out_features;                    /* FC only   */
    int c_in, h_in, w_in, c_out, kh, kw, stride, pad; /* CONV only */
    const float *weight;
    const float *bias;
} cert_layer_desc_t;

/*
 * Builds a network object on the current CUDA device: validates the
 * descriptors, uploads the weights (and the operand forms the contraction
 * kernels want), and allocates a workspace large enough for max_batch boxes.
 * Input boxes are intersected with [clip_lo, clip_hi] (pass -INFINITY and
 * INFINITY for no clipping).  On success *out receives the handle, which the
 * caller releases with cert_net_destroy.  Synchronous.
 */
cert_status_t cert_net_create(const cert_layer_desc_t *layers, int n_layers, int max_batch,
                              float clip_lo, float clip_hi, cert_net_t **out);

/*
 * The same for a network with residual connections (the paper's benchmark table lists one, "Skip";
 * Appendix, table of DNNs).  skip_from is a HOST array of n_layers ints (or NULL for none):
 * skip_from[k] = s >= 0 makes layer k compute W_k a_{k-1} + b_k + a_s, a_s being the outputs of layer s
 * (after its ReLU, if it has one); -1 = no connection into layer k.  Under the DeepPoly listing
 * (Appendix C) such a neuron is an Affine neuron whose prev holds neurons of two layers, and the
 * traversal, which replaces the neurons of the highest layer first (priority -layer), lets the
 * coefficient on a_s wait until the rest of the expression has come down to layer s; that is what the
 * library does: the waiting coefficient matrix stays in a third workspace buffer and is added in the
 * epilogue of the step that reaches layer s, before the ReLU back-step.
 * Requirements (else CERT_ERR_INVALID_ARG): s <= k-2; layers s and k have the same number of neurons;
 * connections follow one another (none starts before the previous one has ended).
 * Such a net is bounded with one launch per back-step and dense coefficient maps (patches and
 * cert_net_enable_reusecert are refused; the banded tensor-core form of conv steps is used on full
 * traversals when every connection ends on a conv layer that takes it and whose map has the shape of its
 * source's).  cert_backsub_bounds works as for other nets: a traversal that
 * stops on a connection's source joins the waiting coefficients before it is simplified, one that stops
 * above it simplifies them against the source's own concrete bounds (map(simplify_*) treats every neuron left
 * in the expression alike).  CERT_CONTRACTION_TC3XFP16 is available for FC nets, for full traversals only
 * (depths that stop early return CERT_ERR_UNSUPPORTED in that mode).
 */
cert_status_t cert_net_create_residual(const cert_layer_desc_t *layers, int n_layers, const int *skip_from,
                                       int max_batch, float clip_lo, float clip_hi, cert_net_t **out);

/*
 * DeepPoly bounds of every affine neuron for `batch` L-infinity boxes.
 *   centers  DEVICE float32 [batch][n0]; box b is
 *            [max(c - eps, clip_lo), min(c + eps, clip_hi)] per coordinate,
 *            with c -/+ eps rounded to float32.
 *   lb_out, ub_out  DEVICE float32 [batch][n_total], n_total =
 *            cert_net_num_neurons(): the pre-activation neurons of affine
 *            layer 1, 2, ... K concatenated in order.  (The bounds of a Relu
 *            layer's neurons are max(l,0), max(u,0) of the layer below and
 *            are not stored.)
 *   stream   a cudaStream_t (NULL = the default stream).
 * The work is enqueued on `stream` and the call returns without waiting; it
 * allocates nothing.  Calls on the same net must not overlap on the device
 * (they share the workspace).  Caller owns centers, lb_out and ub_out.
 */
cert_status_t cert_deeppoly_bounds(cert_net_t *net, const float *centers, float eps, int batch,
                                   float *lb_out, float *ub_out, void *stream);

/*
 * The same flow with a bounded traversal (Section 6.2, DeepPoly_p: "at each
 * Affine layer, the backsubstitution is performed for p iterations"; one
 * iteration = one affine layer together with the Relu layer on top of it).
 *   backsteps  HOST int [n_layers] or NULL.  backsteps[k] >= 0: the expressions
 *            of affine layer k (0-based) are back-substituted through at most
 *            that many layers and then simplified (map(simplify_lower/upper))
 *            against the concrete bounds of the neurons reached: relu(l),
 *            relu(u) of that layer's neurons under a ReLU, else l, u, or the
 *            input box.  Negative, or NULL: to the input (DeepPoly).
 * Certifiers of Appendix C that differ from DeepPoly only in this respect:
 *   IBP listing        backsteps = {0, 0, ..., 0}
 *   CROWN-IBP listing  backsteps = {0, ..., 0, -1}   (curr[last_layer] == 1 -> backsubs_*)
 * The Relu transformer (relaxation from the resulting bounds) is the same in
 * all of them.  Everything else is as for cert_deeppoly_bounds, which is this
 * call with backsteps = NULL.  The array is read before the call returns.
 */
cert_status_t cert_backsub_bounds(cert_net_t *net, const float *centers, float eps, int batch,
                                  const int *backsteps, float *lb_out, float *ub_out, void *stream);

/*
 * ReuseCert (Appendix C, ReuseCert listing; Section 6.1): every neuron's polyhedral bounds are kept
 * over the input layer and reused (stop_traverse(n) = n[layer] <= 1), so each affine layer costs one
 * contraction instead of a traversal through all earlier layers; the bounds are sound but can be
 * looser than DeepPoly's from the third affine layer on.
 *   cert_net_enable_reusecert  allocates what the certifier needs on top of the net (the shapes of one
 *            layer for max_batch boxes, three times; block weight matrices): call it once, outside the
 *            hot path, with the net's device current.  FC layers only, and only where the fp16-split
 *            contraction is available (CERT_ERR_UNSUPPORTED otherwise): every layer's shapes are built
 *            from the rounded shapes of the layer below, so rounding compounds with depth, and of the
 *            two tensor-core forms only the fp16 split holds 1e-4 * (1 + |bound|) on the 6 x 1024 net.
 *   cert_reusecert_bounds      arguments, outputs (l, u of every affine layer as the Relu transformer
 *            computes them: L.map(simplify_lower), U.map(simplify_upper)), branch codes and stream
 *            behaviour as cert_deeppoly_bounds; allocates nothing.  Runs in the fp16 split whatever
 *            CERT_CONTRACTION_AUTO resolves to; a net set to FFMA or TC3XTF32 is refused
 *            (CERT_ERR_UNSUPPORTED).  A shape entry beyond the fp16 range raises CERT_ERR_RANGE in the
 *            status word (cert_net_last_status; the *_host call returns it).
 */
cert_status_t cert_net_enable_reusecert(cert_net_t *net);
cert_status_t cert_reusecert_bounds(cert_net_t *net, const float *centers, float eps, int batch,
                                    float *lb_out, float *ub_out, void *stream);
/* The same with HOST buffers, as cert_deeppoly_bounds_host. */
cert_status_t cert_reusecert_bounds_host(cert_net_t *net, const float *centers_host, float eps, int batch,
                                         float *lb_host, float *ub_host, void *stream);

/* Same, with HOST buffers (pageable or pinned): copies centers to the device,
 * runs cert_deeppoly_bounds, copies the bounds back and waits for the stream.
 * Because it waits anyway it also reads the device-side status word: it
 * returns CERT_ERR_TIMEOUT / CERT_ERR_RANGE (and clears the word) instead of
 * handing back bounds that a run-out wait or an fp16 overflow invalidated;
 * under CERT_CONTRACTION_AUTO an overflow re-runs the call with the TF32 split
 * first.  The three *_host calls all do this. */
cert_status_t cert_deeppoly_bounds_host(cert_net_t *net, const float *centers_host, float eps,
                                        int batch, float *lb_host, float *ub_host, void *stream);

/* cert_backsub_bounds with HOST buffers, in the same way. */
cert_status_t cert_backsub_bounds_host(cert_net_t *net, const float *centers_host, float eps, int batch,
                                       const int *backsteps, float *lb_host, float *ub_host, void *stream);

/* Frees the device and host memory of the net.  Synchronises the device. */
cert_status_t cert_net_destroy(cert_net_t *net);

/* ---- helpers (not part of the paper's problem statement) ---- */

/* n_total: number of affine neurons, summed over layers; -1 for a null net. */
int cert_net_num_neurons(const cert_net_t *net);
/* Number of neurons of affine layers that have a ReLU on top; -1 for null. */
int cert_net_num_relu_neurons(const cert_net_t *net);

/*
 * Relaxation branch of every ReLU neuron in the most recent
 * cert_deeppoly_bounds call (Relu transformer of the DeepPoly listing):
 *   0 stable inactive (u <= 0), 1 stable active (l >= 0),
 *   2 unstable with lower slope 0 (l + u < 0), 3 unstable with lower slope 1.
 * codes_out: DEVICE uint8 [batch][n_relu], ReLU layers concatenated in
 * order; copied on `stream`.
 */
cert_status_t cert_net_branch_codes(cert_net_t *net, unsigned char *codes_out, void *stream);

/*
 * Sticky device-side status.  Waits `stream`, then returns CERT_ERR_TIMEOUT
 * if any kernel of an earlier call on this net gave up a bounded wait,
 * CERT_ERR_RANGE if a coefficient left the fp16 range in TC3XFP16 mode (the
 * results are invalid in both cases), CERT_ERR_BOUNDS if a checked store was
 * refused (checking build, see cert_net_selftest_checked_store), CERT_ERR_CUDA
 * if the stream reports an error, else CERT_OK.  Clears the flag.
 */
cert_status_t cert_net_last_status(cert_net_t *net, void *stream);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  Every device-side wait of the tensor-core
 * kernels (on an mbarrier a TMA copy, an MMA commit or another warp completes) gives up after about a second,
 * raises the net's status word and lets the kernel end normally, so that a lost signal costs a result, not the
 * context.  This call enqueues, on `stream`, one tiny kernel that runs the same wait with a limit of about
 * 0.1 ms on a barrier nothing ever arrives on; afterwards cert_net_last_status returns CERT_ERR_TIMEOUT (and
 * clears the flag), and the net works as before.  Nothing faults, traps or hangs.
 */
cert_status_t cert_net_selftest_bounded_wait(cert_net_t *net, void *stream);

/*
 * Which kernel carries the affine back-step C' = C * W (Section 4.3, Matmul
 * rewrite).  AUTO picks the tensor-core path where the shape allows it.
 *   FFMA:    fp32 FMA units, unfused ReLU step and concretisation kernels.
 *   TC3XTF32: tcgen05 tensor cores with a 3-term TF32 split (fp32-accurate),
 *            ReLU back-step and concretisation fused into the epilogue.
 *   TC3XFP16: the same kernel structure with an fp16 split (x = hi + lo, three fp16
 *            products per multiply-add, exact in the fp32 accumulators): the accuracy of TC3XTF32 at
 *            twice the tensor-core rate and half the operand bytes, for nets of FC layers only and
 *            coefficients below 65504 in magnitude (beyond that cert_net_last_status reports
 *            CERT_ERR_RANGE and the results are invalid; values under 6.1e-5 are held to 1.5e-11
 *            absolute instead of 2^-22 relative).  The coefficients of a traversal travel times a power
 *            of two, 2^a, so that their lo parts are ordinary fp16 numbers and all three products of a
 *            k-block come from one staging of its tiles; the range is then |coefficient| 2^a < 65504:
 *            a = what the layer's proved bound (see AUTO) leaves, at most 14; 4 for a layer that AUTO
 *            runs on trial; 0 (the whole range) for a layer without a proof when this mode is forced.
 *   AUTO:    decided per affine layer k at create.  TC3XFP16 for the traversal of layer k when the net's
 *            weights prove that none of its coefficients can leave that range on any input: a ReLU
 *            back-step scales a coefficient by a slope in [0, 1], so every entry of the traversal's matrix
 *            over layer j-1 is bounded by the matching entry of |W_k| |W_k-1| ... |W_j|, and the largest
 *            entry of those products over j (cert_net_fp16_coefficient_bound) must stay under 60000.  The
 *            products grow with depth, so on deep nets the proof fails for the last layers although their
 *            real coefficients are small.  Such a layer runs in the fp16 split on trial: its kernels report
 *            to a status word of the layer's own, and the same traversal in TC3XTF32 is enqueued right behind
 *            it with kernels that do nothing unless that word came up (an overflow or a run-out wait), in
 *            which case they recompute the layer; either way the call's bounds are valid and the net's
 *            status word is untouched.  FC nets only (with residual connections no layer has a proof, and
 *            every full traversal runs on trial); nets with conv layers run in TC3XTF32, or FFMA where the
 *            tensor-core path is unavailable.  (Environment variables read at create:
 *            CERT_AUTO_FP16=0 keeps AUTO on TC3XTF32, CERT_SPECULATE_FP16=0 runs unproven layers in
 *            TC3XTF32 outright.)
 * Conv back-steps have the same fusions; under FFMA they run on the FMA units, otherwise on the TF32 tensor-core
 * kernel where their geometry allows (see cert_net_set_conv_patches).
 * (The kernels of a call are chained with programmatic dependent launch, so that a kernel's launch and set-up
 * overlap the tail of the one before; the environment variable CERT_PDL=0, read once per process, turns
 * that off.)
 * (The environment variable CERT_TC_CTAS=1, read at create, keeps the
 * tensor-core kernel to one CTA per row panel instead of CTA pairs.)
 */
enum { CERT_CONTRACTION_AUTO = 0, CERT_CONTRACTION_FFMA = 1, CERT_CONTRACTION_TC3XTF32 = 2,
       CERT_CONTRACTION_TC3XFP16 = 3 };
cert_status_t cert_net_set_contraction(cert_net_t *net, int mode);
/* What CERT_CONTRACTION_AUTO stands for on this net: CERT_CONTRACTION_TC3XFP16 if at least one layer's
 * traversal passes the range proof, else CERT_CONTRACTION_TC3XTF32 or CERT_CONTRACTION_FFMA; -1 for a null net. */
int cert_net_auto_contraction(const cert_net_t *net);
/* Largest entry of the products |W_k| ... |W_j|, j = k-1 .. 1, for affine layer k = `layer` (0-based; see AUTO
 * above), or over all layers for layer < 0; INFINITY where no proof was attempted; -1 for bad arguments. */
float cert_net_fp16_coefficient_bound(const cert_net_t *net, int layer);
/* Which contraction kernels the most recent call ran: bit 0 = FFMA, bit 1 = TC3XTF32,
 * bit 2 = the TC3XTF32 kernel ran in its CTA-pair form (tcgen05 cta_group::2), bit 3 = a traversal ran on
 * receptive-field patches, bit 4 = TC3XFP16, bit 5 = TC3XFP16 with a whole traversal per launch (nets whose
 * hidden layers are at most 256 neurons wide keep the coefficient panel in shared memory from the start of
 * a traversal to its concretisation; the environment variable CERT_CHAIN=0, read at create, keeps such nets
 * on one launch per back-step), bit 6 = a conv back-step on dense coefficient maps ran in its banded
 * tensor-core form (the environment variable CERT_CONV_BANDS=0, read at create, keeps those steps on the
 * FMA units), bit 7 = AUTO ran a layer in the fp16 split on trial and enqueued its predicated TC3XTF32 re-run
 * (bits 1 and 2 are then set as well, whether or not the re-run had to do anything). */
int cert_net_last_contraction_paths(const cert_net_t *net);

/*
 * Conv-sourced rows as patches (on by default).  The expressions of a conv layer's neurons over conv
 * layers below are zero outside a receptive-field window (Section 5 keeps such rows as convolution /
 * patches blocks); while the traversal stays in conv layers and the window is at most half the map,
 * the rows travel as [channels][window] patches instead of dense coefficient maps.  Off: every
 * back-step works on dense maps.  The bounds are the same up to summation order.
 * cert_net_last_contraction_paths sets bit 3 when a traversal of the last call ran on patches.
 * Unless the contraction mode is CERT_CONTRACTION_FFMA, both kinds of conv back-step run on the tensor
 * cores where their geometry allows: a patch step as a contraction with the conv layer's dense
 * window-to-window matrix (bit 1 beside bit 3), a step on dense maps band by band with the maps held
 * [row][channel][column] (bit 6; needs channels x width a multiple of 32 floats on both sides of the layer
 * and of every conv layer below it).  Other geometries use the FMA kernels.
 */
cert_status_t cert_net_set_conv_patches(cert_net_t *net, int on);

/*
 * Per-kernel-class device times.  With profiling on, cert_deeppoly_bounds
 * records a CUDA event on `stream` after every launch (the events are created
 * by cert_net_set_profiling, not in the hot call).  cert_net_profile waits for
 * the most recent call and returns, per class, the summed time in ms between
 * consecutive events and the number of launches.  Classes follow the steps of
 * the DeepPoly listing: building the box and the first layer's bounds, the
 * Relu transformer, replace_* through a ReLU layer (and the start of a
 * traversal), replace_* through an FC layer, through a conv layer, and
 * map(simplify_*).  Kernels that fuse steps count under the contraction.
 */
enum { CERT_CLASS_INPUT = 0, CERT_CLASS_RELAX = 1, CERT_CLASS_RELU_STEP = 2, CERT_CLASS_AFFINE = 3,
       CERT_CLASS_CONV = 4, CERT_CLASS_CONCRETIZE = 5, CERT_N_CLASSES = 6 };
cert_status_t cert_net_set_profiling(cert_net_t *net, int on);
cert_status_t cert_net_profile(cert_net_t *net, float *ms_out /* HOST [CERT_N_CLASSES] */,
                               int *launches_out /* HOST [CERT_N_CLASSES] */);

/*
 * Guard words (no counterpart in the paper; memory-safety evidence).  Every device buffer the net owns
 * (weights, coefficient matrices, row constants, relaxation and bound arrays, gathered windows, ...) is
 * allocated with 256 guard bytes before and after it, filled with a fixed pattern at create.  This call
 * waits for `stream` and reads all of them back: 0 = intact, i + 1 = the guard of the i-th allocation was
 * overwritten (a kernel wrote outside its buffer), -1 = null net or a CUDA error.  Test and debugging aid.
 */
int cert_net_check_guards(cert_net_t *net, void *stream);

/*
 * Checked stores (no counterpart in the paper; memory-safety evidence beside the guard words).  A library built
 * with -DCERT_BOUNDS (paper_2507_20055_b200/build.py: build(defines=["CERT_BOUNDS"], lib=...)) looks up the
 * address of every plain global store of its non-TMA kernels in a table of the buffers the call may write (the
 * net's allocations, the caller's lb_out / ub_out); a store outside all of them is skipped and reported as
 * CERT_ERR_BOUNDS by cert_net_last_status.  Slow; for tests on small shapes.
 *   cert_built_with_checked_stores   1 in such a build, else 0.
 *   cert_net_selftest_checked_store  enqueues one kernel that attempts a checked store one float past the end of
 *            one of the net's buffers: the store is skipped (the guard words stay intact) and the next
 *            cert_net_last_status returns CERT_ERR_BOUNDS.  CERT_ERR_UNSUPPORTED in an ordinary build.
 */
int cert_built_with_checked_stores(void);
cert_status_t cert_net_selftest_checked_store(cert_net_t *net, void *stream);

/* Number of kernels the most recent cert_deeppoly_bounds call enqueued. */
int cert_net_last_launch_count(const cert_net_t *net);

/* Floating-point operations of the affine/conv back-steps of one call for
 * `batch` boxes (2 per multiply-add, both bound sides, dense coefficient
 * maps), as the benchmark's roofline numerator. */
double cert_net_backstep_flops(const cert_net_t *net, int batch);

/*
 * (No counterpart in the paper: an addition for embedders.)
 *
 * Interval bounds of a single FC layer over `batch` L-infinity boxes, the
 * same numbers cert_deeppoly_bounds returns for a one-layer net, without any
 * allocation.  It is meant for callers that are not allowed to obtain device
 * memory themselves: code that runs under another framework's memory pool and
 * must not go around it, services whose memory budget is fixed at start-up,
 * and latency-sensitive loops where the implicit synchronisation of
 * cudaMalloc / cudaFree is not acceptable.  Neither this call nor anything it
 * uses calls cudaMalloc, cudaFree or an allocating library routine.
 *
 *   weight   DEVICE float32 [out_features][in_features] row-major (unpadded)
 *   bias     DEVICE float32 [out_features]
 *   centers  DEVICE float32 [batch][in_features]
 *   lb_out, ub_out  DEVICE float32 [batch][out_features]
 * The caller owns all five.  The box endpoints, which the regular path keeps
 * in the net's workspace, are held in a fixed 8 MiB array that is part of the
 * library image (every GPU that loads the library carries it until the
 * process ends).  Limit: batch * round_up(in_features, 32) <= 1048576;
 * beyond it the call returns CERT_ERR_BATCH_TOO_LARGE and does nothing.
 * (batch * out_features beyond 8 * (2^31 - 1), more than one launch can
 * cover, returns CERT_ERR_UNSUPPORTED.)
 *
 * The first call on each device looks up the array's device address (a
 * synchronous runtime query made with that device current); make that first
 * call before starting any stream capture.  All calls on a device share the
 * one array: a call overwrites every element it later reads, so nothing
 * needs clearing between calls, but two calls whose kernels overlap on the
 * GPU (different streams, no ordering between them) race on it.  Work is
 * enqueued on `stream`; the call does not wait for it.
 */
cert_status_t cert_first_layer_bounds_noalloc(const float *weight, const float *bias, int out_features,
                                              int in_features, const float *centers, float eps,
                                              float clip_lo, float clip_hi, int batch, float *lb_out,
                                              float *ub_out, void *stream);

/*
 * (No counterpart in the paper: measurement support for the benchmark's roofline.)
 *
 * Measures, on the current device, the peak rate of the unit a contraction kernel of this library runs on, with
 * a micro-kernel that does nothing else:
 *   kind 0  tcgen05.mma kind::f16,  CTA pairs, 256 x 256 tiles, both operands resident in shared memory
 *   kind 1  tcgen05.mma kind::tf32, the same shape
 *   kind 2  fp32 fused multiply-adds in registers (one 1024-thread block per multiprocessor)
 *   kind 3  bulk copies from L2 into shared memory: one block per multiprocessor keeps eight 16 KB copies in flight
 *           from a 512 KB region of its own (74 MB in all, resident in L2) and nothing reads what lands; this is the
 *           path the operand tiles of the tensor-core contractions travel.  tflops_out then receives TERABYTES per
 *           second over all multiprocessors (divide by their number and by sm_mhz_out for bytes per cycle and SM);
 *           the call allocates and frees that buffer too
 * The kernel is sized by a short calibration run to last about target_ms (0 < target_ms <= 2000); a few ms give
 * a burst figure at boost clocks, a few hundred ms a figure under the power limit.  Outputs (HOST pointers):
 * tflops_out = executed flops / CUDA-event time (2 per multiply-add), sm_mhz_out (may be NULL) = SM cycles per
 * microsecond as the kernel itself saw them, ms_out (may be NULL) = the kernel's duration.  Allocates a few
 * words of device memory and frees them; synchronises `stream`.  Every device-side wait is bounded
 * (CERT_ERR_TIMEOUT if one runs out).
 */
cert_status_t cert_peak_microbench(int kind, double target_ms, double *tflops_out, double *sm_mhz_out,
                                   double *ms_out, void *stream);

const char *cert_status_string(cert_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* CERT_H_ */
