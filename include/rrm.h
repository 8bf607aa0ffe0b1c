/*
 * rrm.h - C ABI of the B200 (sm_100a) Recurrent Residual Module library.
 *
 * The Recurrent Residual Module (RRM) runs a CNN on video by keeping, for every linear
 * layer l, the previous frame's input I_{t-1,l} and projection P_{t-1,l} = F_l*I_{t-1,l} + b_l,
 * and evaluating each new frame as  P_{t,l} = P_{t-1,l} + F_l * (I_{t,l} - I_{t-1,l}),
 * I_{t,l+1} = f(P_{t,l})  (Eq. 4-5, Algorithm 1).  Only the non-zero part of the input
 * delta is visited (Sec. 3.5), so the cost follows the delta density (Table 1) while the
 * result equals a dense recompute of the frame.
 *
 * Conventions
 *   - Every function returns an int status (RRM_OK or a negative RRM_ERR_*), never throws,
 *     never aborts.  Nothing synchronises the stream unless stated.
 *   - "dev" pointers are device pointers on the current CUDA device, "host" pointers are
 *     host memory.  `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - Activation layouts at this boundary, N = number of independent video streams:
 *       RRM_F32 : float   [N][C][H][W]
 *       RRM_I8  : int8_t  [N][C][H][W]     (values in [-127,127]; layer inputs in [0,127]
 *                                           or any range whose frame-to-frame delta fits int8)
 *       RRM_BIN : uint32_t[N][H][W][ceil(C/32)]  bit i of word k = channel 32k+i, 1 = +1, 0 = -1,
 *                                           unused high bits zero
 *       raw int32 projections: int32_t [N][C][H][W]
 *     Filters: [C_out][C_in][kh][kw] row-major; float for RRM_F32, int8_t for RRM_I8 and
 *     RRM_BIN (+1 / -1).  Bias: float (RRM_F32) or int32_t.  Weights and bias are copied and
 *     repacked into library-owned device memory at create time; the caller may free its copy.
 *   - One object may be used from one stream at a time.
 *   - Environment switches, read when an object is created (debugging aids): RRM_NO_GRAPH=1 launches every
 *     kernel of a stack step on its own instead of replaying a captured CUDA graph; RRM_DEBUG=1 names a failing
 *     CUDA call (file, line, error string) on stderr and prints the shape of captured chunk graphs; RRM_PDL=1
 *     launches the kernels of a stack step with programmatic dependent launch (each kernel's set-up overlaps its
 *     predecessor's tail; off by default: measured, it does not pay inside replayed graphs); RRM_CHUNK_INPLACE=1
 *     makes the delta chunks of a stack (rrm_net_step_seq) add each frame's product straight onto the stored
 *     projection, as single steps do, instead of keeping it in a per-frame buffer that the epilogue merges (the
 *     default, which lets the convolution of frame t+1 run beside the epilogue of frame t; same results).
 *     Long delta chunks of few streams (from 16 frames on with up to 2 streams, from 32 on with up to 4) do not
 *     overlap frames at all: every kernel of a layer takes all frames of the chunk in one launch.
 *     RRM_CHUNK_BY_LAYER=1 makes every delta chunk take that form, RRM_CHUNK_PIPELINED=1 none (same results).
 */
#ifndef RRM_H
#define RRM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rrm_net rrm_net;     /* a stack of linear layers with their RRM state */
typedef struct rrm_net rrm_layer;   /* a single layer is a stack of one */

enum {
    RRM_OK = 0,
    RRM_ERR_INVALID_ARG = -1,
    RRM_ERR_SHAPE = -2,
    RRM_ERR_DTYPE = -3,
    RRM_ERR_ALLOC = -4,
    RRM_ERR_CAPACITY = -5,
    RRM_ERR_TIMEOUT = -6,
    RRM_ERR_CUDA = -7,
    RRM_ERR_UNSUPPORTED = -8
};

enum { RRM_CONV = 0, RRM_FC = 1 };
enum { RRM_F32 = 0, RRM_I8 = 1, RRM_BIN = 2 };
enum { RRM_ACT_NONE = 0, RRM_ACT_RELU = 1, RRM_ACT_SIGN = 2,
       RRM_ACT_LEAKY = 3 /* fp32 only: x > 0 ? x : 0.1 x, the leaky ReLU of the YOLOv2-style stacks of Sec. 4.4 */ };
/* How F*dI is evaluated.  As a request in rrm_layer_desc.variant: AUTO lets the library pick per layer: the kernel
 * (tensor cores for int8 and binary layers, CUDA cores for fp32) and, from the measured density, whether the layer
 * runs the sparse product at all.  In a stack whose layers all ask for AUTO every layer's share of projection
 * pixels to update is read back after each delta step (asynchronously); a layer whose share reached
 * rrm_options.layer_dense_activity is evaluated densely inside the following delta steps (P = F*X + b from the
 * current input replaces its stored projection; its input delta is still formed and counted, and its output delta
 * still emitted), and returns to the sparse product below rrm_options.layer_delta_activity.  For a lone int8 FC
 * layer AUTO also means: dense evaluation of a chunk when the previous chunk's measured delta density was high.
 * GATHER forces the CUDA-core / column-gather kernels; TENSOR is AUTO without any density switch; DENSE on a lone
 * FC layer selects the generic (non-fused) path; SPARSE_W: see the enumerator.
 * As a report in rrm_stats.variant: what the most recent step ran for this layer (GATHER, TENSOR, or DENSE for a
 * layer or chunk that was evaluated densely). */
enum { RRM_VARIANT_AUTO = 0, RRM_VARIANT_GATHER = 1, RRM_VARIANT_TENSOR = 2, RRM_VARIANT_DENSE = 3,
       RRM_VARIANT_SPARSE_W = 4 /* lone int8 FC layer: weight-sparse x delta-sparse product (Sec. 3.5 / 4.3: the
                                   compressed models EIE runs).  The zero weights of W (a pruned model) are dropped
                                   at create time: every (input, 512-output slice) keeps a 32-byte header (a 128-bit
                                   map of its non-zero groups of four outputs) and only those groups' bytes, so a non-zero
                                   delta entry gathers a fraction of its column.  Results are the same integers */ };

/*
 * One linear layer and the nonlinear map f that follows it (Eq. 1).
 * f, in order: [requant by `shift`: q = clamp((P + 2^(shift-1)) >> shift, -127, 127)] ->
 * [+ residual tensor] -> act -> max-pool; with act == SIGN the pool comes first and the
 * output bit is (pooled P >= theta).  shift < 0 on an integer layer emits the raw int32
 * projection (no act other than SIGN allowed then).  RRM_F32 ignores shift/theta.
 * An FC layer has h = w = kh = kw = 1, stride 1, pad 0.
 */
typedef struct {
    int32_t kind;        /* RRM_CONV | RRM_FC */
    int32_t dtype;       /* type of the layer's input and weights */
    int32_t n;           /* independent streams processed per call (same for all layers) */
    int32_t c_in, h, w;  /* input tensor */
    int32_t c_out, kh, kw, stride, pad;
    int32_t act;         /* RRM_ACT_* */
    int32_t pool_k, pool_s, pool_p;   /* pool_k == 0: no pooling */
    int32_t shift, theta;
    int32_t src;         /* stacks only: index of the tensor this layer reads (0 = frame, l+1 = output of layer l) */
    int32_t res;         /* stacks only: tensor added before act, or -1 */
    int32_t variant;     /* RRM_VARIANT_* */
} rrm_layer_desc;

/* Counters of the most recent step of one layer (delta density as defined for Table 1). */
typedef struct {
    int64_t in_elems;          /* elements of the layer input (all streams) */
    int64_t nnz_elems;         /* non-zero delta elements: rho = nnz_elems / in_elems */
    int64_t in_pixels;         /* spatial positions of the input (FC: groups of 32 inputs) */
    int64_t active_in_pixels;  /* positions with at least one non-zero delta */
    int64_t out_pixels;        /* spatial positions of the projection */
    int64_t active_out_pixels; /* positions whose projection was updated */
    int64_t active_macs;       /* exact multiply-accumulates the non-zero deltas imply */
    int64_t dense_macs;        /* multiply-accumulates of a dense pass */
    int32_t variant;           /* RRM_VARIANT_* actually used */
    int32_t error_word;        /* device-side error flags, 0 = none */
} rrm_stats;

/* Tunables of one object (a layer or a stack).  The paper leaves all of these to the implementation: it only
 * says that the sparse product pays off below some density (Table 1, Eq. 6) and that a precise inference may
 * replace the state at any time (Sec. 3.4).  rrm_net_get_options returns the defaults of a fresh object. */
typedef struct {
    uint32_t wait_limit;         /* polls a bounded device-side wait (mbarrier, completion of the tensor-core work)
                                    makes before it gives up, sets the time-out bit of rrm_stats.error_word and lets
                                    the thread block leave in an orderly way.  Default 2^20.  0 makes every such wait
                                    give up at once, before the thread block has anything in flight: a test hook */
    float layer_dense_activity;  /* stacks, variant AUTO: a layer whose measured share of projection pixels to update
                                    reached this value is evaluated densely in the following frames ...  Default
                                    1.01, i.e. never: on the stacks measured so far the sparse product of a single
                                    layer was never slower than its dense evaluation inside a delta step; lower it
                                    (e.g. to 0.75) to turn the per-layer choice on */
    float layer_delta_activity;  /* ... and goes back to the sparse product once the share has fallen below this one
                                    (default 1.005) */
    float stack_dense_activity;  /* whole-stack switch (stacks of >= 1 GMAC per frame): MAC-weighted share from which on
                                    every layer of the next frames is evaluated densely */
    int32_t stack_reprobe;       /* dense frames in a row before one delta frame measures the activity again */
    float fc_dense_rows;         /* lone int8 FC layer, chunks: rows x measured density from which on a chunk is
                                    evaluated densely on the tensor cores, per launch that evaluation needs */
    float fc_dense_density;      /* the same for chunks of more rows than the few-row kernel takes: plain density */
    float chunk_dense_activity;  /* stacks whose layers all run on the tensor cores, variant AUTO, chunks of 16 or more
                                    frames of up to 4 streams (rrm_net_step_seq): MAC-weighted share of projection
                                    pixels to update from which on the next chunks are evaluated densely, batched over
                                    their frames (same results; a delta chunk measures again after stack_reprobe dense
                                    ones).  Default 0.40: measured, the two kinds of chunk are level at about a third
                                    of the pixels active */
} rrm_options;

/* ---- single layer (Eq. 2-5) ------------------------------------------------------- */

/* Creates a layer with state I_prev = 0, P_prev = bias (Algorithm 1, line 1), so a first
 * rrm_step without keyframe equals a dense pass.  W_dev / bias_dev: device pointers in the
 * layouts above (bias_dev may be NULL = zeros).  Allocates device memory. */
int rrm_layer_create(rrm_layer** out, const rrm_layer_desc* desc, const void* W_dev, const void* bias_dev);
int rrm_layer_destroy(rrm_layer* layer);

/* Dense ("precise") inference of X0 that resets the state: I_prev = X0, P_prev = F*X0 + b
 * (the re-start that clears accumulated error, Sec. 3.4).  Y0_dev may be NULL; otherwise it
 * receives f(P) like rrm_step.  Asynchronous on `stream`. */
int rrm_keyframe(rrm_layer* layer, const void* X0_dev, void* Y0_dev, void* stream);

/* One RRM frame (Eq. 5): D = X_t - I_prev, compact its non-zeros, P_prev += F*D (no bias),
 * I_prev = X_t, Y_t = f(P_prev).  X_t is read-only and caller-owned; Y_t (caller-owned, may
 * be NULL) is written in full in the boundary layout.  Asynchronous on `stream`; no host
 * synchronisation inside. */
int rrm_step(rrm_layer* layer, const void* Xt_dev, void* Yt_dev, void* stream);

/* The same layer evaluated densely, Y = f(F*X + b), without reading or changing the RRM
 * state: the library's own dense path (the denominator of its delta-path speedup). */
int rrm_dense(rrm_layer* layer, const void* X_dev, void* Y_dev, void* stream);

/* rrm_step with HOST buffers: copies X_t to the device, steps, copies Y_t back, all on
 * `stream`; returns after the stream has been synchronised. */
int rrm_step_host(rrm_layer* layer, const void* Xt_host, void* Yt_host, void* stream);

/* A chunk of T consecutive frames in one call: the frame loop of Algorithm 1 for frames t0 .. t0+T-1
 * (the end of Sec. 3.2 notes that a video may be cut into chunks that are processed on their own).  The result
 * and the state afterwards are exactly those of T rrm_step calls in a row.
 *   X_dev  [T] frames, each in the layer's input layout, back to back; read-only
 *   Y_dev  [T] outputs f(P_t), each in the layer's output layout, back to back; may be NULL
 * For a lone int8 FC layer all T input deltas are known up front (dI_t = X_t - X_{t-1}), so the T
 * sparse products W dI_t run in ONE launch and only the running sum P_t = P_{t-1} + W dI_t is
 * serial.  A stack (and a lone layer of another kind) keeps Algorithm 1's order per layer but lets the frames of
 * the chunk overlap: the T frames are captured as one graph in which layer l of frame t+1 waits only for layer
 * l-1 of frame t+1, for layer l of frame t (its projection) and for the layers of frame t that read the tensor
 * it overwrites; the first call with a new T captures that graph (and allocates T frames of staging).  With eps > 0
 * the frames are stepped one by one.  With variant AUTO the
 * library reads back the measured delta density of each chunk (asynchronously) and evaluates the
 * next chunk densely on the tensor cores instead when that density was high: outputs, state and
 * counters are the same integers either way.  The first call with a larger T than any before
 * allocates scratch memory (T * N * c_out * 4 bytes); later calls do not.
 * T * N must not exceed 65535.  Asynchronous on `stream`.  After the call rrm_get_stats reports the
 * counters summed over the chunk's frames (lone int8 FC layer) or those of the chunk's last frame (other layers). */
int rrm_step_seq(rrm_layer* layer, const void* X_dev, void* Y_dev, int T, void* stream);
/* T frames through the dense path, each on its own (Y_t = f(F*X_t + b)); RRM state untouched. */
int rrm_dense_seq(rrm_layer* layer, const void* X_dev, void* Y_dev, int T, void* stream);
/* rrm_step_seq with HOST buffers (copies in, steps, copies out, synchronises `stream`). */
int rrm_step_seq_host(rrm_layer* layer, const void* X_host, void* Y_host, int T, void* stream);
/* The same without waiting: the call returns once the work is queued.  The copy-in, the frames and the
 * copy-out of a call run on three streams (two of them the library's own) chained by events, through two
 * staging slots, so that consecutive calls overlap: chunk k+1 is copied in and chunk k-1 copied out while
 * chunk k is computed.  X_host and Y_host should be page-locked (pageable memory makes the copies
 * synchronous); X_host must stay unchanged and Y_host unread until rrm_host_sync has returned.  Calls must be
 * issued from one thread, in frame order;
 * the RRM state advances in that order on `stream`.  The first call, and a call with a larger T than any
 * before, allocate the staging slots. */
int rrm_step_seq_host_async(rrm_layer* layer, const void* X_host, void* Y_host, int T, void* stream);
/* Waits until every queued rrm_step_seq_host_async call has delivered its outputs to host memory. */
int rrm_host_sync(rrm_layer* layer);

/* Synchronises the layer's last stream and fills `host_out`.  Returns RRM_ERR_TIMEOUT when a bounded device wait
 * ran out since the last rrm_clear_errors (bit 1 of error_word), RRM_ERR_CAPACITY when an int8 delta did not fit a
 * byte (bit 0): host_out is filled in both cases, and the results of the affected frames are not to be trusted
 * (a dense pass, rrm_keyframe, restores a consistent state). */
int rrm_get_stats(rrm_layer* layer, rrm_stats* host_out);
/* Clears the device error word (synchronises the layer's last stream). */
int rrm_clear_errors(rrm_layer* layer);
/* Reads / replaces the tunables.  rrm_set_options synchronises the device and discards the captured launch
 * sequences (they hold the old values); call it between frames. */
int rrm_get_options(const rrm_layer* layer, rrm_options* out);
int rrm_set_options(rrm_layer* layer, const rrm_options* in);

/* Copies the stored projection P_prev (float or int32, [N][C_out][OH][OW]) to P_dev. */
int rrm_layer_projection(rrm_layer* layer, void* P_dev, void* stream);

/* ---- layer stack (Algorithm 1) ---------------------------------------------------- */

/* descs[l].src / .res give the topology; tensor 0 is the frame, tensor l+1 = f(P_l).
 * W_dev[l] / bias_dev[l] as for rrm_layer_create. */
int rrm_net_create(rrm_net** out, const rrm_layer_desc* descs, int n_layers,
                   const void* const* W_dev, const void* const* bias_dev);
int rrm_net_destroy(rrm_net* net);

/* Dense pass over the whole stack that resets every layer's state. out_dev may be NULL. */
int rrm_net_keyframe(rrm_net* net, const void* frame_dev, void* out_dev, void* stream);
/* Algorithm 1, one iteration of the frame loop; out_dev receives the last tensor.  On a stack of at least
 * 1 GMAC per frame whose layers all ask for RRM_VARIANT_AUTO the library reads back (asynchronously) how many
 * projection pixels the last delta frame had to update; while that share, weighted by the layers' MACs, is
 * 75 % or more it evaluates frames densely instead (a precise inference that replaces the state: the same
 * results), and measures again with a delta frame every 16th frame.  rrm_net_get_stats reports such a frame
 * with variant RRM_VARIANT_DENSE and its counters as -1 (nothing was counted).  Below that share the choice is
 * made layer by layer (see RRM_VARIANT_AUTO): such layers report RRM_VARIANT_DENSE with their counters intact. */
int rrm_net_step(rrm_net* net, const void* frame_dev, void* out_dev, void* stream);
/* Dense evaluation of the stack without touching the RRM state. */
int rrm_net_dense(rrm_net* net, const void* frame_dev, void* out_dev, void* stream);
int rrm_net_step_host(rrm_net* net, const void* frame_host, void* out_host, void* stream);
/* Chunks of T frames, as rrm_step_seq / rrm_dense_seq / rrm_step_seq_host; outs = [T] last tensors.  After the call
 * rrm_net_get_stats reports the counters of the chunk's last frame. */
int rrm_net_step_seq(rrm_net* net, const void* frames_dev, void* outs_dev, int T, void* stream);
int rrm_net_dense_seq(rrm_net* net, const void* frames_dev, void* outs_dev, int T, void* stream);
int rrm_net_step_seq_host(rrm_net* net, const void* frames_host, void* outs_host, int T, void* stream);
/* As rrm_step_seq_host_async / rrm_host_sync. */
int rrm_net_step_seq_host_async(rrm_net* net, const void* frames_host, void* outs_host, int T, void* stream);
int rrm_net_host_sync(rrm_net* net);

int rrm_net_get_stats(rrm_net* net, int layer, rrm_stats* host_out);
int rrm_net_clear_errors(rrm_net* net);
int rrm_net_get_options(const rrm_net* net, rrm_options* out);
int rrm_net_set_options(rrm_net* net, const rrm_options* in);

/* ---- explicit batch normalisation as part of f (the non-linear layer the paper's Discussion names, Sec. 4.5) ----
 * At inference batch normalisation is a per-channel affine on the full projection P_t; it can be folded into
 * the filters, or kept explicit: then f of `layer` becomes [affine] -> [requant] -> [+ residual] -> act -> pool.
 *   RRM_F32 layers: float scale[c_out], shift[c_out]:        y = scale * P + shift
 *   RRM_I8 layers with shift >= 0: int32 m[c_out], a[c_out]: q = clamp((P*m + a + 2^(shift-1)) >> shift, -127, 127),
 *                                                            evaluated in 64 bits
 * Other layers: RRM_ERR_UNSUPPORTED.  Both device arrays are copied.  NULL, NULL removes the affine.  Because f
 * changes, the call puts the stack back into its fresh state (as after rrm_net_create); it synchronises the
 * device and discards the captured launch sequences: call it right after creating the stack. */
int rrm_net_set_affine(rrm_net* net, int layer, const void* scale_dev, const void* shift_dev);

/* ---- approximate mode: sparsity enhancement and accumulated error control (Sec. 3.4) -----------
 * With eps > 0 every delta entry with |d| < eps is truncated to zero before the sparse product (fp32 stacks
 * only, RRM_ERR_DTYPE otherwise).  The snapshot still becomes the new frame, so the truncated part u is lost:
 * the outputs are approximate and the error accumulates until the next rrm_net_keyframe.  eps = 0 (the
 * default) is the exact recurrence.  Synchronises the device; call it between frames. */
int rrm_net_set_epsilon(rrm_net* net, float eps);
/* Eq. 7: *e_t = sum over the frames since the last keyframe and over the linear layers of l2(u), u the
 * truncated part of the layer's input delta (all streams of the batch together).  last_step_l2 (may be NULL)
 * receives the [n_layers] terms of the most recent frame.  Synchronises the net's last stream. */
int rrm_net_truncation(rrm_net* net, double* e_t, double* last_step_l2);
/* Eq. 8 with H a fourth-order polynomial: mu[0] + mu[1] e_t + ... + mu[4] e_t^4 (host arithmetic).  The paper
 * fits mu on its data; the caller supplies it and runs rrm_net_keyframe when the estimate passes its threshold. */
double rrm_aecs_predict(const double mu[5], double e_t);
/* Copies P_prev of `layer` / the current value of tensor `t` (boundary layout) to dst_dev. */
int rrm_net_projection(rrm_net* net, int layer, void* P_dev, void* stream);
int rrm_net_tensor(rrm_net* net, int t, void* dst_dev, void* stream);
/* Bytes rrm_net_tensor / the out_dev argument need for tensor `t` (negative = error). */
int64_t rrm_net_tensor_bytes(const rrm_net* net, int t);

/* ---- allocation-free delta-FC step --------------------------------------------------
 * (The paper has no counterpart; this is a deployment aid of this library.)
 *
 * Some callers of this library are not allowed to allocate device memory: plug-ins whose
 * host hands them a fixed memory budget up front and forbids cudaMalloc afterwards, real-time
 * loops that must not wait on the allocator's lock or on the device-wide synchronisation a
 * cudaFree implies, and processes that share a GPU under a hard memory cap.  This entry point does one int8 delta-FC frame - what rrm_step
 * does for a lone RRM_FC / RRM_I8 layer - without calling cudaMalloc, cudaFree or any
 * allocating routine: the caller owns the whole RRM state, and the one piece of working
 * memory the kernels need (the per-stream lists of non-zero delta entries) is a fixed
 * array compiled into the library, RRM_FC_NOALLOC_MAX_STREAMS * RRM_FC_NOALLOC_MAX_C_IN * 4
 * bytes (1 MiB) plus a 64-byte header.  Every GPU that loads the library keeps that array until
 * the process exits.
 *
 *   Wt_dev    [c_in][c_out] int8   the layer's weights TRANSPOSED (one contiguous row per input)
 *   Xt_dev    [n][c_in]     int8   frame t, read-only
 *   Xprev_dev [n][c_in]     int8   in/out: frame t-1 on entry, frame t on return (start with zeros)
 *   P_dev     [n][c_out]    int32  in/out: stored projection (start with the bias in every row)
 *   Y_dev     [n][c_out]    int32 if shift < 0, else int8 = f(P) as for rrm_step; may be NULL
 * All pointers are device pointers; Wt_dev, Xt_dev and Xprev_dev must be 16-byte aligned; c_in
 * and c_out must be multiples of 16.  act is RRM_ACT_NONE or RRM_ACT_RELU.
 *
 * Errors: RRM_ERR_CAPACITY if n > RRM_FC_NOALLOC_MAX_STREAMS or c_in > RRM_FC_NOALLOC_MAX_C_IN;
 * RRM_ERR_SHAPE / RRM_ERR_INVALID_ARG for the other violations; nothing is launched then.
 *
 * The first call on a device looks up the array's device address (one cudaGetSymbolAddress,
 * no allocation); make that first call before starting any stream capture.  All calls on a
 * device share the one array and it keeps the previous call's contents; nothing in it has to
 * start at zero (each call rewrites every count and entry it later reads), but for the same
 * reason two calls that overlap on the GPU (different streams, no ordering) race on it:
 * serialise them.  Asynchronous on `stream`. */
#define RRM_FC_NOALLOC_MAX_STREAMS 16
#define RRM_FC_NOALLOC_MAX_C_IN 16384
int rrm_fc_step_noalloc(const int8_t* Wt_dev, const int8_t* Xt_dev, int8_t* Xprev_dev, int32_t* P_dev,
                        void* Y_dev, int n, int c_in, int c_out, int shift, int act, void* stream);

/* ---- measured ALU peaks -------------------------------------------------------------
 * (No counterpart in the paper: a reporting aid.)  Runs a register-only loop of independent operations on every
 * SM of the current device and returns the best of four timings as multiply-accumulates per second:
 *   kind 0  fp32 fused multiply-add                       (the fp32 delta convolution, Table 1's MACs)
 *   kind 1  dp4a, counted as 4 int8 multiply-accumulates  (int8 layers on the CUDA cores, the delta-FC products)
 *   kind 2  popc + add, counted as 32 one-bit products    (binary layers on the CUDA cores, Sec. 4.3)
 * The rooflines of ALU-bound kernels are quoted against these numbers.  Allocates 4 bytes, synchronises. */
int rrm_measure_alu_peak(int kind, double* macs_per_s);

const char* rrm_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* RRM_H */
