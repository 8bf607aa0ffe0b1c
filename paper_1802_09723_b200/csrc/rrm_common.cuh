// Internal declarations shared by the translation units of the RRM library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <cstdio>
#include <cstdlib>
#include <functional>
#include <vector>
#include "../../include/rrm.h"

// RRM_DEBUG=1 in the environment: a failing CUDA call is named on stderr (call site and error string)
inline void rrm_note_cuda_error(cudaError_t e, const char* file, int line)
{
    static const bool on = getenv("RRM_DEBUG") != nullptr;
    if (on) fprintf(stderr, "rrm: %s:%d: %s\n", file, line, cudaGetErrorString(e));
}

#define RRM_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) { rrm_note_cuda_error(e__, __FILE__, __LINE__); return RRM_ERR_CUDA; } \
    } while (0)

#define RRM_TRY(expr)                                        \
    do {                                                     \
        int s__ = (expr);                                    \
        if (s__ != RRM_OK) return s__;                       \
    } while (0)

namespace rrm {

// ---- programmatic dependent launch between the kernels of a per-frame sequence --------------------------------
// Every kernel of the sequence lets its successor start launching at once (launch_dependents at its top) and waits
// for its predecessor's results (pdl_wait) only when it first needs global memory: thread-block scheduling, barrier
// initialisation and tensor-memory allocation of kernel k+1 then overlap the tail of kernel k.  Without the launch
// attribute both instructions do nothing.  Measured on B200 inside replayed graphs the attribute moves a step by
// -8 % .. +27 % depending on the stack (the graph's own launch gaps are already small), so it is opt-in:
// RRM_PDL=1 in the environment launches with the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

inline bool pdl_enabled()
{
    static const bool on = [] { const char* e = getenv("RRM_PDL"); return e && e[0] == '1'; }();
    return on;
}

// cluster_z > 1: the CTAs that differ only in blockIdx.z form one thread-block cluster (they can read each other's
// shared memory).
template <typename... P, typename... A>
inline cudaError_t launch_seq_cluster(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_z,
                                      A&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[2];
    int n = 0;
    if (pdl_enabled()) {
        at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster_z > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = 1; at[n].val.clusterDim.y = 1; at[n].val.clusterDim.z = (unsigned)cluster_z;
        ++n;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

template <typename... P, typename... A>
inline cudaError_t launch_seq(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args)
{
    return launch_seq_cluster(kernel, grid, block, smem, st, 1, static_cast<A&&>(args)...);
}

// storage type of a tensor inside the library (always pixel-major: [n][h][w][cs])
enum { T_F32 = 0, T_I8 = 1, T_BIN = 2, T_I32 = 3 };

// device error flags (rrm_stats.error_word)
enum { ERRW_BOUNDS = 1, ERRW_TIMEOUT = 2, ERRW_CAPACITY = 4 };

// tile shape of the CUDA-core implicit GEMM (units: float, 4 x int8, or 32 sign bits)
constexpr int GEMM_TN = 64;   // output channels per CTA
constexpr int GEMM_TK = 32;   // K units per stage

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline int round_up(int a, int b) { return ceil_div(a, b) * b; }

// A layer that reads a tensor, as its input (filter footprint) or as its shortcut (1x1 footprint).
struct Reader {
    uint32_t* oact;                   // the reading layer's bitmap of projection pixels to update
    int oh, ow, kh, kw, stride, pad, c_out;
    unsigned long long* macs;         // the reading layer's counter of exact multiply-accumulates; nullptr for a shortcut reader
};
constexpr int MAX_READERS = 4;
struct Readers { Reader r[MAX_READERS]; int n; };

// Several consecutive frames in one launch (frame = blockIdx.z; frames <= 1: the ordinary single-frame launch): where
// frame g's data lie relative to frame 0's.
struct SeqFrames {
    int frames;
    long long in_stride;      // elements between consecutive frames at the boundary (the frame before frame 0 lies one stride earlier)
    long long row_stride;     // bytes between the frames' sets of delta rows (and of new rows)
    long long arena_stride;   // bytes between the frames' arenas (bitmaps, counters)
};

constexpr int CHUNK_RING = 4;         // sets of delta rows / delta-projection buffers a pipelined chunk cycles through

struct Tensor {
    int dtype = T_F32;
    int n = 0, c = 0, h = 0, w = 0;
    int cs = 0;                       // storage units per pixel (f32/i32: c; i8: c rounded up to 4; bin: words)
    int unit_bytes = 4;               // bytes per storage unit (i8: 1)
    void* X = nullptr;                // current value (= snapshot of the previous frame before a step)
    void* D = nullptr;                // delta rows, valid only for pixels whose `act` bit is set
    uint32_t* act = nullptr;          // bitmap over n*h*w pixels (cleared every step)
    int* pnnz = nullptr;              // per-pixel count of non-zero delta elements (valid where act is set)
    unsigned long long* nnz = nullptr;      // total non-zero delta elements (cleared every step)
    unsigned long long* npix = nullptr;     // active pixels (cleared every step)
    double* trunc = nullptr;                // fp32: sum of squares of the truncated delta entries (cleared every step)
    void* X2 = nullptr;               // value buffer of the stateless dense path
    // pipelined chunks: consecutive frames write their delta rows into a ring of sets ([0] is the set D points at
    // outside the capture of such a chunk), so that a producer does not wait for the previous frames' readers
    void* Dring[CHUNK_RING] = {};
    // binary tensors: the sparse product needs the new value of a changed bit (its sign) next to the delta rows, so the
    // pipelined chunk keeps a copy of the new rows per frame parity; Xn_cur is set only while such a chunk is captured
    void* Xn[CHUNK_RING] = {};
    void* Xn_cur = nullptr;
    // delta chunks taken layer by layer over all frames (rrm_conv_seq.cu): per-frame delta rows, per-frame new rows
    // (binary tensors), and for the stack's last tensor every frame's full rows; SEQ_MAX_FRAMES of each
    void* Dall = nullptr;
    void* Xnall = nullptr;
    void* Xfull = nullptr;
    void* X2b = nullptr;              // value buffer of a dense chunk batched over its frames (as many frames' worth as a launch takes)
    void* Xbefore = nullptr;          // tensors added as a shortcut: the value before the chunk (the snapshot moves on before the reader runs)
    bool shortcut_source = false;
    bool has_consumer = false;        // some layer reads this tensor (its int8 deltas must fit a byte)
    Readers readers{};                // the layers that read it
    int pixels() const { return n * h * w; }
    size_t row_bytes() const { return (size_t)cs * unit_bytes; }
    size_t bytes() const { return (size_t)pixels() * row_bytes(); }
    int act_words() const { return ceil_div(pixels(), 32); }
};

struct Layer {
    rrm_layer_desc d;
    int oh = 0, ow = 0;               // projection spatial size
    int th = 0, tw = 0;               // output tensor spatial size (after pooling)
    int u_in = 0;                     // storage units per input pixel
    int ku = 0, kup = 0;              // K in units, and padded to GEMM_TK
    int np = 0;                       // c_out padded to GEMM_TN
    void* Wk = nullptr;               // packed filters [kup][np] units
    void* bias = nullptr;             // float or int32 [c_out]
    void* bn_scale = nullptr;         // explicit per-channel affine applied to P before the rest of f (batch
    void* bn_shift = nullptr;         // normalisation at inference): float, or int32 multiplier / offset; nullptr: none
    void* P = nullptr;                // projection [n*oh*ow][c_out] float or int32
    void* P2 = nullptr;               // projection buffer of the stateless dense path
    // pipelined delta chunks: the convolution of a frame adds into a delta-projection buffer of its own (one of a ring,
    // zero between uses) and the epilogue merges it, reading the projection from one buffer and writing it to the
    // other, so that the convolution of frame t+1 does not wait for the epilogue of frame t
    void* Palt = nullptr;             // the second projection buffer (a copy of P is made at the start of a chunk)
    void* dP[CHUNK_RING] = {};
    size_t oact_off = 0;              // offset of the update bitmap inside an arena
    void* P2b = nullptr;              // projection buffer of a dense chunk batched over its frames
    void* Aall = nullptr;             // pooled int8 layers of that form: f before the pool window of every frame's projection, as bytes
                                      // ([0]: of the projection before the chunk, every pixel; [1 + g]: frame g's updated pixels)
    void* dPall = nullptr;            // per-frame products of the layer-by-layer chunk form
    uint32_t* oact = nullptr;         // bitmap of projection pixels to update (cleared every step, set by the
                                      // kernels that produce the layer's input and shortcut tensors)
    int* ocount = nullptr;            // their number (cleared every step, written by the convolution kernel)
    unsigned long long* macs = nullptr;     // exact active multiply-accumulates (cleared every step)
    int opixels() const { return d.n * oh * ow; }
    // per-layer choice between the sparse product and a dense evaluation inside a delta step, from the measured
    // share of projection pixels to update (north of rrm_options.layer_dense_activity: dense)
    bool dense_mode = false;          // how the layer runs in the next delta step
    bool ran_dense = false;           // how it ran in the most recent one
    double activity = -1.0;           // last measured share; < 0: unknown
    // fused FC path (int8 FC reading the external input)
    bool fc_fused = false;
    int8_t* Wt = nullptr;             // [c_in][c_out] transposed weights
    int8_t* xs[2] = {nullptr, nullptr};     // ping-pong input snapshots [n][c_in]
    int xs_cur = 0;
    void* fc_scratch = nullptr;             // per-stream non-zero lists of the two-kernel form
    unsigned long long* fc_nnz = nullptr;   // [0] nnz elements, [1] active groups of 32 (cleared by the kernel's last CTA)
    // weight-sparse form (RRM_VARIANT_SPARSE_W): per (input, 512-output slice) a record of sp_stride words:
    // 8 words of header (map of the non-zero groups of four outputs, running counts), then those groups' weights, packed
    uint32_t* Wsp = nullptr;
    int sp_stride = 0;
    long long sp_words = 0;                 // packed weight words of the whole matrix (for reporting)
    // tensor-core variant (int8 / binary layers whose input rows are whole 32-byte K chunks)
    bool tc_ready = false;
    int8_t* tc_Wimg = nullptr;              // [n_tiles][slabs][bn * 128] shared-memory images of the filter tiles
    int tc_kpp = 0;                         // K bytes per tap (padded channels per pixel)
    int tc_bn = 0, tc_ntiles = 0, tc_slabs = 0;
    // few-row dense FC on the tensor cores (weights as the M operand, K split over CTAs)
    int32_t* ft_acc = nullptr;              // [rows][tiles * 128] partial sums, zero between launches
    unsigned* ft_arrive = nullptr;          // [tiles] arrival counters, zero between launches
    bool ft_cluster = false;                // the K shares of an output block run as one thread-block cluster
    // chunk-of-frames form of the fused FC path
    int32_t* seq_dP = nullptr;              // [seq_cap][n][c_out] per-frame projection deltas
    unsigned* seq_stat = nullptr;           // [seq_cap * n][2] per frame and stream: non-zeros, active groups of 32
    unsigned* seq_counters = nullptr;       // [n][slices] arrival counters (zero between launches)
    int seq_cap = 0;                        // frames the scratch arrays hold
    int seq_lanes = 0;                      // 0: pick the slice width per call; 8 / 16 / 32: forced (tuning)
    int seq_last_T = 0;                     // frames of the most recent chunk (0: last call was a single-frame step)
    // measured density of the previous chunk, read back without stalling the stream: chooses between the
    // column gather and the dense tensor-core evaluation of the next chunk
    unsigned* seq_stat_host = nullptr;      // pinned copy of seq_stat
    int seq_stat_host_cap = 0;              // frames it holds
    cudaEvent_t seq_ev = nullptr;           // the copy into seq_stat_host has landed
    bool seq_ev_pending = false;
    int seq_pending_rows = 0;               // frame x stream rows of the pending copy
    double seq_density = -1.0;              // non-zero fraction of the last chunk whose counters were read; < 0: unknown
    int seq_last_variant = RRM_VARIANT_GATHER;
};

}  // namespace rrm

struct rrm_net {
    std::vector<rrm::Layer> layers;
    std::vector<rrm::Tensor> tensors;
    int n = 1;
    void* cleared = nullptr;          // arena zeroed at the start of every step
    char* bound_arena = nullptr;      // the arena the tensors' and layers' bitmap / counter pointers refer to right now
    size_t cleared_bytes = 0;
    int* errw = nullptr;              // device error word
    cudaStream_t last_stream = nullptr;
    void* stage_in = nullptr;         // device staging for the *_host entry points
    void* stage_out = nullptr;
    int stage_frames = 0;             // frames the staging buffers hold
    // pipelined host entry point: two staging slots, copies on streams of their own so that the copy-in of
    // chunk k+1 and the copy-out of chunk k-1 overlap the kernels of chunk k
    cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    void* pipe_in[2] = {nullptr, nullptr};
    void* pipe_out[2] = {nullptr, nullptr};
    int pipe_frames = 0, pipe_slot = 0;
    cudaStream_t cap_stream = nullptr;
    void* frame_buf = nullptr;        // the step's input frame, boundary layout
    void* out_buf = nullptr;          // the step's last tensor, boundary layout
    bool graph_off = false;           // RRM_NO_GRAPH=1: launch kernel by kernel (debugging)
    bool many_in_flight = false;      // set while a chunk graph is captured: its launches share the machine with those of
                                      // neighbouring frames, so grids are sized for throughput instead of latency
    // where a captured sequence reads the frame and writes the output: the nodes (kernel arguments or a copy) that
    // hold frame_buf / out_buf are re-pointed at the caller's buffers before each launch, which saves the two
    // device-to-device copies around the graph; empty when the nodes could not be identified
    struct IoPatch {
        cudaGraphNode_t node = nullptr;
        bool is_copy = false;                      // a 1-D copy node (binary outputs) instead of a kernel
        cudaKernelNodeParams kp = {};
        std::vector<void*> args;                   // the node's argument pointers, ours to edit
        int index = -1;                            // which argument is the buffer
        const void* src = nullptr; size_t bytes = 0;   // copy node: source and size
        void* value = nullptr;                     // storage the patched argument points to
    };
    // the per-frame launch sequences (0: delta step, 1: keyframe, 2: stateless dense pass), each captured once and
    // replayed (fixed frame / output buffers).  A delta step exists in one form per layer mask (bit l: layer l is
    // evaluated densely inside the step); the few most recently used masks are kept.
    struct StepGraph {
        unsigned long long mask = 0, used = 0;
        cudaGraph_t graph = nullptr;
        cudaGraphExec_t exec = nullptr;
        std::vector<IoPatch> patch_in, patch_out;
        bool patch_ok = false;
    };
    std::vector<StepGraph> step_graphs[3];
    unsigned long long step_clock = 0;
    unsigned long long layer_mask = 0;            // the mask of the next delta step
    bool layer_switch = false;                    // every layer asks for RRM_VARIANT_AUTO: the per-layer choice is on
    uint32_t* ones = nullptr;                     // an all-ones bitmap as long as the longest update bitmap
    // pipelined chunks of frames (rrm_net_step_seq on a stack): T frames captured as ONE graph in which layer l of
    // frame t+1 depends only on layer l-1 of frame t+1, on layer l of frame t (its projection) and on the layers of
    // frame t that read the tensor it overwrites - so consecutive frames overlap layer by layer.  Each frame in
    // flight has an arena of its own.
    std::vector<char*> chunk_arena;
    std::vector<cudaStream_t> chunk_streams;      // capture streams, one per frame in flight ([0] is cap_stream)
    // [slot * layers + l]: the most recently captured convolution / epilogue of layer l among the frames of ring slot
    // `slot` (frame mod CHUNK_RING in the split form; slot 0 only otherwise)
    std::vector<cudaEvent_t> ev_conv, ev_epi;
    cudaEvent_t ev_import = nullptr;
    bool dense_batch_ready = false;               // the buffers of the frame-batched dense chunk exist
    bool seq_ready = false;                       // the buffers of the layer-by-layer chunk form exist
    bool chunk_by_layer = false;                  // RRM_CHUNK_BY_LAYER=1: delta chunks always go layer by layer over all frames (where the stack allows)
    bool chunk_pipelined = false;                 // RRM_CHUNK_PIPELINED=1: delta chunks overlap frames instead of batching them per layer
    bool chunk_in_place = false;                  // RRM_CHUNK_INPLACE=1: delta chunks add into the stored projection (no delta-projection buffers)
    uint32_t* zeros = nullptr;                    // an all-zero bitmap as long as the longest update bitmap
    std::vector<cudaEvent_t> ev_join;
    cudaEvent_t ev_fork = nullptr, ev_export = nullptr;
    struct ChunkGraph { int T = 0; unsigned long long mask = 0; cudaGraph_t graph = nullptr; cudaGraphExec_t exec = nullptr; unsigned long long used = 0;
                        int last_arena = 0; /* the arena that holds the chunk's last frame */ };
    std::vector<ChunkGraph> chunk_graphs[3];      // per kind (delta / keyframes / dense): the few most recently used chunk lengths
    unsigned long long chunk_clock = 0;
    void* chunk_in = nullptr;                     // T frames at the boundary; one more frame fits right in front of them
    void* chunk_in_raw = nullptr;                 // (the allocation chunk_in points into)
    void* chunk_out = nullptr;
    int chunk_cap = 0;                            // frames chunk_in / chunk_out hold
    // measured activity of the last delta step, read back without stalling the stream: when nearly every
    // projection pixel has to be updated anyway, the next frames are evaluated densely (same results, less work)
    size_t counters_off = 0, counters_bytes = 0;   // the counters inside the cleared arena
    unsigned char* act_host = nullptr;        // pinned copy of the counters
    cudaEvent_t act_ev = nullptr;
    bool act_pending = false;
    double activity = -1.0;                   // MAC-weighted fraction of projection pixels updated; < 0: unknown
    int dense_streak = 0;                     // dense frames since the last measured delta frame
    bool last_step_dense = false;             // the most recent rrm_net_step was evaluated densely
    bool auto_switch = false;                 // every layer asks for RRM_VARIANT_AUTO and the net is large enough
    bool chunk_switch = false;                // every layer asks for RRM_VARIANT_AUTO and runs on the tensor cores: long chunks may go dense
    // the defaults rrm_net_get_options reports.  (The per-layer thresholds are above 1, i.e. the per-layer choice is off
    // until the caller lowers them: measured on B200, a dense evaluation of one layer inside a delta step is never
    // faster than its sparse product, not even with every pixel active.  What a delta step pays for is change
    // detection and marking, which only a dense pass of the whole stack drops.)
    rrm_options opt = {1u << 20, 1.01f, 1.005f, 0.75f, 15, 0.75f, 0.08f, 0.40f};
    float eps = 0.f;                  // Sec. 3.4: fp32 delta entries below it are truncated (0: exact)
    double* aecs = nullptr;           // [1 + layers]: accumulated truncated value e_t (Eq. 7), then the last step's l2 per layer
    std::vector<void*> allocs;        // everything to free
};

namespace rrm {

// ---- rrm_fc.cu
int fc_fused_create(rrm_net* net, Layer& L, const void* W_dev, const void* bias_dev);
int fc_fused_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, bool dense, bool stateless,
                 cudaStream_t st);
int fc_fused_projection(rrm_net* net, Layer& L, void* P_dev, cudaStream_t st);

// ---- rrm_fc_seq.cu
int fc_seq_create(rrm_net* net, Layer& L);
int fc_sparse_w_create(rrm_net* net, Layer& L);
bool fc_seq_supported(const Layer& L);
int fc_seq_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, int T, bool dense, bool stateless,
               cudaStream_t st);
int fc_seq_stats(Layer& L, unsigned long long* nnz, unsigned long long* groups);
int fc_dense_tc_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, int T, bool stateless, cudaStream_t st);

// ---- rrm_fc_tc.cu
int fc_tc_create(rrm_net* net, Layer& L);
bool fc_tc_usable(const Layer& L, int rows);
int fc_tc_launches(int rows);
int fc_tc_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, int rows, bool stateless, unsigned* stat, cudaStream_t st);

// ---- rrm_conv_tc.cu
bool conv_tc_eligible(const rrm_net* net, const Layer& L);
int conv_tc_create(rrm_net* net, Layer& L, const void* W_dev);
int launch_conv_tc(rrm_net* net, Layer& L, const Tensor& in, bool dense, bool stateless, cudaStream_t st,
                   const uint32_t* count_bitmap = nullptr, void* P_dst = nullptr, int frames = 1, long long arena_stride = 0);
int zero_projection(void* P, long long words, cudaStream_t st);

// ---- rrm_conv.cu
int conv_layer_create(rrm_net* net, Layer& L, const void* W_dev, const void* bias_dev);
int launch_import(rrm_net* net, const void* frame_dev, bool delta, bool stateless, cudaStream_t st, int frames = 1, long long arena_stride = 0);
// Where a delta step of one layer keeps its projection when the frames of a chunk are pipelined (null: in place).
struct SplitProjection {
    void* dP;                         // the convolution adds here (zero wherever the frame has no update)
    const void* R;                    // the projection as of the previous frame
    void* Q;                          // receives R + dP at the pixels updated in this frame or in the previous one
    void* Z;                          // the previous frame's delta-projection buffer, zeroed at that frame's updated pixels
    const uint32_t* prev_oact;        // the previous frame's update bitmap
};
int launch_layer(rrm_net* net, int l, bool dense, bool stateless, cudaStream_t st,
                 const std::function<int(int)>* hook = nullptr, bool dense_in_step = false,
                 const SplitProjection* split = nullptr);
int launch_export_tensor(rrm_net* net, int t, void* dst_dev, bool stateless, cudaStream_t st);
int launch_export_projection(rrm_net* net, int l, void* dst_dev, cudaStream_t st);
int reset_state(rrm_net* net, cudaStream_t st);
int ensure_stateless(rrm_net* net);
int launch_aecs(rrm_net* net, cudaStream_t st);
int ensure_split(rrm_net* net);
int launch_layer_seq(rrm_net* net, int l, int frames, long long arena_stride, cudaStream_t st);
int launch_export_seq(rrm_net* net, int frames, void* dst_dev, cudaStream_t st);

// ---- rrm_conv_seq.cu
int launch_epilogue_seq(rrm_net* net, int l, int frames, long long arena_stride, cudaStream_t st);
int ensure_frame_batch(rrm_net* net);
int seq_max_frames();
int launch_copy_projections(rrm_net* net, cudaStream_t st);
int launch_copy_state_from_batch(rrm_net* net, int slot, cudaStream_t st);
int launch_zero_delta_projections(rrm_net* net, int slot, cudaStream_t st);
int clear_split(rrm_net* net, cudaStream_t st);

}  // namespace rrm
