// C ABI of the RRM library: object construction, validation and the per-frame launch sequences.
#include "rrm_common.cuh"
#include <new>
#include <cstring>
#include <cstdlib>

using namespace rrm;

namespace {

int tensor_bytes_boundary(const Tensor& T, int64_t* out)
{
    if (T.dtype == T_BIN) *out = (int64_t)T.pixels() * T.cs * 4;
    else *out = (int64_t)T.n * T.c * T.h * T.w * (T.dtype == T_I8 ? 1 : 4);
    return RRM_OK;
}

int validate_desc(const rrm_layer_desc& d, int l, int n_layers)
{
    if (d.kind != RRM_CONV && d.kind != RRM_FC) return RRM_ERR_INVALID_ARG;
    if (d.dtype != RRM_F32 && d.dtype != RRM_I8 && d.dtype != RRM_BIN) return RRM_ERR_DTYPE;
    if (d.n < 1 || d.c_in < 1 || d.c_out < 1 || d.h < 1 || d.w < 1) return RRM_ERR_SHAPE;
    if (d.kh < 1 || d.kw < 1 || d.stride < 1 || d.pad < 0) return RRM_ERR_SHAPE;
    if (d.kind == RRM_FC && (d.h != 1 || d.w != 1 || d.kh != 1 || d.kw != 1 || d.stride != 1 || d.pad != 0))
        return RRM_ERR_SHAPE;
    if (d.h + 2 * d.pad < d.kh || d.w + 2 * d.pad < d.kw) return RRM_ERR_SHAPE;
    if (d.pad >= d.kh || d.pad >= d.kw) return RRM_ERR_SHAPE;
    if (d.act != RRM_ACT_NONE && d.act != RRM_ACT_RELU && d.act != RRM_ACT_SIGN && d.act != RRM_ACT_LEAKY) return RRM_ERR_INVALID_ARG;
    if (d.act == RRM_ACT_LEAKY && d.dtype != RRM_F32) return RRM_ERR_UNSUPPORTED;
    if (d.dtype == RRM_F32 && d.act == RRM_ACT_SIGN) return RRM_ERR_UNSUPPORTED;
    if (d.dtype != RRM_F32 && d.shift < 0 && d.act == RRM_ACT_RELU) return RRM_ERR_UNSUPPORTED;
    if (d.shift > 30) return RRM_ERR_INVALID_ARG;
    if (d.pool_k < 0 || (d.pool_k > 0 && (d.pool_s < 1 || d.pool_p < 0 || d.pool_p >= d.pool_k))) return RRM_ERR_SHAPE;
    if (d.pool_k > 3) return RRM_ERR_UNSUPPORTED;
    if (d.src < 0 || d.src > l) return RRM_ERR_INVALID_ARG;
    if (d.res > l) return RRM_ERR_INVALID_ARG;
    if (d.res >= 0 && (d.pool_k > 0 || d.act == RRM_ACT_SIGN)) return RRM_ERR_UNSUPPORTED;
    if (d.res >= 0 && d.dtype != RRM_F32 && d.shift < 0) return RRM_ERR_UNSUPPORTED;
    if (d.variant < RRM_VARIANT_AUTO || d.variant > RRM_VARIANT_SPARSE_W) return RRM_ERR_INVALID_ARG;
    if (d.variant == RRM_VARIANT_SPARSE_W && (n_layers != 1 || d.kind != RRM_FC || d.dtype != RRM_I8)) return RRM_ERR_UNSUPPORTED;
    (void)n_layers;
    return RRM_OK;
}

// Frees a buffer that a larger one is about to replace (the caller has made sure nothing uses it any more).
void dev_release(rrm_net* net, void** p)
{
    if (!*p) return;
    for (size_t i = 0; i < net->allocs.size(); ++i)
        if (net->allocs[i] == *p) { net->allocs.erase(net->allocs.begin() + i); break; }
    cudaFree(*p);
    *p = nullptr;
}

int dev_alloc(rrm_net* net, void** p, size_t bytes)
{
    if (bytes == 0) bytes = 16;
    if (cudaMalloc(p, bytes) != cudaSuccess) { *p = nullptr; cudaGetLastError(); return RRM_ERR_ALLOC; }
    net->allocs.push_back(*p);
    if (cudaMemset(*p, 0, bytes) != cudaSuccess) return RRM_ERR_CUDA;
    return RRM_OK;
}

void set_tensor(Tensor& T, int dtype, int n, int c, int h, int w)
{
    T.dtype = dtype; T.n = n; T.c = c; T.h = h; T.w = w;
    // int8 rows are padded to whole 32-byte K chunks of the tensor-core path (tiny channel counts: to 4)
    if (dtype == T_I8) { T.cs = c <= 4 ? 4 : round_up(c, 32); T.unit_bytes = 1; }
    else if (dtype == T_BIN) { T.cs = ceil_div(c, 32); T.unit_bytes = 4; }
    else { T.cs = c; T.unit_bytes = 4; }
}

// Points every activity bitmap and per-step counter at an arena (one memset clears it): tensors' activity bitmaps,
// layers' update bitmaps, then the counters.  A net has one arena for frame-by-frame stepping and, for pipelined
// chunks of frames, one per frame in flight.
void bind_arena(rrm_net* net, char* base)
{
    size_t off = 0;
    for (auto& T : net->tensors) { T.act = reinterpret_cast<uint32_t*>(base + off); off += (size_t)T.act_words() * 4; }
    for (auto& L : net->layers) { L.oact = reinterpret_cast<uint32_t*>(base + off); L.oact_off = off; off += (size_t)ceil_div(L.opixels(), 32) * 4; }
    off = net->counters_off;
    for (auto& T : net->tensors) {
        T.nnz = reinterpret_cast<unsigned long long*>(base + off);
        T.npix = reinterpret_cast<unsigned long long*>(base + off + 8);
        T.trunc = reinterpret_cast<double*>(base + off + 16);
        off += 32;
    }
    for (auto& L : net->layers) {
        L.macs = reinterpret_cast<unsigned long long*>(base + off);
        L.ocount = reinterpret_cast<int*>(base + off + 8);
        off += 16;
    }
    net->bound_arena = base;
}

// Who reads which tensor: as input (filter footprint) or as shortcut (1x1).  The entries hold arena pointers, so
// this follows every bind_arena.
int bind_readers(rrm_net* net)
{
    for (auto& T : net->tensors) T.readers.n = 0;
    for (auto& L : net->layers) {
        const rrm_layer_desc& d = L.d;
        auto add = [&](int t, Reader r) -> int {
            Readers& R = net->tensors[t].readers;
            if (R.n >= MAX_READERS) return RRM_ERR_UNSUPPORTED;
            R.r[R.n++] = r;
            return RRM_OK;
        };
        RRM_TRY(add(d.src, Reader{L.oact, L.oh, L.ow, d.kh, d.kw, d.stride, d.pad, d.c_out, L.macs}));
        if (d.res >= 0) RRM_TRY(add(d.res, Reader{L.oact, L.oh, L.ow, 1, 1, 1, 0, d.c_out, nullptr}));
    }
    return RRM_OK;
}

int build_net(rrm_net* net, const rrm_layer_desc* descs, int n_layers, const void* const* W, const void* const* B)
{
    const int n = descs[0].n;
    net->n = n;
    net->tensors.resize(n_layers + 1);
    net->layers.resize(n_layers);
    {
        const rrm_layer_desc& d0 = descs[0];
        if (d0.src != 0) return RRM_ERR_INVALID_ARG;
        set_tensor(net->tensors[0], d0.dtype == RRM_F32 ? T_F32 : (d0.dtype == RRM_I8 ? T_I8 : T_BIN), n, d0.c_in, d0.h, d0.w);
    }
    for (int l = 0; l < n_layers; ++l) {
        const rrm_layer_desc& d = descs[l];
        RRM_TRY(validate_desc(d, l, n_layers));
        if (d.n != n) return RRM_ERR_SHAPE;
        if (!W[l]) return RRM_ERR_INVALID_ARG;
        Layer& L = net->layers[l];
        L.d = d;
        L.oh = (d.h + 2 * d.pad - d.kh) / d.stride + 1;
        L.ow = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
        L.th = L.oh; L.tw = L.ow;
        if (d.pool_k > 0) {
            if (L.oh + 2 * d.pool_p < d.pool_k || L.ow + 2 * d.pool_p < d.pool_k) return RRM_ERR_SHAPE;
            L.th = (L.oh + 2 * d.pool_p - d.pool_k) / d.pool_s + 1;
            L.tw = (L.ow + 2 * d.pool_p - d.pool_k) / d.pool_s + 1;
        }
        const Tensor& in = net->tensors[d.src];
        const int want = d.dtype == RRM_F32 ? T_F32 : (d.dtype == RRM_I8 ? T_I8 : T_BIN);
        if (in.dtype != want) return RRM_ERR_DTYPE;
        if (in.c != d.c_in || in.h != d.h || in.w != d.w) return RRM_ERR_SHAPE;
        int ot;
        if (d.dtype == RRM_F32) ot = T_F32;
        else if (d.act == RRM_ACT_SIGN) ot = T_BIN;
        else if (d.shift >= 0) ot = T_I8;
        else ot = T_I32;
        set_tensor(net->tensors[l + 1], ot, n, d.c_out, L.th, L.tw);
        if (d.res >= 0) {
            const Tensor& r = net->tensors[d.res];
            if (r.dtype != ot || r.c != d.c_out || r.h != L.th || r.w != L.tw) return RRM_ERR_SHAPE;
        }
        if ((long long)n * L.oh * L.ow * (long long)d.c_out > (1ll << 31) - 1) return RRM_ERR_CAPACITY;
        if ((long long)n * d.h * d.w * (long long)in.cs > (1ll << 31) - 1) return RRM_ERR_CAPACITY;
    }
    // the fused FC kernel serves a lone int8 FC layer that reads the external input
    bool fused = false;
    if (n_layers == 1 && descs[0].kind == RRM_FC && descs[0].dtype == RRM_I8 && descs[0].pool_k == 0 &&
        descs[0].act != RRM_ACT_SIGN && descs[0].variant != RRM_VARIANT_DENSE) {
        const int s = fc_fused_create(net, net->layers[0], W[0], B ? B[0] : nullptr);
        if (s == RRM_OK) fused = true;
        else if (s != RRM_ERR_UNSUPPORTED) return s;
    }
    RRM_TRY(dev_alloc(net, (void**)&net->errw, 16));
    if (fused) return RRM_OK;
    if (descs[0].variant == RRM_VARIANT_SPARSE_W) return RRM_ERR_UNSUPPORTED;   // (shapes the fused FC path does not take)
    // the import kernel turns 32 pixels x all channels of the frame around in shared memory
    if (net->tensors[0].dtype != T_BIN && net->tensors[0].cs != 4 &&
        (size_t)32 * (net->tensors[0].cs + 1) * net->tensors[0].unit_bytes > 200 * 1024) return RRM_ERR_UNSUPPORTED;

    // tensors
    size_t cleared = 0;
    for (auto& T : net->tensors) {
        RRM_TRY(dev_alloc(net, &T.X, T.bytes()));
        RRM_TRY(dev_alloc(net, &T.D, T.bytes()));
        RRM_TRY(dev_alloc(net, (void**)&T.pnnz, (size_t)T.pixels() * 4));
        cleared += (size_t)T.act_words() * 4;
    }
    for (auto& L : net->layers) cleared += (size_t)ceil_div(L.opixels(), 32) * 4;
    cleared = (cleared + 15) & ~(size_t)15;
    const size_t counters_off = cleared;
    net->counters_off = counters_off;
    net->counters_bytes = net->tensors.size() * 32 + net->layers.size() * 16;
    cleared += net->tensors.size() * 32 + net->layers.size() * 16;
    RRM_TRY(dev_alloc(net, &net->cleared, cleared));
    net->cleared_bytes = cleared;
    bind_arena(net, reinterpret_cast<char*>(net->cleared));
    RRM_TRY(dev_alloc(net, (void**)&net->aecs, (size_t)(1 + n_layers) * 8));
    for (int l = 0; l < n_layers; ++l) RRM_TRY(conv_layer_create(net, net->layers[l], W[l], B ? B[l] : nullptr));
    {
        // dense evaluation of high-activity frames: only where a frame is real work (>= 1 GMAC), so that the
        // per-layer counters stay available on small stacks, and only if no layer pins its variant
        long long macs = 0;
        bool all_auto = true;
        for (auto& L : net->layers) {
            macs += (long long)L.opixels() * L.d.c_out * L.d.c_in * L.d.kh * L.d.kw;
            all_auto = all_auto && L.d.variant == RRM_VARIANT_AUTO;
        }
        net->auto_switch = all_auto && macs >= 1000000000ll;
        net->layer_switch = all_auto && n_layers <= 64;
        {
            bool all_tc = true;
            for (auto& L : net->layers) all_tc = all_tc && L.tc_ready;
            net->chunk_switch = all_auto && all_tc && n_layers <= 64;
        }
        // an all-ones bitmap stands in for a layer's update bitmap when the layer is evaluated densely inside a delta step
        int words = 1;
        for (auto& L : net->layers) words = words > ceil_div(L.opixels(), 32) ? words : ceil_div(L.opixels(), 32);
        RRM_TRY(dev_alloc(net, (void**)&net->ones, (size_t)words * 4));
        RRM_CUDA_TRY(cudaMemset(net->ones, 0xff, (size_t)words * 4));
        RRM_TRY(dev_alloc(net, (void**)&net->zeros, (size_t)words * 4));
    }
    {
        const char* e = getenv("RRM_NO_GRAPH");
        net->graph_off = e && e[0] == '1';
        e = getenv("RRM_CHUNK_INPLACE");
        net->chunk_in_place = e && e[0] == '1';
        e = getenv("RRM_CHUNK_PIPELINED");
        net->chunk_pipelined = e && e[0] == '1';
        e = getenv("RRM_CHUNK_BY_LAYER");
        net->chunk_by_layer = e && e[0] == '1';
    }
    for (auto& L : net->layers) net->tensors[L.d.src].has_consumer = true;
    RRM_TRY(bind_readers(net));
    RRM_TRY(reset_state(net, nullptr));
    RRM_CUDA_TRY(cudaDeviceSynchronize());
    return RRM_OK;
}

int launch_sequence(rrm_net* net, const void* frame, void* out, cudaStream_t st, bool dense, bool stateless,
                    unsigned long long mask = 0);
int run_sequence(rrm_net* net, const void* frame, void* out, cudaStream_t st, bool dense, bool stateless,
                 unsigned long long mask = 0);

// Finds the nodes of a captured sequence that hold the fixed frame / output buffers, so that each launch can
// point them at the caller's buffers instead of copying through the fixed ones.  Any doubt (an API error, no
// node found) leaves patch_ok false and the copies in place.
void find_io_nodes(rrm_net* net, rrm_net::StepGraph& sg)
{
    sg.patch_in.clear(); sg.patch_out.clear(); sg.patch_ok = false;
    size_t n = 0;
    if (cudaGraphGetNodes(sg.graph, nullptr, &n) != cudaSuccess || n == 0) { cudaGetLastError(); return; }
    std::vector<cudaGraphNode_t> nodes(n);
    if (cudaGraphGetNodes(sg.graph, nodes.data(), &n) != cudaSuccess) { cudaGetLastError(); return; }
    for (cudaGraphNode_t node : nodes) {
        cudaGraphNodeType type;
        if (cudaGraphNodeGetType(node, &type) != cudaSuccess) { cudaGetLastError(); return; }
        if (type == cudaGraphNodeTypeKernel) {
            cudaKernelNodeParams kp = {};
            if (cudaGraphKernelNodeGetParams(node, &kp) != cudaSuccess || !kp.kernelParams) { cudaGetLastError(); return; }
            // the kernel's arguments: count and sizes from the function itself
            std::vector<void*> args;
            for (size_t i = 0;; ++i) {
                size_t off = 0, size = 0;
                if (cudaFuncGetParamInfo(kp.func, i, &off, &size) != cudaSuccess) { cudaGetLastError(); break; }
                args.push_back(kp.kernelParams[i]);
            }
            for (size_t i = 0; i < args.size(); ++i) {
                size_t off = 0, size = 0;
                cudaFuncGetParamInfo(kp.func, i, &off, &size);
                if (size != sizeof(void*)) continue;
                void* v = *reinterpret_cast<void* const*>(kp.kernelParams[i]);
                if (v != net->frame_buf && v != net->out_buf) continue;
                rrm_net::IoPatch pt;
                pt.node = node; pt.kp = kp; pt.args = args; pt.index = (int)i;
                (v == net->frame_buf ? sg.patch_in : sg.patch_out).push_back(pt);
            }
        } else if (type == cudaGraphNodeTypeMemcpy) {
            cudaMemcpy3DParms mp = {};
            if (cudaGraphMemcpyNodeGetParams(node, &mp) != cudaSuccess) { cudaGetLastError(); return; }
            if (mp.dstPtr.ptr == net->out_buf && mp.extent.height <= 1 && mp.extent.depth <= 1) {
                rrm_net::IoPatch pt;
                pt.node = node; pt.is_copy = true; pt.src = mp.srcPtr.ptr; pt.bytes = mp.extent.width;
                sg.patch_out.push_back(pt);
            } else if (mp.dstPtr.ptr == net->out_buf || mp.srcPtr.ptr == net->frame_buf) {
                return;                                      // a copy of another shape: leave everything as it is
            }
        }
    }
    sg.patch_ok = sg.patch_in.size() == 1 && sg.patch_out.size() == 1;
}

// Points the frame / output nodes of the instantiated graph at `frame` and `out`.
int patch_io(rrm_net* net, rrm_net::StepGraph& sg, const void* frame, void* out)
{
    for (int side = 0; side < 2; ++side) {
        rrm_net::IoPatch& pt = side == 0 ? sg.patch_in[0] : sg.patch_out[0];
        void* target = side == 0 ? const_cast<void*>(frame) : (out ? out : net->out_buf);
        if (pt.value == target) continue;                    // already there
        if (pt.is_copy) {
            RRM_CUDA_TRY(cudaGraphExecMemcpyNodeSetParams1D(sg.exec, pt.node, target, pt.src, pt.bytes,
                                                            cudaMemcpyDeviceToDevice));
        } else {
            pt.value = target;
            pt.args[pt.index] = &pt.value;
            pt.kp.kernelParams = pt.args.data();
            RRM_CUDA_TRY(cudaGraphExecKernelNodeSetParams(sg.exec, pt.node, &pt.kp));
        }
        pt.value = target;
    }
    return RRM_OK;
}

// Captures one of the per-frame launch sequences into a graph (on a private stream: a capture cannot
// start on the legacy default stream) so that later frames cost one graph launch on the host.
constexpr size_t STEP_GRAPHS_KEPT = 12;         // layer masks whose delta-step graphs are kept

rrm_net::StepGraph* find_step_graph(rrm_net* net, int kind, unsigned long long mask)
{
    for (auto& g : net->step_graphs[kind]) if (g.mask == mask) return &g;
    return nullptr;
}

int build_graph(rrm_net* net, int kind, unsigned long long mask)
{
    const bool dense = kind != 0, stateless = kind == 2;
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    if (!net->frame_buf) RRM_TRY(dev_alloc(net, &net->frame_buf, (size_t)bi));
    if (!net->out_buf) RRM_TRY(dev_alloc(net, &net->out_buf, (size_t)bo));
    if (stateless) RRM_TRY(ensure_stateless(net));           // allocations cannot happen inside a capture
    if (!net->cap_stream) RRM_CUDA_TRY(cudaStreamCreateWithFlags(&net->cap_stream, cudaStreamNonBlocking));
    RRM_CUDA_TRY(cudaStreamBeginCapture(net->cap_stream, cudaStreamCaptureModeThreadLocal));
    const int s = launch_sequence(net, net->frame_buf, net->out_buf, net->cap_stream, dense, stateless, mask);
    cudaGraph_t g = nullptr;
    const cudaError_t e = cudaStreamEndCapture(net->cap_stream, &g);
    if (s != RRM_OK || e != cudaSuccess || !g) { if (g) cudaGraphDestroy(g); cudaGetLastError(); return s != RRM_OK ? s : RRM_ERR_CUDA; }
    auto& cache = net->step_graphs[kind];
    if (cache.size() >= STEP_GRAPHS_KEPT) {                  // drop the mask that has not been used for the longest time
        size_t old = 0;
        for (size_t i = 1; i < cache.size(); ++i) if (cache[i].used < cache[old].used) old = i;
        if (cache[old].exec) cudaGraphExecDestroy(cache[old].exec);
        if (cache[old].graph) cudaGraphDestroy(cache[old].graph);
        cache.erase(cache.begin() + old);
    }
    rrm_net::StepGraph sg;
    sg.mask = mask; sg.graph = g;
    if (cudaGraphInstantiate(&sg.exec, g, 0) != cudaSuccess) { cudaGraphDestroy(g); cudaGetLastError(); return RRM_ERR_CUDA; }
    find_io_nodes(net, sg);
    cache.push_back(std::move(sg));
    return RRM_OK;
}

void drop_chunk_graphs(rrm_net* net, int kind)
{
    for (auto& c : net->chunk_graphs[kind]) {
        if (c.exec) cudaGraphExecDestroy(c.exec);
        if (c.graph) cudaGraphDestroy(c.graph);
    }
    net->chunk_graphs[kind].clear();
}

void drop_graphs(rrm_net* net)
{
    for (int k = 0; k < 3; ++k) {
        drop_chunk_graphs(net, k);
        for (auto& g : net->step_graphs[k]) {
            if (g.exec) cudaGraphExecDestroy(g.exec);
            if (g.graph) cudaGraphDestroy(g.graph);
        }
        net->step_graphs[k].clear();
    }
}


// Copies the step's counters to pinned memory behind the work on the stream (never waited for).
int activity_read_back(rrm_net* net, cudaStream_t st)
{
    if (net->act_pending) return RRM_OK;
    if (!net->act_host && cudaMallocHost(reinterpret_cast<void**>(&net->act_host), net->counters_bytes) != cudaSuccess) { cudaGetLastError(); return RRM_OK; }
    if (!net->act_ev && cudaEventCreateWithFlags(&net->act_ev, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return RRM_OK; }
    RRM_CUDA_TRY(cudaMemcpyAsync(net->act_host, net->bound_arena + net->counters_off, net->counters_bytes,
                                 cudaMemcpyDeviceToHost, st));
    RRM_CUDA_TRY(cudaEventRecord(net->act_ev, st));
    net->act_pending = true;
    return RRM_OK;
}

// Takes in the counters of the last measured delta step, once their copy has landed (never waited for): the
// MAC-weighted activity of the stack, and per layer the share of projection pixels it had to update, from which
// the layer's mode in the following steps is chosen (with a hysteresis between the two thresholds).
void activity_poll(rrm_net* net)
{
    if (!net->act_pending || cudaEventQuery(net->act_ev) != cudaSuccess) { cudaGetLastError(); return; }
    net->act_pending = false;
    double num = 0, den = 0;
    const size_t base = net->tensors.size() * 32;
    unsigned long long mask = 0;
    for (size_t l = 0; l < net->layers.size(); ++l) {
        Layer& L = net->layers[l];
        int oc = 0;
        std::memcpy(&oc, net->act_host + base + l * 16 + 8, 4);
        const double macs = (double)L.opixels() * L.d.c_out * L.d.c_in * L.d.kh * L.d.kw;
        L.activity = oc / (double)L.opixels();
        num += macs * L.activity;
        den += macs;
        if (L.activity >= net->opt.layer_dense_activity) L.dense_mode = true;
        else if (L.activity < net->opt.layer_delta_activity) L.dense_mode = false;
        if (L.dense_mode && l < 64) mask |= 1ull << l;
    }
    net->activity = den > 0 ? num / den : -1.0;
    net->layer_mask = net->layer_switch ? mask : 0;
}

int run(rrm_net* net, const void* frame, void* out, cudaStream_t st, bool dense, bool stateless)
{
    if (!net || !frame) return RRM_ERR_INVALID_ARG;
    net->last_stream = st;
    if (net->layers[0].fc_fused) {
        // (the weight-sparse form lives in the chunk kernel: a single frame is a chunk of one)
        if (net->layers[0].Wsp) return fc_seq_run(net, net->layers[0], frame, out, 1, dense, stateless, st);
        return fc_fused_run(net, net->layers[0], frame, out, dense, stateless, st);
    }
    if (net->bound_arena != reinterpret_cast<char*>(net->cleared)) {    // a pipelined chunk left another arena bound
        bind_arena(net, reinterpret_cast<char*>(net->cleared));
        RRM_TRY(bind_readers(net));
    }
    const bool is_step = !dense && !stateless;
    unsigned long long mask = 0;
    if (is_step) {
        // how this frame is evaluated follows from the measured activity of the last delta frame (temporal
        // coherence).  A whole stack of >= 1 GMAC with nearly every pixel changing is evaluated densely (a precise
        // inference that replaces the state: the same results, and no delta bookkeeping at all); otherwise every
        // layer on its own runs the sparse product or, above its threshold, a dense evaluation inside the delta step.
        net->last_step_dense = false;
        if ((net->auto_switch || net->layer_switch) && net->eps == 0.f) {
            activity_poll(net);
            if (net->auto_switch && net->activity >= net->opt.stack_dense_activity && net->dense_streak < net->opt.stack_reprobe) {
                ++net->dense_streak;
                net->last_step_dense = true;
                dense = true;
            } else {
                net->dense_streak = 0;
                mask = net->layer_mask;
            }
        }
        if (!dense) for (size_t l = 0; l < net->layers.size(); ++l) net->layers[l].ran_dense = l < 64 && (mask >> l & 1ull);
    }
    const int s_run = run_sequence(net, frame, out, st, dense, stateless, mask);
    if (s_run == RRM_OK && is_step && !dense && (net->auto_switch || net->layer_switch) && net->eps == 0.f)
        RRM_TRY(activity_read_back(net, st));
    return s_run;
}

int run_sequence(rrm_net* net, const void* frame, void* out, cudaStream_t st, bool dense, bool stateless,
                 unsigned long long mask)
{
    if (!net->graph_off) {
        const int kind = !dense ? 0 : (stateless ? 2 : 1);
        if (!find_step_graph(net, kind, mask)) {
            const int s = build_graph(net, kind, mask);
            if (s != RRM_OK) { net->graph_off = true; if (s == RRM_ERR_ALLOC) return s; }
        }
        if (rrm_net::StepGraph* sg = find_step_graph(net, kind, mask)) {
            sg->used = ++net->step_clock;
            int64_t bi = 0, bo = 0;
            tensor_bytes_boundary(net->tensors.front(), &bi);
            tensor_bytes_boundary(net->tensors.back(), &bo);
            if (sg->patch_ok && patch_io(net, *sg, frame, out) == RRM_OK) {
                RRM_CUDA_TRY(cudaGraphLaunch(sg->exec, st));
                return RRM_OK;
            }
            if (sg->patch_ok) {
                // an update failed half-way: the graphs are no longer trusted, launch kernel by kernel from now on
                cudaGetLastError();
                drop_graphs(net);
                net->graph_off = true;
                return launch_sequence(net, frame, out, st, dense, stateless, mask);
            }
            RRM_CUDA_TRY(cudaMemcpyAsync(net->frame_buf, frame, (size_t)bi, cudaMemcpyDeviceToDevice, st));
            RRM_CUDA_TRY(cudaGraphLaunch(sg->exec, st));
            if (out) RRM_CUDA_TRY(cudaMemcpyAsync(out, net->out_buf, (size_t)bo, cudaMemcpyDeviceToDevice, st));
            return RRM_OK;
        }
    }
    return launch_sequence(net, frame, out, st, dense, stateless, mask);
}

int launch_sequence(rrm_net* net, const void* frame, void* out, cudaStream_t st, bool dense, bool stateless,
                    unsigned long long mask)
{
    if (!stateless) RRM_CUDA_TRY(cudaMemsetAsync(net->cleared, 0, net->cleared_bytes, st));
    RRM_TRY(launch_import(net, frame, !dense, stateless, st));
    for (int l = 0; l < (int)net->layers.size(); ++l)
        RRM_TRY(launch_layer(net, l, dense, stateless, st, nullptr, !dense && l < 64 && (mask >> l & 1ull)));
    if (!dense && net->eps > 0.f) RRM_TRY(launch_aecs(net, st));
    if (dense && !stateless) RRM_CUDA_TRY(cudaMemsetAsync(net->aecs, 0, (1 + net->layers.size()) * 8, st));   // a precise inference clears e_t
    if (out) RRM_TRY(launch_export_tensor(net, (int)net->layers.size(), out, stateless, st));
    return RRM_OK;
}

constexpr int CHUNK_MAX_SLOTS = 24;             // capture streams = frames in flight
constexpr size_t CHUNK_GRAPHS_KEPT = 8;         // (chunk length, layer mask) pairs whose graphs are kept per kind
constexpr int CHUNK_ARENAS = 64;                // arenas of the chunk graphs (>= CHUNK_MAX_SLOTS)

// Streams, events, arenas and staging buffers of the pipelined chunk graphs.
int ensure_chunk(rrm_net* net, int T)
{
    const int L = (int)net->layers.size();
    // (a frame is ~2 L + 2 launches long and, with the split projection, a new one can start every one or two of them)
    int slots = 2 * L + 2 < CHUNK_MAX_SLOTS ? 2 * L + 2 : CHUNK_MAX_SLOTS;
    if (net->chunk_arena.empty()) {
        if (!net->cap_stream) RRM_CUDA_TRY(cudaStreamCreateWithFlags(&net->cap_stream, cudaStreamNonBlocking));
        // one block of CHUNK_ARENAS arenas: a chunk of up to that many frames gives every frame its own and clears
        // them all with one memset; longer chunks reuse `slots` of them, each cleared by the frame that takes it
        void* block = nullptr;
        RRM_TRY(dev_alloc(net, &block, net->cleared_bytes * CHUNK_ARENAS));
        for (int a = 0; a < CHUNK_ARENAS; ++a) net->chunk_arena.push_back(reinterpret_cast<char*>(block) + (size_t)a * net->cleared_bytes);
        while ((int)net->chunk_streams.size() < slots) {
            cudaStream_t s = net->cap_stream;
            if (!net->chunk_streams.empty()) RRM_CUDA_TRY(cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking));
            net->chunk_streams.push_back(s);
            cudaEvent_t e = nullptr;
            RRM_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
            net->ev_join.push_back(e);
        }
        auto make = [&](cudaEvent_t* e) -> int { RRM_CUDA_TRY(cudaEventCreateWithFlags(e, cudaEventDisableTiming)); return RRM_OK; };
        net->ev_conv.resize(CHUNK_RING * L); net->ev_epi.resize(CHUNK_RING * L);
        for (int l = 0; l < CHUNK_RING * L; ++l) { RRM_TRY(make(&net->ev_conv[l])); RRM_TRY(make(&net->ev_epi[l])); }
        RRM_TRY(make(&net->ev_fork)); RRM_TRY(make(&net->ev_export)); RRM_TRY(make(&net->ev_import));
    }
    if (T > net->chunk_cap) {
        int64_t bi = 0, bo = 0;
        tensor_bytes_boundary(net->tensors.front(), &bi);
        tensor_bytes_boundary(net->tensors.back(), &bo);
        RRM_CUDA_TRY(cudaDeviceSynchronize());               // the old buffers may be in use by a graph in flight
        for (int k = 0; k < 3; ++k) drop_chunk_graphs(net, k);   // graphs hold the old buffers
        dev_release(net, &net->chunk_in_raw);
        dev_release(net, &net->chunk_out);
        {
            // room for one frame in front of the chunk (the layer-by-layer form compares frame 0 with it), aligned
            const size_t front = ((size_t)bi + 255) & ~(size_t)255;
            RRM_TRY(dev_alloc(net, &net->chunk_in_raw, front + (size_t)bi * T));
            net->chunk_in = reinterpret_cast<char*>(net->chunk_in_raw) + front;
        }
        RRM_TRY(dev_alloc(net, &net->chunk_out, (size_t)bo * T));
        net->chunk_cap = T;
    }
    return RRM_OK;
}

// Inserts a captured chunk graph into the cache of its kind (the few most recently used are kept).
static int keep_chunk_graph(rrm_net* net, int kind, int T, unsigned long long mask, cudaGraph_t g, int last_arena)
{
    auto& cache = net->chunk_graphs[kind];
    if (cache.size() >= CHUNK_GRAPHS_KEPT) {
        size_t old = 0;
        for (size_t i = 1; i < cache.size(); ++i) if (cache[i].used < cache[old].used) old = i;
        if (cache[old].exec) cudaGraphExecDestroy(cache[old].exec);
        if (cache[old].graph) cudaGraphDestroy(cache[old].graph);
        cache.erase(cache.begin() + old);
    }
    rrm_net::ChunkGraph c;
    c.T = T; c.mask = mask; c.graph = g; c.last_arena = last_arena;
    if (cudaGraphInstantiate(&c.exec, g, 0) != cudaSuccess) { cudaGraphDestroy(g); cudaGetLastError(); return RRM_ERR_CUDA; }
    c.used = ++net->chunk_clock;
    cache.push_back(c);
    return RRM_OK;
}

// A delta chunk layer by layer: every kernel takes all frames of the chunk (at most seq_max_frames() per launch; a
// longer chunk goes in equal parts one after the other).  2 L + 5 launches per part, no frame-to-frame edges.
// RRM_ERR_UNSUPPORTED: the stack would need too much memory or adds its input as a shortcut (the frame-pipelined graph serves it).
static int build_seq_graph(rrm_net* net, int T)
{
    const int L = (int)net->layers.size();
    RRM_TRY(ensure_chunk(net, T));
    RRM_TRY(ensure_frame_batch(net));
    const int parts = ceil_div(T, seq_max_frames()), per = ceil_div(T, parts);       // (T >= 2: every part holds >= 2 frames)
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    const long long stride = (long long)net->cleared_bytes;
    cudaStream_t st = net->cap_stream;
    std::vector<void*> keep_D;
    for (auto& X : net->tensors) keep_D.push_back(X.D);
    int status = RRM_OK, last_arena = 0;
    auto fail = [&](int s) { if (status == RRM_OK && s != RRM_OK) status = s; };
    RRM_CUDA_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
    for (int m0 = 0; m0 < T && status == RRM_OK; m0 += per) {
        const int F = T - m0 < per ? T - m0 : per;
        if (cudaMemsetAsync(net->chunk_arena[0], 0, net->cleared_bytes * F, st) != cudaSuccess) fail(RRM_ERR_CUDA);
        fail(launch_copy_projections(net, st));              // the epilogues read the projections from the copies and write the stored ones
        for (auto& X : net->tensors)                         // a shortcut's reader needs the value before the chunk
            if (X.shortcut_source && cudaMemcpyAsync(X.Xbefore, X.X, X.bytes(), cudaMemcpyDeviceToDevice, st) != cudaSuccess) fail(RRM_ERR_CUDA);
        bind_arena(net, net->chunk_arena[0]);
        if (bind_readers(net) != RRM_OK) { fail(RRM_ERR_UNSUPPORTED); break; }
        for (auto& X : net->tensors) { X.D = X.Dall; X.Xn_cur = X.Xnall; }
        char* in0 = reinterpret_cast<char*>(net->chunk_in) + (size_t)m0 * bi;
        if (m0 == 0) fail(launch_export_tensor(net, 0, in0 - bi, false, st));        // the frame before the chunk = the input's snapshot
        fail(launch_import(net, in0, true, false, st, F, stride));
        for (int l = 0; l < L && status == RRM_OK; ++l) fail(launch_layer_seq(net, l, F, stride, st));
        fail(launch_export_seq(net, F, reinterpret_cast<char*>(net->chunk_out) + (size_t)m0 * bo, st));
        last_arena = F - 1;
    }
    for (size_t i = 0; i < net->tensors.size(); ++i) { net->tensors[i].D = keep_D[i]; net->tensors[i].Xn_cur = nullptr; }
    cudaGraph_t g = nullptr;
    const cudaError_t e = cudaStreamEndCapture(st, &g);
    if (status != RRM_OK || e != cudaSuccess || !g) {
        if (g) cudaGraphDestroy(g);
        cudaGetLastError();
        return status != RRM_OK ? status : RRM_ERR_CUDA;
    }
    RRM_TRY(keep_chunk_graph(net, 0, T, 0, g, last_arena));
    if (getenv("RRM_DEBUG")) {
        size_t nodes = 0;
        cudaGraphGetNodes(g, nullptr, &nodes);
        fprintf(stderr, "rrm: chunk graph (delta, %d frames, layer by layer): %zu nodes, %d part(s)\n", T, nodes, parts);
    }
    return RRM_OK;
}

// A dense chunk batched over its frames.  The frames of a dense chunk are independent, and T frames of n streams at
// the boundary are laid out exactly like one frame of n*T streams: every kernel of the stateless dense pass is launched
// once for up to DENSE_BATCH frames, on buffers of that size.  kind 1 (the state becomes the last frame) adds one
// stateful dense pass of the last frame.  RRM_ERR_UNSUPPORTED: too large (the frame-pipelined graph serves it).
constexpr int DENSE_BATCH = 32;

static int ensure_dense_batch(rrm_net* net)
{
    if (net->dense_batch_ready) return RRM_OK;
    size_t need = 0;
    for (auto& X : net->tensors) {
        if ((long long)X.pixels() * DENSE_BATCH * (long long)X.cs > (1ll << 31) - 1) return RRM_ERR_UNSUPPORTED;
        need += X.bytes() * DENSE_BATCH;
    }
    for (auto& Y : net->layers) {
        if ((long long)Y.opixels() * DENSE_BATCH * (long long)Y.d.c_out > (1ll << 31) - 1) return RRM_ERR_UNSUPPORTED;
        need += (size_t)Y.opixels() * Y.d.c_out * 4 * DENSE_BATCH;
    }
    if (need > ((size_t)8 << 30)) return RRM_ERR_UNSUPPORTED;
    for (auto& X : net->tensors) if (!X.X2b) RRM_TRY(dev_alloc(net, &X.X2b, X.bytes() * DENSE_BATCH));
    for (auto& Y : net->layers) if (!Y.P2b) RRM_TRY(dev_alloc(net, &Y.P2b, (size_t)Y.opixels() * Y.d.c_out * 4 * DENSE_BATCH));
    net->dense_batch_ready = true;
    return RRM_OK;
}

static int build_dense_batch_graph(rrm_net* net, int kind, int T)
{
    const int L = (int)net->layers.size();
    RRM_TRY(ensure_chunk(net, T));
    RRM_TRY(ensure_stateless(net));
    RRM_TRY(ensure_dense_batch(net));
    const int parts = ceil_div(T, DENSE_BATCH), per = ceil_div(T, parts);
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    cudaStream_t st = net->cap_stream;
    const int n0 = net->n;
    // the stack with F times as many streams, on the large buffers (restored below)
    auto scale = [&](int F) {
        net->n = n0 * F;
        for (auto& X : net->tensors) { X.n = n0 * F; std::swap(X.X2, X.X2b); }
        for (auto& Y : net->layers) { Y.d.n = n0 * F; std::swap(Y.P2, Y.P2b); }
    };
    auto unscale = [&]() {
        net->n = n0;
        for (auto& X : net->tensors) { X.n = n0; std::swap(X.X2, X.X2b); }
        for (auto& Y : net->layers) { Y.d.n = n0; std::swap(Y.P2, Y.P2b); }
    };
    int status = RRM_OK;
    auto fail = [&](int s) { if (status == RRM_OK && s != RRM_OK) status = s; };
    RRM_CUDA_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
    if (cudaMemsetAsync(net->chunk_arena[0], 0, net->cleared_bytes, st) != cudaSuccess) fail(RRM_ERR_CUDA);
    for (int m0 = 0; m0 < T && status == RRM_OK; m0 += per) {
        const int F = T - m0 < per ? T - m0 : per;
        scale(F);
        fail(launch_import(net, reinterpret_cast<const char*>(net->chunk_in) + (size_t)m0 * bi, false, true, st));
        for (int l = 0; l < L && status == RRM_OK; ++l) fail(launch_layer(net, l, true, true, st));
        fail(launch_export_tensor(net, L, reinterpret_cast<char*>(net->chunk_out) + (size_t)m0 * bo, true, st));
        unscale();
    }
    if (kind == 1 && status == RRM_OK) {
        // the state becomes the last frame (a precise inference: the accumulated truncation error is cleared): its
        // tensors and projections are copied out of the last part's batched buffers
        bind_arena(net, net->chunk_arena[0]);
        if (bind_readers(net) != RRM_OK) fail(RRM_ERR_UNSUPPORTED);
        const int last_part_frames = T - (parts - 1) * per;
        fail(launch_copy_state_from_batch(net, last_part_frames - 1, st));
        if (cudaMemsetAsync(net->aecs, 0, (1 + net->layers.size()) * 8, st) != cudaSuccess) fail(RRM_ERR_CUDA);
    }
    cudaGraph_t g = nullptr;
    const cudaError_t e = cudaStreamEndCapture(st, &g);
    if (status != RRM_OK || e != cudaSuccess || !g) {
        if (g) cudaGraphDestroy(g);
        cudaGetLastError();
        return status != RRM_OK ? status : RRM_ERR_CUDA;
    }
    RRM_TRY(keep_chunk_graph(net, kind, T, 0, g, 0));
    if (getenv("RRM_DEBUG")) {
        size_t nodes = 0;
        cudaGraphGetNodes(g, nullptr, &nodes);
        fprintf(stderr, "rrm: chunk graph (%s, %d frames, batched over the frames): %zu nodes, %d part(s)\n",
                kind == 1 ? "keyframes" : "dense", T, nodes, parts);
    }
    return RRM_OK;
}

// T frames as one graph.  Frame t is captured on stream t mod S with arena t mod S; inside a frame the launches
// follow each other on that stream.  Across frames, in the in-place form (keyframes, dense passes, delta chunks with
// a layer evaluated densely, RRM_CHUNK_INPLACE=1):
//   the convolution of layer l waits for the previous frame's epilogue of layer l (which reads the projection it adds to);
//   the producer of a tensor (the import for tensor 0, the epilogue of layer l for tensor l+1) waits for the previous
//   frame's readers of that tensor (convolutions that take it as input, epilogues that add it as shortcut, the export
//   of the last tensor), because it overwrites the snapshot and the delta rows they read.
// Delta chunks otherwise take the split form, which removes both waits from the frame-to-frame cycle (a layer then
// advances one frame per epilogue instead of one per convolution + epilogue):
//   the convolution of frame t adds its product into delta-projection buffer t mod R (R = CHUNK_RING) and waits only
//   for the epilogue of frame t-R+1, whose merge role zeroed that buffer; the epilogue evaluates f from (projection
//   as of t-1) + (the product), writes the merged rows to the other projection buffer and waits for the epilogue of
//   frame t-1;
//   delta rows (and the new rows of binary tensors) cycle through R sets, so a producer waits for the convolutions
//   of frame t-R that read its tensor, and for the previous frame's shortcut readers and export, which read the
//   snapshot it overwrites in place.
// Everything else of consecutive frames may overlap.
int build_chunk_graph(rrm_net* net, int kind, int T, unsigned long long mask)
{
    const bool dense = kind != 0, stateless = kind == 2;
    const int L = (int)net->layers.size();
    // Delta chunks go layer by layer over all frames where that pays: its epilogue gives every frame a lane of a warp, so
    // short chunks waste lanes, and with many streams per call the frame-pipelined graph's kernels are large enough by
    // themselves (measured on cfg1 and cfg3 int8, 1-8 streams x 8-32 frames: ahead from 16 frames on with up to 2
    // streams, from 32 frames on with up to 4)
    const int per_launch = T < seq_max_frames() ? T : seq_max_frames();
    const bool by_layer = net->chunk_by_layer || (per_launch >= 16 && net->n <= 2) || (per_launch >= 32 && net->n <= 4);
    if (kind == 0 && mask == 0 && !net->chunk_in_place && !net->chunk_pipelined && by_layer) {
        const int s = build_seq_graph(net, T);
        if (s != RRM_ERR_UNSUPPORTED && s != RRM_ERR_ALLOC) return s;
        cudaGetLastError();
    }
    if (kind != 0 && !net->chunk_pipelined) {
        const int s = build_dense_batch_graph(net, kind, T);
        if (s != RRM_ERR_UNSUPPORTED && s != RRM_ERR_ALLOC) return s;
        cudaGetLastError();
    }
    RRM_TRY(ensure_chunk(net, T));
    if (stateless) RRM_TRY(ensure_stateless(net));
    // (with many streams per call the merge work of the split form costs more than the overlap gains: measured level at 8
    // streams, behind at 16 on cfg3 int8)
    const bool split = kind == 0 && mask == 0 && !net->chunk_in_place && net->n <= 8;
    if (split) RRM_TRY(ensure_split(net));
    const int S = (int)net->chunk_streams.size() < T ? (int)net->chunk_streams.size() : T;
    const bool own_arena = T <= CHUNK_ARENAS;                // every frame has an arena of its own
    const int R = CHUNK_RING;
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    cudaStream_t origin = net->cap_stream;
    // [slot * L + l]: an event of that layer has been recorded for a frame of that ring slot (in-place form: slot 0 only)
    std::vector<char> conv_rec(R * L, 0), epi_rec(R * L, 0);
    bool export_rec = false, import_rec = false;
    int status = RRM_OK;
    RRM_CUDA_TRY(cudaStreamBeginCapture(origin, cudaStreamCaptureModeThreadLocal));
    net->many_in_flight = true;
    auto fail = [&](int s) { if (status == RRM_OK) status = s; };
    auto wait = [&](cudaStream_t s, cudaEvent_t e) { if (cudaStreamWaitEvent(s, e, 0) != cudaSuccess) fail(RRM_ERR_CUDA); };
    auto record = [&](cudaEvent_t e, cudaStream_t s) { if (cudaEventRecord(e, s) != cudaSuccess) fail(RRM_ERR_CUDA); };
    if (own_arena && !stateless && cudaMemsetAsync(net->chunk_arena[0], 0, net->cleared_bytes * T, origin) != cudaSuccess) fail(RRM_ERR_CUDA);
    // the second projection buffers start as copies of the stored projections; whichever buffer the first frame reads,
    // the last frame's merge lands in the stored one
    if (split) { const int q = launch_copy_projections(net, origin); if (q != RRM_OK) fail(q); }
    record(net->ev_fork, origin);
    for (int k = 1; k < S; ++k) wait(net->chunk_streams[k], net->ev_fork);
    // what the producer of tensor j waits for in a frame of ring slot `cur` (the previous frame has slot `prv`)
    auto wait_readers = [&](cudaStream_t s, int j, int cur, int prv) {
        for (int r = 0; r < L; ++r) {
            // (split form: slot `cur` still holds the events of frame t-R, whose convolutions read the set of delta
            // rows about to be overwritten)
            if (net->layers[r].d.src == j && conv_rec[cur * L + r]) wait(s, net->ev_conv[cur * L + r]);
            if (net->layers[r].d.res == j && epi_rec[prv * L + r]) wait(s, net->ev_epi[prv * L + r]);
        }
        if (j == L && export_rec) wait(s, net->ev_export);
    };
    for (int t = 0; t < T && status == RRM_OK; ++t) {
        cudaStream_t s = net->chunk_streams[t % S];
        const int cur = split ? t % R : 0, prv = split ? (t + R - 1) % R : 0, nxt = split ? (t + 1) % R : 0;
        char* const prev_arena = net->chunk_arena[own_arena ? (t > 0 ? t - 1 : 0) : (t + S - 1) % S];
        bind_arena(net, net->chunk_arena[own_arena ? t : t % S]);
        if (bind_readers(net) != RRM_OK) { fail(RRM_ERR_UNSUPPORTED); break; }
        if (!own_arena && !stateless) {
            // a reused arena: the frame that used it before ran on this same stream, so it is complete before the clear;
            // in the split form the frame after that one read its update bitmaps as well
            if (split && t >= S) wait(s, net->ev_join[(t + 1) % S]);
            if (cudaMemsetAsync(net->bound_arena, 0, net->cleared_bytes, s) != cudaSuccess) fail(RRM_ERR_CUDA);
        }
        if (split) for (auto& X : net->tensors) { X.D = X.Dring[cur]; X.Xn_cur = X.Xn[cur]; }
        wait_readers(s, 0, cur, prv);
        if (split && import_rec) wait(s, net->ev_import);        // (the import reads and overwrites the input's snapshot)
        { const int q = launch_import(net, reinterpret_cast<const char*>(net->chunk_in) + (size_t)t * bi, !dense, stateless, s); if (q != RRM_OK) fail(q); }
        if (split) { record(net->ev_import, s); import_rec = true; }
        for (int l = 0; l < L && status == RRM_OK; ++l) {
            Layer& Y = net->layers[l];
            SplitProjection sp{};
            if (split) {
                // frame T-1 writes the stored projection, the frames before it alternate
                const bool to_stored = ((T - 1 - t) & 1) == 0;
                sp.dP = Y.dP[cur];
                sp.R = to_stored ? Y.Palt : Y.P;
                sp.Q = to_stored ? Y.P : Y.Palt;
                sp.Z = Y.dP[prv];
                sp.prev_oact = t > 0 ? reinterpret_cast<const uint32_t*>(prev_arena + Y.oact_off) : net->zeros;
            }
            const std::function<int(int)> hook = [&, l, s](int phase) -> int {
                if (phase == 0) {
                    // split form: slot `nxt` holds the epilogue of frame t-R+1, whose merge role zeroed the buffer this product goes to
                    if (epi_rec[nxt * L + l]) wait(s, net->ev_epi[nxt * L + l]);
                } else if (phase == 1) {
                    record(net->ev_conv[cur * L + l], s); conv_rec[cur * L + l] = 1;
                    wait_readers(s, l + 1, cur, prv);
                    if (split && epi_rec[prv * L + l]) wait(s, net->ev_epi[prv * L + l]);   // frame t-1: projection buffers, the output's snapshot
                } else { record(net->ev_epi[cur * L + l], s); epi_rec[cur * L + l] = 1; }
                return status;
            };
            const int q = launch_layer(net, l, dense, stateless, s, &hook, !dense && l < 64 && (mask >> l & 1ull), split ? &sp : nullptr);
            if (q != RRM_OK) fail(q);
        }
        if (dense && !stateless && cudaMemsetAsync(net->aecs, 0, (1 + net->layers.size()) * 8, s) != cudaSuccess) fail(RRM_ERR_CUDA);
        { const int q = launch_export_tensor(net, L, reinterpret_cast<char*>(net->chunk_out) + (size_t)t * bo, stateless, s); if (q != RRM_OK) fail(q); }
        record(net->ev_export, s);
        export_rec = true;
        if (split && !own_arena) record(net->ev_join[t % S], s);                // the frame is complete (its arena may be cleared one frame later)
    }
    if (split) for (auto& X : net->tensors) { X.D = X.Dring[0]; X.Xn_cur = nullptr; }
    for (int k = 1; k < S; ++k) { record(net->ev_join[k], net->chunk_streams[k]); wait(origin, net->ev_join[k]); }
    // the last frame's products were merged but not zeroed (the arena bound now is that frame's)
    if (split && status == RRM_OK) { const int q = launch_zero_delta_projections(net, (T - 1) % CHUNK_RING, origin); if (q != RRM_OK) fail(q); }
    cudaGraph_t g = nullptr;
    const cudaError_t e = cudaStreamEndCapture(origin, &g);
    net->many_in_flight = false;
    if (status != RRM_OK || e != cudaSuccess || !g) {
        if (g) cudaGraphDestroy(g);
        cudaGetLastError();
        return status != RRM_OK ? status : RRM_ERR_CUDA;
    }
    // keep the few most recently used chunk lengths (a video's last chunk is usually shorter than the others)
    RRM_TRY(keep_chunk_graph(net, kind, T, mask, g, own_arena ? T - 1 : (T - 1) % S));
    if (getenv("RRM_DEBUG")) {
        size_t nodes = 0;
        cudaGraphGetNodes(g, nullptr, &nodes);
        fprintf(stderr, "rrm: chunk graph (%s, %d frames): %zu nodes, %d frames in flight\n",
                kind == 0 ? "delta" : (kind == 1 ? "keyframes" : "dense"), T, nodes, S);
    }
    return RRM_OK;
}

// T consecutive frames of a stack as one pipelined graph; RRM_ERR_UNSUPPORTED when the per-frame loop has to do it.
int run_chunk(rrm_net* net, const void* frames, void* outs, int T, cudaStream_t st, bool dense, bool stateless)
{
    if (net->graph_off || net->eps > 0.f || T < 2) return RRM_ERR_UNSUPPORTED;
    const bool is_step = !dense && !stateless;
    unsigned long long mask = 0;
    if (is_step) {
        // one decision per chunk, from the measured activity of the last delta frame (as rrm_net_step does per frame)
        net->last_step_dense = false;
        if (net->auto_switch || net->layer_switch) {
            activity_poll(net);
            // long chunks of few streams have a batched dense form that needs no change detection, marking or prefix
            // sums: on tensor-core stacks it is ahead from a lower activity on than the whole-stack switch of single steps
            const bool long_chunk = net->chunk_switch && T >= 16 && net->n <= 4 && !net->chunk_pipelined;
            const bool go_dense = (net->auto_switch && net->activity >= net->opt.stack_dense_activity) ||
                                  (long_chunk && net->activity >= net->opt.chunk_dense_activity);
            if (go_dense && net->dense_streak < net->opt.stack_reprobe) {
                ++net->dense_streak;                         // (counted in calls: a delta chunk measures again after 15 dense ones)
                net->last_step_dense = true;
                dense = true;
            } else {
                net->dense_streak = 0;
                mask = net->layer_mask;
            }
        }
        if (!dense) for (size_t l = 0; l < net->layers.size(); ++l) net->layers[l].ran_dense = l < 64 && (mask >> l & 1ull);
    }
    const int kind = !dense ? 0 : (stateless ? 2 : 1);
    auto find = [&]() -> rrm_net::ChunkGraph* {
        for (auto& c : net->chunk_graphs[kind]) if (c.T == T && c.mask == mask) return &c;
        return nullptr;
    };
    if (!find()) {
        const int s = build_chunk_graph(net, kind, T, mask);
        if (s != RRM_OK) {
            cudaGetLastError();
            bind_arena(net, reinterpret_cast<char*>(net->cleared));
            RRM_TRY(bind_readers(net));
            return s == RRM_ERR_ALLOC ? s : RRM_ERR_UNSUPPORTED;
        }
    }
    // the structures describe the last frame of the chunk from here on (statistics, activity read-back)
    bind_arena(net, net->chunk_arena[find()->last_arena]);
    RRM_TRY(bind_readers(net));
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    RRM_CUDA_TRY(cudaMemcpyAsync(net->chunk_in, frames, (size_t)bi * T, cudaMemcpyDeviceToDevice, st));
    rrm_net::ChunkGraph* cg = find();
    cg->used = ++net->chunk_clock;
    RRM_CUDA_TRY(cudaGraphLaunch(cg->exec, st));
    if (outs) RRM_CUDA_TRY(cudaMemcpyAsync(outs, net->chunk_out, (size_t)bo * T, cudaMemcpyDeviceToDevice, st));
    if (is_step && !dense && (net->auto_switch || net->layer_switch)) RRM_TRY(activity_read_back(net, st));
    return RRM_OK;
}

// T consecutive frames: one launch for the fused FC layer, the per-frame launch sequence otherwise
int run_seq(rrm_net* net, const void* frames, void* outs, int T, cudaStream_t st, bool dense, bool stateless)
{
    if (!net || !frames || T < 1) return RRM_ERR_INVALID_ARG;
    Layer& L0 = net->layers[0];
    // (a chunk too small to fill the machine goes frame by frame through the split-list kernel instead)
    if (L0.fc_fused && fc_seq_supported(L0) && (T * net->n >= 4 || L0.Wsp)) {
        net->last_stream = st;
        return fc_seq_run(net, L0, frames, outs, T, dense, stateless, st);
    }
    if (!L0.fc_fused) {
        // a stack: the frames of the chunk overlap layer by layer inside one graph
        net->last_stream = st;
        const int s = run_chunk(net, frames, outs, T, st, dense, stateless);
        if (s != RRM_ERR_UNSUPPORTED) return s;
    }
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    for (int t = 0; t < T; ++t)
        RRM_TRY(run(net, reinterpret_cast<const char*>(frames) + (size_t)t * bi,
                    outs ? reinterpret_cast<char*>(outs) + (size_t)t * bo : nullptr, st, dense, stateless));
    return RRM_OK;
}

// device staging of the *_host entry points, grown on demand to `frames` frames
int ensure_stage(rrm_net* net, int frames = 1)
{
    if (net->stage_in && frames <= net->stage_frames) return RRM_OK;
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    if (net->stage_in) {                                     // growing: the old buffers may still be in use
        RRM_CUDA_TRY(cudaDeviceSynchronize());
        dev_release(net, &net->stage_in);
        dev_release(net, &net->stage_out);
    }
    RRM_TRY(dev_alloc(net, &net->stage_in, (size_t)bi * frames));
    RRM_TRY(dev_alloc(net, &net->stage_out, (size_t)bo * frames));
    net->stage_frames = frames;
    return RRM_OK;
}

// Staging slots, copy streams and events of the pipelined host entry point.
int ensure_pipe(rrm_net* net, int frames)
{
    if (!net->h2d_stream) {
        RRM_CUDA_TRY(cudaStreamCreateWithFlags(&net->h2d_stream, cudaStreamNonBlocking));
        RRM_CUDA_TRY(cudaStreamCreateWithFlags(&net->d2h_stream, cudaStreamNonBlocking));
        for (int s = 0; s < 2; ++s) {
            RRM_CUDA_TRY(cudaEventCreateWithFlags(&net->ev_in[s], cudaEventDisableTiming));
            RRM_CUDA_TRY(cudaEventCreateWithFlags(&net->ev_done[s], cudaEventDisableTiming));
            RRM_CUDA_TRY(cudaEventCreateWithFlags(&net->ev_out[s], cudaEventDisableTiming));
        }
    }
    if (frames <= net->pipe_frames) return RRM_OK;
    // larger slots: the old ones may still be in use by copies in flight
    RRM_CUDA_TRY(cudaStreamSynchronize(net->h2d_stream));
    RRM_CUDA_TRY(cudaStreamSynchronize(net->d2h_stream));
    if (net->last_stream) RRM_CUDA_TRY(cudaStreamSynchronize(net->last_stream));
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    for (int s = 0; s < 2; ++s) {
        dev_release(net, &net->pipe_in[s]);
        dev_release(net, &net->pipe_out[s]);
        RRM_TRY(dev_alloc(net, &net->pipe_in[s], (size_t)bi * frames));
        RRM_TRY(dev_alloc(net, &net->pipe_out[s], (size_t)bo * frames));
    }
    net->pipe_frames = frames;
    return RRM_OK;
}

}  // namespace

extern "C" {

int rrm_net_create(rrm_net** out, const rrm_layer_desc* descs, int n_layers,
                   const void* const* W_dev, const void* const* bias_dev)
{
    if (!out || !descs || n_layers < 1 || !W_dev) return RRM_ERR_INVALID_ARG;
    *out = nullptr;
    rrm_net* net = new (std::nothrow) rrm_net();
    if (!net) return RRM_ERR_ALLOC;
    int s;
    try {
        s = build_net(net, descs, n_layers, W_dev, bias_dev);
    } catch (...) {
        s = RRM_ERR_ALLOC;
    }
    if (s != RRM_OK) {
        for (void* p : net->allocs) cudaFree(p);
        delete net;
        cudaGetLastError();
        return s;
    }
    *out = net;
    return RRM_OK;
}

int rrm_net_destroy(rrm_net* net)
{
    if (!net) return RRM_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    for (auto& L : net->layers) {
        if (L.seq_ev) cudaEventDestroy(L.seq_ev);
        if (L.seq_stat_host) cudaFreeHost(L.seq_stat_host);
    }
    drop_graphs(net);
    if (net->act_ev) cudaEventDestroy(net->act_ev);
    if (net->act_host) cudaFreeHost(net->act_host);
    if (net->cap_stream) cudaStreamDestroy(net->cap_stream);
    for (size_t k = 1; k < net->chunk_streams.size(); ++k) cudaStreamDestroy(net->chunk_streams[k]);   // [0] is cap_stream
    for (cudaEvent_t e : net->ev_conv) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : net->ev_epi) if (e) cudaEventDestroy(e);
    if (net->ev_import) cudaEventDestroy(net->ev_import);
    for (cudaEvent_t e : net->ev_join) if (e) cudaEventDestroy(e);
    if (net->ev_fork) cudaEventDestroy(net->ev_fork);
    if (net->ev_export) cudaEventDestroy(net->ev_export);
    if (net->h2d_stream) cudaStreamDestroy(net->h2d_stream);
    if (net->d2h_stream) cudaStreamDestroy(net->d2h_stream);
    for (int s = 0; s < 2; ++s) {
        if (net->ev_in[s]) cudaEventDestroy(net->ev_in[s]);
        if (net->ev_done[s]) cudaEventDestroy(net->ev_done[s]);
        if (net->ev_out[s]) cudaEventDestroy(net->ev_out[s]);
    }
    for (void* p : net->allocs) cudaFree(p);
    delete net;
    return RRM_OK;
}

int rrm_layer_create(rrm_layer** out, const rrm_layer_desc* desc, const void* W_dev, const void* bias_dev)
{
    if (!out || !desc) return RRM_ERR_INVALID_ARG;
    rrm_layer_desc d = *desc;
    d.src = 0;
    d.res = -1;
    const void* W[1] = {W_dev};
    const void* B[1] = {bias_dev};
    return rrm_net_create(out, &d, 1, W, B);
}

int rrm_layer_destroy(rrm_layer* layer) { return rrm_net_destroy(layer); }

int rrm_net_keyframe(rrm_net* net, const void* frame_dev, void* out_dev, void* stream)
{
    return run(net, frame_dev, out_dev, (cudaStream_t)stream, true, false);
}
int rrm_net_step(rrm_net* net, const void* frame_dev, void* out_dev, void* stream)
{
    return run(net, frame_dev, out_dev, (cudaStream_t)stream, false, false);
}
int rrm_net_dense(rrm_net* net, const void* frame_dev, void* out_dev, void* stream)
{
    return run(net, frame_dev, out_dev, (cudaStream_t)stream, true, true);
}
int rrm_keyframe(rrm_layer* layer, const void* X0_dev, void* Y0_dev, void* stream)
{
    return rrm_net_keyframe(layer, X0_dev, Y0_dev, stream);
}
int rrm_step(rrm_layer* layer, const void* Xt_dev, void* Yt_dev, void* stream)
{
    return rrm_net_step(layer, Xt_dev, Yt_dev, stream);
}
int rrm_dense(rrm_layer* layer, const void* X_dev, void* Y_dev, void* stream)
{
    return rrm_net_dense(layer, X_dev, Y_dev, stream);
}

int rrm_net_step_host(rrm_net* net, const void* frame_host, void* out_host, void* stream)
{
    if (!net || !frame_host) return RRM_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    RRM_TRY(ensure_stage(net));
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    RRM_CUDA_TRY(cudaMemcpyAsync(net->stage_in, frame_host, (size_t)bi, cudaMemcpyHostToDevice, st));
    RRM_TRY(run(net, net->stage_in, out_host ? net->stage_out : nullptr, st, false, false));
    if (out_host) RRM_CUDA_TRY(cudaMemcpyAsync(out_host, net->stage_out, (size_t)bo, cudaMemcpyDeviceToHost, st));
    RRM_CUDA_TRY(cudaStreamSynchronize(st));
    return RRM_OK;
}
int rrm_step_host(rrm_layer* layer, const void* Xt_host, void* Yt_host, void* stream)
{
    return rrm_net_step_host(layer, Xt_host, Yt_host, stream);
}

int rrm_net_step_seq(rrm_net* net, const void* frames_dev, void* outs_dev, int T, void* stream)
{
    return run_seq(net, frames_dev, outs_dev, T, (cudaStream_t)stream, false, false);
}
int rrm_net_dense_seq(rrm_net* net, const void* frames_dev, void* outs_dev, int T, void* stream)
{
    return run_seq(net, frames_dev, outs_dev, T, (cudaStream_t)stream, true, true);
}
int rrm_step_seq(rrm_layer* layer, const void* X_dev, void* Y_dev, int T, void* stream)
{
    return rrm_net_step_seq(layer, X_dev, Y_dev, T, stream);
}
int rrm_dense_seq(rrm_layer* layer, const void* X_dev, void* Y_dev, int T, void* stream)
{
    return rrm_net_dense_seq(layer, X_dev, Y_dev, T, stream);
}
int rrm_net_step_seq_host(rrm_net* net, const void* frames_host, void* outs_host, int T, void* stream)
{
    if (!net || !frames_host || T < 1) return RRM_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    RRM_TRY(ensure_stage(net, T));
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    RRM_CUDA_TRY(cudaMemcpyAsync(net->stage_in, frames_host, (size_t)bi * T, cudaMemcpyHostToDevice, st));
    RRM_TRY(run_seq(net, net->stage_in, outs_host ? net->stage_out : nullptr, T, st, false, false));
    if (outs_host) RRM_CUDA_TRY(cudaMemcpyAsync(outs_host, net->stage_out, (size_t)bo * T, cudaMemcpyDeviceToHost, st));
    RRM_CUDA_TRY(cudaStreamSynchronize(st));
    return RRM_OK;
}
int rrm_step_seq_host(rrm_layer* layer, const void* X_host, void* Y_host, int T, void* stream)
{
    return rrm_net_step_seq_host(layer, X_host, Y_host, T, stream);
}

int rrm_net_step_seq_host_async(rrm_net* net, const void* frames_host, void* outs_host, int T, void* stream)
{
    if (!net || !frames_host || T < 1) return RRM_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    RRM_TRY(ensure_pipe(net, T));
    int64_t bi = 0, bo = 0;
    tensor_bytes_boundary(net->tensors.front(), &bi);
    tensor_bytes_boundary(net->tensors.back(), &bo);
    const int s = net->pipe_slot;
    net->pipe_slot ^= 1;
    // copy-in, once the kernels that read this slot two calls ago are done (waiting for an event that was never
    // recorded returns at once)
    RRM_CUDA_TRY(cudaStreamWaitEvent(net->h2d_stream, net->ev_done[s], 0));
    RRM_CUDA_TRY(cudaMemcpyAsync(net->pipe_in[s], frames_host, (size_t)bi * T, cudaMemcpyHostToDevice, net->h2d_stream));
    RRM_CUDA_TRY(cudaEventRecord(net->ev_in[s], net->h2d_stream));
    // the frames themselves, on the caller's stream: after their copy-in and after the copy-out that last read this
    // slot's output buffer
    RRM_CUDA_TRY(cudaStreamWaitEvent(st, net->ev_in[s], 0));
    RRM_CUDA_TRY(cudaStreamWaitEvent(st, net->ev_out[s], 0));
    RRM_TRY(run_seq(net, net->pipe_in[s], outs_host ? net->pipe_out[s] : nullptr, T, st, false, false));
    RRM_CUDA_TRY(cudaEventRecord(net->ev_done[s], st));
    if (outs_host) {
        RRM_CUDA_TRY(cudaStreamWaitEvent(net->d2h_stream, net->ev_done[s], 0));
        RRM_CUDA_TRY(cudaMemcpyAsync(outs_host, net->pipe_out[s], (size_t)bo * T, cudaMemcpyDeviceToHost, net->d2h_stream));
        RRM_CUDA_TRY(cudaEventRecord(net->ev_out[s], net->d2h_stream));
    }
    return RRM_OK;
}
int rrm_step_seq_host_async(rrm_layer* layer, const void* X_host, void* Y_host, int T, void* stream)
{
    return rrm_net_step_seq_host_async(layer, X_host, Y_host, T, stream);
}
int rrm_net_host_sync(rrm_net* net)
{
    if (!net) return RRM_ERR_INVALID_ARG;
    if (net->last_stream) RRM_CUDA_TRY(cudaStreamSynchronize(net->last_stream));
    if (net->d2h_stream) RRM_CUDA_TRY(cudaStreamSynchronize(net->d2h_stream));
    return RRM_OK;
}
int rrm_host_sync(rrm_layer* layer) { return rrm_net_host_sync(layer); }

int rrm_net_set_epsilon(rrm_net* net, float eps)
{
    if (!net || !(eps >= 0.f)) return RRM_ERR_INVALID_ARG;
    if (net->layers[0].fc_fused) return RRM_ERR_UNSUPPORTED;
    for (auto& L : net->layers) if (L.d.dtype != RRM_F32) return RRM_ERR_DTYPE;
    if (eps == net->eps) return RRM_OK;
    RRM_CUDA_TRY(cudaDeviceSynchronize());
    net->eps = eps;
    // the threshold is a kernel argument: captured sequences have to be captured again
    drop_graphs(net);
    return RRM_OK;
}

int rrm_net_set_affine(rrm_net* net, int layer, const void* scale_dev, const void* shift_dev)
{
    if (!net || layer < 0 || layer >= (int)net->layers.size() || (!scale_dev) != (!shift_dev)) return RRM_ERR_INVALID_ARG;
    Layer& L = net->layers[layer];
    if (L.fc_fused) return RRM_ERR_UNSUPPORTED;
    // the integer form lives inside the requantisation: layers that emit raw projections or signs have none
    if (L.d.dtype != RRM_F32 && (L.d.shift < 0 || L.d.act == RRM_ACT_SIGN)) return RRM_ERR_UNSUPPORTED;
    RRM_CUDA_TRY(cudaDeviceSynchronize());
    const size_t bytes = (size_t)L.d.c_out * 4;
    if (scale_dev) {
        if (!L.bn_scale) { RRM_TRY(dev_alloc(net, &L.bn_scale, bytes)); RRM_TRY(dev_alloc(net, &L.bn_shift, bytes)); }
        RRM_CUDA_TRY(cudaMemcpy(L.bn_scale, scale_dev, bytes, cudaMemcpyDeviceToDevice));
        RRM_CUDA_TRY(cudaMemcpy(L.bn_shift, shift_dev, bytes, cudaMemcpyDeviceToDevice));
    } else {
        dev_release(net, &L.bn_scale);
        dev_release(net, &L.bn_shift);
    }
    drop_graphs(net);                                        // captured sequences hold the old arguments
    if (net->bound_arena != reinterpret_cast<char*>(net->cleared)) {
        bind_arena(net, reinterpret_cast<char*>(net->cleared));
        RRM_TRY(bind_readers(net));
    }
    RRM_TRY(reset_state(net, nullptr));                      // f changed: back to the fresh state, consistent with the new f
    RRM_CUDA_TRY(cudaDeviceSynchronize());
    return RRM_OK;
}

int rrm_net_truncation(rrm_net* net, double* e_t, double* last_step_l2)
{
    if (!net || !e_t) return RRM_ERR_INVALID_ARG;
    if (net->layers[0].fc_fused) return RRM_ERR_UNSUPPORTED;
    RRM_CUDA_TRY(cudaStreamSynchronize(net->last_stream));
    std::vector<double> h(1 + net->layers.size());
    RRM_CUDA_TRY(cudaMemcpy(h.data(), net->aecs, h.size() * 8, cudaMemcpyDeviceToHost));
    *e_t = h[0];
    if (last_step_l2) for (size_t l = 0; l < net->layers.size(); ++l) last_step_l2[l] = h[1 + l];
    return RRM_OK;
}

double rrm_aecs_predict(const double mu[5], double e_t)
{
    if (!mu) return 0.0;
    return mu[0] + e_t * (mu[1] + e_t * (mu[2] + e_t * (mu[3] + e_t * mu[4])));
}

static int stats_fill(rrm_net* net, int layer, rrm_stats* h);

int rrm_net_get_stats(rrm_net* net, int layer, rrm_stats* h)
{
    if (!net || !h || layer < 0 || layer >= (int)net->layers.size()) return RRM_ERR_INVALID_ARG;
    RRM_TRY(stats_fill(net, layer, h));
    // device-side errors since the last rrm_net_clear_errors surface here (the steps themselves are asynchronous)
    if (h->error_word & ERRW_TIMEOUT) return RRM_ERR_TIMEOUT;
    if (h->error_word & (ERRW_BOUNDS | ERRW_CAPACITY)) return RRM_ERR_CAPACITY;
    return RRM_OK;
}

static int stats_fill(rrm_net* net, int layer, rrm_stats* h)
{
    RRM_CUDA_TRY(cudaStreamSynchronize(net->last_stream));
    std::memset(h, 0, sizeof(*h));
    const Layer& L = net->layers[layer];
    const rrm_layer_desc& d = L.d;
    const int oh = (d.h + 2 * d.pad - d.kh) / d.stride + 1, ow = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
    h->in_elems = (int64_t)d.n * d.c_in * d.h * d.w;
    h->out_pixels = (int64_t)d.n * oh * ow;
    h->dense_macs = h->out_pixels * d.c_out * d.c_in * d.kh * d.kw;
    int errw = 0;
    RRM_CUDA_TRY(cudaMemcpy(&errw, net->errw, 4, cudaMemcpyDeviceToHost));
    h->error_word = errw;
    if (L.fc_fused) {
        unsigned long long tot[2] = {0, 0};
        int frames = 1;
        if (L.seq_last_T > 0) {                  // the last call was a chunk: counters cover all its frames
            frames = L.seq_last_T;
            RRM_TRY(fc_seq_stats(net->layers[layer], &tot[0], &tot[1]));
            h->in_elems *= frames;
            h->out_pixels *= frames;
            h->dense_macs *= frames;
        } else {
            std::vector<unsigned long long> v((size_t)d.n * 2);
            RRM_CUDA_TRY(cudaMemcpy(v.data(), L.fc_nnz, v.size() * 8, cudaMemcpyDeviceToHost));
            for (int s = 0; s < d.n; ++s) { tot[0] += v[s * 2]; tot[1] += v[s * 2 + 1]; }
        }
        h->nnz_elems = (int64_t)tot[0];
        h->in_pixels = (int64_t)frames * d.n * ((d.c_in + 31) / 32);
        h->active_in_pixels = (int64_t)tot[1];
        h->active_out_pixels = tot[0] ? (int64_t)frames * d.n : 0;
        h->active_macs = (int64_t)tot[0] * d.c_out;
        h->variant = L.seq_last_T > 0 ? L.seq_last_variant : RRM_VARIANT_GATHER;
        return RRM_OK;
    }
    if (net->last_step_dense) {                  // the most recent step was evaluated densely: nothing was counted
        h->nnz_elems = h->active_in_pixels = h->active_out_pixels = h->active_macs = -1;
        h->in_pixels = net->tensors[d.src].pixels();
        h->variant = RRM_VARIANT_DENSE;
        return RRM_OK;
    }
    const Tensor& in = net->tensors[d.src];
    unsigned long long v[2] = {0, 0};
    RRM_CUDA_TRY(cudaMemcpy(v, in.nnz, 16, cudaMemcpyDeviceToHost));
    h->nnz_elems = (int64_t)v[0];
    h->active_in_pixels = (int64_t)v[1];
    h->in_pixels = in.pixels();
    unsigned long long m = 0;
    int oc = 0;
    RRM_CUDA_TRY(cudaMemcpy(&m, L.macs, 8, cudaMemcpyDeviceToHost));
    RRM_CUDA_TRY(cudaMemcpy(&oc, L.ocount, 4, cudaMemcpyDeviceToHost));
    h->active_macs = (int64_t)m;
    h->active_out_pixels = oc;
    // (a layer that was evaluated densely inside the delta step keeps its counters: the deltas were still formed and counted)
    h->variant = L.ran_dense ? RRM_VARIANT_DENSE : (L.tc_ready ? RRM_VARIANT_TENSOR : RRM_VARIANT_GATHER);
    return RRM_OK;
}
int rrm_get_stats(rrm_layer* layer, rrm_stats* host_out) { return rrm_net_get_stats(layer, 0, host_out); }

int rrm_net_clear_errors(rrm_net* net)
{
    if (!net) return RRM_ERR_INVALID_ARG;
    if (net->last_stream) RRM_CUDA_TRY(cudaStreamSynchronize(net->last_stream));
    RRM_CUDA_TRY(cudaMemset(net->errw, 0, 4));
    RRM_TRY(clear_split(net, nullptr));          // (a pipelined chunk that gave up may have left products unmerged)
    RRM_CUDA_TRY(cudaDeviceSynchronize());
    return RRM_OK;
}
int rrm_clear_errors(rrm_layer* layer) { return rrm_net_clear_errors(layer); }

int rrm_net_get_options(const rrm_net* net, rrm_options* out)
{
    if (!net || !out) return RRM_ERR_INVALID_ARG;
    *out = net->opt;
    return RRM_OK;
}
int rrm_net_set_options(rrm_net* net, const rrm_options* in)
{
    if (!net || !in) return RRM_ERR_INVALID_ARG;
    if (!(in->layer_dense_activity >= 0.f) || !(in->layer_delta_activity >= 0.f) || in->layer_delta_activity > in->layer_dense_activity ||
        !(in->stack_dense_activity >= 0.f) || in->stack_reprobe < 1 || !(in->fc_dense_rows >= 0.f) || !(in->fc_dense_density >= 0.f) ||
        !(in->chunk_dense_activity >= 0.f))
        return RRM_ERR_INVALID_ARG;
    RRM_CUDA_TRY(cudaDeviceSynchronize());
    net->opt = *in;
    drop_graphs(net);                                        // captured sequences hold the old wait limit
    return RRM_OK;
}
int rrm_get_options(const rrm_layer* layer, rrm_options* out) { return rrm_net_get_options(layer, out); }
int rrm_set_options(rrm_layer* layer, const rrm_options* in) { return rrm_net_set_options(layer, in); }

int rrm_net_projection(rrm_net* net, int layer, void* P_dev, void* stream)
{
    if (!net || !P_dev || layer < 0 || layer >= (int)net->layers.size()) return RRM_ERR_INVALID_ARG;
    if (net->layers[layer].fc_fused) return fc_fused_projection(net, net->layers[layer], P_dev, (cudaStream_t)stream);
    return launch_export_projection(net, layer, P_dev, (cudaStream_t)stream);
}
int rrm_layer_projection(rrm_layer* layer, void* P_dev, void* stream) { return rrm_net_projection(layer, 0, P_dev, stream); }

int rrm_net_tensor(rrm_net* net, int t, void* dst_dev, void* stream)
{
    if (!net || !dst_dev || t < 0 || t >= (int)net->tensors.size()) return RRM_ERR_INVALID_ARG;
    if (net->layers[0].fc_fused) return RRM_ERR_UNSUPPORTED;
    return launch_export_tensor(net, t, dst_dev, false, (cudaStream_t)stream);
}

int64_t rrm_net_tensor_bytes(const rrm_net* net, int t)
{
    if (!net || t < 0 || t >= (int)net->tensors.size()) return RRM_ERR_INVALID_ARG;
    int64_t b = 0;
    tensor_bytes_boundary(net->tensors[t], &b);
    return b;
}

const char* rrm_strerror(int status)
{
    switch (status) {
        case RRM_OK: return "ok";
        case RRM_ERR_INVALID_ARG: return "invalid argument";
        case RRM_ERR_SHAPE: return "shape mismatch";
        case RRM_ERR_DTYPE: return "dtype mismatch";
        case RRM_ERR_ALLOC: return "device allocation failed";
        case RRM_ERR_CAPACITY: return "size exceeds the library's index range";
        case RRM_ERR_TIMEOUT: return "bounded device wait ran out";
        case RRM_ERR_CUDA: return "CUDA runtime error";
        case RRM_ERR_UNSUPPORTED: return "unsupported combination";
        default: return "unknown status";
    }
}

}  // extern "C"
