// Fused delta-FC step for int8 layers (Algorithm 1, FC branch; Sec. 3.5 column products).
//
// One launch does the whole frame of one FC layer:
//   1. every CTA scans X_t against the snapshot with 128-bit loads and builds, by ballot-free
//      per-chunk counts + a block prefix sum, the ordered list of non-zero delta entries;
//   2. the list is split evenly over the CTAs of a column group; each CTA gathers only the
//      weight columns W[:, j] of its entries (weights are stored transposed, one contiguous
//      C_out-byte row per input j) and accumulates d_j * W[:, j] in int32;
//   3. partial sums are added into the stored projection P with integer atomics (exact,
//      order-independent);
//   4. the last CTA to finish an output slice applies f and writes Y_t; CTA 0 of a stream
//      writes the new snapshot into the other half of a ping-pong pair.
// Cost is HBM-bound: nnz * C_out weight bytes per frame.
#include "rrm_common.cuh"

namespace rrm {

constexpr int FC_THREADS = 256;
constexpr int FC_OW = 512;                 // outputs per CTA (32 lanes x 16 bytes)
constexpr int FC_GROUPS = FC_THREADS / 32; // column groups working in parallel inside a CTA
constexpr int FC_LCAP = 1024;              // list entries one CTA can own
constexpr int FC_MAX_CHUNKS = 4096;        // 16-byte chunks of one input row (C_in <= 65536)

struct FcParams {
    const int8_t* xt;        // [n][c_in]
    const int8_t* xprev;     // [n][c_in] snapshot, or nullptr: treat every entry as active with d = x
    int8_t* xnext;           // [n][c_in] snapshot to write, or nullptr
    const int8_t* Wt;        // [c_in][c_out]
    int32_t* P;              // [n][c_out]
    void* Y;                 // [n][c_out] int32 or int8, or nullptr
    unsigned int* counters;  // [n][slices]
    unsigned long long* stat;// [n][2]: nnz elements, active groups of 32 inputs (or nullptr)
    int c_in, c_out, ksplit, shift, act;
};

__device__ __forceinline__ int fc_apply_f(int v, int shift, int act) {
    if (shift > 0) v = (v + (1 << (shift - 1))) >> shift;
    v = max(-127, min(127, v));
    if (act == RRM_ACT_RELU) v = max(v, 0);
    return v;
}

__global__ void __launch_bounds__(FC_THREADS) fc_delta_i8_kernel(FcParams p)
{
    __shared__ int s_warp[FC_THREADS / 32];
    __shared__ int s_list_j[FC_LCAP];
    __shared__ int s_list_d[FC_LCAP];
    __shared__ int s_red[FC_GROUPS][FC_OW];
    __shared__ int s_flag;

    const int tid = threadIdx.x;
    const int kg = blockIdx.x, slice = blockIdx.y, s = blockIdx.z;
    const int C = p.c_in, K = p.c_out;
    const int nchunks = C >> 4;
    const uint4* xt4 = reinterpret_cast<const uint4*>(p.xt + (size_t)s * C);
    const uint4* xp4 = p.xprev ? reinterpret_cast<const uint4*>(p.xprev + (size_t)s * C) : nullptr;

    // ---- 1. count non-zero delta bytes per 16-byte chunk; each thread owns a contiguous range of chunks
    const int per_thread = (nchunks + FC_THREADS - 1) / FC_THREADS;
    const int c_begin = min(nchunks, tid * per_thread), c_end = min(nchunks, c_begin + per_thread);
    int local = 0;
    for (int c = c_begin; c < c_end; ++c) {
        if (xp4) {
            const uint4 a = __ldg(xt4 + c), b = __ldg(xp4 + c);
            // a byte differs <=> its delta is non-zero
            auto nzb = [](unsigned v) { v |= v >> 4; v |= v >> 2; v |= v >> 1; return __popc(v & 0x01010101u); };
            local += nzb(a.x ^ b.x) + nzb(a.y ^ b.y) + nzb(a.z ^ b.z) + nzb(a.w ^ b.w);
        } else {
            local += 16;
        }
    }
    // block exclusive scan of `local`
    const int lane = tid & 31, warp = tid >> 5;
    int incl = local;
    #pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int warp_off = 0, total = 0;
    #pragma unroll
    for (int w = 0; w < FC_THREADS / 32; ++w) {
        int v = s_warp[w];
        if (w < warp) warp_off += v;
        total += v;
    }
    int offset = warp_off + incl - local;          // index of this thread's first entry in the global list

    // ---- 2. this CTA's share of the ordered list
    const int per_cta = (total + p.ksplit - 1) / p.ksplit;
    const int lo = kg * per_cta, hi = min(total, lo + per_cta);
    const int mine = max(0, hi - lo);              // <= FC_LCAP by the host's choice of ksplit
    if (offset < hi && offset + local > lo) {
        for (int c = c_begin; c < c_end; ++c) {
            uint4 a = __ldg(xt4 + c);
            uint4 b = xp4 ? __ldg(xp4 + c) : make_uint4(0, 0, 0, 0);
            const unsigned aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
            #pragma unroll
            for (int i = 0; i < 16; ++i) {
                int av = (int)(int8_t)(aw[i >> 2] >> ((i & 3) * 8));
                int bv = (int)(int8_t)(bw[i >> 2] >> ((i & 3) * 8));
                bool on = xp4 ? (av != bv) : true;
                if (on) {
                    if (offset >= lo && offset < hi) {
                        s_list_j[offset - lo] = c * 16 + i;
                        s_list_d[offset - lo] = av - bv;
                    }
                    ++offset;
                }
            }
        }
    }
    // new snapshot and statistics: one CTA per stream
    if (kg == 0 && slice == 0) {
        int groups32 = 0;
        for (int base = 0; base < nchunks; base += FC_THREADS) {      // uniform trip count: shuffles inside
            const int c = base + tid;
            const bool in = c < nchunks;
            uint4 a = make_uint4(0, 0, 0, 0), b = a;
            if (in) {
                a = __ldg(xt4 + c);
                if (p.xnext) reinterpret_cast<uint4*>(p.xnext + (size_t)s * C)[c] = a;
                if (xp4) b = __ldg(xp4 + c);
            }
            const unsigned diff = (a.x ^ b.x) | (a.y ^ b.y) | (a.z ^ b.z) | (a.w ^ b.w);
            // a group of 32 inputs spans two chunks held by neighbouring lanes
            const unsigned other = __shfl_xor_sync(0xffffffffu, diff, 1);
            groups32 += in && ((c & 1) == 0) && ((diff | other) != 0);
        }
        if (p.stat) {
            #pragma unroll
            for (int o = 16; o > 0; o >>= 1) groups32 += __shfl_down_sync(0xffffffffu, groups32, o);
            if (lane == 0 && groups32) atomicAdd(&p.stat[s * 2 + 1], (unsigned long long)groups32);
            if (tid == 0) atomicAdd(&p.stat[s * 2 + 0], (unsigned long long)total);
        }
    }
    __syncthreads();

    // ---- 3. gather the columns of the owned entries: lane -> 16 outputs, warp -> column group
    const int o0 = slice * FC_OW + lane * 16;
    const bool o_ok = o0 < K;                       // K is a multiple of 16
    int acc[16];
    #pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0;
    const int8_t* wbase = p.Wt + o0;
    // acc[i] += w_i * d for the 16 int8 weights in w.  dp4a against a selector that holds d in
    // one byte lane; a delta outside int8 range (|d| <= 254) is split into two in-range halves.
    auto fma16 = [&](const uint4& w, int d) {
        const unsigned ww[4] = {w.x, w.y, w.z, w.w};
        if (d >= -128 && d <= 127) {                 // warp-uniform: d belongs to the column
            const unsigned db = (unsigned)d & 0xffu;
            #pragma unroll
            for (int q = 0; q < 4; ++q) {
                #pragma unroll
                for (int b = 0; b < 4; ++b) acc[q * 4 + b] = __dp4a((int)ww[q], (int)(db << (8 * b)), acc[q * 4 + b]);
            }
        } else {
            const int dh = d / 2, dl = d - dh;
            const unsigned hb = (unsigned)dh & 0xffu, lb = (unsigned)dl & 0xffu;
            #pragma unroll
            for (int q = 0; q < 4; ++q) {
                #pragma unroll
                for (int b = 0; b < 4; ++b) {
                    acc[q * 4 + b] = __dp4a((int)ww[q], (int)(hb << (8 * b)), acc[q * 4 + b]);
                    acc[q * 4 + b] = __dp4a((int)ww[q], (int)(lb << (8 * b)), acc[q * 4 + b]);
                }
            }
        }
    };
    if (o_ok) {
        int e = warp;
        for (; e + 3 * FC_GROUPS < mine; e += 4 * FC_GROUPS) {
            const int j0 = s_list_j[e], j1 = s_list_j[e + FC_GROUPS], j2 = s_list_j[e + 2 * FC_GROUPS],
                      j3 = s_list_j[e + 3 * FC_GROUPS];
            const uint4 w0 = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)j0 * K));
            const uint4 w1 = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)j1 * K));
            const uint4 w2 = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)j2 * K));
            const uint4 w3 = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)j3 * K));
            fma16(w0, s_list_d[e]);
            fma16(w1, s_list_d[e + FC_GROUPS]);
            fma16(w2, s_list_d[e + 2 * FC_GROUPS]);
            fma16(w3, s_list_d[e + 3 * FC_GROUPS]);
        }
        for (; e < mine; e += FC_GROUPS) {
            const uint4 w0 = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)s_list_j[e] * K));
            fma16(w0, s_list_d[e]);
        }
    }
    #pragma unroll
    for (int i = 0; i < 16; ++i) s_red[warp][lane * 16 + i] = acc[i];
    __syncthreads();

    // ---- 4. add into the stored projection (exact integer atomics)
    int32_t* Ps = p.P + (size_t)s * K + slice * FC_OW;
    const int width = min(FC_OW, K - slice * FC_OW);
    if (mine > 0) {
        for (int o = tid; o < width; o += FC_THREADS) {
            int v = 0;
            #pragma unroll
            for (int g = 0; g < FC_GROUPS; ++g) v += s_red[g][o];
            if (v) atomicAdd(&Ps[o], v);
        }
    }

    // ---- 5. last CTA of this (stream, slice) applies f and writes Y_t
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned int* ctr = &p.counters[s * gridDim.y + slice];
        const unsigned int ticket = atomicAdd(ctr, 1u);
        const int last = (ticket == (unsigned)p.ksplit - 1);
        if (last) *ctr = 0;                          // ready for the next launch (stream-ordered)
        s_flag = last;
    }
    __syncthreads();
    if (s_flag && p.Y) {
        __threadfence();
        for (int o = tid; o < width; o += FC_THREADS) {
            const int v = __ldcg(&Ps[o]);
            const size_t oi = (size_t)s * K + slice * FC_OW + o;
            if (p.shift < 0) reinterpret_cast<int32_t*>(p.Y)[oi] = v;
            else reinterpret_cast<int8_t*>(p.Y)[oi] = (int8_t)fc_apply_f(v, p.shift, p.act);
        }
    }
}

// P[s][o] = bias[o]; optionally zero a snapshot
__global__ void fc_init_kernel(int32_t* P, const int32_t* bias, int n, int K, int8_t* snap, int C)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n * K) P[i] = bias ? bias[i % K] : 0;
    if (snap && i < n * C) snap[i] = 0;
}

// Wt[j][o] = W[o][j]
__global__ void fc_transpose_kernel(const int8_t* W, int8_t* Wt, int K, int C)
{
    __shared__ int8_t tile[32][33];
    const int j0 = blockIdx.x * 32, o0 = blockIdx.y * 32;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int o = o0 + r, j = j0 + threadIdx.x;
        tile[r][threadIdx.x] = (o < K && j < C) ? W[(size_t)o * C + j] : 0;
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int j = j0 + r, o = o0 + threadIdx.x;
        if (j < C && o < K) Wt[(size_t)j * K + o] = tile[threadIdx.x][r];
    }
}

static int fc_ksplit(const Layer& L)
{
    const int slices = ceil_div(L.d.c_out, FC_OW);
    int ks = ceil_div(2 * 148, slices * L.d.n);
    ks = ks < 1 ? 1 : ks;
    const int need = ceil_div(L.d.c_in, FC_LCAP);      // a CTA's share must fit its list
    return ks < need ? need : ks;
}

int fc_fused_create(rrm_net* net, Layer& L, const void* W_dev, const void* bias_dev)
{
    const int C = L.d.c_in, K = L.d.c_out, n = L.d.n;
    if (C % 16 || K % 16 || C / 16 > FC_MAX_CHUNKS * 4) return RRM_ERR_UNSUPPORTED;
    auto alloc = [&](void** p, size_t bytes) -> int {
        if (cudaMalloc(p, bytes) != cudaSuccess) return RRM_ERR_ALLOC;
        net->allocs.push_back(*p);
        return RRM_OK;
    };
    const int slices = ceil_div(K, FC_OW);
    RRM_TRY(alloc((void**)&L.Wt, (size_t)C * K));
    RRM_TRY(alloc((void**)&L.xs[0], (size_t)n * C));
    RRM_TRY(alloc((void**)&L.xs[1], (size_t)n * C));
    RRM_TRY(alloc((void**)&L.P, (size_t)n * K * 4));
    RRM_TRY(alloc((void**)&L.P2, (size_t)n * K * 4));
    RRM_TRY(alloc((void**)&L.bias, (size_t)K * 4));
    RRM_TRY(alloc((void**)&L.fc_counters, (size_t)n * slices * 4 * 2));
    RRM_TRY(alloc((void**)&L.fc_nnz, (size_t)n * 2 * 8));
    RRM_CUDA_TRY(cudaMemset(L.fc_counters, 0, (size_t)n * slices * 4 * 2));
    RRM_CUDA_TRY(cudaMemset(L.fc_nnz, 0, (size_t)n * 2 * 8));
    if (bias_dev) RRM_CUDA_TRY(cudaMemcpy(L.bias, bias_dev, (size_t)K * 4, cudaMemcpyDeviceToDevice));
    else RRM_CUDA_TRY(cudaMemset(L.bias, 0, (size_t)K * 4));
    dim3 tb(32, 8), tg(ceil_div(C, 32), ceil_div(K, 32));
    fc_transpose_kernel<<<tg, tb>>>(reinterpret_cast<const int8_t*>(W_dev), L.Wt, K, C);
    const int tot = n * (K > C ? K : C);
    fc_init_kernel<<<ceil_div(tot, 256), 256>>>(reinterpret_cast<int32_t*>(L.P), reinterpret_cast<int32_t*>(L.bias),
                                                n, K, L.xs[0], C);
    RRM_CUDA_TRY(cudaGetLastError());
    RRM_CUDA_TRY(cudaDeviceSynchronize());
    L.xs_cur = 0;
    L.fc_fused = true;
    return RRM_OK;
}

// dense:     every input entry is visited (keyframe or the stateless dense path)
// stateless: results go to the scratch projection P2, the RRM state is left untouched
int fc_fused_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, bool dense, bool stateless, cudaStream_t st)
{
    const int C = L.d.c_in, K = L.d.c_out, n = L.d.n;
    const int slices = ceil_div(K, FC_OW);
    FcParams p;
    p.xt = reinterpret_cast<const int8_t*>(X_dev);
    p.Wt = L.Wt;
    p.c_in = C; p.c_out = K; p.shift = L.d.shift; p.act = L.d.act;
    p.ksplit = fc_ksplit(L);
    p.Y = Y_dev;
    const int tot = n * (K > C ? K : C);
    if (dense) {
        int32_t* Pd = reinterpret_cast<int32_t*>(stateless ? L.P2 : L.P);
        fc_init_kernel<<<ceil_div(tot, 256), 256, 0, st>>>(Pd, reinterpret_cast<int32_t*>(L.bias), n, K, nullptr, C);
        p.xprev = nullptr;
        p.P = Pd;
        p.stat = nullptr;
        p.counters = L.fc_counters + (stateless ? n * slices : 0);
        if (stateless) p.xnext = nullptr;
        else { p.xnext = L.xs[L.xs_cur ^ 1]; L.xs_cur ^= 1; }
    } else {
        cudaMemsetAsync(L.fc_nnz, 0, (size_t)n * 2 * 8, st);
        p.xprev = L.xs[L.xs_cur];
        p.xnext = L.xs[L.xs_cur ^ 1];
        L.xs_cur ^= 1;
        p.P = reinterpret_cast<int32_t*>(L.P);
        p.stat = L.fc_nnz;
        p.counters = L.fc_counters;
    }
    dim3 grid(p.ksplit, slices, n);
    fc_delta_i8_kernel<<<grid, FC_THREADS, 0, st>>>(p);
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

int fc_fused_projection(rrm_net* net, Layer& L, void* P_dev, cudaStream_t st)
{
    RRM_CUDA_TRY(cudaMemcpyAsync(P_dev, L.P, (size_t)L.d.n * L.d.c_out * 4, cudaMemcpyDeviceToDevice, st));
    return RRM_OK;
}

}  // namespace rrm
