// Fused delta-FC step for int8 layers (Algorithm 1, FC branch; Sec. 3.5 column products).
//
// One launch does the whole frame of one FC layer.  The grid is made of clusters of FC_CL CTAs;
// a cluster owns FC_OW consecutive outputs of one stream:
//   1. every CTA scans X_t against the snapshot with 128-bit loads (all loads issued up front) and
//      finds, by per-thread counts and a block prefix sum, its share of the ordered list of
//      non-zero delta entries (the list is split evenly over the CTAs of the cluster);
//   2. each CTA gathers only the weight columns W[:, j] of its entries (weights are stored
//      transposed, one contiguous C_out-byte row per input j) and accumulates d_j * W[:, j] in int32;
//   3. partial sums are reduced inside the CTA, then across the cluster through distributed shared
//      memory; CTA 0 of the cluster adds them onto the stored projection P (owner computes, no
//      atomics), applies f and writes Y_t;
//   4. one CTA per stream writes the new snapshot into the other half of a ping-pong pair.
// Cost is HBM-bound: nnz * C_out weight bytes per frame.
#include "rrm_common.cuh"
#include "rrm_dev.cuh"
#include <cooperative_groups.h>
#include <mutex>

namespace cg = cooperative_groups;

namespace rrm {

constexpr int FC_THREADS = 256;
constexpr int FC_CL = 8;                   // CTAs per cluster = split of the non-zero list
constexpr int FC_OW = 128;                 // outputs per cluster (8 lanes x 16 bytes)
constexpr int FC_GROUPS = FC_THREADS / 8;  // columns gathered in parallel inside a CTA
constexpr int FC_LCAP = 2048;              // list entries one CTA can own  (C_in <= FC_CL * FC_LCAP)
constexpr int FC_TWO_KERNEL_MIN_STREAMS = 3;   // from this many streams per call on, build the list once per stream
constexpr int FC_PT = 4;                   // 16-byte chunks scanned per thread (C_in <= 16 * FC_PT * FC_THREADS)

struct FcParams {
    const int8_t* xt;        // [n][c_in]
    const int8_t* xprev;     // [n][c_in] snapshot, or nullptr: treat every entry as active with d = x
    int8_t* xnext;           // [n][c_in] snapshot to write, or nullptr
    const int8_t* Wt;        // [c_in][c_out]
    int32_t* P;              // [n][c_out]
    void* Y;                 // [n][c_out] int32 or int8, or nullptr
    unsigned long long* stat;// [n][2]: nnz elements, active groups of 32 inputs (or nullptr)
    int c_in, c_out, shift, act;
};

// Split cluster barrier.  Every thread alternates arrive and wait; a thread may exit after an arrive.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__global__ void __cluster_dims__(FC_CL, 1, 1) __launch_bounds__(FC_THREADS) fc_delta_i8_kernel(FcParams p)
{
    __shared__ int s_warp[FC_THREADS / 32];
    __shared__ int s_off[FC_THREADS];
    __shared__ unsigned long long s_mask[FC_THREADS];
    __shared__ unsigned short s_list_j[FC_LCAP];   // C_in <= 16384 fits 16 bits
    __shared__ __align__(16) int8_t s_xt[16 * FC_PT * FC_THREADS];
    __shared__ __align__(16) int8_t s_xp[16 * FC_PT * FC_THREADS];
    __shared__ int s_red[FC_THREADS / 32][FC_OW];
    __shared__ int s_part[FC_CL][FC_OW];          // used in rank 0 only: partial sums pushed by every rank

    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int kg = blockIdx.x;                       // rank inside the cluster (cluster spans x)
    const int slice = blockIdx.y, s = blockIdx.z;
    const int C = p.c_in, K = p.c_out;
    const int nchunks = C >> 4;
    const uint4* xt4 = reinterpret_cast<const uint4*>(p.xt + (size_t)s * C);
    const uint4* xp4 = p.xprev ? reinterpret_cast<const uint4*>(p.xprev + (size_t)s * C) : nullptr;
    int32_t* Ps = p.P + (size_t)s * K + slice * FC_OW;
    const int width = min(FC_OW, K - slice * FC_OW);

    cluster_arrive_relaxed();                        // waited for just before the first remote store
    // stored projection of this slice: fetched now, needed at the very end
    int p_old = 0;
    if (kg == 0 && tid < width) p_old = Ps[tid];

    // ---- 1. non-zero delta bytes per 16-byte chunk; each thread owns FC_PT consecutive chunks
    const int c_begin = tid * FC_PT;
    uint4 xa[FC_PT], xb[FC_PT];
    #pragma unroll
    for (int i = 0; i < FC_PT; ++i) {
        xa[i] = make_uint4(0, 0, 0, 0);
        xb[i] = xa[i];
        if (c_begin + i < nchunks) {
            xa[i] = __ldg(xt4 + c_begin + i);
            if (xp4) xb[i] = __ldg(xp4 + c_begin + i);
        }
    }
    // raw bytes to shared memory (the gather looks the delta of an entry up there) and a 64-bit mask
    // of the non-zero delta bytes of this thread's 64 inputs (a byte differs <=> its delta is non-zero)
    unsigned long long m = 0;
    #pragma unroll
    for (int i = 0; i < FC_PT; ++i) {
        if (c_begin + i < nchunks) {
            reinterpret_cast<uint4*>(s_xt)[c_begin + i] = xa[i];
            reinterpret_cast<uint4*>(s_xp)[c_begin + i] = xb[i];
            const unsigned cm = xp4 ? differing_bytes(xa[i], xb[i]) : 0xffffu;
            m |= (unsigned long long)cm << (16 * i);
        }
    }
    const int local = __popcll(m);
    // block exclusive scan of `local`
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
    int offset = warp_off + incl - local;          // index of this thread's first entry in the ordered list

    s_off[tid] = offset;
    s_mask[tid] = m;
    __syncthreads();
    // ---- 2. this CTA's share of the list, one entry per thread: find the thread that scanned entry e
    // (largest t with s_off[t] <= e) and pick the matching set bit of its mask
    const int per_cta = (total + FC_CL - 1) / FC_CL;
    const int lo = kg * per_cta, hi = min(total, lo + per_cta);
    const int mine = max(0, hi - lo);              // <= FC_LCAP: checked on the host
    for (int e = lo + tid; e < hi; e += FC_THREADS) {
        int t = 0;
        #pragma unroll
        for (int step = FC_THREADS / 2; step > 0; step >>= 1)
            if (s_off[t + step] <= e) t += step;
        const unsigned long long mk = s_mask[t];
        const int r = e - s_off[t];                  // r-th set bit (0-based) of mk
        const unsigned lo32 = (unsigned)mk, hi32 = (unsigned)(mk >> 32);
        const int cl = __popc(lo32);
        const int bit = r < cl ? (int)__fns(lo32, 0, r + 1) : 32 + (int)__fns(hi32, 0, r - cl + 1);
        s_list_j[e - lo] = (unsigned short)(t * (16 * FC_PT) + bit);
    }
    // new snapshot: in the clusters of slice 0, CTA r stores the chunks scanned by its warp r
    if (slice == 0 && p.xnext && warp == kg) {
        #pragma unroll
        for (int i = 0; i < FC_PT; ++i)
            if (c_begin + i < nchunks) reinterpret_cast<uint4*>(p.xnext + (size_t)s * C)[c_begin + i] = xa[i];
    }
    // statistics: one CTA per stream
    if (kg == 0 && slice == 0 && p.stat) {
        int groups32 = __popc((unsigned)((m | m >> 16) & 0xffffu) != 0) + __popc((unsigned)(((m >> 32) | (m >> 48)) & 0xffffu) != 0);
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) groups32 += __shfl_down_sync(0xffffffffu, groups32, o);
        __shared__ int s_grp[FC_THREADS / 32];
        if (lane == 0) s_grp[warp] = groups32;
        __syncthreads();
        if (tid == 0) {
            int g = 0;
            #pragma unroll
            for (int w = 0; w < FC_THREADS / 32; ++w) g += s_grp[w];
            p.stat[s * 2 + 0] = (unsigned long long)total;
            p.stat[s * 2 + 1] = (unsigned long long)g;
        }
    }
    __syncthreads();

    // ---- 3. gather the columns of the owned entries: 8 lanes x 16 bytes span the slice, 32 columns in flight
    const int sub = tid & 7, grp = tid >> 3;
    const int o0 = slice * FC_OW + sub * 16;
    const bool o_ok = o0 < K;                       // K is a multiple of 16
    int acc[16];
    #pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0;
    const int8_t* wbase = p.Wt + o0;
    if (o_ok) {
        constexpr int U = 8;                           // columns in flight per thread
        for (int e = grp; e < mine; e += U * FC_GROUPS) {
            int j[U];
            uint4 w[U];
            #pragma unroll
            for (int u = 0; u < U; ++u) {
                const int eu = e + u * FC_GROUPS;
                j[u] = eu < mine ? s_list_j[eu] : -1;
            }
            #pragma unroll
            for (int u = 0; u < U; ++u)
                w[u] = j[u] >= 0 ? __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)j[u] * K)) : make_uint4(0, 0, 0, 0);
            #pragma unroll
            for (int u = 0; u < U; ++u)
                if (j[u] >= 0) fma16(acc, w[u], (int)s_xt[j[u]] - (int)s_xp[j[u]]);
        }
    }
    // ---- 4. reduce: the 4 column groups of a warp by shuffles, the 8 warps through shared memory
    #pragma unroll
    for (int i = 0; i < 16; ++i) {
        acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 8);
        acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 16);
    }
    if (lane < 8) {
        #pragma unroll
        for (int i = 0; i < 16; ++i) s_red[warp][lane * 16 + i] = acc[i];
    }
    __syncthreads();
    // ---- 5. across the cluster: every CTA pushes its partial sums into rank 0's shared memory, then
    // arrives at the cluster barrier; only rank 0 waits, adds them onto the projection slice it owns
    // (owner computes, no atomics), applies f and writes Y_t.
    cluster_wait();                                  // pairs with the arrive at kernel entry: all CTAs are running
    if (tid < FC_OW) {
        int v = 0;
        #pragma unroll
        for (int w = 0; w < FC_THREADS / 32; ++w) v += s_red[w][tid];
        *cluster.map_shared_rank(&s_part[kg][tid], 0) = v;
    }
    cluster_arrive_release();
    if (kg != 0) return;                             // nobody reads a non-zero rank's shared memory
    cluster_wait_acquire();
    if (tid < width) {
        int v = p_old;
        #pragma unroll
        for (int r = 0; r < FC_CL; ++r) v += s_part[r][tid];
        if (total > 0) Ps[tid] = v;
        if (p.Y) {
            const size_t oi = (size_t)s * K + slice * FC_OW + tid;
            if (p.shift < 0) reinterpret_cast<int32_t*>(p.Y)[oi] = v;
            else reinterpret_cast<int8_t*>(p.Y)[oi] = (int8_t)fc_apply_f(v, p.shift, p.act);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Two-kernel form of the same step, used when many streams are processed per call: the list of
// non-zero delta entries is built once per stream into global scratch memory instead of once per
// CTA, and the gather kernel needs no cross-CTA reduction (one CTA owns FC_OW outputs of a stream).
//   scratch layout: count[n] (int), then entries[n][c_in] (uint32: input index | (delta + 256) << 16)
// ------------------------------------------------------------------------------------------------
__host__ __device__ inline size_t fc_scratch_bytes(int n, int c_in) { return ((size_t)n * 4 + 15) / 16 * 16 + (size_t)n * c_in * 4; }
__host__ __device__ inline uint32_t* fc_scratch_entries(void* scratch, int n) {
    return reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(scratch) + ((size_t)n * 4 + 15) / 16 * 16);
}

__global__ void __launch_bounds__(FC_THREADS) fc_scan_kernel(FcParams p, void* scratch, int n)
{
    __shared__ int s_warp[FC_THREADS / 32];
    __shared__ int s_off[FC_THREADS];
    __shared__ unsigned long long s_mask[FC_THREADS];
    __shared__ __align__(16) int8_t s_xt[16 * FC_PT * FC_THREADS];
    __shared__ __align__(16) int8_t s_xp[16 * FC_PT * FC_THREADS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int s = blockIdx.x;
    const int C = p.c_in;
    const int nchunks = C >> 4;
    const uint4* xt4 = reinterpret_cast<const uint4*>(p.xt + (size_t)s * C);
    const uint4* xp4 = p.xprev ? reinterpret_cast<const uint4*>(p.xprev + (size_t)s * C) : nullptr;
    const int c_begin = tid * FC_PT;
    unsigned long long m = 0;
    #pragma unroll
    for (int i = 0; i < FC_PT; ++i) {
        if (c_begin + i < nchunks) {
            const uint4 a = __ldg(xt4 + c_begin + i);
            const uint4 b = xp4 ? xp4[c_begin + i] : make_uint4(0, 0, 0, 0);
            reinterpret_cast<uint4*>(s_xt)[c_begin + i] = a;
            reinterpret_cast<uint4*>(s_xp)[c_begin + i] = b;
            // the thread that read a chunk of the snapshot is the one that overwrites it: in place is safe
            if (p.xnext) reinterpret_cast<uint4*>(p.xnext + (size_t)s * C)[c_begin + i] = a;
            const unsigned cm = xp4 ? differing_bytes(a, b) : 0xffffu;
            m |= (unsigned long long)cm << (16 * i);
        }
    }
    const int local = __popcll(m);
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
    s_off[tid] = warp_off + incl - local;
    s_mask[tid] = m;
    __syncthreads();
    uint32_t* entries = fc_scratch_entries(scratch, n) + (size_t)s * C;
    for (int e = tid; e < total; e += FC_THREADS) {
        int t = 0;
        #pragma unroll
        for (int step = FC_THREADS / 2; step > 0; step >>= 1)
            if (s_off[t + step] <= e) t += step;
        const unsigned long long mk = s_mask[t];
        const int r = e - s_off[t];
        const unsigned lo32 = (unsigned)mk, hi32 = (unsigned)(mk >> 32);
        const int cl = __popc(lo32);
        const int bit = r < cl ? (int)__fns(lo32, 0, r + 1) : 32 + (int)__fns(hi32, 0, r - cl + 1);
        const int j = t * (16 * FC_PT) + bit;
        const int d = (int)s_xt[j] - (int)s_xp[j];
        entries[e] = (uint32_t)j | ((uint32_t)(d + 256) << 16);
    }
    if (tid == 0) reinterpret_cast<int*>(scratch)[s] = total;
    if (p.stat) {
        int groups32 = __popc((unsigned)((m | m >> 16) & 0xffffu) != 0) + __popc((unsigned)(((m >> 32) | (m >> 48)) & 0xffffu) != 0);
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) groups32 += __shfl_down_sync(0xffffffffu, groups32, o);
        if (lane == 0) s_warp[warp] = groups32;      // s_warp is free again: every thread is past its reads
        __syncthreads();
        if (tid == 0) {
            int g = 0;
            #pragma unroll
            for (int w = 0; w < FC_THREADS / 32; ++w) g += s_warp[w];
            p.stat[s * 2 + 0] = (unsigned long long)total;
            p.stat[s * 2 + 1] = (unsigned long long)g;
        }
    }
}

__global__ void __launch_bounds__(FC_THREADS) fc_gather_kernel(FcParams p, const void* scratch, int n)
{
    __shared__ int s_red[FC_THREADS / 32][FC_OW];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slice = blockIdx.x, s = blockIdx.y;
    const int C = p.c_in, K = p.c_out;
    const int total = reinterpret_cast<const int*>(scratch)[s];
    const uint32_t* entries = fc_scratch_entries(const_cast<void*>(scratch), n) + (size_t)s * C;
    int32_t* Ps = p.P + (size_t)s * K + slice * FC_OW;
    const int width = min(FC_OW, K - slice * FC_OW);
    int p_old = 0;
    if (tid < width) p_old = Ps[tid];
    const int sub = tid & 7, grp = tid >> 3;
    const int o0 = slice * FC_OW + sub * 16;
    int acc[16];
    #pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0;
    const int8_t* wbase = p.Wt + o0;
    if (o0 < K) {
        constexpr int U = 8;
        for (int e = grp; e < total; e += U * FC_GROUPS) {
            uint32_t ent[U];
            uint4 w[U];
            #pragma unroll
            for (int u = 0; u < U; ++u) {
                const int eu = e + u * FC_GROUPS;
                ent[u] = eu < total ? __ldg(entries + eu) : 0xffffffffu;
            }
            #pragma unroll
            for (int u = 0; u < U; ++u)
                w[u] = ent[u] != 0xffffffffu ? __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)(ent[u] & 0xffffu) * K))
                                             : make_uint4(0, 0, 0, 0);
            #pragma unroll
            for (int u = 0; u < U; ++u)
                if (ent[u] != 0xffffffffu) fma16(acc, w[u], (int)(ent[u] >> 16) - 256);
        }
    }
    #pragma unroll
    for (int i = 0; i < 16; ++i) {
        acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 8);
        acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 16);
    }
    if (lane < 8) {
        #pragma unroll
        for (int i = 0; i < 16; ++i) s_red[warp][lane * 16 + i] = acc[i];
    }
    __syncthreads();
    if (tid < width) {
        int v = p_old;
        #pragma unroll
        for (int w = 0; w < FC_THREADS / 32; ++w) v += s_red[w][tid];
        if (total > 0) Ps[tid] = v;
        if (p.Y) {
            const size_t oi = (size_t)s * K + slice * FC_OW + tid;
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

int fc_fused_create(rrm_net* net, Layer& L, const void* W_dev, const void* bias_dev)
{
    const int C = L.d.c_in, K = L.d.c_out, n = L.d.n;
    if (C % 16 || K % 16 || C > FC_CL * FC_LCAP || C > 16 * FC_PT * FC_THREADS) return RRM_ERR_UNSUPPORTED;
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
    RRM_TRY(alloc((void**)&L.fc_nnz, (size_t)n * 2 * 8));
    RRM_TRY(alloc((void**)&L.fc_scratch, fc_scratch_bytes(n, C)));
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
    RRM_TRY(fc_seq_create(net, L));
    if (L.d.variant == RRM_VARIANT_SPARSE_W) return fc_sparse_w_create(net, L);
    // the dense path (keyframe, rrm_dense) runs on the tensor cores when the inputs are whole 32-byte K chunks
    if (C % 32 == 0 && L.d.variant != RRM_VARIANT_GATHER) {
        RRM_TRY(conv_tc_create(net, L, W_dev));
        RRM_TRY(fc_tc_create(net, L));
    }
    return RRM_OK;
}

// dense:     every input entry is visited (keyframe or the stateless dense path)
// stateless: results go to the scratch projection P2, the RRM state is left untouched
int fc_fused_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, bool dense, bool stateless, cudaStream_t st)
{
    const int C = L.d.c_in, K = L.d.c_out, n = L.d.n;
    const int slices = ceil_div(K, FC_OW);
    // (without the few-row tensor-core form a handful of rows is served faster by the gather kernel with every entry active)
    if (dense && L.tc_ready && (n >= 4 || fc_tc_usable(L, n))) return fc_dense_tc_run(net, L, X_dev, Y_dev, 1, stateless, st);
    FcParams p;
    p.xt = reinterpret_cast<const int8_t*>(X_dev);
    p.Wt = L.Wt;
    p.c_in = C; p.c_out = K; p.shift = L.d.shift; p.act = L.d.act;
    p.Y = Y_dev;
    const int tot = n * (K > C ? K : C);
    if (dense) {
        int32_t* Pd = reinterpret_cast<int32_t*>(stateless ? L.P2 : L.P);
        fc_init_kernel<<<ceil_div(tot, 256), 256, 0, st>>>(Pd, reinterpret_cast<int32_t*>(L.bias), n, K, nullptr, C);
        p.xprev = nullptr;
        p.P = Pd;
        p.stat = nullptr;
        if (stateless) p.xnext = nullptr;
        else { p.xnext = L.xs[L.xs_cur ^ 1]; L.xs_cur ^= 1; }
    } else {
        p.xprev = L.xs[L.xs_cur];
        p.xnext = L.xs[L.xs_cur ^ 1];
        L.xs_cur ^= 1;
        p.P = reinterpret_cast<int32_t*>(L.P);
        p.stat = L.fc_nnz;
        L.seq_last_T = 0;
    }
    if (n < FC_TWO_KERNEL_MIN_STREAMS) {
        dim3 grid(FC_CL, slices, n);
        fc_delta_i8_kernel<<<grid, FC_THREADS, 0, st>>>(p);
    } else {
        fc_scan_kernel<<<n, FC_THREADS, 0, st>>>(p, L.fc_scratch, n);
        fc_gather_kernel<<<dim3(slices, n), FC_THREADS, 0, st>>>(p, L.fc_scratch, n);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

int fc_fused_projection(rrm_net* net, Layer& L, void* P_dev, cudaStream_t st)
{
    RRM_CUDA_TRY(cudaMemcpyAsync(P_dev, L.P, (size_t)L.d.n * L.d.c_out * 4, cudaMemcpyDeviceToDevice, st));
    return RRM_OK;
}

}  // namespace rrm

// ------------------------------------------------------------------------------------------------
// Allocation-free delta-FC step.  The per-stream non-zero lists live in a fixed array that is part
// of the loaded module, so the call needs no device allocation at all.
// ------------------------------------------------------------------------------------------------
namespace {

constexpr int NOALLOC_MAX_STREAMS = RRM_FC_NOALLOC_MAX_STREAMS;
constexpr int NOALLOC_MAX_C_IN = RRM_FC_NOALLOC_MAX_C_IN;
constexpr size_t NOALLOC_BYTES = ((size_t)NOALLOC_MAX_STREAMS * 4 + 15) / 16 * 16 +
                                 (size_t)NOALLOC_MAX_STREAMS * NOALLOC_MAX_C_IN * 4;

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_fc_noalloc_scratch[NOALLOC_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
void* g_noalloc_ptr[NOALLOC_MAX_DEVICES];          // device address of the array, per device
std::mutex g_noalloc_mutex;

// In host code the array's name is only a handle: the address a kernel can use has to be asked for,
// once per device, with that device current.
int noalloc_scratch(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return RRM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_fc_noalloc_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return RRM_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return RRM_OK;
}

}  // namespace

extern "C" int rrm_fc_step_noalloc(const int8_t* Wt_dev, const int8_t* Xt_dev, int8_t* Xprev_dev, int32_t* P_dev,
                                   void* Y_dev, int n, int c_in, int c_out, int shift, int act, void* stream)
{
    using namespace rrm;
    if (!Wt_dev || !Xt_dev || !Xprev_dev || !P_dev) return RRM_ERR_INVALID_ARG;
    if (n < 1 || c_in < 1 || c_out < 1) return RRM_ERR_SHAPE;
    if (n > NOALLOC_MAX_STREAMS || c_in > NOALLOC_MAX_C_IN) return RRM_ERR_CAPACITY;
    if (c_in % 16 || c_out % 16) return RRM_ERR_SHAPE;
    if (act != RRM_ACT_NONE && act != RRM_ACT_RELU) return RRM_ERR_INVALID_ARG;
    if (shift > 30 || (shift < 0 && act != RRM_ACT_NONE)) return RRM_ERR_INVALID_ARG;
    if (((uintptr_t)Wt_dev | (uintptr_t)Xt_dev | (uintptr_t)Xprev_dev) & 15) return RRM_ERR_INVALID_ARG;
    if (((uintptr_t)P_dev & 3) || (Y_dev && shift < 0 && ((uintptr_t)Y_dev & 3))) return RRM_ERR_INVALID_ARG;
    void* scratch = nullptr;
    RRM_TRY(noalloc_scratch(&scratch));
    FcParams p;
    p.xt = Xt_dev; p.xprev = Xprev_dev; p.xnext = Xprev_dev;   // snapshot updated in place
    p.Wt = Wt_dev; p.P = P_dev; p.Y = Y_dev; p.stat = nullptr;
    p.c_in = c_in; p.c_out = c_out; p.shift = shift; p.act = act;
    cudaStream_t st = (cudaStream_t)stream;
    fc_scan_kernel<<<n, FC_THREADS, 0, st>>>(p, scratch, n);
    fc_gather_kernel<<<dim3(ceil_div(c_out, FC_OW), n), FC_THREADS, 0, st>>>(p, scratch, n);
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

