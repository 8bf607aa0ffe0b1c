// Convolution path of the RRM step (Algorithm 1, conv branch), CUDA-core variant.
//
// All tensors inside the library are pixel-major ([n][h][w][units]); a "unit" is one float,
// four int8 channels, or 32 sign bits.  Per frame and layer:
//   import_delta   (layer input = the external frame only)  D = X_t - X_prev, per-pixel activity
//                  bitmap, X_prev := X_t in place for changed pixels;
//   delta_conv     implicit GEMM over the projection pixels that can change: every CTA finds its
//                  rows by a prefix sum over the layer's bitmap of such pixels; K = taps x input
//                  units gathered from the delta rows of active input pixels (zero otherwise),
//                  N = output channels; P_prev += result (owner computes: no float atomics);
//   epilogue       recomputes f only where its window touches an updated projection pixel,
//                  compares with the stored activation and emits the next layer's delta rows,
//                  activity bitmap and snapshot update in one pass.
// A kernel that finds a changed pixel of a tensor (import, epilogue) also marks, in the bitmap of every
// layer that reads the tensor, the projection pixels whose filter footprint covers it, and counts the
// exact multiply-accumulates the non-zero deltas imply (Table 1): no separate pass over the activity.
// The same GEMM kernel with DENSE=true (all pixels, input values instead of deltas, bias added)
// is the library's dense path and the keyframe.
#include "rrm_common.cuh"
#include "rrm_rows.cuh"
#include "rrm_tc.cuh"
#include "rrm_dev.cuh"
#include <type_traits>
#include <array>
#include <vector>

namespace rrm {

constexpr int TM = 64;            // projection pixels per CTA
constexpr int TN = GEMM_TN;       // output channels per CTA
constexpr int TK = GEMM_TK;       // K units per stage
constexpr int CONV_THREADS = 128;
constexpr int RM = TM * 16 / CONV_THREADS;   // rows of the tile per thread (x 4 output channels): 16 threads span the TN = 64 channels
static_assert(TN == 64 && CONV_THREADS >= TM && TM % (CONV_THREADS / 8) == 0, "thread layout of conv_gemm_kernel");

struct ConvParams {
    const void* D;            // delta rows (delta mode) / unused (dense)
    const void* X;            // input values (dense mode; binary delta mode: new sign bits)
    const uint32_t* in_act;   // input activity bitmap (delta mode)
    const uint32_t* oact;     // projection pixels to update (delta mode)
    int* ocount;              // receives their number
    const void* Wk;           // [kup][np] units
    const void* bias;
    void* P;                  // [opixels][c_out]
    int* errw;
    int n, c_in, h, w, u_in, oh, ow, kh, kw, stride, pad, c_out, np, ku, kup, opixels;
    int ksplit;               // gridDim.z: CTAs that share one output tile, each with a contiguous range of K stages
    unsigned wait_limit;      // polls of one bounded wait
    const uint32_t* count_bitmap;   // dense evaluation inside a delta step: the layer's update bitmap, whose set bits the
                                    // first CTA counts into *ocount (the measured activity); nullptr otherwise
    // several frames in one launch (delta only, K not split; gridDim.z = frames): frame g reads its delta rows, new
    // rows and bitmaps, and stores its product, at these distances from frame 0's
    int frames;
    long long row_stride;     // bytes between the frames' sets of delta rows (and of new rows)
    long long arena_stride;   // bytes between the frames' arenas (bitmaps, counters)
    long long p_stride;       // elements between the frames' products
    unsigned magic_u, magic_kw;     // ceil(2^32 / u_in), ceil(2^32 / kw): quotients by a multiply-high (0: the divisor is 1); set by launch_gemm
};

// The number of set bits of bm[0 .. words) -> *out, by one CTA (the activity of a layer that is evaluated densely).
__device__ __forceinline__ void count_bits_cta(const uint32_t* __restrict__ bm, int words, int* out, int* s_scratch)
{
    int c = 0;
    for (int i = threadIdx.x; i < words; i += blockDim.x) c += __popc(__ldg(bm + i));
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if ((threadIdx.x & 31) == 0) s_scratch[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < (int)((blockDim.x + 31) >> 5); ++w) t += s_scratch[w];
        *out = t;
    }
    __syncthreads();
}

__device__ __forceinline__ bool bit_test(const uint32_t* bm, int i) { return (bm[i >> 5] >> (i & 31)) & 1u; }

// ------------------------------------------------------------------------------------------------
// Implicit GEMM on the CUDA cores.  DT: T_F32 (float FMA), T_I8 (dp4a on 4-channel words), T_BIN
// (popcount on 32-channel words: sum(d*w) = 2*(popc(changed) - 2*popc(changed & (new ^ wbits))), dense:
// valid instead of changed and no factor 2).
//
// A CTA owns TM projection pixels x TN output channels and walks K = taps x input units in stages of
// TK units through a ring of GEMM_STAGES shared-memory buffers:
//   - the filter slice of a stage ([TK][TN] words, contiguous in the packed filters) is staged with one
//     bulk copy (cp.async.bulk) that completes on an mbarrier;
//   - the activation slice is gathered with asynchronous copies (16 bytes = 4 K units of one row at a
//     time when the units per pixel allow it, 8 lanes covering 128 contiguous bytes of a pixel row; else
//     4 bytes), zero-filled where the input pixel is outside the image or did not change; which taps
//     are usable is decided once per row (a 128-bit mask in shared memory), so the gather addresses
//     depend on no further load;
//   - stages none of whose taps is usable under any row of the tile are skipped.
// Copies of later stages are in flight while the current one is multiplied (RM x 4 outputs per thread).
// ------------------------------------------------------------------------------------------------
constexpr int GEMM_STAGES = 3;
constexpr int GEMM_LDA = TK + 4;                   // words per activation row in shared memory (16-byte aligned, bank-staggered)
constexpr int GEMM_A_WORDS = TM * GEMM_LDA, GEMM_B_WORDS = TK * TN;

__device__ __forceinline__ uint32_t g_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void g_cp_async4(uint32_t dst, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void g_cp_async16(uint32_t dst, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// Two fp32 multiply-adds per instruction (each rounded as fmaf rounds): acc = a * b + acc on both halves of 64-bit pairs.
__device__ __forceinline__ unsigned long long g_pack2(uint32_t lo, uint32_t hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void g_fma2(unsigned long long& acc, unsigned long long a, unsigned long long b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}

template <int DT, bool DENSE, bool VEC>
__global__ void __launch_bounds__(CONV_THREADS) conv_gemm_kernel(ConvParams p)
{
    using acc_t = typename std::conditional<DT == T_F32, float, int>::type;
    constexpr int A_BUFS = (DT == T_BIN) ? 2 : 1;
    extern __shared__ __align__(128) uint32_t g_smem[];    // [stages][B | A | (A2)]
    constexpr int STAGE_WORDS = GEMM_B_WORDS + A_BUFS * GEMM_A_WORDS;
    __shared__ __align__(8) unsigned long long s_full[GEMM_STAGES];
    __shared__ int s_q[TM];
    __shared__ int s_tmp[256 + 34];
    __shared__ unsigned s_tapmask[4];
    __shared__ uint32_t s_live[8];                           // bit r: stage s_first + r has a usable tap (the first 256 stages of the CTA's range)
    __shared__ unsigned long long s_rmask[TM][2];
    __shared__ int s_pix0[TM];
    __shared__ int s_fcnt[32];                               // several frames per launch: every frame's number of rows

    const int tid = threadIdx.x, lane = tid & 31;
    int tile = blockIdx.x;
    const int n0 = blockIdx.y * TN;
    const bool batched = !DENSE && p.frames > 1;             // gridDim.z counts frames x shares of K (shares: fp32 only)
    const int zshare = batched ? (int)(blockIdx.z % p.ksplit) : (int)blockIdx.z;
    pdl_launch_dependents();
    if (!DENSE) {
        pdl_wait();                                          // the update bitmap is the predecessors' work
        if (batched) {
            // Which (frame, tile) this CTA takes: the tiles that have rows, numbered frame by frame, go to the CTAs in
            // launch order (gridDim.x * gridDim.z of them per N tile), so that the CTAs with work come first and spread
            // evenly over the SMs instead of landing wherever an active frame's block index happens to fall.  Every
            // CTA counts all frames' update bitmaps for that (a few words per frame and lane).
            const int words = (p.opixels + 31) >> 5, nfr = (int)gridDim.z / p.ksplit;
            for (int g = tid >> 5; g < nfr; g += CONV_THREADS / 32) {
                const uint32_t* bm = reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(p.oact) + (long long)g * p.arena_stride);
                int c = 0;
                for (int i = lane; i < words; i += 32) c += __popc(__ldg(bm + i));
                c = __reduce_add_sync(0xffffffffu, c);
                if (lane == 0) s_fcnt[g] = c;
            }
            __syncthreads();
            int id = (int)((blockIdx.z / p.ksplit) * gridDim.x + blockIdx.x), frame = -1;   // (the shares of a tile agree)
            if (id == 0 && blockIdx.y == 0 && zshare == 0 && tid < nfr)     // every frame's count, also of frames without a tile
                *reinterpret_cast<int*>(reinterpret_cast<char*>(p.ocount) + (long long)tid * p.arena_stride) = s_fcnt[tid];
            for (int g = 0; g < nfr; ++g) {
                const int t = (s_fcnt[g] + TM - 1) / TM;
                if (id < t) { frame = g; break; }
                id -= t;
            }
            if (frame < 0) return;
            tile = id;
            const long long g = frame;
            p.D = reinterpret_cast<const char*>(p.D) + g * p.row_stride;
            p.X = reinterpret_cast<const char*>(p.X) + g * p.row_stride;
            p.in_act = reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(p.in_act) + g * p.arena_stride);
            p.oact = reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(p.oact) + g * p.arena_stride);
            p.P = reinterpret_cast<char*>(p.P) + g * p.p_stride * 4;
        }
        // this CTA's rows: the tile-th group of TM set bits of the layer's update bitmap
        const int count = select_rows<TM>(p.oact, (p.opixels + 31) >> 5, tile, s_q, s_tmp);
        if (!batched && tile == 0 && blockIdx.y == 0 && zshare == 0 && tid == 0) *p.ocount = count;
        if (tile * TM >= count) return;
    }
    if (tid == 0) {
        for (int s = 0; s < GEMM_STAGES; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(g_smem_u32(&s_full[s])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 4) s_tapmask[tid] = 0;
    if (tid < 8) s_live[tid] = 0;
    __syncthreads();

    // ---- per row: the input pixel under tap (0,0) and the usable taps
    const int taps = p.kh * p.kw;
    if (tid < TM) {
        const int r = tile * TM + tid;
        const int q = DENSE ? (r < p.opixels ? r : -1) : s_q[tid];
        s_q[tid] = q;
        int pix0 = 0;
        unsigned long long m0 = 0, m1 = 0;
        if (q >= 0) {
            const int ox = q % p.ow, oy = (q / p.ow) % p.oh, ns = q / (p.ow * p.oh);
            const int y0 = oy * p.stride - p.pad, x0 = ox * p.stride - p.pad;
            pix0 = ns * p.h * p.w + y0 * p.w + x0;
            row_tap_masks<DENSE>(p.in_act, pix0, y0, x0, p.h, p.w, p.kh, p.kw, m0, m1);
        }
        s_pix0[tid] = pix0;
        s_rmask[tid][0] = m0; s_rmask[tid][1] = m1;
        const unsigned a0 = __reduce_or_sync(0xffffffffu, (unsigned)m0), a1 = __reduce_or_sync(0xffffffffu, (unsigned)(m0 >> 32));
        const unsigned a2 = __reduce_or_sync(0xffffffffu, (unsigned)m1), a3 = __reduce_or_sync(0xffffffffu, (unsigned)(m1 >> 32));
        if (lane == 0) {
            if (a0) atomicOr(&s_tapmask[0], a0);
            if (a1) atomicOr(&s_tapmask[1], a1);
            if (a2) atomicOr(&s_tapmask[2], a2);
            if (a3) atomicOr(&s_tapmask[3], a3);
        }
    }
    __syncthreads();
    const unsigned long long tm0 = (unsigned long long)s_tapmask[0] | (unsigned long long)s_tapmask[1] << 32;
    const unsigned long long tm1 = (unsigned long long)s_tapmask[2] | (unsigned long long)s_tapmask[3] << 32;
    if (DENSE) pdl_wait();                                   // barriers and row tables are set up; the inputs come next
    if (DENSE && p.count_bitmap && tile == 0 && blockIdx.y == 0 && zshare == 0)
        count_bits_cta(p.count_bitmap, (p.opixels + 31) >> 5, p.ocount, s_tmp);
    // this CTA's share of the K stages
    const int all_stages = p.kup / TK, per_split = (all_stages + p.ksplit - 1) / p.ksplit;
    const int s_first = zshare * per_split, n_stages = min(all_stages, s_first + per_split);
    auto div_u = [&](int x) -> int { return p.magic_u ? (int)__umulhi((unsigned)x, p.magic_u) : x; };
    auto div_kw = [&](int x) -> int { return p.magic_kw ? (int)__umulhi((unsigned)x, p.magic_kw) : x; };
    auto stage_live = [&](int ks) -> bool {                 // any usable tap among the stage's K units?
        const int t_lo = div_u(ks * TK), t_hi = min(taps - 1, div_u(ks * TK + TK - 1));
        for (int t = t_lo; t <= t_hi; ++t)
            if (t < 64 ? (tm0 >> t) & 1ull : (tm1 >> (t - 64)) & 1ull) return true;
        return false;
    };
    // which stages are live is worked out once, by all threads, and kept as a bitmap: the loop then finds its next
    // stage with a shift (ranges beyond 256 stages test the rest stage by stage)
    const int n_range = max(0, n_stages - s_first);
    for (int r = tid; r < min(n_range, 256); r += CONV_THREADS)
        if (stage_live(s_first + r)) atomicOr(&s_live[r >> 5], 1u << (r & 31));
    __syncthreads();
    auto next_live = [&](int ks) -> int {                   // first live stage >= ks, or n_stages
        int r = ks - s_first;
        while (r < min(n_range, 256)) {
            const uint32_t wbits = s_live[r >> 5] >> (r & 31);
            if (wbits) return s_first + r + __ffs(wbits) - 1;
            r = (r | 31) + 1;
        }
        ks = s_first + max(r, ks - s_first);
        while (ks < n_stages && !stage_live(ks)) ++ks;
        return min(ks, n_stages);
    };

    const uint32_t* Du = reinterpret_cast<const uint32_t*>(p.D);
    const uint32_t* Xu = reinterpret_cast<const uint32_t*>(p.X);
    const uint32_t* Wu = reinterpret_cast<const uint32_t*>(p.Wk) + (size_t)blockIdx.y * p.kup * TN;   // this N tile's filters
    const uint32_t smem_base = g_smem_u32(g_smem);
    const uint32_t tail_mask = (p.c_in & 31) ? ((1u << (p.c_in & 31)) - 1u) : 0xffffffffu;

    // issues the copies of stage `ks` into ring slot `slot`
    auto issue = [&](int ks, int slot) {
        const uint32_t sB = smem_base + (uint32_t)(slot * STAGE_WORDS) * 4u, sA = sB + GEMM_B_WORDS * 4u;
        if (tid == 0) {
            const uint32_t bar = g_smem_u32(&s_full[slot]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier reads of the slot precede the bulk write
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)(GEMM_B_WORDS * 4)) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(sB), "l"(Wu + (size_t)ks * GEMM_B_WORDS), "r"((uint32_t)(GEMM_B_WORDS * 4)), "r"(bar) : "memory");
        }
        // thread -> (row = tid / 8 [+ a pass of CONV_THREADS / 8 rows], piece = tid % 8): 8 lanes cover the 32 K units of one row
        const int piece = tid & 7;
        #pragma unroll
        for (int half = 0; half < TM / (CONV_THREADS / 8); ++half) {
            const int row = (tid >> 3) + half * (CONV_THREADS / 8);
            const unsigned long long rm0 = s_rmask[row][0], rm1 = s_rmask[row][1];
            const int pix0 = s_pix0[row];
            #pragma unroll
            for (int i = 0; i < (VEC ? 1 : 4); ++i) {
                const int kk = VEC ? piece * 4 : piece + 8 * i, k = ks * TK + kk;
                const int tap = div_u(k), u = k - tap * p.u_in;
                const int ky = div_kw(tap), kx = tap - ky * p.kw;
                const bool use = tap < taps && ((tap < 64 ? rm0 >> tap : rm1 >> (tap - 64)) & 1ull);
                const size_t off = use ? (size_t)(pix0 + ky * p.w + kx) * p.u_in + u : 0;
                const int sidx = row * GEMM_LDA + kk;
                const uint32_t dst = sA + (uint32_t)sidx * 4u;
                if (DT == T_BIN) {
                    // first buffer: changed bits (dense: the valid-channel mask, written directly), second: sign bits
                    if (DENSE) {
                        uint32_t* d = g_smem + slot * STAGE_WORDS + GEMM_B_WORDS + sidx;
                        #pragma unroll
                        for (int j = 0; j < (VEC ? 4 : 1); ++j) d[j] = use ? ((u + j == p.u_in - 1) ? tail_mask : 0xffffffffu) : 0u;
                    } else if (VEC) g_cp_async16(dst, Du + off, use ? 16u : 0u);
                    else g_cp_async4(dst, Du + off, use ? 4u : 0u);
                    if (VEC) g_cp_async16(dst + GEMM_A_WORDS * 4u, Xu + off, use ? 16u : 0u);
                    else g_cp_async4(dst + GEMM_A_WORDS * 4u, Xu + off, use ? 4u : 0u);
                } else if (VEC) {
                    g_cp_async16(dst, (DENSE ? Xu : Du) + off, use ? 16u : 0u);
                } else {
                    g_cp_async4(dst, (DENSE ? Xu : Du) + off, use ? 4u : 0u);
                }
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    const int tm = (tid >> 4) * RM, tn = (tid & 15) * 4;   // RM x 4 outputs per thread
    acc_t acc[RM][4];
    unsigned long long acc2[RM][2];                        // fp32: the same accumulators as pairs (channels 0-1, 2-3)
    int rowpop[RM];                                        // binary: changed (dense: valid) bits of the thread's rows
    #pragma unroll
    for (int i = 0; i < RM; ++i) {
        rowpop[i] = 0;
        acc2[i][0] = acc2[i][1] = 0ull;
        #pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;
    }
    bool ok = true;

    // prologue: the first GEMM_STAGES - 1 live stages
    int ks_issue = next_live(s_first), issued = 0;
    for (int s = 0; s < GEMM_STAGES - 1; ++s) {
        if (ks_issue < n_stages) { issue(ks_issue, issued % GEMM_STAGES); ++issued; ks_issue = next_live(ks_issue + 1); }
        else asm volatile("cp.async.commit_group;" ::: "memory");
    }
    int it = 0;
    for (int ks = next_live(s_first); ks < n_stages; ks = next_live(ks + 1), ++it) {
        const int slot = it % GEMM_STAGES;
        asm volatile("cp.async.wait_group %0;" ::"n"(GEMM_STAGES - 2) : "memory");   // this thread's copies of stage `it` landed
        if (!mbar_wait(g_smem_u32(&s_full[slot]), (it / GEMM_STAGES) & 1, p.wait_limit)) ok = false;
        // everyone's copies landed; everyone is done with stage it - 1.  A wait that ran out in any thread ends the
        // loop for all of them: nothing more is issued
        if (__syncthreads_or(!ok)) { ok = false; break; }
        if (ks_issue < n_stages) { issue(ks_issue, issued % GEMM_STAGES); ++issued; ks_issue = next_live(ks_issue + 1); }
        else asm volatile("cp.async.commit_group;" ::: "memory");
        const uint32_t* Bs = g_smem + slot * STAGE_WORDS;
        const uint32_t* As = Bs + GEMM_B_WORDS;
        #pragma unroll 4
        for (int k4 = 0; k4 < TK; k4 += 4) {
            uint4 ar[RM], an[RM];                             // 4 K units of each of the thread's rows
            #pragma unroll
            for (int i = 0; i < RM; ++i) {
                ar[i] = *reinterpret_cast<const uint4*>(&As[(tm + i) * GEMM_LDA + k4]);
                if (DT == T_BIN) an[i] = *reinterpret_cast<const uint4*>(&As[GEMM_A_WORDS + (tm + i) * GEMM_LDA + k4]);
            }
            #pragma unroll
            for (int kq = 0; kq < 4; ++kq) {
                const uint4 bw = *reinterpret_cast<const uint4*>(&Bs[(k4 + kq) * TN + tn]);
                const uint32_t b[4] = {bw.x, bw.y, bw.z, bw.w};
                #pragma unroll
                for (int i = 0; i < RM; ++i) {
                    const uint32_t a = kq == 0 ? ar[i].x : kq == 1 ? ar[i].y : kq == 2 ? ar[i].z : ar[i].w;
                    uint32_t nw = 0;
                    if (DT == T_BIN) {
                        nw = kq == 0 ? an[i].x : kq == 1 ? an[i].y : kq == 2 ? an[i].z : an[i].w;
                        rowpop[i] += __popc(a);
                    }
                    if (DT == T_F32) {
                        const unsigned long long aa = g_pack2(a, a);
                        g_fma2(acc2[i][0], aa, g_pack2(b[0], b[1]));
                        g_fma2(acc2[i][1], aa, g_pack2(b[2], b[3]));
                    } else {
                        #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (DT == T_I8) acc[i][j] = __dp4a((int)a, (int)b[j], (int)acc[i][j]);
                            else acc[i][j] += __popc(a & (nw ^ b[j]));
                        }
                    }
                }
            }
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (DT == T_F32) {
        #pragma unroll
        for (int i = 0; i < RM; ++i)
            #pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t lo, hi;
                asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(acc2[i][h]));
                acc[i][2 * h] = (acc_t)__uint_as_float(lo); acc[i][2 * h + 1] = (acc_t)__uint_as_float(hi);
            }
    }
    if (!ok) {
        // giving up: the filter slices still on their way (stages issued, not consumed) must land before the CTA's
        // shared memory goes away; thread 0 issued them and waits for them, the others wait for thread 0
        if (tid == 0) {
            atomicOr(p.errw, ERRW_TIMEOUT);
            for (int j = it; j < issued; ++j)
                mbar_wait(g_smem_u32(&s_full[j % GEMM_STAGES]), (j / GEMM_STAGES) & 1, WAIT_LIMIT_DEFAULT);
        }
        __syncthreads();
        if (!(DT == T_F32 && p.ksplit > 1)) return;          // (an fp32 share still meets its cluster at the barriers below)
    }

    // ---- fp32 with the K range split over CTAs: the shares of a tile form one thread-block cluster and their partial
    // sums meet through distributed shared memory in a FIXED order (share 0, 1, ...), so the stored projection is
    // reproducible bit for bit and no float atomics are needed.  Every share parks its partial tile in its own
    // shared memory; share r then adds up rows [r * TM / shares, (r + 1) * TM / shares) of all shares and updates
    // the projection for them.
    if (DT == T_F32 && p.ksplit > 1) {
        float* tilebuf = reinterpret_cast<float*>(g_smem);   // [TM][TN]; the ring is free: every issued stage was consumed
        __syncthreads();
        #pragma unroll
        for (int i = 0; i < RM; ++i)
            *reinterpret_cast<float4*>(&tilebuf[(tm + i) * TN + tn]) = make_float4((float)acc[i][0], (float)acc[i][1], (float)acc[i][2], (float)acc[i][3]);
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        const int rank = zshare, rows_per = TM / p.ksplit;
        const uint32_t tile_u32 = g_smem_u32(tilebuf);
        float* P = reinterpret_cast<float*>(p.P);
        for (int item = tid; item < rows_per * (TN / 4); item += CONV_THREADS) {
            const int row = rank * rows_per + item / (TN / 4), c4 = (item % (TN / 4)) * 4;
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int z = 0; z < p.ksplit; ++z) {
                uint32_t remote;
                float4 v;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(tile_u32 + (uint32_t)(row * TN + c4) * 4u), "r"(z));
                asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
                sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
            }
            const int q = s_q[row];
            if (q < 0 || !ok) continue;
            const float sv[4] = {sum.x, sum.y, sum.z, sum.w};
            #pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int co = n0 + c4 + j;
                if (co >= p.c_out) continue;
                const size_t o = (size_t)q * p.c_out + co;
                if (DENSE) P[o] = sv[j] + (p.bias ? reinterpret_cast<const float*>(p.bias)[co] : 0.f);
                else if (batched) P[o] = sv[j];              // (several frames per launch: the product is stored, not added)
                else P[o] += sv[j];
            }
        }
        // nobody leaves while its tile may still be read
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        return;
    }

    // ---- update of the stored projection: the owner of a tile writes it; CTAs that share a tile
    // (split K) add their partial sums with atomics (dense: onto a zeroed projection, split 0 adds the bias)
    const bool shared_tile = p.ksplit > 1;
    #pragma unroll
    for (int i = 0; i < RM; ++i) {
        const int q = s_q[tm + i];
        if (q < 0) continue;
        #pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int co = n0 + tn + j;
            if (co >= p.c_out) continue;
            const size_t o = (size_t)q * p.c_out + co;
            if (DT == T_F32) {                                 // (a tile owned by one CTA; shared fp32 tiles were closed above)
                float* P = reinterpret_cast<float*>(p.P);
                float v = acc[i][j];
                if (DENSE && p.bias) v += reinterpret_cast<const float*>(p.bias)[co];
                if (DENSE || batched) P[o] = v;            // (several frames per launch: the product is stored, not added)
                else P[o] += v;
            } else {
                int* P = reinterpret_cast<int*>(p.P);
                int v = (int)acc[i][j];
                if (DT == T_BIN) v = DENSE ? (rowpop[i] - 2 * v) : 2 * (rowpop[i] - 2 * v);
                if (DENSE && zshare == 0 && p.bias) v += reinterpret_cast<const int*>(p.bias)[co];
                if (shared_tile) atomicAdd(P + o, v);
                else if (DENSE || batched) P[o] = v;
                else P[o] += v;
            }
        }
    }
}

static size_t gemm_smem_bytes(int dt)
{
    return (size_t)GEMM_STAGES * (GEMM_B_WORDS + (dt == T_BIN ? 2 : 1) * GEMM_A_WORDS) * 4;
}

template <int DT, bool DENSE>
static void launch_gemm(const ConvParams& p_in, dim3 grid, cudaStream_t st)
{
    ConvParams p = p_in;
    const int cluster_z = (DT == T_F32 && p.ksplit > 1) ? p.ksplit : 1;       // fp32 shares of a tile: one cluster
    // (exact while the dividend stays below 2^32 / divisor: K units and taps are far below that)
    p.magic_u = p.u_in > 1 ? (unsigned)(((1ull << 32) + p.u_in - 1) / p.u_in) : 0u;
    p.magic_kw = p.kw > 1 ? (unsigned)(((1ull << 32) + p.kw - 1) / p.kw) : 0u;
    if (p.u_in % 4 == 0) launch_seq_cluster(conv_gemm_kernel<DT, DENSE, true>, dim3(grid), dim3(CONV_THREADS), gemm_smem_bytes(DT), st, cluster_z, p);
    else launch_seq_cluster(conv_gemm_kernel<DT, DENSE, false>, dim3(grid), dim3(CONV_THREADS), gemm_smem_bytes(DT), st, cluster_z, p);
}

template <int DT>
static int gemm_allow_smem()
{
    const int b = (int)gemm_smem_bytes(DT);
    if (DT == T_F32) {                                       // clusters of 16 CTAs are beyond the portable size of 8
        RRM_CUDA_TRY(cudaFuncSetAttribute(conv_gemm_kernel<DT, true, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        RRM_CUDA_TRY(cudaFuncSetAttribute(conv_gemm_kernel<DT, false, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        RRM_CUDA_TRY(cudaFuncSetAttribute(conv_gemm_kernel<DT, true, false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        RRM_CUDA_TRY(cudaFuncSetAttribute(conv_gemm_kernel<DT, false, false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    }
    RRM_CUDA_TRY(cudaFuncSetAttribute(conv_gemm_kernel<DT, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b));
    RRM_CUDA_TRY(cudaFuncSetAttribute(conv_gemm_kernel<DT, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b));
    RRM_CUDA_TRY(cudaFuncSetAttribute(conv_gemm_kernel<DT, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, b));
    RRM_CUDA_TRY(cudaFuncSetAttribute(conv_gemm_kernel<DT, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, b));
    return RRM_OK;
}

// ------------------------------------------------------------------------------------------------
// Filter repack: W[c_out][c_in][kh][kw] -> Wk[n tile][k][TN] with k = tap * u_in + unit (zero padded), so
// that the filter slice of one GEMM stage ([TK][TN] words of one N tile) is one contiguous block.
// ------------------------------------------------------------------------------------------------
__global__ void pack_weights_kernel(const void* W, uint32_t* Wk, int dt, int c_in, int c_out, int kh, int kw,
                                    int u_in, int kup, int np)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= kup * np) return;
    const int nt = idx / (kup * TN), k = (idx / TN) % kup, co = nt * TN + idx % TN;
    uint32_t out = 0;
    const int taps = kh * kw;
    const int tap = k / u_in, u = k - tap * u_in;
    if (tap < taps && co < c_out) {
        const size_t base = (size_t)co * c_in * taps + tap;        // + ci * taps
        if (dt == T_F32) {
            out = __float_as_uint(reinterpret_cast<const float*>(W)[base + (size_t)u * taps]);
        } else if (dt == T_I8) {
            for (int b = 0; b < 4; ++b) {
                const int ci = 4 * u + b;
                const int v = ci < c_in ? reinterpret_cast<const int8_t*>(W)[base + (size_t)ci * taps] : 0;
                out |= ((uint32_t)v & 0xffu) << (8 * b);
            }
        } else {
            for (int b = 0; b < 32; ++b) {
                const int ci = 32 * u + b;
                if (ci < c_in && reinterpret_cast<const int8_t*>(W)[base + (size_t)ci * taps] > 0) out |= 1u << b;
            }
        }
    }
    Wk[idx] = out;
}

// ------------------------------------------------------------------------------------------------
// Import of the external frame (boundary layout [n][c][h][w]) into tensor 0, with or without delta.
// One CTA handles 32 consecutive pixels of one stream: coalesced reads along w, transposed through
// shared memory, coalesced pixel-major writes.
// ------------------------------------------------------------------------------------------------
constexpr int IMP_TP = 32;                  // pixels per tile = lanes of the warp that marks their footprints

template <typename T, bool DELTA>
__global__ void __launch_bounds__(256) import_nchw_kernel(const T* __restrict__ src, T* X, T* D, uint32_t* act,
                                                          int* pnnz, unsigned long long* nnz,
                                                          unsigned long long* npix, int* errw,
                                                          int c, int cs, int hw, int w, Readers readers,
                                                          float eps, double* trunc, SeqFrames sf)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* s_x = reinterpret_cast<T*>(smem_raw);               // [IMP_TP][cs + 1] (several frames per launch: a second tile, the frame before)
    __shared__ int s_cnt[IMP_TP];
    const int ld = cs + 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ns = blockIdx.y, pix0 = blockIdx.x * IMP_TP;
    // several frames per launch: frame g is compared with frame g-1 at the boundary, not with the snapshot, which
    // only the last frame writes (all of it)
    const bool seq = DELTA && sf.frames > 1;
    T* s_p = s_x + IMP_TP * ld;
    if (seq) {
        const long long g = blockIdx.z;
        src += g * sf.in_stride;
        D = shift_bytes(D, g * sf.row_stride);
        act = shift_bytes(act, g * sf.arena_stride); nnz = shift_bytes(nnz, g * sf.arena_stride);
        npix = shift_bytes(npix, g * sf.arena_stride);
    }
    const long long arena_off = seq ? (long long)blockIdx.z * sf.arena_stride : 0;
    const bool write_x = !seq || (int)blockIdx.z == sf.frames - 1;
    pdl_launch_dependents();
    pdl_wait();
    if (tid < IMP_TP) s_cnt[tid] = 0;
    for (int ch = warp; ch < cs; ch += 8) {
        T v = 0, pv = 0;
        if (ch < c && pix0 + lane < hw) {
            v = src[((size_t)ns * c + ch) * hw + pix0 + lane];
            if (seq) pv = (src - sf.in_stride)[((size_t)ns * c + ch) * hw + pix0 + lane];
        }
        s_x[lane * ld + ch] = v;
        if (seq) s_p[lane * ld + ch] = pv;
    }
    __syncthreads();
    const size_t gp0 = (size_t)ns * hw + pix0;
    float sq = 0.f;                                          // squares of the truncated delta entries
    for (int idx = tid; idx < IMP_TP * cs; idx += 256) {
        const int pl = idx / cs, ch = idx - pl * cs;
        if (pix0 + pl >= hw) continue;
        const size_t o = (gp0 + pl) * cs + ch;
        const T xt = s_x[pl * ld + ch];
        if (DELTA) {
            const T xp = seq ? s_p[pl * ld + ch] : X[o];
            T dv = (T)(xt - xp);
            if (seq && write_x) X[o] = xt;
            if (xt != xp) {
                if (!seq) X[o] = xt;                         // the snapshot always moves on to the new frame
                bool keep = true;
                if (sizeof(T) == 4 && eps > 0.f) keep = fabsf((float)dv) >= eps;   // Sec. 3.4: small deltas are truncated
                if (keep) atomicAdd(&s_cnt[pl], 1);
                else { sq += (float)dv * (float)dv; dv = (T)0; }
                if (sizeof(T) == 1) {
                    const int d = (int)xt - (int)xp;
                    if (d < -128 || d > 127) atomicOr(errw, ERRW_BOUNDS);
                }
            }
            s_x[pl * ld + ch] = dv;
        } else {
            X[o] = xt;
        }
    }
    if (!DELTA) return;
    __syncthreads();
    for (int idx = tid; idx < IMP_TP * cs; idx += 256) {
        const int pl = idx / cs, ch = idx - pl * cs;
        if (pix0 + pl >= hw || s_cnt[pl] == 0) continue;
        D[(gp0 + pl) * cs + ch] = s_x[pl * ld + ch];
    }
    if (tid < IMP_TP) {
        const int cnt = (pix0 + tid < hw) ? s_cnt[tid] : 0;
        const unsigned m = __ballot_sync(0xffffffffu, cnt > 0);
        if (cnt > 0) {
            const size_t gp = gp0 + tid;
            atomicOr(&act[gp >> 5], 1u << (gp & 31));
            pnnz[gp] = cnt;
        }
        int tot = cnt;
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) tot += __shfl_down_sync(0xffffffffu, tot, o);
        if (tid == 0 && m) {
            atomicAdd(nnz, (unsigned long long)tot);
            atomicAdd(npix, (unsigned long long)__popc(m));
        }
    }
    // every changed pixel marks the projection pixels of the reading layers that it touches
    __shared__ unsigned long long s_macs[MAX_READERS];
    __shared__ float s_sq;
    if (tid < MAX_READERS) s_macs[tid] = 0;
    if (tid == 0) s_sq = 0.f;
    __syncthreads();
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if (lane == 0 && sq > 0.f) atomicAdd(&s_sq, sq);
    if (warp == 0) {                                         // lane = pixel of the tile
        const int pix = pix0 + lane;
        const int cnt = pix < hw ? s_cnt[lane] : 0;
        unsigned long long macs[MAX_READERS];
        scatter_changed_warp(readers, ns, pix / w, pix % w, cnt, lane, macs, arena_off);
        if (lane == 0) {
            #pragma unroll
            for (int i = 0; i < MAX_READERS; ++i) if (macs[i]) s_macs[i] = macs[i];
        }
    }
    __syncthreads();
    if (tid < readers.n && s_macs[tid] && readers.r[tid].macs) atomicAdd(shift_bytes(readers.r[tid].macs, arena_off), s_macs[tid]);
    if (tid == 0 && trunc && s_sq > 0.f) atomicAdd(trunc, (double)s_sq);
}

// int8 frames with up to 4 channels (one 4-byte word per pixel): one thread per pixel, plane reads coalesced
// across the warp, the activity word of 32 consecutive pixels written by one lane from a ballot.
template <bool DELTA>
__global__ void __launch_bounds__(256) import_i8_word_kernel(const int8_t* __restrict__ src, uint32_t* X, uint32_t* D,
                                                            uint32_t* act, int* pnnz, unsigned long long* nnz,
                                                            unsigned long long* npix, int* errw, int c, int h, int w,
                                                            int pixels, Readers readers)
{
    const int gp = blockIdx.x * blockDim.x + threadIdx.x, lane = threadIdx.x & 31;
    const int hw = h * w;
    pdl_launch_dependents();
    pdl_wait();
    int cnt = 0;
    if (gp < pixels) {
        const int ns = gp / hw, pix = gp - ns * hw;
        uint32_t nw = 0;
        for (int ch = 0; ch < c; ++ch) nw |= ((uint32_t)(uint8_t)src[((size_t)ns * c + ch) * hw + pix]) << (8 * ch);
        if (DELTA) {
            const uint32_t ow = X[gp];
            if (nw != ow) {
                uint32_t dw = 0;
                #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int d = (int)(int8_t)(nw >> (8 * j)) - (int)(int8_t)(ow >> (8 * j));
                    if (d < -128 || d > 127) atomicOr(errw, ERRW_BOUNDS);
                    dw |= ((uint32_t)d & 0xffu) << (8 * j);
                    cnt += d != 0;
                }
                D[gp] = dw;
                X[gp] = nw;
                pnnz[gp] = cnt;
            }
        } else {
            X[gp] = nw;
        }
    }
    if (!DELTA) return;
    const unsigned m = __ballot_sync(0xffffffffu, cnt > 0);
    if (m == 0) return;                                      // uniform inside the warp
    if (lane == 0) act[gp >> 5] = m;                         // gp of lane 0 is a multiple of 32: the word is this warp's alone
    int tot = cnt;
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) tot += __shfl_down_sync(0xffffffffu, tot, o);
    if (lane == 0) {
        atomicAdd(nnz, (unsigned long long)tot);
        atomicAdd(npix, (unsigned long long)__popc(m));
    }
    unsigned long long wsum[MAX_READERS];
    {
        const int ns = gp / hw, pix = gp - ns * hw;
        scatter_changed_warp(readers, ns, pix / w, pix % w, cnt, lane, wsum);
    }
    if (lane == 0) {
        #pragma unroll
        for (int i = 0; i < MAX_READERS; ++i) if (i < readers.n && wsum[i]) atomicAdd(readers.r[i].macs, wsum[i]);
    }
}

// The same for several consecutive frames in one launch (frame = blockIdx.z): frame g is compared with frame g-1 at
// the boundary (see import_nchw_kernel), the snapshot is written by the last frame.  A warp takes 128 consecutive
// pixels, lane l the pixels l, l + 32, l + 64, l + 96 of them: all 24 plane reads of a thread are in flight together,
// and each group of 32 pixels still owns its activity word.
__global__ void __launch_bounds__(256, 4) import_i8_word_frames_kernel(const int8_t* __restrict__ src, uint32_t* X, uint32_t* D,
                                                                      uint32_t* act, unsigned long long* nnz,
                                                                      unsigned long long* npix, int* errw, int c, int h, int w,
                                                                      int pixels, Readers readers, SeqFrames sf)
{
    const int lane = threadIdx.x & 31;
    const int base = (blockIdx.x * 8 + (threadIdx.x >> 5)) * 128;
    const int hw = h * w;
    {
        const long long g = blockIdx.z;
        src += g * sf.in_stride;
        D = shift_bytes(D, g * sf.row_stride);
        act = shift_bytes(act, g * sf.arena_stride); nnz = shift_bytes(nnz, g * sf.arena_stride);
        npix = shift_bytes(npix, g * sf.arena_stride);
    }
    const long long arena_off = (long long)blockIdx.z * sf.arena_stride;
    const bool write_x = (int)blockIdx.z == sf.frames - 1;
    pdl_launch_dependents();
    pdl_wait();
    uint32_t nw[4], pw[4];
    #pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int gp = base + 32 * k + lane;
        nw[k] = pw[k] = 0;
        if (gp >= pixels) continue;
        const int ns = gp / hw, pix = gp - ns * hw;
        for (int ch = 0; ch < c; ++ch) {
            const size_t o = ((size_t)ns * c + ch) * hw + pix;
            nw[k] |= ((uint32_t)(uint8_t)src[o]) << (8 * ch);
            pw[k] |= ((uint32_t)(uint8_t)(src - sf.in_stride)[o]) << (8 * ch);
        }
    }
    #pragma unroll 1
    for (int k = 0; k < 4; ++k) {
        const int gp = base + 32 * k + lane;
        if (base + 32 * k >= pixels) break;                  // uniform inside the warp
        int cnt = 0;
        if (gp < pixels) {
            if (write_x) X[gp] = nw[k];
            if (nw[k] != pw[k]) {
                uint32_t dw = 0;
                #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int d = (int)(int8_t)(nw[k] >> (8 * j)) - (int)(int8_t)(pw[k] >> (8 * j));
                    if (d < -128 || d > 127) atomicOr(errw, ERRW_BOUNDS);
                    dw |= ((uint32_t)d & 0xffu) << (8 * j);
                    cnt += d != 0;
                }
                D[gp] = dw;
            }
        }
        const unsigned m = __ballot_sync(0xffffffffu, cnt > 0);
        if (m == 0) continue;                                // uniform inside the warp
        if (lane == 0) act[gp >> 5] = m;                     // gp of lane 0 is a multiple of 32: the word is this group's alone
        const int tot = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0) {
            atomicAdd(nnz, (unsigned long long)tot);
            atomicAdd(npix, (unsigned long long)__popc(m));
        }
        unsigned long long wsum[MAX_READERS];
        {
            const int ns = gp / hw, pix = gp - ns * hw;
            scatter_changed_warp(readers, ns, pix / w, pix % w, cnt, lane, wsum, arena_off);
        }
        if (lane == 0) {
            #pragma unroll
            for (int i = 0; i < MAX_READERS; ++i)
                if (i < readers.n && readers.r[i].macs && wsum[i]) atomicAdd(shift_bytes(readers.r[i].macs, arena_off), wsum[i]);
        }
    }
}

// fp32 frames of at most 4 channels, several frames per launch, no truncation (Sec. 3.4 off): the same walk as
// import_i8_word_frames_kernel - a thread per pixel reads its channel planes of frame g and g - 1 (coalesced along the
// pixels), writes the delta row of a changed pixel and, in the last frame, the snapshot.
__global__ void __launch_bounds__(256, 4) import_f32_px_frames_kernel(const float* __restrict__ src, float* X, float* D, uint32_t* act,
                                                                     unsigned long long* nnz, unsigned long long* npix,
                                                                     int c, int h, int w, int pixels, Readers readers, SeqFrames sf)
{
    const int lane = threadIdx.x & 31;
    const int base = (blockIdx.x * 8 + (threadIdx.x >> 5)) * 128;
    const int hw = h * w;
    {
        const long long g = blockIdx.z;
        src += g * sf.in_stride;
        D = shift_bytes(D, g * sf.row_stride);
        act = shift_bytes(act, g * sf.arena_stride); nnz = shift_bytes(nnz, g * sf.arena_stride);
        npix = shift_bytes(npix, g * sf.arena_stride);
    }
    const long long arena_off = (long long)blockIdx.z * sf.arena_stride;
    const bool write_x = (int)blockIdx.z == sf.frames - 1;
    pdl_launch_dependents();
    pdl_wait();
    float nv[4][4], pv[4][4];
    #pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int gp = base + 32 * k + lane;
        #pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            nv[k][ch] = pv[k][ch] = 0.f;
            if (gp >= pixels || ch >= c) continue;
            const int ns = gp / hw, pix = gp - ns * hw;
            const size_t o = ((size_t)ns * c + ch) * hw + pix;
            nv[k][ch] = src[o];
            pv[k][ch] = (src - sf.in_stride)[o];
        }
    }
    #pragma unroll 1
    for (int k = 0; k < 4; ++k) {
        const int gp = base + 32 * k + lane;
        if (base + 32 * k >= pixels) break;                  // uniform inside the warp
        int cnt = 0;
        if (gp < pixels) {
            #pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                if (ch >= c) break;
                if (write_x) X[(size_t)gp * c + ch] = nv[k][ch];
                cnt += nv[k][ch] != pv[k][ch];
            }
            if (cnt) {
                #pragma unroll
                for (int ch = 0; ch < 4; ++ch) if (ch < c) D[(size_t)gp * c + ch] = nv[k][ch] - pv[k][ch];
            }
        }
        const unsigned m = __ballot_sync(0xffffffffu, cnt > 0);
        if (m == 0) continue;                                // uniform inside the warp
        if (lane == 0) act[gp >> 5] = m;                     // gp of lane 0 is a multiple of 32: the word is this group's alone
        const int tot = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0) {
            atomicAdd(nnz, (unsigned long long)tot);
            atomicAdd(npix, (unsigned long long)__popc(m));
        }
        unsigned long long wsum[MAX_READERS];
        {
            const int ns = gp / hw, pix = gp - ns * hw;
            scatter_changed_warp(readers, ns, pix / w, pix % w, cnt, lane, wsum, arena_off);
        }
        if (lane == 0) {
            #pragma unroll
            for (int i = 0; i < MAX_READERS; ++i)
                if (i < readers.n && readers.r[i].macs && wsum[i]) atomicAdd(shift_bytes(readers.r[i].macs, arena_off), wsum[i]);
        }
    }
}

// Binary frames arrive already pixel-major and bit-packed: one thread per pixel.
template <bool DELTA>
__global__ void import_bin_kernel(const uint32_t* __restrict__ src, uint32_t* X, uint32_t* D, uint32_t* act,
                                  int* pnnz, unsigned long long* nnz, unsigned long long* npix, int cw, int pixels,
                                  int h, int w, Readers readers, uint32_t* Xn, SeqFrames sf)
{
    const int gp = blockIdx.x * blockDim.x + threadIdx.x;
    const bool seq = DELTA && sf.frames > 1;                 // (see import_nchw_kernel)
    if (seq) {
        const long long g = blockIdx.z;
        src += g * sf.in_stride;
        D = shift_bytes(D, g * sf.row_stride);
        if (Xn) Xn = shift_bytes(Xn, g * sf.row_stride);
        act = shift_bytes(act, g * sf.arena_stride); nnz = shift_bytes(nnz, g * sf.arena_stride);
        npix = shift_bytes(npix, g * sf.arena_stride);
    }
    const long long arena_off = seq ? (long long)blockIdx.z * sf.arena_stride : 0;
    const bool write_x = !seq || (int)blockIdx.z == sf.frames - 1;
    pdl_launch_dependents();
    pdl_wait();
    int cnt = 0;
    if (gp < pixels) {
        for (int k = 0; k < cw; ++k) {
            const uint32_t xt = src[(size_t)gp * cw + k];
            if (DELTA) {
                const uint32_t ch = xt ^ (seq ? (src - sf.in_stride)[(size_t)gp * cw + k] : X[(size_t)gp * cw + k]);
                D[(size_t)gp * cw + k] = ch;
                cnt += __popc(ch);
            }
            if (write_x) X[(size_t)gp * cw + k] = xt;
            if (DELTA && Xn) Xn[(size_t)gp * cw + k] = xt;   // (pipelined chunk: the frame's own copy of the new rows)
        }
        if (DELTA && cnt) {
            atomicOr(&act[gp >> 5], 1u << (gp & 31));
            pnnz[gp] = cnt;
        }
    }
    if (!DELTA) return;
    const unsigned m = __ballot_sync(0xffffffffu, cnt > 0);
    int tot = cnt;
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) tot += __shfl_down_sync(0xffffffffu, tot, o);
    if ((threadIdx.x & 31) == 0 && m) {
        atomicAdd(nnz, (unsigned long long)tot);
        atomicAdd(npix, (unsigned long long)__popc(m));
    }
    // every changed pixel marks the projection pixels of the reading layers that it touches
    const int lane = threadIdx.x & 31;
    unsigned long long wsum[MAX_READERS];
    {
        const int ns = gp / (w * h), pix = gp - ns * (w * h);
        scatter_changed_warp(readers, ns, pix / w, pix % w, cnt, lane, wsum, arena_off);
    }
    if (lane == 0) {
        #pragma unroll
        for (int i = 0; i < MAX_READERS; ++i)
            if (i < readers.n && readers.r[i].macs && wsum[i]) atomicAdd(shift_bytes(readers.r[i].macs, arena_off), wsum[i]);
    }
}

// ------------------------------------------------------------------------------------------------
// Epilogue: f on the stored projection, next layer's delta.  A pixel of the output tensor belongs to `wpp` warps
// of one CTA (1, 2, 4 or 8: the chunks of 128 channels are dealt out to them, so that a pixel of a wide layer
// costs one memory round trip, not one per chunk); a lane owns 4 neighbouring channels at a time, so the
// 4-channel words of all window positions are fetched with independent 128-bit loads.
// ------------------------------------------------------------------------------------------------
struct EpiParams {
    const void* P;            // [opixels][c_out] float / int
    const uint32_t* oact;     // updated projection pixels (delta mode)
    const void* resX;         // residual tensor values (same storage as the output tensor) or nullptr
    void* X;                  // output tensor values
    void* D;                  // output tensor delta rows
    uint32_t* act;
    int* pnnz;
    unsigned long long* nnz;
    unsigned long long* npix;
    int* errw;
    int n, oh, ow, th, tw, c_out, cs, pool_k, pool_s, pool_p, act_fn, shift, theta;
    int wpp;                  // warps that share one output pixel (1, 2, 4 or 8); a CTA of 8 warps holds 8 / wpp pixels
    Readers readers;          // layers that read the output tensor
    float eps;                // fp32: delta entries below it are truncated to zero (Sec. 3.4)
    double* trunc;            // fp32: receives the sum of squares of the truncated entries
    const void* bn_scale;     // explicit batch normalisation, the first step of f: per-channel float scale / shift
    const void* bn_shift;     // (fp32) or int32 multiplier / offset inside the requantisation (int8); nullptr: none
    // SPLIT form (pipelined chunks): P is the projection as of the previous frame and is only read; the frame's product
    // waits in dP (zero wherever oact has no bit).  CTAs from f_blocks on merge: Q = P + dP at the pixels of oact and
    // of oact_prev (the other buffer missed the previous frame's update), and Z, the previous frame's dP, is zeroed
    // at the pixels of oact_prev so that the buffer can be added into again.
    const void* dP;
    void* Q;
    void* Z;
    void* Xn;                 // binary outputs: receives a copy of the new rows of the pixels looked at (or nullptr)
    const uint32_t* oact_prev;
    int f_blocks;             // CTAs that evaluate f
    int opix;                 // projection pixels
};

// PT: projection type (T_F32 or T_I32).  OT: output tensor storage type.  KW: pool window edge (1 = no pool).
// READERS: some layer reads the output tensor (a last layer's kernel leaves the marking code, and its registers, out).
// BN: f starts with the explicit per-channel affine (the kernels of layers without one are compiled without it).
// SPLIT: the projection is read from one buffer plus the frame's delta projection and merged into another (see EpiParams).
template <int PT, int OT, bool DENSE, int KW, bool READERS, bool BN, bool SPLIT>
__global__ void __launch_bounds__(256) epilogue_kernel(EpiParams p)
{
    using pt = typename std::conditional<PT == T_F32, float, int>::type;
    using pt4 = typename std::conditional<PT == T_F32, float4, int4>::type;
    __shared__ unsigned long long s_macs[MAX_READERS];
    __shared__ unsigned int s_nnz, s_npix;
    __shared__ int s_cnt[8];                                 // changed elements of the CTA's pixels
    __shared__ float s_sq;
    const int lane = threadIdx.x & 31;
    pdl_launch_dependents();
    if (SPLIT && (int)blockIdx.x >= p.f_blocks) {
        // ---- merge role: a CTA per word of the update bitmaps, a warp per four of its pixels, whose rows are in flight together
        pdl_wait();
        const int w = (int)blockIdx.x - p.f_blocks;
        const unsigned bp = p.oact_prev[w];
        const unsigned u = (p.oact[w] | bp) >> ((threadIdx.x >> 5) * 4);
        if ((u & 15u) == 0) return;
        const unsigned zp = bp >> ((threadIdx.x >> 5) * 4);
        const pt* R = reinterpret_cast<const pt*>(p.P);
        const pt* dP = reinterpret_cast<const pt*>(p.dP);
        pt* Q = reinterpret_cast<pt*>(p.Q);
        pt* Z = reinterpret_cast<pt*>(p.Z);
        const size_t row0 = (size_t)(w * 32 + (threadIdx.x >> 5) * 4) * p.c_out;
        if ((p.c_out & 3) == 0) {
            for (int c = lane * 4; c < p.c_out; c += 128) {
                pt4 r[4], d[4];
                #pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (!(u >> k & 1u)) continue;
                    r[k] = *reinterpret_cast<const pt4*>(R + row0 + (size_t)k * p.c_out + c);
                    d[k] = *reinterpret_cast<const pt4*>(dP + row0 + (size_t)k * p.c_out + c);
                }
                #pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (!(u >> k & 1u)) continue;
                    pt4 t = r[k];
                    t.x += d[k].x; t.y += d[k].y; t.z += d[k].z; t.w += d[k].w;
                    *reinterpret_cast<pt4*>(Q + row0 + (size_t)k * p.c_out + c) = t;
                    if (zp >> k & 1u) { pt4 z; z.x = z.y = z.z = z.w = 0; *reinterpret_cast<pt4*>(Z + row0 + (size_t)k * p.c_out + c) = z; }
                }
            }
        } else {
            #pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (!(u >> k & 1u)) continue;
                for (int c = lane; c < p.c_out; c += 32) {
                    const size_t o = row0 + (size_t)k * p.c_out + c;
                    Q[o] = R[o] + dP[o];
                    if (zp >> k & 1u) Z[o] = 0;
                }
            }
        }
        return;
    }
    if (threadIdx.x < MAX_READERS) s_macs[threadIdx.x] = 0;
    if (threadIdx.x < 8) s_cnt[threadIdx.x] = 0;
    if (threadIdx.x == 0) { s_nnz = 0; s_npix = 0; s_sq = 0.f; }
    pdl_wait();                                              // the projection (and its update bitmap) is the convolution's work
    __syncthreads();
    const int ppc = (blockDim.x >> 5) / p.wpp;               // pixels per CTA
    const int slot = (threadIdx.x >> 5) / p.wpp, sub = (threadIdx.x >> 5) % p.wpp;   // this warp's pixel of the CTA, and its share of the chunks
    const int r = blockIdx.x * ppc + slot;
    const int tpix = p.n * p.th * p.tw;
    const int tx = r % p.tw, ty = (r / p.tw) % p.th, ns = r / (p.tw * p.th);
    const int st = KW > 1 ? p.pool_s : 1, pp = KW > 1 ? p.pool_p : 0;
    const int y0 = ty * st - pp, x0 = tx * st - pp;
    const int qbase = ns * p.oh * p.ow;
    // window positions inside the projection (bit wy * KW + wx), and whether any of them was updated
    unsigned inside = 0, updm = 0;
    bool on = false;
    if (r < tpix) {
        bool mine = false, upd = false;
        if (lane < KW * KW) {
            const int y = y0 + lane / KW, x = x0 + lane % KW;
            mine = y >= 0 && y < p.oh && x >= 0 && x < p.ow;
            if (mine && !DENSE) { const int q = qbase + y * p.ow + x; upd = (p.oact[q >> 5] >> (q & 31)) & 1u; }
        }
        inside = __ballot_sync(0xffffffffu, mine);
        updm = __ballot_sync(0xffffffffu, upd);
        on = DENSE ? true : updm != 0;
    }
    int cnt = 0;
    float sq = 0.f;                                          // squares of the truncated delta entries (fp32)
    if (on) {
        const pt* P = reinterpret_cast<const pt*>(p.P);
        const bool vec = (p.c_out & 3) == 0;
        const int c_iter = (OT == T_BIN) ? p.cs * 32 : p.cs;
        for (int c0 = sub * 128; c0 < c_iter; c0 += p.wpp * 128) {
            const int c = c0 + lane * 4;
            // the stored int8 activation word is fetched together with the projection, not after it
            uint32_t old_word = 0;
            if (OT == T_I8 && !DENSE && c < p.cs)
                old_word = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const int8_t*>(p.X) + (size_t)r * p.cs + c);
            // ---- the 4-channel words of every window position
            pt v[KW * KW][4];
            #pragma unroll
            for (int wi = 0; wi < KW * KW; ++wi) {
                v[wi][0] = v[wi][1] = v[wi][2] = v[wi][3] = 0;
                if (!(inside >> wi & 1u) || c >= p.c_out) continue;
                const size_t o = (size_t)(qbase + (y0 + wi / KW) * p.ow + x0 + wi % KW) * p.c_out + c;
                if (vec) {
                    if (PT == T_F32) { const float4 t = *reinterpret_cast<const float4*>(P + o); v[wi][0] = (pt)t.x; v[wi][1] = (pt)t.y; v[wi][2] = (pt)t.z; v[wi][3] = (pt)t.w; }
                    else { const int4 t = *reinterpret_cast<const int4*>(P + o); v[wi][0] = (pt)t.x; v[wi][1] = (pt)t.y; v[wi][2] = (pt)t.z; v[wi][3] = (pt)t.w; }
                } else {
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) if (c + j < p.c_out) v[wi][j] = P[o + j];
                }
                if (SPLIT && (updm >> wi & 1u)) {            // this frame's product is still on its own
                    const pt* dP = reinterpret_cast<const pt*>(p.dP);
                    if (vec) { const pt4 t = *reinterpret_cast<const pt4*>(dP + o); v[wi][0] += t.x; v[wi][1] += t.y; v[wi][2] += t.z; v[wi][3] += t.w; }
                    else {
                        #pragma unroll
                        for (int j = 0; j < 4; ++j) if (c + j < p.c_out) v[wi][j] += dP[o + j];
                    }
                }
            }
            // ---- f: [affine] -> [requant] -> [+ shortcut] -> act -> max over the window (sign: max first, threshold last)
            pt best[4], res[4] = {0, 0, 0, 0};
            if (p.resX) {
                #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (c + j >= p.c_out) continue;
                    if (PT == T_F32) res[j] = (pt)reinterpret_cast<const float*>(p.resX)[(size_t)r * p.cs + c + j];
                    else if (OT == T_I8) res[j] = (pt)reinterpret_cast<const int8_t*>(p.resX)[(size_t)r * p.cs + c + j];
                }
            }
            epi_f<PT, OT, KW, BN, pt>(v, inside, c, res, p.c_out, p.act_fn, p.shift, p.bn_scale, p.bn_shift, best);
            // ---- compare with the stored activation, emit delta row and snapshot
            if (OT == T_BIN) {
                unsigned bits = 0;
                #pragma unroll
                for (int j = 0; j < 4; ++j) if (c + j < p.c_out && (int)best[j] >= p.theta) bits |= 1u << j;
                unsigned word = bits << (4 * (lane & 7));
                word |= __shfl_xor_sync(0xffffffffu, word, 1);
                word |= __shfl_xor_sync(0xffffffffu, word, 2);
                word |= __shfl_xor_sync(0xffffffffu, word, 4);
                const int wd = (c0 >> 5) + (lane >> 3);
                if ((lane & 7) == 0 && wd < p.cs) {
                    uint32_t* X = reinterpret_cast<uint32_t*>(p.X);
                    const size_t o = (size_t)r * p.cs + wd;
                    if (DENSE) X[o] = word;
                    else {
                        const uint32_t ch = word ^ X[o];
                        reinterpret_cast<uint32_t*>(p.D)[o] = ch;
                        X[o] = word;
                        if (SPLIT && p.Xn) reinterpret_cast<uint32_t*>(p.Xn)[o] = word;
                        cnt += __popc(ch);
                    }
                }
            } else if (c < p.cs) {
                const size_t o = (size_t)r * p.cs + c;
                if (OT == T_I8) {            // cs is a multiple of 4: one 4-channel word per lane
                    const uint32_t nw = ((uint32_t)(int)best[0] & 0xffu) | ((uint32_t)(int)best[1] & 0xffu) << 8 |
                                        ((uint32_t)(int)best[2] & 0xffu) << 16 | ((uint32_t)(int)best[3] & 0xffu) << 24;
                    uint32_t* X = reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(p.X) + o);
                    if (DENSE) *X = nw;
                    else {
                        const uint32_t ow_ = old_word;
                        uint32_t dw = 0;
                        #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int nv = (int)(int8_t)(nw >> (8 * j)), ov = (int)(int8_t)(ow_ >> (8 * j));
                            const int d = nv - ov;
                            if (p.errw && (d < -128 || d > 127)) atomicOr(p.errw, ERRW_BOUNDS);
                            dw |= ((uint32_t)d & 0xffu) << (8 * j);
                            cnt += nv != ov;
                        }
                        *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(p.D) + o) = dw;
                        if (nw != ow_) *X = nw;
                    }
                } else {
                    pt* X = reinterpret_cast<pt*>(p.X);
                    pt* Dp = reinterpret_cast<pt*>(p.D);
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (c + j >= p.cs) break;
                        if (DENSE) X[o + j] = best[j];
                        else {
                            const pt old = X[o + j];
                            pt dv = best[j] - old;
                            if (best[j] != old) {
                                X[o + j] = best[j];          // the snapshot always moves on
                                if (PT == T_F32 && p.eps > 0.f && fabsf((float)dv) < p.eps) { sq += (float)dv * (float)dv; dv = 0; }
                                else ++cnt;
                            }
                            Dp[o + j] = dv;
                        }
                    }
                }
            }
        }
    }
    if (DENSE) return;
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) { cnt += __shfl_xor_sync(0xffffffffu, cnt, o); sq += __shfl_xor_sync(0xffffffffu, sq, o); }
    if (PT == T_F32 && lane == 0 && sq > 0.f) atomicAdd(&s_sq, sq);
    if (cnt && lane == 0) atomicAdd(&s_cnt[slot], cnt);      // (cnt is uniform inside the warp) the pixel's warps add up
    __syncthreads();
    if (sub == 0 && lane == 0 && r < tpix && s_cnt[slot]) {
        atomicOr(&p.act[r >> 5], 1u << (r & 31));
        p.pnnz[r] = s_cnt[slot];
        atomicAdd(&s_nnz, (unsigned)s_cnt[slot]);
        atomicAdd(&s_npix, 1u);
    }
    // the CTA's consecutive pixels mark the reading layers' projection pixels together (lane = pixel)
    if (READERS && threadIdx.x < 32) {
        const int rl = blockIdx.x * ppc + lane;
        const bool have = lane < ppc && rl < tpix;
        unsigned long long macs[MAX_READERS];
        scatter_changed_warp(p.readers, have ? rl / (p.tw * p.th) : 0, have ? (rl / p.tw) % p.th : 0, have ? rl % p.tw : 1,
                             have ? s_cnt[lane] : 0, lane, macs);
        if (lane == 0) {
            #pragma unroll
            for (int i = 0; i < MAX_READERS; ++i) s_macs[i] = macs[i];
        }
    }
    __syncthreads();
    if (threadIdx.x < p.readers.n && s_macs[threadIdx.x]) atomicAdd(p.readers.r[threadIdx.x].macs, s_macs[threadIdx.x]);
    if (threadIdx.x == 0 && s_npix) {
        atomicAdd(p.nnz, (unsigned long long)s_nnz);
        atomicAdd(p.npix, (unsigned long long)s_npix);
    }
    if (PT == T_F32 && threadIdx.x == 0 && p.trunc && s_sq > 0.f) atomicAdd(p.trunc, (double)s_sq);
}

// ------------------------------------------------------------------------------------------------
// Exports to the boundary layout.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void export_nchw_kernel(const T* __restrict__ src, T* dst, int c, int cs, int hw, long long total,
                                   long long src_stride = 0, long long dst_stride = 0)   // elements between frames (frame = blockIdx.y)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    src += blockIdx.y * src_stride;
    dst += blockIdx.y * dst_stride;
    pdl_launch_dependents();
    pdl_wait();
    if (i >= total) return;
    const int pix = (int)(i % hw);
    const int ch = (int)((i / hw) % c);
    const long long ns = i / ((long long)hw * c);
    dst[i] = src[(ns * hw + pix) * cs + ch];
}

// The same through a 32 x 32 tile in shared memory (4-byte elements): rows read along the channels, planes written
// along the pixels, both coalesced.  grid = (pixel tiles, channel tiles x n, frames), block = (32, 8).
__global__ void __launch_bounds__(256) export_nchw_tiled_kernel(const uint32_t* __restrict__ src, uint32_t* dst, int c, int cs, int hw,
                                                                int ctiles, long long src_stride, long long dst_stride)
{
    __shared__ uint32_t tile[32][33];
    const int p0 = blockIdx.x * 32, c0 = (int)(blockIdx.y % ctiles) * 32;
    const long long ns = blockIdx.y / ctiles;
    src += blockIdx.z * src_stride;
    dst += blockIdx.z * dst_stride;
    pdl_launch_dependents();
    pdl_wait();
    for (int k = threadIdx.y; k < 32; k += 8) {
        const int pix = p0 + k, ch = c0 + (int)threadIdx.x;
        if (pix < hw && ch < c) tile[k][threadIdx.x] = src[(ns * hw + pix) * cs + ch];
    }
    __syncthreads();
    for (int k = threadIdx.y; k < 32; k += 8) {
        const int ch = c0 + k, pix = p0 + (int)threadIdx.x;
        if (pix < hw && ch < c) dst[(ns * c + ch) * hw + pix] = tile[threadIdx.x][k];
    }
}

template <typename T>
__global__ void fill_projection_kernel(T* P, const T* bias, int c_out, long long total)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total) P[i] = bias ? bias[i % c_out] : (T)0;
}

// Eq. 7, one frame: e_t += sum over the linear layers of l2(truncated part of the layer's input).
// Copies of whole projections (start of a pipelined chunk: the second buffer of every layer), one launch for up to 32 layers.
struct CopyJobs { const int* src[32]; int* dst[32]; long long words[32]; int n; };
__global__ void __launch_bounds__(256) copy_projections_kernel(CopyJobs j)
{
    const int k = blockIdx.y;
    const long long n = j.words[k], step = (long long)gridDim.x * blockDim.x;
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    if ((n & 3) == 0) {
        const int4* s = reinterpret_cast<const int4*>(j.src[k]);
        int4* d = reinterpret_cast<int4*>(j.dst[k]);
        for (long long i = i0; i < n / 4; i += step) d[i] = s[i];
    } else {
        for (long long i = i0; i < n; i += step) j.dst[k][i] = j.src[k][i];
    }
}

// End of a pipelined chunk: the last frame's delta projections go back to zero (rows of the pixels in `bits`).
struct ZeroJobs { int* dst[32]; const uint32_t* bits[32]; int words[32]; int c_out[32]; int n; };
__global__ void __launch_bounds__(256) zero_rows_kernel(ZeroJobs j)
{
    const int k = blockIdx.y, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    pdl_wait();
    const int c_out = j.c_out[k];
    for (int w = blockIdx.x * 8 + (threadIdx.x >> 5); w < j.words[k]; w += gridDim.x * 8) {
        unsigned u = j.bits[k][w];
        while (u) {
            const int q = w * 32 + __ffs(u) - 1;
            u &= u - 1;
            int* row = j.dst[k] + (size_t)q * c_out;
            if ((c_out & 3) == 0) for (int c = lane * 4; c < c_out; c += 128) *reinterpret_cast<int4*>(row + c) = make_int4(0, 0, 0, 0);
            else for (int c = lane; c < c_out; c += 32) row[c] = 0;
        }
    }
}

struct AecsParams { const double* sumsq[64]; int n; double* e_t; double* last_l2; };
__global__ void aecs_accumulate_kernel(AecsParams p)
{
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double add = 0.0;
    for (int l = 0; l < p.n; ++l) { const double v = sqrt(*p.sumsq[l]); p.last_l2[l] = v; add += v; }
    *p.e_t += add;
}

// ================================================================================================
// host side
// ================================================================================================
static int dev_alloc(rrm_net* net, void** p, size_t bytes, bool zero = true)
{
    if (bytes == 0) bytes = 16;
    if (cudaMalloc(p, bytes) != cudaSuccess) { *p = nullptr; return RRM_ERR_ALLOC; }
    net->allocs.push_back(*p);
    if (zero && cudaMemset(*p, 0, bytes) != cudaSuccess) return RRM_ERR_CUDA;
    return RRM_OK;
}

static int proj_type(const Layer& L) { return L.d.dtype == RRM_F32 ? T_F32 : T_I32; }

// CTAs that share one output tile of the CUDA-core kernel, each with a contiguous range of K stages: K is split
// while the tiles alone leave most of the machine idle (each share keeps >= 2 stages).  A delta pass is sized as
// if half of the tiles had rows: the others leave right after the row scan.
static int gemm_ksplit(const Layer& L, bool dense)
{
    const int stages = L.kup / TK;
    const long long gx = ceil_div(L.opixels(), TM), gy = L.np / TN;
    const long long tiles = dense ? gx * gy : (gx + 1) / 2 * gy;
    int ks = 1;
    while (tiles * ks < 2 * 148 && stages / (ks * 2) >= 2) ks *= 2;
    if (L.d.dtype == RRM_F32 && ks > 16) ks = 16;            // fp32 shares form a thread-block cluster (at most 16 CTAs on this GPU)
    return ks;
}

int conv_layer_create(rrm_net* net, Layer& L, const void* W_dev, const void* bias_dev)
{
    const rrm_layer_desc& d = L.d;
    const Tensor& in = net->tensors[d.src];
    L.u_in = (d.dtype == RRM_F32) ? in.cs : (d.dtype == RRM_I8 ? in.cs / 4 : in.cs);
    L.ku = d.kh * d.kw * L.u_in;
    L.kup = round_up(L.ku, TK);
    L.np = round_up(d.c_out, TN);
    RRM_TRY(dev_alloc(net, &L.Wk, (size_t)L.kup * L.np * 4));
    RRM_TRY(dev_alloc(net, &L.bias, (size_t)d.c_out * 4));
    RRM_TRY(dev_alloc(net, &L.P, (size_t)L.opixels() * d.c_out * 4));
    if (bias_dev) RRM_CUDA_TRY(cudaMemcpy(L.bias, bias_dev, (size_t)d.c_out * 4, cudaMemcpyDeviceToDevice));
    const int tot = L.kup * L.np;
    pack_weights_kernel<<<ceil_div(tot, 256), 256>>>(W_dev, reinterpret_cast<uint32_t*>(L.Wk),
                                                    d.dtype == RRM_F32 ? T_F32 : (d.dtype == RRM_I8 ? T_I8 : T_BIN),
                                                    d.c_in, d.c_out, d.kh, d.kw, L.u_in, L.kup, L.np);
    RRM_CUDA_TRY(cudaGetLastError());
    if (d.kh * d.kw > 128) return RRM_ERR_UNSUPPORTED;       // the kernels keep a row's usable taps in a 128-bit mask

    RRM_TRY(gemm_allow_smem<T_F32>());
    RRM_TRY(gemm_allow_smem<T_I8>());
    RRM_TRY(gemm_allow_smem<T_BIN>());
    if (d.variant != RRM_VARIANT_GATHER && conv_tc_eligible(net, L)) RRM_TRY(conv_tc_create(net, L, W_dev));
    return RRM_OK;
}

// Fresh state = the stack's response to the all-zero input pattern (zero pixels; all -1 for a binary
// input): layer 0 then holds I_prev = 0 and P_prev = b as Algorithm 1 starts, and every deeper layer
// holds a snapshot that is consistent with it.
int reset_state(rrm_net* net, cudaStream_t st)
{
    RRM_CUDA_TRY(cudaMemsetAsync(net->tensors[0].X, 0, net->tensors[0].bytes(), st));
    for (int l = 0; l < (int)net->layers.size(); ++l) RRM_TRY(launch_layer(net, l, true, false, st));
    return RRM_OK;
}

int ensure_stateless(rrm_net* net)
{
    for (auto& T : net->tensors)
        if (!T.X2) RRM_TRY(dev_alloc(net, &T.X2, T.bytes()));
    for (auto& L : net->layers)
        if (!L.P2) RRM_TRY(dev_alloc(net, &L.P2, (size_t)L.opixels() * L.d.c_out * 4));
    return RRM_OK;
}

// frames > 1 (delta only): `frame` is the first of that many consecutive frames at the boundary, the frame before it
// lies right in front of them; frame g's delta rows, new rows and arena follow frame 0's (the bound ones) at the
// tensor's size / arena_stride bytes each.  The snapshot ends up as the last frame.
int launch_import(rrm_net* net, const void* frame, bool delta, bool stateless, cudaStream_t st, int frames, long long arena_stride)
{
    if (stateless) RRM_TRY(ensure_stateless(net));
    Tensor& T = net->tensors[0];
    void* X = stateless ? T.X2 : T.X;
    const int hw = T.h * T.w;
    const bool seq = frames > 1 && delta && !stateless;
    const unsigned gz = seq ? (unsigned)frames : 1u;
    SeqFrames sf{};
    if (seq) {
        sf.frames = frames; sf.row_stride = (long long)T.bytes(); sf.arena_stride = arena_stride;
        sf.in_stride = T.dtype == T_BIN ? (long long)T.pixels() * T.cs : (long long)T.n * T.c * hw;
    }
    if (T.dtype == T_BIN) {
        const int blocks = ceil_div(T.pixels(), 256);
        if (delta) launch_seq(import_bin_kernel<true>, dim3(blocks, 1, gz), dim3(256), 0, st, (const uint32_t*)frame, (uint32_t*)X, (uint32_t*)T.D,
                                                                  T.act, T.pnnz, T.nnz, T.npix, T.cs, T.pixels(),
                                                                  T.h, T.w, T.readers, (uint32_t*)(stateless ? nullptr : T.Xn_cur), sf);
        else launch_seq(import_bin_kernel<false>, dim3(blocks), dim3(256), 0, st, (const uint32_t*)frame, (uint32_t*)X, nullptr, nullptr,
                                                              nullptr, nullptr, nullptr, T.cs, T.pixels(), T.h, T.w,
                                                              Readers{}, (uint32_t*)nullptr, sf);
    } else if (T.dtype == T_I8 && T.cs == 4) {
        const int blocks = ceil_div(T.pixels(), 256);
        if (seq) launch_seq(import_i8_word_frames_kernel, dim3(ceil_div(T.pixels(), 1024), 1, gz), dim3(256), 0, st, (const int8_t*)frame, (uint32_t*)X,
                            (uint32_t*)T.D, T.act, T.nnz, T.npix, net->errw, T.c, T.h, T.w, T.pixels(), T.readers, sf);
        else if (delta) launch_seq(import_i8_word_kernel<true>, dim3(blocks), dim3(256), 0, st, (const int8_t*)frame, (uint32_t*)X, (uint32_t*)T.D, T.act,
                                                                      T.pnnz, T.nnz, T.npix, net->errw, T.c, T.h, T.w,
                                                                      T.pixels(), T.readers);
        else launch_seq(import_i8_word_kernel<false>, dim3(blocks), dim3(256), 0, st, (const int8_t*)frame, (uint32_t*)X, nullptr, nullptr, nullptr,
                                                                  nullptr, nullptr, net->errw, T.c, T.h, T.w, T.pixels(),
                                                                  Readers{});
    } else {
        dim3 grid(ceil_div(hw, IMP_TP), T.n, gz);
        const size_t smem = (size_t)IMP_TP * (T.cs + 1) * T.unit_bytes * (seq ? 2 : 1);
        if (smem > 200 * 1024) return RRM_ERR_UNSUPPORTED;
        if (T.dtype == T_F32 && seq && T.c <= 4 && !(net->eps > 0.f)) {
            launch_seq(import_f32_px_frames_kernel, dim3(ceil_div(T.pixels(), 1024), 1, gz), dim3(256), 0, st, (const float*)frame, (float*)X,
                       (float*)T.D, T.act, T.nnz, T.npix, T.c, T.h, T.w, T.pixels(), T.readers, sf);
        } else if (T.dtype == T_F32) {
            auto kd = import_nchw_kernel<float, true>;
            auto kn = import_nchw_kernel<float, false>;
            if (smem > 48 * 1024) {
                cudaFuncSetAttribute(kd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
                cudaFuncSetAttribute(kn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            }
            if (delta) launch_seq(kd, dim3(grid), dim3(256), smem, st, (const float*)frame, (float*)X, (float*)T.D, T.act, T.pnnz, T.nnz,
                                                   T.npix, net->errw, T.c, T.cs, hw, T.w, T.readers, net->eps, T.trunc, sf);
            else launch_seq(kn, dim3(grid), dim3(256), smem, st, (const float*)frame, (float*)X, nullptr, nullptr, nullptr, nullptr,
                                             nullptr, net->errw, T.c, T.cs, hw, T.w, Readers{}, 0.f, nullptr, sf);
        } else {
            auto kd = import_nchw_kernel<int8_t, true>;
            auto kn = import_nchw_kernel<int8_t, false>;
            if (smem > 48 * 1024) {
                cudaFuncSetAttribute(kd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
                cudaFuncSetAttribute(kn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            }
            if (delta) launch_seq(kd, dim3(grid), dim3(256), smem, st, (const int8_t*)frame, (int8_t*)X, (int8_t*)T.D, T.act, T.pnnz,
                                                   T.nnz, T.npix, net->errw, T.c, T.cs, hw, T.w, T.readers, 0.f, nullptr, sf);
            else launch_seq(kn, dim3(grid), dim3(256), smem, st, (const int8_t*)frame, (int8_t*)X, nullptr, nullptr, nullptr, nullptr,
                                             nullptr, net->errw, T.c, T.cs, hw, T.w, Readers{}, 0.f, nullptr, sf);
        }
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

template <int PT, int OT, bool DENSE, bool BN, int KW>
static void launch_epi_kw(const EpiParams& e, int blocks, cudaStream_t st)
{
    const bool rd = !DENSE && e.readers.n > 0;               // (a dense pass marks nothing)
    if (!DENSE && e.dP) {                                    // pipelined chunk: f from P + dP, merge CTAs behind the f CTAs
        if (rd) launch_seq(epilogue_kernel<PT, OT, DENSE, KW, !DENSE, BN, !DENSE>, dim3(blocks), dim3(256), 0, st, e);
        else launch_seq(epilogue_kernel<PT, OT, DENSE, KW, false, BN, !DENSE>, dim3(blocks), dim3(256), 0, st, e);
    } else {
        if (rd) launch_seq(epilogue_kernel<PT, OT, DENSE, KW, !DENSE, BN, false>, dim3(blocks), dim3(256), 0, st, e);
        else launch_seq(epilogue_kernel<PT, OT, DENSE, KW, false, BN, false>, dim3(blocks), dim3(256), 0, st, e);
    }
}

template <int PT, int OT, bool DENSE, bool BN>
static int launch_epi_kb(const EpiParams& e, int blocks, cudaStream_t st)
{
    switch (e.pool_k > 0 ? e.pool_k : 1) {
        case 1: launch_epi_kw<PT, OT, DENSE, BN, 1>(e, blocks, st); break;
        case 2: launch_epi_kw<PT, OT, DENSE, BN, 2>(e, blocks, st); break;
        case 3: launch_epi_kw<PT, OT, DENSE, BN, 3>(e, blocks, st); break;
        default: return RRM_ERR_UNSUPPORTED;                 // pool windows are 2x2 or 3x3
    }
    return RRM_OK;
}

template <int PT, int OT, bool DENSE>
static int launch_epi_k(const EpiParams& e, int blocks, cudaStream_t st)
{
    // (the affine exists for fp32 outputs and for requantised int8 outputs only)
    if ((OT == T_F32 || OT == T_I8) && e.bn_scale) return launch_epi_kb<PT, OT, DENSE, (OT == T_F32 || OT == T_I8)>(e, blocks, st);
    return launch_epi_kb<PT, OT, DENSE, false>(e, blocks, st);
}

template <int PT, bool DENSE>
static int launch_epi(const EpiParams& e, int ot, int blocks, cudaStream_t st)
{
    if (PT == T_F32) return launch_epi_k<PT, T_F32, DENSE>(e, blocks, st);
    switch (ot) {
        case T_I8: return launch_epi_k<PT, T_I8, DENSE>(e, blocks, st);
        case T_BIN: return launch_epi_k<PT, T_BIN, DENSE>(e, blocks, st);
        default: return launch_epi_k<PT, T_I32, DENSE>(e, blocks, st);
    }
}

// hook (may be null): called with 0 before the layer's first launch, with 1 between the convolution and the
// epilogue, with 2 after the epilogue (the pipelined chunk graph inserts its cross-frame dependencies there).
// dense_in_step: the layer is evaluated densely inside a delta step (its measured activity is above the
// threshold): P = F*X + b from the input's current value replaces the stored projection (a precise inference of
// this layer), and the epilogue still compares f(P) with the stored output and emits the next layer's delta.
// split (delta steps of pipelined chunks): the product goes to a delta-projection buffer and the epilogue merges it.
int launch_layer(rrm_net* net, int l, bool dense, bool stateless, cudaStream_t st, const std::function<int(int)>* hook,
                 bool dense_in_step, const SplitProjection* split)
{
    if (hook) RRM_TRY((*hook)(0));
    if (split && (dense || stateless || dense_in_step)) return RRM_ERR_INVALID_ARG;
    const bool step_dense = dense_in_step && !dense && !stateless;
    const bool conv_dense = dense || step_dense;
    Layer& L = net->layers[l];
    const rrm_layer_desc& d = L.d;
    Tensor& in = net->tensors[d.src];
    Tensor& out = net->tensors[l + 1];
    Tensor* res = d.res >= 0 ? &net->tensors[d.res] : nullptr;

    ConvParams p{};
    p.frames = 1;
    p.D = in.D; p.X = stateless ? in.X2 : (split && in.Xn_cur ? in.Xn_cur : in.X); p.in_act = in.act; p.oact = L.oact; p.ocount = L.ocount;
    p.Wk = L.Wk; p.bias = L.bias; p.P = split ? split->dP : (stateless ? L.P2 : L.P);
    p.n = d.n; p.c_in = d.c_in; p.h = d.h; p.w = d.w; p.u_in = L.u_in; p.oh = L.oh; p.ow = L.ow;
    p.kh = d.kh; p.kw = d.kw; p.stride = d.stride; p.pad = d.pad; p.c_out = d.c_out; p.np = L.np;
    p.ku = L.ku; p.kup = L.kup; p.opixels = L.opixels();
    p.wait_limit = net->opt.wait_limit;
    p.count_bitmap = step_dense ? L.oact : nullptr;
    dim3 grid(ceil_div(L.opixels(), TM), L.np / TN);
    p.errw = net->errw;
    {
        const int ks = gemm_ksplit(L, conv_dense);
        p.ksplit = ks;
        grid.z = ks;
        // (integer shares add onto a zeroed projection; fp32 shares meet in their cluster's shared memory, in a fixed order)
        if (!L.tc_ready && conv_dense && ks > 1 && d.dtype != RRM_F32) RRM_TRY(zero_projection(p.P, (long long)L.opixels() * d.c_out, st));
    }
    if (L.tc_ready) RRM_TRY(launch_conv_tc(net, L, in, conv_dense, stateless, st, p.count_bitmap, split ? split->dP : nullptr));
    else if (d.dtype == RRM_F32) { if (conv_dense) launch_gemm<T_F32, true>(p, grid, st); else launch_gemm<T_F32, false>(p, grid, st); }
    else if (d.dtype == RRM_I8) { if (conv_dense) launch_gemm<T_I8, true>(p, grid, st); else launch_gemm<T_I8, false>(p, grid, st); }
    else { if (conv_dense) launch_gemm<T_BIN, true>(p, grid, st); else launch_gemm<T_BIN, false>(p, grid, st); }

    if (hook) RRM_TRY((*hook)(1));
    EpiParams e{};
    e.P = split ? split->R : p.P; e.oact = step_dense ? net->ones : L.oact;     // (dense inside a delta step: every window is looked at)
    e.dP = split ? split->dP : nullptr; e.Q = split ? split->Q : nullptr; e.Z = split ? split->Z : nullptr;
    e.oact_prev = split ? split->prev_oact : nullptr; e.opix = L.opixels(); e.Xn = split ? out.Xn_cur : nullptr;
    e.resX = res ? (stateless ? res->X2 : res->X) : nullptr;
    e.X = stateless ? out.X2 : out.X; e.D = out.D; e.act = out.act; e.pnnz = out.pnnz; e.nnz = out.nnz;
    e.npix = out.npix; e.errw = out.has_consumer ? net->errw : nullptr;
    e.n = d.n; e.oh = L.oh; e.ow = L.ow; e.th = L.th; e.tw = L.tw; e.c_out = d.c_out; e.cs = out.cs;
    e.pool_k = d.pool_k; e.pool_s = d.pool_s; e.pool_p = d.pool_p; e.act_fn = d.act; e.shift = d.shift; e.theta = d.theta;
    e.readers = dense ? Readers{} : out.readers;
    e.eps = net->eps; e.trunc = out.trunc;
    e.bn_scale = L.bn_scale; e.bn_shift = L.bn_shift;
    {
        const int chunks = ceil_div(out.dtype == T_BIN ? out.cs * 32 : out.cs, 128);
        // (several warps per pixel shorten a lone frame's step, where the launch is a handful of CTAs; with enough pixels
        // to fill the machine, or inside a chunk graph where launches of several frames overlap anyway, one warp per
        // pixel does the same work with fewer CTAs: measured 10.5 against 18.5 us for a 32-stream layer)
        const bool latency_bound = !net->many_in_flight && out.pixels() <= 8 * 2 * 148;
        e.wpp = !latency_bound ? 1 : (chunks >= 8 ? 8 : (chunks > 2 ? 4 : (chunks > 1 ? 2 : 1)));
    }
    e.f_blocks = ceil_div(out.pixels(), 8 / e.wpp);
    const int blocks = e.f_blocks + (split ? ceil_div(L.opixels(), 32) : 0);   // merge CTAs: one per word of the update bitmap
    int es;
    if (proj_type(L) == T_F32) es = dense ? launch_epi<T_F32, true>(e, out.dtype, blocks, st) : launch_epi<T_F32, false>(e, out.dtype, blocks, st);
    else es = dense ? launch_epi<T_I32, true>(e, out.dtype, blocks, st) : launch_epi<T_I32, false>(e, out.dtype, blocks, st);
    RRM_TRY(es);
    RRM_CUDA_TRY(cudaGetLastError());
    if (hook) RRM_TRY((*hook)(2));
    return RRM_OK;
}

// The buffers of the pipelined delta chunks (second projection, the rings of delta projections and of delta rows).
int ensure_split(rrm_net* net)
{
    for (auto& L : net->layers) {
        const size_t bytes = (size_t)L.opixels() * L.d.c_out * 4;
        if (!L.Palt) RRM_TRY(dev_alloc(net, &L.Palt, bytes, false));
        for (int k = 0; k < CHUNK_RING; ++k) if (!L.dP[k]) RRM_TRY(dev_alloc(net, &L.dP[k], bytes));      // zero
    }
    for (auto& T : net->tensors) {
        if (!T.Dring[0]) T.Dring[0] = T.D;
        for (int k = 1; k < CHUNK_RING; ++k) if (!T.Dring[k]) RRM_TRY(dev_alloc(net, &T.Dring[k], T.bytes()));
        if (T.dtype == T_BIN) for (int k = 0; k < CHUNK_RING; ++k) if (!T.Xn[k]) RRM_TRY(dev_alloc(net, &T.Xn[k], T.bytes()));
    }
    return RRM_OK;
}

// P -> Palt for every layer.
int launch_copy_projections(rrm_net* net, cudaStream_t st)
{
    const int n = (int)net->layers.size();
    for (int l0 = 0; l0 < n; l0 += 32) {
        CopyJobs j;
        j.n = n - l0 < 32 ? n - l0 : 32;
        long long most = 0;
        for (int k = 0; k < j.n; ++k) {
            const Layer& L = net->layers[l0 + k];
            j.src[k] = reinterpret_cast<const int*>(L.P);
            j.dst[k] = reinterpret_cast<int*>(L.Palt);
            j.words[k] = (long long)L.opixels() * L.d.c_out;
            most = most > j.words[k] ? most : j.words[k];
        }
        for (int k = j.n; k < 32; ++k) { j.src[k] = nullptr; j.dst[k] = nullptr; j.words[k] = 0; }
        long long gx = (most / 4 + 255) / 256;
        gx = gx < 1 ? 1 : (gx > 148 ? 148 : gx);                 // (a few 16-byte words per thread at most layers' sizes)
        launch_seq(copy_projections_kernel, dim3((unsigned)gx, (unsigned)j.n), dim3(256), 0, st, j);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

// Zeroes delta-projection buffer `slot` of every layer at the pixels of the bound arena's update bitmaps.
int launch_zero_delta_projections(rrm_net* net, int slot, cudaStream_t st)
{
    const int n = (int)net->layers.size();
    for (int l0 = 0; l0 < n; l0 += 32) {
        ZeroJobs j;
        j.n = n - l0 < 32 ? n - l0 : 32;
        int most = 1;
        for (int k = 0; k < 32; ++k) {
            if (k < j.n) {
                const Layer& L = net->layers[l0 + k];
                j.dst[k] = reinterpret_cast<int*>(L.dP[slot]); j.bits[k] = L.oact;
                j.words[k] = ceil_div(L.opixels(), 32); j.c_out[k] = L.d.c_out;
                most = most > j.words[k] ? most : j.words[k];
            } else { j.dst[k] = nullptr; j.bits[k] = nullptr; j.words[k] = 0; j.c_out[k] = 0; }
        }
        const int gx = ceil_div(most, 8) < 148 ? ceil_div(most, 8) : 148;
        launch_seq(zero_rows_kernel, dim3((unsigned)gx, (unsigned)j.n), dim3(256), 0, st, j);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

// All delta-projection buffers back to zero (after a step that gave up may have left rows behind).
int clear_split(rrm_net* net, cudaStream_t st)
{
    for (auto& L : net->layers)
        for (int k = 0; k < CHUNK_RING; ++k)
            if (L.dP[k]) RRM_CUDA_TRY(cudaMemsetAsync(L.dP[k], 0, (size_t)L.opixels() * L.d.c_out * 4, st));
    return RRM_OK;
}

// The state becomes frame `slot` of a dense pass that was batched over frames: every tensor's value and every layer's
// projection are copied out of the batched buffers.
int launch_copy_state_from_batch(rrm_net* net, int slot, cudaStream_t st)
{
    std::vector<std::array<const void*, 2>> ptr;
    std::vector<long long> words;
    for (auto& T : net->tensors) {
        if (!T.X2b) return RRM_ERR_INVALID_ARG;
        ptr.push_back({reinterpret_cast<const char*>(T.X2b) + (size_t)slot * T.bytes(), T.X});
        words.push_back((long long)(T.bytes() / 4));
    }
    for (auto& L : net->layers) {
        if (!L.P2b) return RRM_ERR_INVALID_ARG;
        const size_t bytes = (size_t)L.opixels() * L.d.c_out * 4;
        ptr.push_back({reinterpret_cast<const char*>(L.P2b) + (size_t)slot * bytes, L.P});
        words.push_back((long long)(bytes / 4));
    }
    for (size_t j0 = 0; j0 < ptr.size(); j0 += 32) {
        CopyJobs j;
        j.n = (int)(ptr.size() - j0 < 32 ? ptr.size() - j0 : 32);
        long long most = 0;
        for (int k = 0; k < 32; ++k) {
            if (k < j.n) {
                j.src[k] = reinterpret_cast<const int*>(ptr[j0 + k][0]);
                j.dst[k] = reinterpret_cast<int*>(const_cast<void*>(ptr[j0 + k][1]));
                j.words[k] = words[j0 + k];
                most = most > j.words[k] ? most : j.words[k];
            } else { j.src[k] = nullptr; j.dst[k] = nullptr; j.words[k] = 0; }
        }
        long long gx = (most / 4 + 255) / 256;
        gx = gx < 1 ? 1 : (gx > 148 ? 148 : gx);
        launch_seq(copy_projections_kernel, dim3((unsigned)gx, (unsigned)j.n), dim3(256), 0, st, j);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

int launch_aecs(rrm_net* net, cudaStream_t st)
{
    AecsParams a;
    a.n = (int)net->layers.size();
    if (a.n > 64) return RRM_ERR_UNSUPPORTED;
    for (int l = 0; l < a.n; ++l) a.sumsq[l] = net->tensors[net->layers[l].d.src].trunc;
    a.e_t = net->aecs; a.last_l2 = net->aecs + 1;
    launch_seq(aecs_accumulate_kernel, dim3(1), dim3(32), 0, st, a);
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

int launch_export_tensor(rrm_net* net, int t, void* dst, bool stateless, cudaStream_t st)
{
    Tensor& T = net->tensors[t];
    const void* X = stateless ? T.X2 : T.X;
    if (T.dtype == T_BIN) {
        RRM_CUDA_TRY(cudaMemcpyAsync(dst, X, T.bytes(), cudaMemcpyDeviceToDevice, st));
        return RRM_OK;
    }
    const int hw = T.h * T.w;
    const long long total = (long long)T.n * T.c * hw;
    const int blocks = (int)((total + 255) / 256);
    if (T.dtype == T_I8) launch_seq(export_nchw_kernel<int8_t>, dim3(blocks), dim3(256), 0, st, (const int8_t*)X, (int8_t*)dst, T.c, T.cs, hw, total, 0ll, 0ll);
    else {
        const int ctiles = ceil_div(T.c, 32);
        launch_seq(export_nchw_tiled_kernel, dim3(ceil_div(hw, 32), ctiles * T.n, 1), dim3(32, 8), 0, st, (const uint32_t*)X, (uint32_t*)dst,
                   T.c, T.cs, hw, ctiles, 0ll, 0ll);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

// Every frame's output of the layer-by-layer chunk form (the last tensor's full rows) to the boundary layout.
int launch_export_seq(rrm_net* net, int frames, void* dst, cudaStream_t st)
{
    Tensor& T = net->tensors.back();
    if (!T.Xfull) return RRM_ERR_INVALID_ARG;
    if (T.dtype == T_BIN) {
        RRM_CUDA_TRY(cudaMemcpyAsync(dst, T.Xfull, T.bytes() * frames, cudaMemcpyDeviceToDevice, st));
        return RRM_OK;
    }
    const int hw = T.h * T.w;
    const long long total = (long long)T.n * T.c * hw;
    const dim3 grid((unsigned)((total + 255) / 256), (unsigned)frames);
    if (T.dtype == T_I8) launch_seq(export_nchw_kernel<int8_t>, grid, dim3(256), 0, st, (const int8_t*)T.Xfull, (int8_t*)dst, T.c, T.cs, hw, total,
                                    (long long)T.bytes(), total);
    else {
        const int ctiles = ceil_div(T.c, 32);
        launch_seq(export_nchw_tiled_kernel, dim3(ceil_div(hw, 32), ctiles * T.n, frames), dim3(32, 8), 0, st, (const uint32_t*)T.Xfull, (uint32_t*)dst,
                   T.c, T.cs, hw, ctiles, (long long)T.bytes() / 4, total);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

// Layer l over `frames` consecutive frames in two launches: the sparse products of all frames, each stored in a buffer
// of its own (rows of the updated pixels), then the epilogue that walks the frames in order (rrm_conv_seq.cu).  The
// bound arena and the tensors' D / Xn_cur are frame 0's.
int launch_layer_seq(rrm_net* net, int l, int frames, long long arena_stride, cudaStream_t st)
{
    Layer& L = net->layers[l];
    const rrm_layer_desc& d = L.d;
    Tensor& in = net->tensors[d.src];
    if (!L.dPall || frames < 1) return RRM_ERR_INVALID_ARG;
    if (L.tc_ready) RRM_TRY(launch_conv_tc(net, L, in, false, false, st, nullptr, L.dPall, frames, arena_stride));
    else {
        ConvParams p{};
        p.D = in.D; p.X = in.Xn_cur ? in.Xn_cur : in.X; p.in_act = in.act; p.oact = L.oact; p.ocount = L.ocount;
        p.Wk = L.Wk; p.bias = L.bias; p.P = L.dPall;
        p.n = d.n; p.c_in = d.c_in; p.h = d.h; p.w = d.w; p.u_in = L.u_in; p.oh = L.oh; p.ow = L.ow;
        p.kh = d.kh; p.kw = d.kw; p.stride = d.stride; p.pad = d.pad; p.c_out = d.c_out; p.np = L.np;
        p.ku = L.ku; p.kup = L.kup; p.opixels = L.opixels();
        p.wait_limit = net->opt.wait_limit;
        p.errw = net->errw;
        p.ksplit = 1;
        p.frames = frames > 1 ? frames : 2;                  // (one frame still takes the storing form: the kernel tests frames > 1)
        p.row_stride = (long long)in.bytes(); p.arena_stride = arena_stride; p.p_stride = (long long)L.opixels() * d.c_out;
        dim3 grid(ceil_div(L.opixels(), TM), L.np / TN, frames);
        if (d.dtype == RRM_F32) {
            // fp32 with a grid of less than ~3 waves: 2 or 4 shares of K per tile (a cluster that adds its partial tiles in
            // a fixed order), while a share keeps at least 4 stages: CTAs with rows are few and long otherwise
            const long long ctas = (long long)grid.x * grid.y * grid.z, slots = 4ll * 148;
            const int stages = L.kup / TK;
            while (p.ksplit < 4 && ctas * p.ksplit < 3 * slots && stages / (p.ksplit * 2) >= 4) p.ksplit *= 2;
            grid.z = frames * p.ksplit;
        }
        if (d.dtype == RRM_F32) launch_gemm<T_F32, false>(p, grid, st);
        else if (d.dtype == RRM_I8) launch_gemm<T_I8, false>(p, grid, st);
        else launch_gemm<T_BIN, false>(p, grid, st);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return launch_epilogue_seq(net, l, frames, arena_stride, st);
}

int launch_export_projection(rrm_net* net, int l, void* dst, cudaStream_t st)
{
    Layer& L = net->layers[l];
    const int hw = L.oh * L.ow;
    const long long total = (long long)L.d.n * L.d.c_out * hw;
    launch_seq(export_nchw_kernel<uint32_t>, dim3((int)((total + 255) / 256)), dim3(256), 0, st, (const uint32_t*)L.P, (uint32_t*)dst,
                                                                            L.d.c_out, L.d.c_out, hw, total, 0ll, 0ll);
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

}  // namespace rrm
