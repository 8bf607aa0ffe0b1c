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
#include <type_traits>

namespace rrm {

constexpr int TM = 64;            // projection pixels per CTA
constexpr int TN = GEMM_TN;       // output channels per CTA
constexpr int TK = GEMM_TK;       // K units per stage
constexpr int CONV_THREADS = 256;

struct ConvParams {
    const void* D;            // delta rows (delta mode) / unused (dense)
    const void* X;            // input values (dense mode; binary delta mode: new sign bits)
    const uint32_t* in_act;   // input activity bitmap (delta mode)
    const uint32_t* oact;     // projection pixels to update (delta mode)
    int* ocount;              // receives their number
    const void* Wk;           // [kup][np] units
    const void* bias;
    void* P;                  // [opixels][c_out]
    int n, c_in, h, w, u_in, oh, ow, kh, kw, stride, pad, c_out, np, ku, kup, opixels;
};

__device__ __forceinline__ bool bit_test(const uint32_t* bm, int i) { return (bm[i >> 5] >> (i & 31)) & 1u; }

// ------------------------------------------------------------------------------------------------
// Implicit GEMM.  DT: T_F32 (float FMA), T_I8 (dp4a on 4-channel words), T_BIN (popcount on 32-channel
// words: sum(d*w) = 2*(popc(changed) - 2*popc(changed & (new ^ wbits))), dense: valid instead of changed
// and no factor 2).  VEC: units per pixel divisible by 4 -> 128-bit gathers.
// ------------------------------------------------------------------------------------------------
template <int DT, bool DENSE, bool VEC>
__global__ void __launch_bounds__(CONV_THREADS) conv_gemm_kernel(ConvParams p)
{
    using acc_t = typename std::conditional<DT == T_F32, float, int>::type;
    __shared__ __align__(16) uint32_t As[TK][TM];
    __shared__ __align__(16) uint32_t As2[(DT == T_BIN) ? TK : 1][TM];
    __shared__ __align__(16) uint32_t Bs[TK][TN];
    __shared__ int s_q[TM], s_nbase[TM], s_iy0[TM], s_ix0[TM];
    __shared__ int s_rowsum[TM];
    __shared__ int s_tmp[33];

    const int tid = threadIdx.x;
    const int tile = blockIdx.x, n0 = blockIdx.y * TN;
    if (!DENSE) {
        // this CTA's rows: the tile-th group of TM set bits of the layer's update bitmap
        const int count = select_rows<TM>(p.oact, (p.opixels + 31) >> 5, tile, s_q, s_tmp);
        if (tile == 0 && blockIdx.y == 0 && tid == 0) *p.ocount = count;
        if (tile * TM >= count) return;
    }
    if (tid < TM) {
        const int r = tile * TM + tid;
        const int q = DENSE ? (r < p.opixels ? r : -1) : s_q[tid];
        s_q[tid] = q;
        s_rowsum[tid] = 0;
        if (q >= 0) {
            const int ox = q % p.ow, oy = (q / p.ow) % p.oh, ns = q / (p.ow * p.oh);
            s_nbase[tid] = ns * p.h * p.w;
            s_iy0[tid] = oy * p.stride - p.pad;
            s_ix0[tid] = ox * p.stride - p.pad;
        } else {
            s_nbase[tid] = 0; s_iy0[tid] = -(1 << 20); s_ix0[tid] = -(1 << 20);
        }
    }
    __syncthreads();

    const int a_row = tid >> 2, a_k = (tid & 3) * 4;       // A gather: 4 consecutive units of one row
    const int b_row = tid >> 4, b_col = (tid & 15) * 4;    // B load: 4 consecutive output channels
    const int tm = (tid >> 4) * 4, tn = (tid & 15) * 4;    // 4x4 outputs per thread
    const int my_nbase = s_nbase[a_row], my_iy0 = s_iy0[a_row], my_ix0 = s_ix0[a_row];
    const uint32_t tail_mask = (p.c_in & 31) ? ((1u << (p.c_in & 31)) - 1u) : 0xffffffffu;

    acc_t acc[4][4];
    #pragma unroll
    for (int i = 0; i < 4; ++i)
        #pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;
    int my_popc = 0;

    const uint32_t* Du = reinterpret_cast<const uint32_t*>(p.D);
    const uint32_t* Xu = reinterpret_cast<const uint32_t*>(p.X);
    const uint32_t* Wu = reinterpret_cast<const uint32_t*>(p.Wk);

    for (int k0 = 0; k0 < p.kup; k0 += TK) {
        // ---- gather 4 units of A into registers
        uint32_t a1[4] = {0, 0, 0, 0}, a2[4] = {0, 0, 0, 0};
        int any = 0;
        auto locate = [&](int k, int& u) -> long long {     // pixel-row offset (in units) or -1
            if (k >= p.ku) return -1;
            const int tap = k / p.u_in;
            u = k - tap * p.u_in;
            const int ky = tap / p.kw, kx = tap - ky * p.kw;
            const int iy = my_iy0 + ky, ix = my_ix0 + kx;
            if (iy < 0 || iy >= p.h || ix < 0 || ix >= p.w) return -1;
            const int pix = my_nbase + iy * p.w + ix;
            if (!DENSE && !bit_test(p.in_act, pix)) return -1;
            return (long long)pix * p.u_in;
        };
        if (VEC) {
            int u;
            const long long off = locate(k0 + a_k, u);
            if (off >= 0) {
                any = 1;
                if (DT == T_BIN) {
                    const uint4 nw = *reinterpret_cast<const uint4*>(Xu + off + u);
                    uint4 ch;
                    if (DENSE) {
                        ch = make_uint4(~0u, ~0u, ~0u, ~0u);
                        if (u + 3 == p.u_in - 1) ch.w = tail_mask;
                    } else {
                        ch = *reinterpret_cast<const uint4*>(Du + off + u);
                    }
                    a1[0] = ch.x; a1[1] = ch.y; a1[2] = ch.z; a1[3] = ch.w;
                    a2[0] = nw.x; a2[1] = nw.y; a2[2] = nw.z; a2[3] = nw.w;
                } else {
                    const uint4 v = *reinterpret_cast<const uint4*>((DENSE ? Xu : Du) + off + u);
                    a1[0] = v.x; a1[1] = v.y; a1[2] = v.z; a1[3] = v.w;
                }
            }
        } else {
            #pragma unroll
            for (int i = 0; i < 4; ++i) {
                int u;
                const long long off = locate(k0 + a_k + i, u);
                if (off >= 0) {
                    any = 1;
                    if (DT == T_BIN) {
                        a2[i] = Xu[off + u];
                        a1[i] = DENSE ? ((u == p.u_in - 1) ? tail_mask : 0xffffffffu) : Du[off + u];
                    } else {
                        a1[i] = (DENSE ? Xu : Du)[off + u];
                    }
                }
            }
        }
        // a stage with no active row contributes nothing: skip it (uniform decision; the barrier
        // also protects the shared tiles from the previous stage's readers)
        if (!__syncthreads_or(any)) continue;
        const uint4 bv = *reinterpret_cast<const uint4*>(Wu + (size_t)(k0 + b_row) * p.np + n0 + b_col);
        #pragma unroll
        for (int i = 0; i < 4; ++i) {
            As[a_k + i][a_row] = a1[i];
            if (DT == T_BIN) { As2[a_k + i][a_row] = a2[i]; my_popc += __popc(a1[i]); }
        }
        *reinterpret_cast<uint4*>(&Bs[b_row][b_col]) = bv;
        __syncthreads();
        #pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            const uint4 av = *reinterpret_cast<const uint4*>(&As[kk][tm]);
            const uint4 bw = *reinterpret_cast<const uint4*>(&Bs[kk][tn]);
            const uint32_t a[4] = {av.x, av.y, av.z, av.w}, b[4] = {bw.x, bw.y, bw.z, bw.w};
            uint32_t a_nw[4] = {0, 0, 0, 0};
            if (DT == T_BIN) {
                const uint4 nv = *reinterpret_cast<const uint4*>(&As2[kk][tm]);
                a_nw[0] = nv.x; a_nw[1] = nv.y; a_nw[2] = nv.z; a_nw[3] = nv.w;
            }
            #pragma unroll
            for (int i = 0; i < 4; ++i)
                #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (DT == T_F32) acc[i][j] = fmaf(__uint_as_float(a[i]), __uint_as_float(b[j]), acc[i][j]);
                    else if (DT == T_I8) acc[i][j] = __dp4a((int)a[i], (int)b[j], (int)acc[i][j]);
                    else acc[i][j] += __popc(a[i] & (a_nw[i] ^ b[j]));
                }
        }
    }
    if (DT == T_BIN) {
        if (my_popc) atomicAdd(&s_rowsum[a_row], my_popc);
    }
    __syncthreads();

    // ---- owner-computes update of the stored projection
    #pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int q = s_q[tm + i];
        if (q < 0) continue;
        #pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int co = n0 + tn + j;
            if (co >= p.c_out) continue;
            const size_t o = (size_t)q * p.c_out + co;
            if (DT == T_F32) {
                float* P = reinterpret_cast<float*>(p.P);
                if (DENSE) P[o] = acc[i][j] + (p.bias ? reinterpret_cast<const float*>(p.bias)[co] : 0.f);
                else P[o] += acc[i][j];
            } else {
                int* P = reinterpret_cast<int*>(p.P);
                int v = (int)acc[i][j];
                if (DT == T_BIN) v = DENSE ? (s_rowsum[tm + i] - 2 * v) : 2 * (s_rowsum[tm + i] - 2 * v);
                if (DENSE) P[o] = v + (p.bias ? reinterpret_cast<const int*>(p.bias)[co] : 0);
                else P[o] += v;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Filter repack: W[c_out][c_in][kh][kw] -> Wk[k][np] with k = tap * u_in + unit (zero padded).
// ------------------------------------------------------------------------------------------------
__global__ void pack_weights_kernel(const void* W, uint32_t* Wk, int dt, int c_in, int c_out, int kh, int kw,
                                    int u_in, int kup, int np)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= kup * np) return;
    const int k = idx / np, co = idx - k * np;
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
constexpr int IMP_TP = 32;

template <typename T, bool DELTA>
__global__ void __launch_bounds__(256) import_nchw_kernel(const T* __restrict__ src, T* X, T* D, uint32_t* act,
                                                          int* pnnz, unsigned long long* nnz,
                                                          unsigned long long* npix, int* errw,
                                                          int c, int cs, int hw, int w, Readers readers)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* s_x = reinterpret_cast<T*>(smem_raw);               // [IMP_TP][cs + 1]
    __shared__ int s_cnt[IMP_TP];
    const int ld = cs + 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ns = blockIdx.y, pix0 = blockIdx.x * IMP_TP;
    if (tid < IMP_TP) s_cnt[tid] = 0;
    for (int ch = warp; ch < cs; ch += 8) {
        T v = 0;
        if (ch < c && pix0 + lane < hw) v = src[((size_t)ns * c + ch) * hw + pix0 + lane];
        s_x[lane * ld + ch] = v;
    }
    __syncthreads();
    const size_t gp0 = (size_t)ns * hw + pix0;
    for (int idx = tid; idx < IMP_TP * cs; idx += 256) {
        const int pl = idx / cs, ch = idx - pl * cs;
        if (pix0 + pl >= hw) continue;
        const size_t o = (gp0 + pl) * cs + ch;
        const T xt = s_x[pl * ld + ch];
        if (DELTA) {
            const T xp = X[o];
            if (xt != xp) {
                atomicAdd(&s_cnt[pl], 1);
                X[o] = xt;
                if (sizeof(T) == 1) {
                    const int d = (int)xt - (int)xp;
                    if (d < -128 || d > 127) atomicOr(errw, ERRW_BOUNDS);
                }
            }
            s_x[pl * ld + ch] = (T)(xt - xp);
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
    if (tid < MAX_READERS) s_macs[tid] = 0;
    __syncthreads();
    for (int pl = warp; pl < IMP_TP; pl += 8) {
        const int cnt = (pix0 + pl < hw) ? s_cnt[pl] : 0;
        if (cnt == 0) continue;
        const int pix = pix0 + pl;
        unsigned long long macs[MAX_READERS];
        scatter_changed(readers, ns, pix / w, pix % w, cnt, lane, macs);
        if (lane == 0) {
            #pragma unroll
            for (int i = 0; i < MAX_READERS; ++i) if (macs[i]) atomicAdd(&s_macs[i], macs[i]);
        }
    }
    __syncthreads();
    if (tid < readers.n && s_macs[tid]) atomicAdd(readers.r[tid].macs, s_macs[tid]);
}

// Binary frames arrive already pixel-major and bit-packed: one thread per pixel.
template <bool DELTA>
__global__ void import_bin_kernel(const uint32_t* __restrict__ src, uint32_t* X, uint32_t* D, uint32_t* act,
                                  int* pnnz, unsigned long long* nnz, unsigned long long* npix, int cw, int pixels,
                                  int h, int w, Readers readers)
{
    const int gp = blockIdx.x * blockDim.x + threadIdx.x;
    int cnt = 0;
    if (gp < pixels) {
        for (int k = 0; k < cw; ++k) {
            const uint32_t xt = src[(size_t)gp * cw + k];
            if (DELTA) {
                const uint32_t ch = xt ^ X[(size_t)gp * cw + k];
                D[(size_t)gp * cw + k] = ch;
                cnt += __popc(ch);
            }
            X[(size_t)gp * cw + k] = xt;
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
    #pragma unroll
    for (int i = 0; i < MAX_READERS; ++i) wsum[i] = 0;
    for (unsigned mm = m; mm; mm &= mm - 1) {
        const int src_lane = __ffs(mm) - 1;
        const int pix = __shfl_sync(0xffffffffu, gp, src_lane), c = __shfl_sync(0xffffffffu, cnt, src_lane);
        const int x = pix % w, y = (pix / w) % h, ns = pix / (w * h);
        unsigned long long macs[MAX_READERS];
        scatter_changed(readers, ns, y, x, c, lane, macs);
        #pragma unroll
        for (int i = 0; i < MAX_READERS; ++i) wsum[i] += macs[i];
    }
    if (lane == 0) {
        #pragma unroll
        for (int i = 0; i < MAX_READERS; ++i) if (i < readers.n && wsum[i]) atomicAdd(readers.r[i].macs, wsum[i]);
    }
}

// ------------------------------------------------------------------------------------------------
// Epilogue: f on the stored projection, next layer's delta.  One warp per output-tensor pixel; a lane
// owns 4 neighbouring channels at a time, so the 4-channel words of all window positions are fetched
// with independent 128-bit loads (one memory round trip per 128 channels).
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
    Readers readers;          // layers that read the output tensor
};

// PT: projection type (T_F32 or T_I32).  OT: output tensor storage type.  KW: pool window edge (1 = no pool).
template <int PT, int OT, bool DENSE, int KW>
__global__ void __launch_bounds__(256) epilogue_kernel(EpiParams p)
{
    using pt = typename std::conditional<PT == T_F32, float, int>::type;
    __shared__ unsigned long long s_macs[MAX_READERS];
    __shared__ unsigned int s_nnz, s_npix;
    const int lane = threadIdx.x & 31;
    if (threadIdx.x < MAX_READERS) s_macs[threadIdx.x] = 0;
    if (threadIdx.x == 0) { s_nnz = 0; s_npix = 0; }
    __syncthreads();
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int tpix = p.n * p.th * p.tw;
    const int tx = r % p.tw, ty = (r / p.tw) % p.th, ns = r / (p.tw * p.th);
    const int st = KW > 1 ? p.pool_s : 1, pp = KW > 1 ? p.pool_p : 0;
    const int y0 = ty * st - pp, x0 = tx * st - pp;
    const int qbase = ns * p.oh * p.ow;
    // window positions inside the projection (bit wy * KW + wx), and whether any of them was updated
    unsigned inside = 0;
    bool on = false;
    if (r < tpix) {
        bool mine = false, upd = false;
        if (lane < KW * KW) {
            const int y = y0 + lane / KW, x = x0 + lane % KW;
            mine = y >= 0 && y < p.oh && x >= 0 && x < p.ow;
            if (mine && !DENSE) { const int q = qbase + y * p.ow + x; upd = (p.oact[q >> 5] >> (q & 31)) & 1u; }
        }
        inside = __ballot_sync(0xffffffffu, mine);
        on = DENSE ? true : (__ballot_sync(0xffffffffu, upd) != 0);
    }
    int cnt = 0;
    if (on) {
        const pt* P = reinterpret_cast<const pt*>(p.P);
        const bool vec = (p.c_out & 3) == 0;
        const int c_iter = (OT == T_BIN) ? p.cs * 32 : p.cs;
        for (int c0 = 0; c0 < c_iter; c0 += 128) {
            const int c = c0 + lane * 4;
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
            }
            // ---- f: [requant] -> [+ shortcut] -> act -> max over the window (sign: max first, threshold last)
            pt best[4];
            #pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool live = c + j < p.c_out;
                pt res = 0;
                if (live && p.resX) {
                    if (PT == T_F32) res = (pt)reinterpret_cast<const float*>(p.resX)[(size_t)r * p.cs + c + j];
                    else if (OT == T_I8) res = (pt)reinterpret_cast<const int8_t*>(p.resX)[(size_t)r * p.cs + c + j];
                }
                bool have = false;
                pt b = 0;
                #pragma unroll
                for (int wi = 0; wi < KW * KW; ++wi) {
                    if (!(inside >> wi & 1u)) continue;
                    pt x = v[wi][j];
                    if (PT == T_F32) {
                        x += res;
                        if (p.act_fn == RRM_ACT_RELU) x = x > 0 ? x : 0;
                    } else if (OT == T_I8) {
                        int iv = (int)x;
                        if (p.shift > 0) iv = (iv + (1 << (p.shift - 1))) >> p.shift;
                        iv = max(-127, min(127, iv));
                        iv += (int)res;
                        iv = (p.act_fn == RRM_ACT_RELU) ? max(0, min(127, iv)) : max(-127, min(127, iv));
                        x = (pt)iv;
                    }
                    if (!have || x > b) { b = x; have = true; }
                }
                best[j] = live ? b : (pt)0;
            }
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
                        const uint32_t ow_ = *X;
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
                            Dp[o + j] = best[j] - old;
                            if (best[j] != old) { X[o + j] = best[j]; ++cnt; }
                        }
                    }
                }
            }
        }
    }
    if (DENSE) return;
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (cnt) {                                               // uniform inside the warp
        if (lane == 0) {
            atomicOr(&p.act[r >> 5], 1u << (r & 31));
            p.pnnz[r] = cnt;
            atomicAdd(&s_nnz, (unsigned)cnt);
            atomicAdd(&s_npix, 1u);
        }
        unsigned long long macs[MAX_READERS];
        scatter_changed(p.readers, ns, ty, tx, cnt, lane, macs);
        if (lane == 0) {
            #pragma unroll
            for (int i = 0; i < MAX_READERS; ++i) if (macs[i]) atomicAdd(&s_macs[i], macs[i]);
        }
    }
    __syncthreads();
    if (threadIdx.x < p.readers.n && s_macs[threadIdx.x]) atomicAdd(p.readers.r[threadIdx.x].macs, s_macs[threadIdx.x]);
    if (threadIdx.x == 0 && s_npix) {
        atomicAdd(p.nnz, (unsigned long long)s_nnz);
        atomicAdd(p.npix, (unsigned long long)s_npix);
    }
}

// ------------------------------------------------------------------------------------------------
// Exports to the boundary layout.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void export_nchw_kernel(const T* __restrict__ src, T* dst, int c, int cs, int hw, long long total)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int pix = (int)(i % hw);
    const int ch = (int)((i / hw) % c);
    const long long ns = i / ((long long)hw * c);
    dst[i] = src[(ns * hw + pix) * cs + ch];
}

template <typename T>
__global__ void fill_projection_kernel(T* P, const T* bias, int c_out, long long total)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total) P[i] = bias ? bias[i % c_out] : (T)0;
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

static int ensure_stateless(rrm_net* net)
{
    for (auto& T : net->tensors)
        if (!T.X2) RRM_TRY(dev_alloc(net, &T.X2, T.bytes()));
    for (auto& L : net->layers)
        if (!L.P2) RRM_TRY(dev_alloc(net, &L.P2, (size_t)L.opixels() * L.d.c_out * 4));
    return RRM_OK;
}

int launch_import(rrm_net* net, const void* frame, bool delta, bool stateless, cudaStream_t st)
{
    if (stateless) RRM_TRY(ensure_stateless(net));
    Tensor& T = net->tensors[0];
    void* X = stateless ? T.X2 : T.X;
    const int hw = T.h * T.w;
    if (T.dtype == T_BIN) {
        const int blocks = ceil_div(T.pixels(), 256);
        if (delta) import_bin_kernel<true><<<blocks, 256, 0, st>>>((const uint32_t*)frame, (uint32_t*)X, (uint32_t*)T.D,
                                                                  T.act, T.pnnz, T.nnz, T.npix, T.cs, T.pixels(),
                                                                  T.h, T.w, T.readers);
        else import_bin_kernel<false><<<blocks, 256, 0, st>>>((const uint32_t*)frame, (uint32_t*)X, nullptr, nullptr,
                                                              nullptr, nullptr, nullptr, T.cs, T.pixels(), T.h, T.w,
                                                              Readers{});
    } else {
        dim3 grid(ceil_div(hw, IMP_TP), T.n);
        const size_t smem = (size_t)IMP_TP * (T.cs + 1) * T.unit_bytes;
        if (T.dtype == T_F32) {
            auto kd = import_nchw_kernel<float, true>;
            auto kn = import_nchw_kernel<float, false>;
            if (smem > 48 * 1024) {
                cudaFuncSetAttribute(kd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
                cudaFuncSetAttribute(kn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            }
            if (delta) kd<<<grid, 256, smem, st>>>((const float*)frame, (float*)X, (float*)T.D, T.act, T.pnnz, T.nnz,
                                                   T.npix, net->errw, T.c, T.cs, hw, T.w, T.readers);
            else kn<<<grid, 256, smem, st>>>((const float*)frame, (float*)X, nullptr, nullptr, nullptr, nullptr,
                                             nullptr, net->errw, T.c, T.cs, hw, T.w, Readers{});
        } else {
            auto kd = import_nchw_kernel<int8_t, true>;
            auto kn = import_nchw_kernel<int8_t, false>;
            if (delta) kd<<<grid, 256, smem, st>>>((const int8_t*)frame, (int8_t*)X, (int8_t*)T.D, T.act, T.pnnz,
                                                   T.nnz, T.npix, net->errw, T.c, T.cs, hw, T.w, T.readers);
            else kn<<<grid, 256, smem, st>>>((const int8_t*)frame, (int8_t*)X, nullptr, nullptr, nullptr, nullptr,
                                             nullptr, net->errw, T.c, T.cs, hw, T.w, Readers{});
        }
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

template <int DT, bool DENSE>
static void launch_gemm(const ConvParams& p, bool vec, dim3 grid, cudaStream_t st)
{
    if (vec) conv_gemm_kernel<DT, DENSE, true><<<grid, CONV_THREADS, 0, st>>>(p);
    else conv_gemm_kernel<DT, DENSE, false><<<grid, CONV_THREADS, 0, st>>>(p);
}

template <int PT, int OT, bool DENSE>
static int launch_epi_k(const EpiParams& e, int blocks, cudaStream_t st)
{
    switch (e.pool_k > 0 ? e.pool_k : 1) {
        case 1: epilogue_kernel<PT, OT, DENSE, 1><<<blocks, 256, 0, st>>>(e); break;
        case 2: epilogue_kernel<PT, OT, DENSE, 2><<<blocks, 256, 0, st>>>(e); break;
        case 3: epilogue_kernel<PT, OT, DENSE, 3><<<blocks, 256, 0, st>>>(e); break;
        default: return RRM_ERR_UNSUPPORTED;                 // pool windows are 2x2 or 3x3
    }
    return RRM_OK;
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

int launch_layer(rrm_net* net, int l, bool dense, bool stateless, cudaStream_t st)
{
    Layer& L = net->layers[l];
    const rrm_layer_desc& d = L.d;
    Tensor& in = net->tensors[d.src];
    Tensor& out = net->tensors[l + 1];
    Tensor* res = d.res >= 0 ? &net->tensors[d.res] : nullptr;

    ConvParams p;
    p.D = in.D; p.X = stateless ? in.X2 : in.X; p.in_act = in.act; p.oact = L.oact; p.ocount = L.ocount;
    p.Wk = L.Wk; p.bias = L.bias; p.P = stateless ? L.P2 : L.P;
    p.n = d.n; p.c_in = d.c_in; p.h = d.h; p.w = d.w; p.u_in = L.u_in; p.oh = L.oh; p.ow = L.ow;
    p.kh = d.kh; p.kw = d.kw; p.stride = d.stride; p.pad = d.pad; p.c_out = d.c_out; p.np = L.np;
    p.ku = L.ku; p.kup = L.kup; p.opixels = L.opixels();
    dim3 grid(ceil_div(L.opixels(), TM), L.np / TN);
    const bool vec = (L.u_in % 4) == 0;
    if (L.tc_ready) RRM_TRY(launch_conv_tc(net, L, in, dense, stateless, st));
    else if (d.dtype == RRM_F32) { if (dense) launch_gemm<T_F32, true>(p, vec, grid, st); else launch_gemm<T_F32, false>(p, vec, grid, st); }
    else if (d.dtype == RRM_I8) { if (dense) launch_gemm<T_I8, true>(p, vec, grid, st); else launch_gemm<T_I8, false>(p, vec, grid, st); }
    else { if (dense) launch_gemm<T_BIN, true>(p, vec, grid, st); else launch_gemm<T_BIN, false>(p, vec, grid, st); }

    EpiParams e;
    e.P = p.P; e.oact = L.oact;
    e.resX = res ? (stateless ? res->X2 : res->X) : nullptr;
    e.X = stateless ? out.X2 : out.X; e.D = out.D; e.act = out.act; e.pnnz = out.pnnz; e.nnz = out.nnz;
    e.npix = out.npix; e.errw = out.has_consumer ? net->errw : nullptr;
    e.n = d.n; e.oh = L.oh; e.ow = L.ow; e.th = L.th; e.tw = L.tw; e.c_out = d.c_out; e.cs = out.cs;
    e.pool_k = d.pool_k; e.pool_s = d.pool_s; e.pool_p = d.pool_p; e.act_fn = d.act; e.shift = d.shift; e.theta = d.theta;
    e.readers = dense ? Readers{} : out.readers;
    const int blocks = ceil_div(out.pixels(), 8);
    int es;
    if (proj_type(L) == T_F32) es = dense ? launch_epi<T_F32, true>(e, out.dtype, blocks, st) : launch_epi<T_F32, false>(e, out.dtype, blocks, st);
    else es = dense ? launch_epi<T_I32, true>(e, out.dtype, blocks, st) : launch_epi<T_I32, false>(e, out.dtype, blocks, st);
    RRM_TRY(es);
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
    if (T.dtype == T_I8) export_nchw_kernel<int8_t><<<blocks, 256, 0, st>>>((const int8_t*)X, (int8_t*)dst, T.c, T.cs, hw, total);
    else export_nchw_kernel<uint32_t><<<blocks, 256, 0, st>>>((const uint32_t*)X, (uint32_t*)dst, T.c, T.cs, hw, total);
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

int launch_export_projection(rrm_net* net, int l, void* dst, cudaStream_t st)
{
    Layer& L = net->layers[l];
    const int hw = L.oh * L.ow;
    const long long total = (long long)L.d.n * L.d.c_out * hw;
    export_nchw_kernel<uint32_t><<<(int)((total + 255) / 256), 256, 0, st>>>((const uint32_t*)L.P, (uint32_t*)dst,
                                                                            L.d.c_out, L.d.c_out, hw, total);
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

}  // namespace rrm
