// Convolution path of the RRM step (Algorithm 1, conv branch), CUDA-core variant.
//
// All tensors inside the library are pixel-major ([n][h][w][units]); a "unit" is one float,
// four int8 channels, or 32 sign bits.  Per frame and layer:
//   import_delta   (layer input = the external frame only)  D = X_t - X_prev, per-pixel activity
//                  bitmap, X_prev := X_t in place for changed pixels;
//   active_pixels  dilates the input activity by the filter footprint into the set of projection
//                  pixels that can change, compacts it with warp ballots into a list, and counts
//                  the exact multiply-accumulates the non-zero deltas imply (Table 1);
//   delta_conv     implicit GEMM over the compacted pixels: rows = listed pixels, K = taps x input
//                  units gathered from the delta rows of active input pixels (zero otherwise),
//                  N = output channels; P_prev += result (owner computes: no float atomics);
//   epilogue       recomputes f only where its window touches an updated projection pixel,
//                  compares with the stored activation and emits the next layer's delta rows,
//                  activity bitmap and snapshot update in one pass.
// The same GEMM kernel with DENSE=true (all pixels, input values instead of deltas, bias added)
// is the library's dense path and the keyframe.
#include "rrm_common.cuh"
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
    const int* olist;         // compacted projection pixels (delta mode)
    const int* ocount;
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

    const int tid = threadIdx.x;
    const int tile = blockIdx.x, n0 = blockIdx.y * TN;
    int count = p.opixels;
    if (!DENSE) {
        count = *p.ocount;
        if (tile * TM >= count) return;
    }
    if (tid < TM) {
        const int r = tile * TM + tid;
        int q = -1;
        if (r < count) q = DENSE ? r : p.olist[r];
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
                                                          int c, int cs, int hw)
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
}

// Binary frames arrive already pixel-major and bit-packed: one thread per pixel.
template <bool DELTA>
__global__ void import_bin_kernel(const uint32_t* __restrict__ src, uint32_t* X, uint32_t* D, uint32_t* act,
                                  int* pnnz, unsigned long long* nnz, unsigned long long* npix, int cw, int pixels)
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
}

// ------------------------------------------------------------------------------------------------
// Active projection pixels: q is active iff some input pixel under its filter footprint is active,
// or the residual tensor changed at q.  Warp ballots give the bitmap word and the compacted list.
// The second half counts the exact multiply-accumulates implied by the non-zero deltas.
// ------------------------------------------------------------------------------------------------
struct ActiveParams {
    const uint32_t* in_act;
    const int* in_pnnz;
    const uint32_t* res_act;      // or nullptr
    uint32_t* oact;
    int* olist;
    int* ocount;
    unsigned long long* macs;
    int n, h, w, oh, ow, kh, kw, stride, pad, c_out;
};

__global__ void __launch_bounds__(256) active_pixels_kernel(ActiveParams p)
{
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    const int opix = p.n * p.oh * p.ow, ipix = p.n * p.h * p.w;
    const int lane = threadIdx.x & 31;
    bool on = false;
    if (q < opix) {
        const int ox = q % p.ow, oy = (q / p.ow) % p.oh, ns = q / (p.ow * p.oh);
        const int base = ns * p.h * p.w;
        for (int ky = 0; ky < p.kh && !on; ++ky) {
            const int iy = oy * p.stride - p.pad + ky;
            if (iy < 0 || iy >= p.h) continue;
            for (int kx = 0; kx < p.kw; ++kx) {
                const int ix = ox * p.stride - p.pad + kx;
                if (ix < 0 || ix >= p.w) continue;
                if (bit_test(p.in_act, base + iy * p.w + ix)) { on = true; break; }
            }
        }
        if (!on && p.res_act) on = bit_test(p.res_act, q);
    }
    const unsigned m = __ballot_sync(0xffffffffu, on);
    if (m) {
        int slot = 0;
        if (lane == 0) {
            slot = atomicAdd(p.ocount, __popc(m));
            p.oact[q >> 5] = m;                       // q of lane 0 is a multiple of 32
        }
        slot = __shfl_sync(0xffffffffu, slot, 0);
        if (on) p.olist[slot + __popc(m & ((1u << lane) - 1u))] = q;
    }
    // exact active MACs: every non-zero delta element at (y,x) meets ty(y)*tx(x) filter taps
    unsigned long long macs = 0;
    if (q < ipix && bit_test(p.in_act, q)) {
        const int x = q % p.w, y = (q / p.w) % p.h;
        int ty = 0, tx = 0;
        for (int ky = 0; ky < p.kh; ++ky) {
            const int t = y + p.pad - ky;
            ty += (t >= 0 && t % p.stride == 0 && t / p.stride < p.oh);
        }
        for (int kx = 0; kx < p.kw; ++kx) {
            const int t = x + p.pad - kx;
            tx += (t >= 0 && t % p.stride == 0 && t / p.stride < p.ow);
        }
        macs = (unsigned long long)p.in_pnnz[q] * ty * tx * p.c_out;
    }
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) macs += __shfl_down_sync(0xffffffffu, macs, o);
    if (lane == 0 && macs) atomicAdd(p.macs, macs);
}

// ------------------------------------------------------------------------------------------------
// Epilogue: f on the stored projection, next layer's delta.  One warp per output-tensor pixel.
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
};

// PT: projection type (T_F32 or T_I32).  OT: output tensor storage type.
template <int PT, int OT, bool DENSE>
__global__ void __launch_bounds__(256) epilogue_kernel(EpiParams p)
{
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int tpix = p.n * p.th * p.tw;
    if (r >= tpix) return;
    const int tx = r % p.tw, ty = (r / p.tw) % p.th, ns = r / (p.tw * p.th);
    const int k = p.pool_k > 0 ? p.pool_k : 1, st = p.pool_k > 0 ? p.pool_s : 1, pp = p.pool_k > 0 ? p.pool_p : 0;
    const int y0 = ty * st - pp, x0 = tx * st - pp;
    const int qbase = ns * p.oh * p.ow;
    if (!DENSE) {
        bool on = false;
        for (int wy = 0; wy < k && !on; ++wy) {
            const int y = y0 + wy;
            if (y < 0 || y >= p.oh) continue;
            for (int wx = 0; wx < k; ++wx) {
                const int x = x0 + wx;
                if (x < 0 || x >= p.ow) continue;
                if (bit_test(p.oact, qbase + y * p.ow + x)) { on = true; break; }
            }
        }
        if (!on) return;
    }
    using pt = typename std::conditional<PT == T_F32, float, int>::type;
    const pt* P = reinterpret_cast<const pt*>(p.P);
    int cnt = 0;
    const int c_iter = (OT == T_BIN) ? p.cs * 32 : p.cs;
    for (int c0 = 0; c0 < c_iter; c0 += 32) {
        const int c = c0 + lane;
        const bool live = c < p.c_out;
        // pooled value of channel c (before sign / after requant+residual+act for int8)
        pt best = 0;
        bool have = false;
        if (live) {
            for (int wy = 0; wy < k; ++wy) {
                const int y = y0 + wy;
                if (y < 0 || y >= p.oh) continue;
                for (int wx = 0; wx < k; ++wx) {
                    const int x = x0 + wx;
                    if (x < 0 || x >= p.ow) continue;
                    pt v = P[(size_t)(qbase + y * p.ow + x) * p.c_out + c];
                    if (PT == T_F32) {
                        if (p.resX) v += reinterpret_cast<const float*>(p.resX)[(size_t)r * p.cs + c];
                        if (p.act_fn == RRM_ACT_RELU) v = v > 0 ? v : 0;
                    } else if (OT == T_I8) {
                        int iv = (int)v;
                        if (p.shift > 0) iv = (iv + (1 << (p.shift - 1))) >> p.shift;
                        iv = max(-127, min(127, iv));
                        if (p.resX) iv += (int)reinterpret_cast<const int8_t*>(p.resX)[(size_t)r * p.cs + c];
                        iv = (p.act_fn == RRM_ACT_RELU) ? max(0, min(127, iv)) : max(-127, min(127, iv));
                        v = (pt)iv;
                    }
                    if (!have || v > best) { best = v; have = true; }
                }
            }
        }
        const size_t o = (size_t)r * p.cs + (OT == T_BIN ? (c0 >> 5) : c);
        if (OT == T_BIN) {
            const unsigned word = __ballot_sync(0xffffffffu, live && (int)best >= p.theta);
            if (lane == 0) {
                uint32_t* X = reinterpret_cast<uint32_t*>(p.X);
                if (DENSE) X[o] = word;
                else {
                    const uint32_t ch = word ^ X[o];
                    reinterpret_cast<uint32_t*>(p.D)[o] = ch;
                    X[o] = word;
                    cnt += __popc(ch);
                }
            }
        } else if (c < p.cs) {
            if (OT == T_F32) {
                float* X = reinterpret_cast<float*>(p.X);
                const float v = live ? (float)best : 0.f;
                if (DENSE) X[o] = v;
                else {
                    const float old = X[o];
                    reinterpret_cast<float*>(p.D)[o] = v - old;
                    if (v != old) { X[o] = v; ++cnt; }
                }
            } else if (OT == T_I32) {
                int* X = reinterpret_cast<int*>(p.X);
                const int v = live ? (int)best : 0;
                if (DENSE) X[o] = v;
                else {
                    const int old = X[o];
                    reinterpret_cast<int*>(p.D)[o] = v - old;
                    if (v != old) { X[o] = v; ++cnt; }
                }
            } else {   // T_I8
                int8_t* X = reinterpret_cast<int8_t*>(p.X);
                const int v = live ? (int)best : 0;
                if (DENSE) X[o] = (int8_t)v;
                else {
                    const int old = X[o];
                    const int d = v - old;
                    if (p.errw && (d < -128 || d > 127)) atomicOr(p.errw, ERRW_BOUNDS);
                    reinterpret_cast<int8_t*>(p.D)[o] = (int8_t)d;
                    if (v != old) { X[o] = (int8_t)v; ++cnt; }
                }
            }
        }
    }
    if (DENSE) return;
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_down_sync(0xffffffffu, cnt, o);
    if (lane == 0 && cnt) {
        atomicOr(&p.act[r >> 5], 1u << (r & 31));
        p.pnnz[r] = cnt;
        atomicAdd(p.nnz, (unsigned long long)cnt);
        atomicAdd(p.npix, 1ull);
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
    RRM_TRY(dev_alloc(net, (void**)&L.olist, (size_t)L.opixels() * 4));
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
                                                                  T.act, T.pnnz, T.nnz, T.npix, T.cs, T.pixels());
        else import_bin_kernel<false><<<blocks, 256, 0, st>>>((const uint32_t*)frame, (uint32_t*)X, nullptr, nullptr,
                                                              nullptr, nullptr, nullptr, T.cs, T.pixels());
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
                                                   T.npix, net->errw, T.c, T.cs, hw);
            else kn<<<grid, 256, smem, st>>>((const float*)frame, (float*)X, nullptr, nullptr, nullptr, nullptr,
                                             nullptr, net->errw, T.c, T.cs, hw);
        } else {
            auto kd = import_nchw_kernel<int8_t, true>;
            auto kn = import_nchw_kernel<int8_t, false>;
            if (delta) kd<<<grid, 256, smem, st>>>((const int8_t*)frame, (int8_t*)X, (int8_t*)T.D, T.act, T.pnnz,
                                                   T.nnz, T.npix, net->errw, T.c, T.cs, hw);
            else kn<<<grid, 256, smem, st>>>((const int8_t*)frame, (int8_t*)X, nullptr, nullptr, nullptr, nullptr,
                                             nullptr, net->errw, T.c, T.cs, hw);
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

template <int PT, bool DENSE>
static void launch_epi(const EpiParams& e, int ot, int blocks, cudaStream_t st)
{
    switch (ot) {
        case T_F32: epilogue_kernel<PT, T_F32, DENSE><<<blocks, 256, 0, st>>>(e); break;
        case T_I8: epilogue_kernel<PT, T_I8, DENSE><<<blocks, 256, 0, st>>>(e); break;
        case T_BIN: epilogue_kernel<PT, T_BIN, DENSE><<<blocks, 256, 0, st>>>(e); break;
        default: epilogue_kernel<PT, T_I32, DENSE><<<blocks, 256, 0, st>>>(e); break;
    }
}

int launch_layer(rrm_net* net, int l, bool dense, bool stateless, cudaStream_t st)
{
    Layer& L = net->layers[l];
    const rrm_layer_desc& d = L.d;
    Tensor& in = net->tensors[d.src];
    Tensor& out = net->tensors[l + 1];
    Tensor* res = d.res >= 0 ? &net->tensors[d.res] : nullptr;

    if (!dense) {
        ActiveParams a;
        a.in_act = in.act; a.in_pnnz = in.pnnz; a.res_act = res ? res->act : nullptr;
        a.oact = L.oact; a.olist = L.olist; a.ocount = L.ocount; a.macs = L.macs;
        a.n = d.n; a.h = d.h; a.w = d.w; a.oh = L.oh; a.ow = L.ow; a.kh = d.kh; a.kw = d.kw;
        a.stride = d.stride; a.pad = d.pad; a.c_out = d.c_out;
        const int work = L.opixels() > in.pixels() ? L.opixels() : in.pixels();
        active_pixels_kernel<<<ceil_div(work, 256), 256, 0, st>>>(a);
    }
    ConvParams p;
    p.D = in.D; p.X = stateless ? in.X2 : in.X; p.in_act = in.act; p.olist = L.olist; p.ocount = L.ocount;
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
    const int blocks = ceil_div(out.pixels(), 8);
    if (proj_type(L) == T_F32) { if (dense) launch_epi<T_F32, true>(e, out.dtype, blocks, st); else launch_epi<T_F32, false>(e, out.dtype, blocks, st); }
    else { if (dense) launch_epi<T_I32, true>(e, out.dtype, blocks, st); else launch_epi<T_I32, false>(e, out.dtype, blocks, st); }
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
