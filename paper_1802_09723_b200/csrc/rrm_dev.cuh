// Small device functions shared by several kernels of the library: the int8 delta scan (non-zero bytes of a word),
// the column product of the delta-FC kernels, the integer form of f for an FC output, and the per-row tap masks of
// the two convolution kernels.
#pragma once
#include <cstdint>
#include <type_traits>
#include <cuda_runtime.h>
#include "../../include/rrm.h"

namespace rrm {

// one flag bit per non-zero byte of v, packed into the low 4 bits
__device__ __forceinline__ unsigned nonzero_bytes(unsigned v)
{
    v |= v >> 4; v |= v >> 2; v |= v >> 1;
    return ((v & 0x01010101u) * 0x01020408u) >> 24 & 0xfu;
}

// 16-bit mask of the bytes in which two 16-byte chunks differ (a byte differs <=> its delta is non-zero)
__device__ __forceinline__ unsigned differing_bytes(const uint4& a, const uint4& b)
{
    return nonzero_bytes(a.x ^ b.x) | nonzero_bytes(a.y ^ b.y) << 4 | nonzero_bytes(a.z ^ b.z) << 8 | nonzero_bytes(a.w ^ b.w) << 12;
}

// acc[i] += w_i * d for the 16 int8 weights in w (one 16-byte piece of a weight column, Sec. 3.5): dp4a against a
// selector that holds d in one byte lane; a delta outside the int8 range (|d| <= 254) is split into two in-range halves.
__device__ __forceinline__ void fma16(int (&acc)[16], const uint4& w, int d)
{
    const unsigned ww[4] = {w.x, w.y, w.z, w.w};
    const int dh = (d >= -128 && d <= 127) ? 0 : d / 2;
    const int dl = d - dh;
    const unsigned lb = (unsigned)dl & 0xffu, hb = (unsigned)dh & 0xffu;
    #pragma unroll
    for (int q = 0; q < 4; ++q) {
        #pragma unroll
        for (int b = 0; b < 4; ++b) acc[q * 4 + b] = __dp4a((int)ww[q], (int)(lb << (8 * b)), acc[q * 4 + b]);
    }
    if (dh != 0) {
        #pragma unroll
        for (int q = 0; q < 4; ++q) {
            #pragma unroll
            for (int b = 0; b < 4; ++b) acc[q * 4 + b] = __dp4a((int)ww[q], (int)(hb << (8 * b)), acc[q * 4 + b]);
        }
    }
}

// f of an int8 FC output: requantise by `shift` (round half up), clamp to [-127, 127], optional ReLU
__device__ __forceinline__ int fc_apply_f(int v, int shift, int act)
{
    if (shift > 0) v = (v + (1 << (shift - 1))) >> shift;
    v = max(-127, min(127, v));
    if (act == RRM_ACT_RELU) v = max(v, 0);
    return v;
}

// The usable filter taps of one projection pixel as a 128-bit mask (bit t = tap ky * kw + kx): the tap's input pixel
// lies inside the image and, in a delta pass, changed in this frame (its bit in the input activity bitmap is set).
// (y0, x0) is the input pixel under tap (0, 0) and pix0 its flat index (both may lie outside the image).
// One filter row at a time: its usable taps are a run of consecutive input pixels, whose activity bits come out of
// one or two bitmap words together; filters wider than 32 taps go tap by tap, 8 bitmap loads in flight.
template <bool DENSE>
__device__ __forceinline__ void row_tap_masks(const uint32_t* __restrict__ in_act, int pix0, int y0, int x0, int h, int w, int kh, int kw,
                                              unsigned long long& m0, unsigned long long& m1)
{
    m0 = 0; m1 = 0;
    const int taps = kh * kw;
    if (kw <= 32) {
        const int kx_lo = max(0, -x0), kx_hi = min(kw, w - x0), nk = kx_hi - kx_lo;
        const unsigned run = nk >= 32 ? 0xffffffffu : ((1u << max(nk, 0)) - 1u);
        for (int ky = 0; ky < kh && nk > 0; ++ky) {
            const int iy = y0 + ky;
            if (iy < 0 || iy >= h) continue;
            unsigned bits = run;
            if (!DENSE) {
                const int g = pix0 + ky * w + kx_lo, sh = g & 31;
                unsigned long long two = in_act[g >> 5];
                if (sh + nk > 32) two |= (unsigned long long)in_act[(g >> 5) + 1] << 32;
                bits = (unsigned)(two >> sh) & run;
            }
            if (bits == 0) continue;
            const int t = ky * kw + kx_lo;                   // tap index of the run's first bit
            if (t < 64) {
                m0 |= (unsigned long long)bits << t;
                if (t + nk > 64) m1 |= (unsigned long long)bits >> (64 - t);
            } else {
                m1 |= (unsigned long long)bits << (t - 64);
            }
        }
        return;
    }
    for (int t0 = 0; t0 < taps; t0 += 8) {
        uint32_t word[8];
        int sh[8];
        #pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int t = t0 + u, ky = t / kw, kx = t - ky * kw;
            const int iy = y0 + ky, ix = x0 + kx;
            const bool in = t < taps && iy >= 0 && iy < h && ix >= 0 && ix < w;
            const int pix = pix0 + ky * w + kx;
            sh[u] = in ? (pix & 31) : -1;
            word[u] = DENSE ? 0xffffffffu : (in ? in_act[pix >> 5] : 0u);
        }
        #pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (sh[u] >= 0 && ((word[u] >> sh[u]) & 1u)) {
                const int t = t0 + u;
                if (t < 64) m0 |= 1ull << t; else m1 |= 1ull << (t - 64);
            }
        }
    }
}

// pointer + byte offset
template <typename P>
__device__ __forceinline__ P* shift_bytes(P* p, long long bytes)
{
    return reinterpret_cast<P*>(reinterpret_cast<char*>(const_cast<typename std::remove_const<P>::type*>(p)) + bytes);
}

// f of Algorithm 1 on the 4 neighbouring channels c .. c+3 of one output pixel: [affine] -> [requantisation] -> [+ shortcut]
// -> activation -> max over the pool window (a sign activation takes the max first, its threshold is the caller's).
// v: the projection at the window's positions (bit wi of `inside`: position wi lies inside the projection);
// res: the shortcut's values; PT: projection type, OT: output storage type, KW: window edge, BN: the explicit
// per-channel affine of Sec. 4.5 (fp32: y = scale * P + shift; int8: multiplier and offset inside the requantisation).
template <int PT, int OT, int KW, bool BN, typename pt>
__device__ __forceinline__ void epi_f(const pt (&v)[KW * KW][4], unsigned inside, int c, const pt (&res)[4], int c_out,
                                      int act_fn, int shift, const void* bn_scale, const void* bn_shift, pt (&best)[4])
{
    #pragma unroll
    for (int j = 0; j < 4; ++j) {
        const bool live = c + j < c_out;
        pt bn_m = 1, bn_a = 0;
        if (BN && live) {
            bn_m = reinterpret_cast<const pt*>(bn_scale)[c + j];
            bn_a = reinterpret_cast<const pt*>(bn_shift)[c + j];
        }
        bool have = false;
        pt b = 0;
        #pragma unroll
        for (int wi = 0; wi < KW * KW; ++wi) {
            if (!(inside >> wi & 1u)) continue;
            pt x = v[wi][j];
            if (PT == T_F32) {
                if (BN) x = (pt)fmaf((float)x, (float)bn_m, (float)bn_a);
                x += res[j];
                if (act_fn == RRM_ACT_RELU) x = x > 0 ? x : 0;
                else if (act_fn == RRM_ACT_LEAKY) x = x > 0 ? x : (pt)(0.1f * (float)x);
            } else if (OT == T_I8) {
                int iv = (int)x;
                if (BN) {                                    // 64-bit exact
                    long long t = (long long)iv * (long long)(int)bn_m + (long long)(int)bn_a;
                    if (shift > 0) t = (t + (1ll << (shift - 1))) >> shift;
                    iv = (int)max(-127ll, min(127ll, t));
                } else {
                    if (shift > 0) iv = (iv + (1 << (shift - 1))) >> shift;
                    iv = max(-127, min(127, iv));
                }
                iv += (int)res[j];
                iv = (act_fn == RRM_ACT_RELU) ? max(0, min(127, iv)) : max(-127, min(127, iv));
                x = (pt)iv;
            }
            if (!have || x > b) { b = x; have = true; }
        }
        best[j] = live ? b : (pt)0;
    }
}

}  // namespace rrm
