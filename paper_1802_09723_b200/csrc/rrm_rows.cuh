// Device helpers shared by the convolution kernels: how activity travels from a tensor to the layers
// that read it, and how a CTA finds its rows in a layer's bitmap of projection pixels to update.
#pragma once
#include "rrm_common.cuh"
#include "rrm_dev.cuh"

namespace rrm {

// Executed by a full warp for 32 CONSECUTIVE pixels of a tensor: lane j owns one pixel (ns, y, x) (consecutive in
// the flattened [n][h][w] order) with `cnt` non-zero delta elements (0: unchanged or past the end).  Marks, in every
// reading layer's bitmap, the projection pixels whose filter footprint covers a changed pixel (a layer that adds
// the tensor as its shortcut is a 1x1 reader), and returns in macs[i] (same value in every lane) the exact
// multiply-accumulates the changed pixels imply in reader i: non-zeros x (output, tap) pairs that meet the pixel x
// output channels (Table 1 without its border approximation).
// The projection pixels that meet (y, x) form a rectangle [oy_lo, oy_hi] x [ox_lo, ox_hi], and changed pixels come
// in runs along an image row, so the marking is done per row segment of the warp, not per pixel: lane j tests
// candidate projection column ox_min + j against the segment's mask of changed pixels, a ballot gives the columns
// as a run of bits, and lane r ORs that run into projection row oy_lo + r (one or two word-wide atomic ORs).
// arena_off: byte offset of the arena whose bitmaps are marked from the one the readers' pointers refer to (several
// frames per launch: frame g's arena).
__device__ __forceinline__ void scatter_changed_warp(const Readers& R, int ns, int y, int x, int cnt, int lane,
                                                     unsigned long long (&macs)[MAX_READERS], long long arena_off = 0)
{
    const unsigned m = __ballot_sync(0xffffffffu, cnt > 0);
    #pragma unroll
    for (int i = 0; i < MAX_READERS; ++i) macs[i] = 0;
    if (m == 0) return;                                      // nothing changed: uniform inside the warp
    const unsigned seg_starts = __ballot_sync(0xffffffffu, x == 0 || lane == 0);
    #pragma unroll 1
    for (int i = 0; i < R.n; ++i) {
        const Reader& c = R.r[i];
        // this lane's own pixel: rows x columns of projection pixels it meets (for the exact count)
        if (c.macs) {
            unsigned long long mine = 0;
            if (cnt > 0) {
                const int ay = y + c.pad, ax = x + c.pad;
                const int rows = min(c.oh - 1, ay / c.stride) - max(0, (ay - c.kh + c.stride) / c.stride) + 1;
                const int cols = min(c.ow - 1, ax / c.stride) - max(0, (ax - c.kw + c.stride) / c.stride) + 1;
                if (rows > 0 && cols > 0) mine = (unsigned long long)cnt * rows * cols * c.c_out;
            }
            #pragma unroll
            for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
            macs[i] = mine;
        }
        // one row segment [a, b] of lanes at a time
        for (unsigned ss = seg_starts; ss; ss &= ss - 1) {
            const int a = __ffs(ss) - 1;
            const unsigned rest = ss & (ss - 1);
            const int b = rest ? __ffs(rest) - 2 : 31;
            const unsigned seg = (b - a == 31 ? 0xffffffffu : ((1u << (b - a + 1)) - 1u) << a);
            const unsigned ms = m & seg;
            if (ms == 0) continue;
            const int sns = __shfl_sync(0xffffffffu, ns, a), sy = __shfl_sync(0xffffffffu, y, a), xa = __shfl_sync(0xffffffffu, x, a);
            const int ay = sy + c.pad;
            const int oy_lo = max(0, (ay - c.kh + c.stride) / c.stride), oy_hi = min(c.oh - 1, ay / c.stride);
            if (oy_hi < oy_lo) continue;
            const int x_first = xa + (__ffs(ms) - 1 - a), x_last = xa + (31 - __clz(ms) - a);
            const int ox_min = max(0, (x_first + c.pad - c.kw + c.stride) / c.stride);
            const int ox_max = min(c.ow - 1, (x_last + c.pad) / c.stride);
            for (int c0 = ox_min; c0 <= ox_max; c0 += 32) {
                const int ox = c0 + lane;
                bool touched = false;
                if (ox <= ox_max) {
                    // input columns under this projection column, as lanes of the segment
                    const int la = max(a, ox * c.stride - c.pad - xa + a), lb = min(b, ox * c.stride - c.pad + c.kw - 1 - xa + a);
                    if (la <= lb) {
                        const unsigned bits = (lb - la == 31 ? 0xffffffffu : ((1u << (lb - la + 1)) - 1u) << la);
                        touched = (ms & bits) != 0;
                    }
                }
                const unsigned run = __ballot_sync(0xffffffffu, touched);
                if (run == 0) continue;
                for (int r = oy_lo + lane; r <= oy_hi; r += 32) {
                    const int q0 = (sns * c.oh + r) * c.ow + c0;
                    const unsigned long long v = (unsigned long long)run << (q0 & 31);
                    uint32_t* bm = shift_bytes(c.oact, arena_off);
                    atomicOr(&bm[q0 >> 5], (unsigned)v);
                    if (v >> 32) atomicOr(&bm[(q0 >> 5) + 1], (unsigned)(v >> 32));
                }
            }
        }
    }
}

// Rows [tile * TM, tile * TM + TM) of the set bits of bm[0 .. words), in increasing pixel order, go to
// s_q[0 .. TM) (-1 where the bitmap has fewer).  Returns the total number of set bits.  Every thread
// of the CTA calls it (blockDim.x <= 256, TM <= blockDim.x); s_pref holds 256 + 34 ints.
// Each thread counts a contiguous share of the words; an exclusive prefix sum over the threads tells
// every row which thread's share holds its bit, and the row walks that share (a few words) itself:
// all TM rows are located in parallel.
template <int TM>
__device__ int select_rows(const uint32_t* __restrict__ bm, int words, int tile, int* s_q, int* s_pref)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nt = blockDim.x, nwarps = (nt + 31) >> 5;
    int* s_warp = s_pref + 257;
    const int nper = (words + nt - 1) / nt;
    const int lo = min(words, tid * nper), hi = min(words, lo + nper);
    int mine = 0;
    for (int i = lo; i < hi; ++i) mine += __popc(__ldg(bm + i));
    int incl = mine;
    #pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int before = incl - mine, total = 0;
    for (int w = 0; w < nwarps; ++w) {
        const int v = s_warp[w];
        if (w < warp) before += v;
        total += v;
    }
    s_pref[tid] = before;                                    // set bits in the shares of threads 0 .. tid-1
    if (tid == nt - 1) s_pref[nt] = total;
    __syncthreads();
    if (tid < TM) {
        const int rank = tile * TM + tid;
        int q = -1;
        if (rank < total) {
            int t = 0;                                       // largest t with s_pref[t] <= rank
            for (int step = 128; step > 0; step >>= 1)
                if (t + step < nt && s_pref[t + step] <= rank) t += step;
            int k = rank - s_pref[t];
            for (int i = t * nper; i < words; ++i) {
                const uint32_t w = __ldg(bm + i);
                const int c = __popc(w);
                if (k < c) { q = i * 32 + (int)__fns(w, 0, k + 1); break; }
                k -= c;
            }
        }
        s_q[tid] = q;
    }
    __syncthreads();
    return total;
}

}  // namespace rrm
