// Device helpers shared by the convolution kernels: how activity travels from a tensor to the layers
// that read it, and how a CTA finds its rows in a layer's bitmap of projection pixels to update.
#pragma once
#include "rrm_common.cuh"

namespace rrm {

// Executed by a full warp for ONE changed pixel (ns, y, x) of a tensor with `nnz` non-zero delta
// elements: marks, in every reading layer's bitmap, the projection pixels whose filter footprint
// covers the pixel (a layer that adds the tensor as its shortcut is a 1x1 reader), and returns in
// macs[i] (same value in every lane) the exact multiply-accumulates the pixel implies in reader i:
// nnz x (output, tap) pairs that meet it x output channels (Table 1 without its border approximation).
__device__ __forceinline__ void scatter_changed(const Readers& R, int ns, int y, int x, int nnz, int lane,
                                                unsigned long long (&macs)[MAX_READERS])
{
    #pragma unroll
    for (int i = 0; i < MAX_READERS; ++i) {
        macs[i] = 0;
        if (i >= R.n) continue;
        const Reader& c = R.r[i];
        const int taps = c.kh * c.kw;
        int hits = 0;
        for (int t = lane; t < taps; t += 32) {
            const int ky = t / c.kw, kx = t - ky * c.kw;
            const int ty = y + c.pad - ky, tx = x + c.pad - kx;
            if (ty < 0 || tx < 0 || ty % c.stride || tx % c.stride) continue;
            const int oy = ty / c.stride, ox = tx / c.stride;
            if (oy >= c.oh || ox >= c.ow) continue;
            const int q = (ns * c.oh + oy) * c.ow + ox;
            atomicOr(&c.oact[q >> 5], 1u << (q & 31));
            ++hits;
        }
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) hits += __shfl_xor_sync(0xffffffffu, hits, o);
        if (c.macs) macs[i] = (unsigned long long)nnz * hits * c.c_out;
    }
}

// Rows [tile * TM, tile * TM + TM) of the set bits of bm[0 .. words), in increasing pixel order, go to
// s_q[0 .. TM) (-1 where the bitmap has fewer).  Returns the total number of set bits.  Every thread
// of the CTA calls it; s_tmp holds 33 ints.
template <int TM>
__device__ int select_rows(const uint32_t* __restrict__ bm, int words, int tile, int* s_q, int* s_tmp)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nt = blockDim.x, nwarps = (nt + 31) >> 5;
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
    if (lane == 31) s_tmp[warp] = incl;
    if (tid < TM) s_q[tid] = -1;
    __syncthreads();
    int run = incl - mine, total = 0;
    for (int w = 0; w < nwarps; ++w) {
        const int v = s_tmp[w];
        if (w < warp) run += v;
        total += v;
    }
    const int first = tile * TM;
    if (run < first + TM && run + mine > first) {
        for (int i = lo; i < hi; ++i) {
            uint32_t w = __ldg(bm + i);
            while (w) {
                const int b = __ffs(w) - 1;
                w &= w - 1;
                if (run >= first && run < first + TM) s_q[run - first] = i * 32 + b;
                ++run;
            }
        }
    }
    __syncthreads();
    return total;
}

}  // namespace rrm
