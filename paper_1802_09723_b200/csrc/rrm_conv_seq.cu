// A chunk of consecutive frames through a stack, layer by layer (rrm_net_step_seq on delta chunks; the remark at the
// end of Sec. 3.2: a video may be handed over in chunks).
//
// Algorithm 1 is serial in t only through the state a layer keeps: the T input deltas of layer 0 are known as soon as
// the chunk is, and once a layer has emitted its T output deltas the next layer's T sparse products F*dI_t are
// independent of one another.  So every kernel of a step takes all frames of the chunk in one launch:
//   import      frame g against frame g-1 at the boundary (rrm_conv.cu), delta rows and bitmaps per frame;
//   convolution frame = blockIdx.z: the product of frame g is stored in a buffer of its own, rows of updated pixels only;
//   projection  (here) lane g of a warp is frame g: P_g = P_before + sum_{t<=g} F*dI_t (Eq. 5 unrolled) is an inclusive
//               prefix sum over the lanes, once per updated projection pixel; the last frame's goes to the stored projection;
//   epilogue    (here) lane = frame again: f is evaluated in every frame at once, the previous frame's output comes
//               from the neighbouring lane, and lane g emits frame g's delta row, bitmap bit and counters.
// A 32-frame chunk of a five-layer stack is 20 launches instead of 384, and the chains of dependent memory round trips
// that bound a single-frame launch are paid once per layer and chunk instead of once per layer and frame.
#include "rrm_common.cuh"
#include "rrm_rows.cuh"
#include "rrm_dev.cuh"
#include <type_traits>

namespace rrm {

constexpr int SEQ_MAX_FRAMES = 32;            // frames per launch: one lane of a warp per frame

struct EpiSeqParams {
    const void* P;            // the projection as of the frame before the chunk (a copy: read only)
    void* Q;                  // the stored projection: receives P + the products of all frames at the updated pixels
    const void* dP;           // frame 0's product (rows of the pixels in frame 0's update bitmap)
    const uint32_t* oact;     // frame 0's update bitmap
    void* X;                  // the output tensor's snapshot: read as the value before the chunk, left as the last frame's
    void* D;                  // frame 0's delta rows of the output tensor
    void* Xn;                 // frame 0's new rows (binary outputs that a layer reads: the sign of a changed bit) or nullptr
    void* Xfull;              // or nullptr: receives every pixel's row of every frame (the stack's last tensor)
    // shortcut (the layer adds another tensor of the output's shape before the activation): that tensor's value before
    // the chunk, frame 0's new rows of it and frame 0's activity bitmap of it; nullptr: none
    const void* res_before;
    const void* res_new;
    const uint32_t* res_act;
    long long res_stride;     // bytes between the frames' new rows of the shortcut tensor
    uint32_t* act;            // frame 0's activity bitmap of the output tensor
    unsigned long long* nnz;
    unsigned long long* npix;
    int* errw;
    int n, oh, ow, th, tw, c_out, cs, pool_k, pool_s, pool_p, act_fn, shift, theta;
    Readers readers;          // layers that read the output tensor (frame 0's arena)
    const void* bn_scale;
    const void* bn_shift;
    int frames;
    long long row_stride;     // bytes between the frames' delta rows / new rows / full rows of the output tensor
    long long arena_stride;   // bytes between the frames' arenas
    long long p_stride;       // elements between the frames' products
    int opix;                 // projection pixels
    const int8_t* A0;         // epilogue_seq_pool8_kernel: the pointwise part of f as bytes, before the chunk (every projection pixel) ...
    const int8_t* A;          // ... and of frame 0 (updated pixels), the frames a_stride bytes apart
    long long a_stride;
};

// Inclusive prefix sum over the lanes of a warp (lane g: sum of lanes 0 .. g), in a fixed order: the merge role and the
// f role use the same one, so the stored projection is bit for bit the one f saw for the last frame (fp32).
template <typename pt>
__device__ __forceinline__ void scan4(pt (&d)[4], int lane)
{
    #pragma unroll
    for (int k = 1; k < 32; k <<= 1) {
        #pragma unroll
        for (int j = 0; j < 4; ++j) {
            const pt t = __shfl_up_sync(0xffffffffu, d[j], k);
            if (lane >= k) d[j] += t;
        }
    }
}

// 4 neighbouring elements at P + o (o a multiple of 4 when vec); elements from `limit` on read as zero
template <typename pt, typename pt4>
__device__ __forceinline__ void load4(const pt* P, size_t o, bool vec, int c, int limit, pt (&v)[4])
{
    v[0] = v[1] = v[2] = v[3] = 0;
    if (c >= limit) return;
    if (vec) { const pt4 t = *reinterpret_cast<const pt4*>(P + o); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
    else {
        #pragma unroll
        for (int j = 0; j < 4; ++j) if (c + j < limit) v[j] = P[o + j];
    }
}

// The projections of all frames, once per projection pixel: P_g = P_before + sum_{t<=g} F*dI_t (Eq. 5 unrolled) as an
// inclusive prefix sum over the lanes (lane g = frame g).  P_g overwrites frame g's product where frame g updated
// the pixel; the last frame's value goes to the stored projection.  A CTA per pixel of the union of the frames'
// update bitmaps, its warps spread over the channels.
struct ProjSeqParams {
    const void* R;            // the projection before the chunk (a copy: read only)
    void* Q;                  // the stored projection
    void* dP;                 // frame 0's product; in: F*dI_g, out: P_g
    const uint32_t* oact;     // frame 0's update bitmap
    int frames, c_out, opix;
    long long arena_stride, p_stride;
    // ACT (int8 outputs behind a pool window): the pointwise part of f ([affine] -> requantisation -> activation) is
    // applied here, once per projection pixel, and kept as bytes: A0 for the projection before the chunk (every pixel),
    // A + g * a_stride for frame g (its updated pixels); the epilogue then only takes maxima of bytes
    int8_t* A0;
    int8_t* A;
    long long a_stride;
    int act_fn, shift;
    const void* bn_scale;
    const void* bn_shift;
};

template <int PT, bool ACT, bool BN>
__global__ void __launch_bounds__(256) project_seq_kernel(ProjSeqParams p)
{
    using pt = typename std::conditional<PT == T_F32, float, int>::type;
    using pt4 = typename std::conditional<PT == T_F32, float4, int4>::type;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool vec = (p.c_out & 3) == 0;
    const int q = blockIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    bool mine = false;
    if (lane < p.frames) mine = (shift_bytes(p.oact, lane * p.arena_stride)[q >> 5] >> (q & 31)) & 1u;
    const bool any = __any_sync(0xffffffffu, mine);          // (the same in every warp of the CTA)
    if (!any && !ACT) return;
    const pt* R = reinterpret_cast<const pt*>(p.R);
    pt* Q = reinterpret_cast<pt*>(p.Q);
    pt* dPg = reinterpret_cast<pt*>(p.dP) + (size_t)(lane < p.frames ? lane : 0) * p.p_stride;
    const size_t row = (size_t)q * p.c_out;
    const int quads = (p.c_out + 3) >> 2;
    constexpr int NQ = 4;                                    // groups of four channels per turn (one memory round trip)
    for (int u0 = warp * NQ; u0 < quads; u0 += 8 * NQ) {
        pt base[NQ][4], d[NQ][4];
        #pragma unroll
        for (int k = 0; k < NQ; ++k) {
            const int c = (u0 + k) * 4;
            base[k][0] = base[k][1] = base[k][2] = base[k][3] = 0;
            d[k][0] = d[k][1] = d[k][2] = d[k][3] = 0;
            if (u0 + k >= quads) continue;
            load4<pt, pt4>(R, row + c, vec, c, p.c_out, base[k]);
            if (mine) load4<pt, pt4>(dPg, row + c, vec, c, p.c_out, d[k]);
        }
        #pragma unroll
        for (int k = 0; k < NQ; ++k) {
            const int c = (u0 + k) * 4;
            if (u0 + k >= quads) continue;                   // uniform inside the warp
            if (ACT) {
                // f before the pool window, as bytes: of the projection before the chunk (lane 0 writes it) ...
                pt y[4];
                const pt none[4] = {0, 0, 0, 0};
                const pt (&b1)[1][4] = reinterpret_cast<const pt (&)[1][4]>(base[k]);
                epi_f<PT, T_I8, 1, BN, pt>(b1, 1u, c, none, p.c_out, p.act_fn, p.shift, p.bn_scale, p.bn_shift, y);
                if (lane == 0)
                    *reinterpret_cast<uint32_t*>(p.A0 + row + c) = ((uint32_t)(int)y[0] & 0xffu) | ((uint32_t)(int)y[1] & 0xffu) << 8 |
                                                                   ((uint32_t)(int)y[2] & 0xffu) << 16 | ((uint32_t)(int)y[3] & 0xffu) << 24;
                if (!any) continue;                          // a pixel no frame updates: nothing else to do
            }
            scan4(d[k], lane);
            #pragma unroll
            for (int j = 0; j < 4; ++j) d[k][j] += base[k][j];
            if (ACT && mine) {                               // ... and of this lane's frame
                pt y[4];
                const pt none[4] = {0, 0, 0, 0};
                const pt (&d1)[1][4] = reinterpret_cast<const pt (&)[1][4]>(d[k]);
                epi_f<PT, T_I8, 1, BN, pt>(d1, 1u, c, none, p.c_out, p.act_fn, p.shift, p.bn_scale, p.bn_shift, y);
                *reinterpret_cast<uint32_t*>(p.A + (long long)lane * p.a_stride + row + c) =
                    ((uint32_t)(int)y[0] & 0xffu) | ((uint32_t)(int)y[1] & 0xffu) << 8 | ((uint32_t)(int)y[2] & 0xffu) << 16 | ((uint32_t)(int)y[3] & 0xffu) << 24;
            }
            if (mine || lane == 31) {
                pt* dst = mine ? dPg : Q;
                if (vec) {
                    pt4 t; t.x = d[k][0]; t.y = d[k][1]; t.z = d[k][2]; t.w = d[k][3];
                    *reinterpret_cast<pt4*>(dst + row + c) = t;
                    if (mine && lane == 31) *reinterpret_cast<pt4*>(Q + row + c) = t;
                } else {
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (c + j >= p.c_out) continue;
                        dst[row + c + j] = d[k][j];
                        if (mine && lane == 31) Q[row + c + j] = d[k][j];
                    }
                }
            }
        }
    }
}

// Per frame in which the CTA's output pixel r changed (lane = frame, all frames at once): activity bit, counters, and in
// every reading layer's update bitmap of that frame the projection pixels whose filter footprint covers the pixel, with
// the exact multiply-accumulates they imply (non-zeros x covering (output, tap) pairs x output channels).
template <bool READERS>
__device__ __forceinline__ void seq_mark_frames(const EpiSeqParams& p, const int* s_cnt, int r, int ns, int ty, int tx, int lane, int warp)
{
    if (warp != 0) return;
    {
        const int cnt = lane < p.frames ? s_cnt[lane] : 0;
        if (cnt > 0) {
            const long long off = lane * p.arena_stride;
            // (the CTAs of the grid's y dimension share the pixel, each with a slice of the channels: counts add up, marks
            // are idempotent, and whoever sets the activity bit first counts the pixel)
            const unsigned had = atomicOr(shift_bytes(p.act, off) + (r >> 5), 1u << (r & 31));
            atomicAdd(shift_bytes(p.nnz, off), (unsigned long long)cnt);
            if (!(had >> (r & 31) & 1u)) atomicAdd(shift_bytes(p.npix, off), 1ull);
            if (READERS) {
                #pragma unroll 1
                for (int i = 0; i < p.readers.n; ++i) {
                    const Reader& rd = p.readers.r[i];
                    const int ay = ty + rd.pad, ax = tx + rd.pad;
                    const int oy_lo = max(0, (ay - rd.kh + rd.stride) / rd.stride), oy_hi = min(rd.oh - 1, ay / rd.stride);
                    const int ox_lo = max(0, (ax - rd.kw + rd.stride) / rd.stride), ox_hi = min(rd.ow - 1, ax / rd.stride);
                    if (oy_hi < oy_lo || ox_hi < ox_lo) continue;
                    uint32_t* bm = shift_bytes(rd.oact, off);
                    for (int oy = oy_lo; oy <= oy_hi; ++oy) {
                        int q0 = (ns * rd.oh + oy) * rd.ow + ox_lo, left = ox_hi - ox_lo + 1;
                        while (left > 0) {                   // the run of columns, word by word
                            const int bit = q0 & 31, take = min(left, 32 - bit);
                            const unsigned run = (take == 32 ? 0xffffffffu : ((1u << take) - 1u)) << bit;
                            atomicOr(&bm[q0 >> 5], run);
                            q0 += take; left -= take;
                        }
                    }
                    if (rd.macs)
                        atomicAdd(shift_bytes(rd.macs, off),
                                  (unsigned long long)cnt * (unsigned long long)((oy_hi - oy_lo + 1) * (ox_hi - ox_lo + 1)) * (unsigned long long)rd.c_out);
                }
            }
        }
    }
}

template <int PT, int OT, int KW, bool READERS, bool BN>
__global__ void __launch_bounds__(256) epilogue_seq_kernel(EpiSeqParams p)
{
    using pt = typename std::conditional<PT == T_F32, float, int>::type;
    using pt4 = typename std::conditional<PT == T_F32, float4, int4>::type;
    __shared__ int s_cnt[SEQ_MAX_FRAMES];                    // changed elements of the CTA's pixel, per frame
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (int)(blockDim.x >> 5);
    const bool vec = (p.c_out & 3) == 0;
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x < SEQ_MAX_FRAMES) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    // ---- f role: this CTA's output pixel; lane = frame
    const int r = blockIdx.x;
    const int tx = r % p.tw, ty = (r / p.tw) % p.th, ns = r / (p.tw * p.th);
    const int st = KW > 1 ? p.pool_s : 1, pp = KW > 1 ? p.pool_p : 0;
    const int y0 = ty * st - pp, x0 = tx * st - pp;
    const int qbase = ns * p.oh * p.ow;
    // window positions inside the projection (bit wy * KW + wx); ub: the positions this lane's frame updates
    unsigned inside, ub = 0;
    {
        bool mine = false;
        if (lane < KW * KW) {
            const int y = y0 + lane / KW, x = x0 + lane % KW;
            mine = y >= 0 && y < p.oh && x >= 0 && x < p.ow;
        }
        inside = __ballot_sync(0xffffffffu, mine);
        if (lane < p.frames) {
            const uint32_t* oa = shift_bytes(p.oact, lane * p.arena_stride);
            #pragma unroll
            for (int wi = 0; wi < KW * KW; ++wi) {
                if (!(inside >> wi & 1u)) continue;
                const int q = qbase + (y0 + wi / KW) * p.ow + x0 + wi % KW;
                if ((oa[q >> 5] >> (q & 31)) & 1u) ub |= 1u << wi;
            }
        }
    }
    const unsigned on_frames = __ballot_sync(0xffffffffu, ub != 0);
    const bool full = p.Xfull != nullptr;
    if (on_frames || full) {
        const bool live = lane < p.frames;                   // this lane stands for a frame
        const bool on = (on_frames >> lane) & 1u;            // ... whose window was updated: it emits a delta row
        const bool last = lane == p.frames - 1;
        const pt* P = reinterpret_cast<const pt*>(p.P);
        const pt* dP = reinterpret_cast<const pt*>(p.dP);
        unsigned uf[KW * KW];                                // per window position: the frames that update it
        #pragma unroll
        for (int wi = 0; wi < KW * KW; ++wi) uf[wi] = __ballot_sync(0xffffffffu, (ub >> wi) & 1u);
        unsigned res_upto = 0;                               // the frames up to this lane's in which the shortcut's pixel changed
        if (p.res_before) {
            bool ch = false;
            if (live) ch = (shift_bytes(p.res_act, lane * p.arena_stride)[r >> 5] >> (r & 31)) & 1u;
            res_upto = __ballot_sync(0xffffffffu, ch) & (0xffffffffu >> (31 - lane));
        }
        const long long roff = (long long)(live ? lane : 0) * p.row_stride;
        int cnt = 0;
        // f on NQ groups of four channels in every frame at once (a turn is one memory round trip): per window position
        // the frame's projection is fetched, the pointwise part of f applied, then the max over the window.
        // c[q] < 0: no such group.
        constexpr int NQ = KW == 1 ? 4 : (KW == 2 ? 2 : 1);
        auto eval = [&](const int (&c)[NQ], pt (&best)[NQ][4]) {
            pt x[NQ][KW * KW][4], res[NQ][4];
            pt dsum[KW == 1 ? NQ : 1][4];                    // no pool window: this frame's product, prefix-summed below
            #pragma unroll
            for (int q = 0; q < NQ; ++q) {
                res[q][0] = res[q][1] = res[q][2] = res[q][3] = 0;
                if (p.res_before && c[q] >= 0) {
                    // the shortcut's value in this lane's frame: the new row of the latest frame up to it in which the
                    // shortcut's pixel changed, else the value before the chunk
                    const char* src = res_upto ? reinterpret_cast<const char*>(p.res_new) + (long long)(31 - __clz(res_upto)) * p.res_stride
                                               : reinterpret_cast<const char*>(p.res_before);
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (c[q] + j >= p.c_out) continue;
                        if (PT == T_F32) res[q][j] = (pt)reinterpret_cast<const float*>(src)[(size_t)r * p.cs + c[q] + j];
                        else if (OT == T_I8) res[q][j] = (pt)reinterpret_cast<const int8_t*>(src)[(size_t)r * p.cs + c[q] + j];
                    }
                }
                #pragma unroll
                for (int wi = 0; wi < KW * KW; ++wi) {
                    x[q][wi][0] = x[q][wi][1] = x[q][wi][2] = x[q][wi][3] = 0;
                    if (c[q] < 0 || !(inside >> wi & 1u)) continue;
                    const size_t o = (size_t)(qbase + (y0 + wi / KW) * p.ow + x0 + wi % KW) * p.c_out + c[q];
                    // the position's projection in this lane's frame: that of the latest frame up to it that updated the
                    // position (written there by project_seq_kernel), else the projection before the chunk
                    if (KW == 1) {
                        // without a pool window a projection pixel belongs to one output pixel, so the prefix sum over the
                        // frames is taken right here (project_seq_kernel is not run for such a layer)
                        load4<pt, pt4>(P, o, vec, c[q], p.c_out, x[q][wi]);
                        dsum[q][0] = dsum[q][1] = dsum[q][2] = dsum[q][3] = 0;
                        if (ub & 1u) load4<pt, pt4>(dP + (size_t)lane * p.p_stride, o, vec, c[q], p.c_out, dsum[q]);
                    } else {
                        const unsigned upto = uf[wi] & (0xffffffffu >> (31 - lane));
                        const pt* src = upto ? dP + (size_t)(31 - __clz(upto)) * p.p_stride : P;
                        load4<pt, pt4>(src, o, vec, c[q], p.c_out, x[q][wi]);
                    }
                }
            }
            if (KW == 1 && on_frames) {
                pt* Q = reinterpret_cast<pt*>(p.Q);
                #pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    if (c[q] < 0) continue;                  // uniform inside the warp
                    scan4(dsum[q], lane);
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) x[q][0][j] += dsum[q][j];
                    if (lane == 31 && c[q] < p.c_out) {      // the sum over all frames: the stored projection (not for padding channels)
                        const size_t o = (size_t)(qbase + y0 * p.ow + x0) * p.c_out + c[q];
                        if (vec) { pt4 t; t.x = x[q][0][0]; t.y = x[q][0][1]; t.z = x[q][0][2]; t.w = x[q][0][3]; *reinterpret_cast<pt4*>(Q + o) = t; }
                        else {
                            #pragma unroll
                            for (int j = 0; j < 4; ++j) if (c[q] + j < p.c_out) Q[o + j] = x[q][0][j];
                        }
                    }
                }
            }
            #pragma unroll
            for (int q = 0; q < NQ; ++q) {
                bool have = false;
                best[q][0] = best[q][1] = best[q][2] = best[q][3] = 0;
                if (c[q] < 0) continue;                      // uniform inside the warp
                #pragma unroll
                for (int wi = 0; wi < KW * KW; ++wi) {
                    if (!(inside >> wi & 1u)) continue;
                    pt y[4];
                    const pt (&x1)[1][4] = reinterpret_cast<const pt (&)[1][4]>(x[q][wi]);
                    epi_f<PT, OT, 1, BN, pt>(x1, 1u, c[q], res[q], p.c_out, p.act_fn, p.shift, p.bn_scale, p.bn_shift, y);
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) best[q][j] = (!have || y[j] > best[q][j]) ? y[j] : best[q][j];
                    have = true;
                }
            }
        };
        if (OT == T_BIN) {
            for (int u = blockIdx.y * nwarps + warp; u < p.cs; u += nwarps * gridDim.y) {   // one 32-channel word of the output per turn
                const size_t o = (size_t)r * p.cs + u;
                const uint32_t before = reinterpret_cast<const uint32_t*>(p.X)[o];
                uint32_t word = 0;
                for (int qd = 0; qd < 8; qd += NQ) {
                    int c[NQ];
                    #pragma unroll
                    for (int q = 0; q < NQ; ++q) { c[q] = u * 32 + (qd + q) * 4; if (c[q] >= p.c_out) c[q] = -1; }
                    if (c[0] < 0) break;
                    pt best[NQ][4];
                    eval(c, best);
                    #pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        #pragma unroll
                        for (int j = 0; j < 4; ++j) if (c[q] >= 0 && c[q] + j < p.c_out && (int)best[q][j] >= p.theta) word |= 1u << ((qd + q) * 4 + j);
                    }
                }
                uint32_t prev = __shfl_up_sync(0xffffffffu, word, 1);
                if (lane == 0) prev = before;
                const uint32_t ch = word ^ prev;
                if (live) {
                    if (on) {
                        shift_bytes(reinterpret_cast<uint32_t*>(p.D), roff)[o] = ch;
                        if (p.Xn) shift_bytes(reinterpret_cast<uint32_t*>(p.Xn), roff)[o] = word;
                        cnt += __popc(ch);
                    }
                    if (full) shift_bytes(reinterpret_cast<uint32_t*>(p.Xfull), roff)[o] = word;
                }
                if (last && on_frames) reinterpret_cast<uint32_t*>(p.X)[o] = word;       // (every lane read the old word before the turn's shuffles)
            }
        } else {
            const int units = (p.cs + 3) >> 2;
            for (int u0 = (blockIdx.y * nwarps + warp) * NQ; u0 < units; u0 += nwarps * NQ * gridDim.y) {   // NQ groups of four output channels per turn
                int c[NQ];
                #pragma unroll
                for (int q = 0; q < NQ; ++q) c[q] = (u0 + q < units) ? (u0 + q) * 4 : -1;
                // the output's value before the chunk (lane 0's previous frame), fetched with the turn's other loads
                uint32_t before_w[NQ];
                pt before[NQ][4];
                #pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    before_w[q] = 0;
                    before[q][0] = before[q][1] = before[q][2] = before[q][3] = 0;
                    if (c[q] < 0) continue;
                    const size_t o = (size_t)r * p.cs + c[q];
                    if (OT == T_I8) before_w[q] = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const int8_t*>(p.X) + o);
                    else if ((p.cs & 3) == 0) {              // (rows of whole 16-byte groups: one load)
                        const pt4 t = *reinterpret_cast<const pt4*>(reinterpret_cast<const pt*>(p.X) + o);
                        before[q][0] = t.x; before[q][1] = t.y; before[q][2] = t.z; before[q][3] = t.w;
                    } else {
                        #pragma unroll
                        for (int j = 0; j < 4; ++j) if (c[q] + j < p.cs) before[q][j] = reinterpret_cast<const pt*>(p.X)[o + j];
                    }
                }
                pt best[NQ][4];
                eval(c, best);
                #pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    if (c[q] < 0) continue;                  // uniform inside the warp
                    const size_t o = (size_t)r * p.cs + c[q];
                    if (OT == T_I8) {                        // (cs is a multiple of 4)
                        const uint32_t nw = ((uint32_t)(int)best[q][0] & 0xffu) | ((uint32_t)(int)best[q][1] & 0xffu) << 8 |
                                            ((uint32_t)(int)best[q][2] & 0xffu) << 16 | ((uint32_t)(int)best[q][3] & 0xffu) << 24;
                        uint32_t ow_ = __shfl_up_sync(0xffffffffu, nw, 1);
                        if (lane == 0) ow_ = before_w[q];
                        if (live) {
                            if (on) {
                                uint32_t dw = 0;
                                #pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const int nv = (int)(int8_t)(nw >> (8 * j)), ov = (int)(int8_t)(ow_ >> (8 * j));
                                    const int dd = nv - ov;
                                    if (p.errw && (dd < -128 || dd > 127)) atomicOr(p.errw, ERRW_BOUNDS);
                                    dw |= ((uint32_t)dd & 0xffu) << (8 * j);
                                    cnt += nv != ov;
                                }
                                *reinterpret_cast<uint32_t*>(shift_bytes(reinterpret_cast<int8_t*>(p.D), roff) + o) = dw;
                                if (p.Xn) *reinterpret_cast<uint32_t*>(shift_bytes(reinterpret_cast<int8_t*>(p.Xn), roff) + o) = nw;
                            }
                            if (full) *reinterpret_cast<uint32_t*>(shift_bytes(reinterpret_cast<int8_t*>(p.Xfull), roff) + o) = nw;
                        }
                        if (last && on_frames) *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(p.X) + o) = nw;
                    } else {
                        pt old[4];
                        if (PT == T_F32) {
                            // a frame that leaves the window alone keeps the value of the frame before it, bit for bit (its
                            // own f would see the same projection, but the snapshot may stem from a differently rounded sum)
                            const unsigned below = on_frames & (0xffffffffu >> (31 - lane));
                            const int src = below ? 31 - __clz(below) : -1;      // the nearest frame at or below this one that re-evaluates
                            #pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const pt carried = __shfl_sync(0xffffffffu, best[q][j], src < 0 ? 0 : src);
                                best[q][j] = src < 0 ? before[q][j] : carried;
                            }
                        }
                        #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            old[j] = __shfl_up_sync(0xffffffffu, best[q][j], 1);
                            if (lane == 0) old[j] = before[q][j];
                        }
                        const bool v4 = (p.cs & 3) == 0;     // rows of whole 16-byte groups: one store per row and group
                        pt4 bv; bv.x = best[q][0]; bv.y = best[q][1]; bv.z = best[q][2]; bv.w = best[q][3];
                        if (live) {
                            pt* Dg = shift_bytes(reinterpret_cast<pt*>(p.D), roff);
                            pt* Fg = full ? shift_bytes(reinterpret_cast<pt*>(p.Xfull), roff) : nullptr;
                            pt* Ng = p.Xn ? shift_bytes(reinterpret_cast<pt*>(p.Xn), roff) : nullptr;
                            if (v4) {
                                if (on) {
                                    pt4 dv; dv.x = best[q][0] - old[0]; dv.y = best[q][1] - old[1]; dv.z = best[q][2] - old[2]; dv.w = best[q][3] - old[3];
                                    *reinterpret_cast<pt4*>(Dg + o) = dv;
                                    #pragma unroll
                                    for (int j = 0; j < 4; ++j) cnt += best[q][j] != old[j];
                                    if (Ng) *reinterpret_cast<pt4*>(Ng + o) = bv;
                                }
                                if (full) *reinterpret_cast<pt4*>(Fg + o) = bv;
                            } else {
                                #pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    if (c[q] + j >= p.cs) break;
                                    if (on) { Dg[o + j] = best[q][j] - old[j]; cnt += best[q][j] != old[j]; if (Ng) Ng[o + j] = best[q][j]; }
                                    if (full) Fg[o + j] = best[q][j];
                                }
                            }
                        }
                        if (last && on_frames) {
                            if (v4) *reinterpret_cast<pt4*>(reinterpret_cast<pt*>(p.X) + o) = bv;
                            else {
                                #pragma unroll
                                for (int j = 0; j < 4; ++j) if (c[q] + j < p.cs) reinterpret_cast<pt*>(p.X)[o + j] = best[q][j];
                            }
                        }
                    }
                }
            }
        }
        if (cnt) atomicAdd(&s_cnt[lane], cnt);
    }
    __syncthreads();
    seq_mark_frames<READERS>(p, s_cnt, r, ns, ty, tx, lane, warp);
}

// The epilogue of an int8 layer behind a pool window whose projection kernel has already applied the pointwise part of
// f (EpiSeqParams.A0 / A: bytes): lane = frame; per window position the lane takes its frame's row (the latest frame up
// to it that updated the position, else the row before the chunk), the window's max is a byte-wise max of 16 channels
// at a time, the previous frame's output comes from the neighbouring lane.  c_out is a multiple of 16.
template <int KW, bool READERS>
__global__ void __launch_bounds__(256) epilogue_seq_pool8_kernel(EpiSeqParams p)
{
    __shared__ int s_cnt[SEQ_MAX_FRAMES];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x < SEQ_MAX_FRAMES) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    const int r = blockIdx.x;
    const int tx = r % p.tw, ty = (r / p.tw) % p.th, ns = r / (p.tw * p.th);
    const int y0 = ty * p.pool_s - p.pool_p, x0 = tx * p.pool_s - p.pool_p;
    const int qbase = ns * p.oh * p.ow;
    unsigned inside, ub = 0;
    {
        bool mine = false;
        if (lane < KW * KW) {
            const int y = y0 + lane / KW, x = x0 + lane % KW;
            mine = y >= 0 && y < p.oh && x >= 0 && x < p.ow;
        }
        inside = __ballot_sync(0xffffffffu, mine);
        if (lane < p.frames) {
            const uint32_t* oa = shift_bytes(p.oact, lane * p.arena_stride);
            #pragma unroll
            for (int wi = 0; wi < KW * KW; ++wi) {
                if (!(inside >> wi & 1u)) continue;
                const int q = qbase + (y0 + wi / KW) * p.ow + x0 + wi % KW;
                if ((oa[q >> 5] >> (q & 31)) & 1u) ub |= 1u << wi;
            }
        }
    }
    const unsigned on_frames = __ballot_sync(0xffffffffu, ub != 0);
    const bool full = p.Xfull != nullptr;
    if (on_frames || full) {
        const bool live = lane < p.frames, on = (on_frames >> lane) & 1u, last = lane == p.frames - 1;
        const long long roff = (long long)(live ? lane : 0) * p.row_stride;
        // per window position: the row this lane's frame sees
        const int8_t* rowp[KW * KW];
        #pragma unroll
        for (int wi = 0; wi < KW * KW; ++wi) {
            const unsigned uf = __ballot_sync(0xffffffffu, (ub >> wi) & 1u);
            const unsigned upto = uf & (0xffffffffu >> (31 - lane));
            const size_t pos = (size_t)(qbase + (y0 + wi / KW) * p.ow + x0 + wi % KW) * p.c_out;
            rowp[wi] = (upto ? p.A + (long long)(31 - __clz(upto)) * p.a_stride : p.A0) + pos;
        }
        int cnt = 0;
        const int units = p.cs >> 4;                         // (cs is a multiple of 32)
        for (int u = blockIdx.y * 8 + warp; u < units; u += 8 * gridDim.y) {
            const int c = u * 16;
            const size_t o = (size_t)r * p.cs + c;
            const uint4 before = *reinterpret_cast<const uint4*>(reinterpret_cast<const int8_t*>(p.X) + o);
            uint4 best = make_uint4(0, 0, 0, 0);
            if (c < p.c_out) {                               // (channels past c_out are padding: zero)
                uint4 v[KW * KW];
                #pragma unroll
                for (int wi = 0; wi < KW * KW; ++wi)
                    if (inside >> wi & 1u) v[wi] = *reinterpret_cast<const uint4*>(rowp[wi] + c);
                bool have = false;
                #pragma unroll
                for (int wi = 0; wi < KW * KW; ++wi) {
                    if (!(inside >> wi & 1u)) continue;
                    if (!have) best = v[wi];
                    else {
                        best.x = __vmaxs4(best.x, v[wi].x); best.y = __vmaxs4(best.y, v[wi].y);
                        best.z = __vmaxs4(best.z, v[wi].z); best.w = __vmaxs4(best.w, v[wi].w);
                    }
                    have = true;
                }
            }
            uint4 old;
            old.x = __shfl_up_sync(0xffffffffu, best.x, 1); old.y = __shfl_up_sync(0xffffffffu, best.y, 1);
            old.z = __shfl_up_sync(0xffffffffu, best.z, 1); old.w = __shfl_up_sync(0xffffffffu, best.w, 1);
            if (lane == 0) old = before;
            if (live) {
                if (on) {
                    uint4 dw;
                    dw.x = __vsub4(best.x, old.x); dw.y = __vsub4(best.y, old.y); dw.z = __vsub4(best.z, old.z); dw.w = __vsub4(best.w, old.w);
                    // a difference outside a byte shows as a wrapped subtraction that differs from the saturating one
                    if (p.errw && (dw.x != __vsubss4(best.x, old.x) || dw.y != __vsubss4(best.y, old.y) ||
                                   dw.z != __vsubss4(best.z, old.z) || dw.w != __vsubss4(best.w, old.w))) atomicOr(p.errw, ERRW_BOUNDS);
                    cnt += __popc(nonzero_bytes(dw.x)) + __popc(nonzero_bytes(dw.y)) + __popc(nonzero_bytes(dw.z)) + __popc(nonzero_bytes(dw.w));
                    *reinterpret_cast<uint4*>(shift_bytes(reinterpret_cast<int8_t*>(p.D), roff) + o) = dw;
                    if (p.Xn) *reinterpret_cast<uint4*>(shift_bytes(reinterpret_cast<int8_t*>(p.Xn), roff) + o) = best;
                }
                if (full) *reinterpret_cast<uint4*>(shift_bytes(reinterpret_cast<int8_t*>(p.Xfull), roff) + o) = best;
            }
            if (last && on_frames) *reinterpret_cast<uint4*>(reinterpret_cast<int8_t*>(p.X) + o) = best;
        }
        if (cnt) atomicAdd(&s_cnt[lane], cnt);
    }
    __syncthreads();
    seq_mark_frames<READERS>(p, s_cnt, r, ns, ty, tx, lane, warp);
}

// ================================================================================================
// host side
// ================================================================================================
template <int PT, int OT, bool BN, int KW>
static void launch_epi_seq_kw(const EpiSeqParams& e, int blocks, cudaStream_t st)
{
    // a pixel's channels are dealt out to so many CTAs that a warp has about two turns (memory round trips) to make
    constexpr int NQ = KW == 1 ? 4 : (KW == 2 ? 2 : 1);
    const int turns = OT == T_BIN ? ceil_div(e.cs, 8) : ceil_div(ceil_div(e.cs, 4), 8 * NQ);    // per warp of a lone CTA
    int slices = ceil_div(turns, 2);
    slices = slices < 1 ? 1 : (slices > 16 ? 16 : slices);
    // (a layer of few channels: no more warps than have a turn to make)
    const int busy = OT == T_BIN ? e.cs : ceil_div(ceil_div(e.cs, 4), NQ);
    const int threads = 32 * (busy < 1 ? 1 : (busy > 8 ? 8 : busy));
    if (e.readers.n > 0) launch_seq(epilogue_seq_kernel<PT, OT, KW, true, BN>, dim3(blocks, slices), dim3(threads), 0, st, e);
    else launch_seq(epilogue_seq_kernel<PT, OT, KW, false, BN>, dim3(blocks, slices), dim3(threads), 0, st, e);
}

template <int PT, int OT, bool BN>
static int launch_epi_seq_b(const EpiSeqParams& e, int blocks, cudaStream_t st)
{
    switch (e.pool_k > 0 ? e.pool_k : 1) {
        case 1: launch_epi_seq_kw<PT, OT, BN, 1>(e, blocks, st); break;
        case 2: launch_epi_seq_kw<PT, OT, BN, 2>(e, blocks, st); break;
        case 3: launch_epi_seq_kw<PT, OT, BN, 3>(e, blocks, st); break;
        default: return RRM_ERR_UNSUPPORTED;
    }
    return RRM_OK;
}

template <int PT, int OT>
static int launch_epi_seq_t(const EpiSeqParams& e, int blocks, cudaStream_t st)
{
    if ((OT == T_F32 || OT == T_I8) && e.bn_scale) return launch_epi_seq_b<PT, OT, (OT == T_F32 || OT == T_I8)>(e, blocks, st);
    return launch_epi_seq_b<PT, OT, false>(e, blocks, st);
}

// The epilogue of layer l over `frames` consecutive frames (the bound arena is frame 0's).
int launch_epilogue_seq(rrm_net* net, int l, int frames, long long arena_stride, cudaStream_t st)
{
    Layer& L = net->layers[l];
    const rrm_layer_desc& d = L.d;
    Tensor& out = net->tensors[l + 1];
    if (frames < 1 || frames > SEQ_MAX_FRAMES || !L.Palt || !L.dPall || !out.Dall) return RRM_ERR_INVALID_ARG;
    EpiSeqParams e{};
    e.P = L.Palt; e.Q = L.P; e.dP = L.dPall; e.oact = L.oact;
    e.X = out.X; e.D = out.Dall;
    e.Xn = ((out.dtype == T_BIN && out.has_consumer) || out.shortcut_source) ? out.Xnall : nullptr;
    if (d.res >= 0) {
        const Tensor& rt = net->tensors[d.res];
        if (!rt.Xbefore || !rt.Xnall) return RRM_ERR_INVALID_ARG;
        e.res_before = rt.Xbefore; e.res_new = rt.Xnall; e.res_act = rt.act; e.res_stride = (long long)rt.bytes();
    }
    e.Xfull = (l + 1 == (int)net->layers.size()) ? out.Xfull : nullptr;
    e.act = out.act; e.nnz = out.nnz; e.npix = out.npix;
    e.errw = out.has_consumer ? net->errw : nullptr;
    e.n = d.n; e.oh = L.oh; e.ow = L.ow; e.th = L.th; e.tw = L.tw; e.c_out = d.c_out; e.cs = out.cs;
    e.pool_k = d.pool_k; e.pool_s = d.pool_s; e.pool_p = d.pool_p; e.act_fn = d.act; e.shift = d.shift; e.theta = d.theta;
    e.readers = out.readers;
    e.bn_scale = L.bn_scale; e.bn_shift = L.bn_shift;
    e.frames = frames; e.row_stride = (long long)out.bytes(); e.arena_stride = arena_stride;
    e.p_stride = (long long)L.opixels() * d.c_out;
    e.opix = L.opixels();
    // int8 outputs behind a pool window: the projection kernel applies the pointwise part of f and the epilogue works on bytes
    const bool bytes = L.Aall != nullptr;
    if (d.pool_k > 1) {                                      // (without a pool window the epilogue sums the frames' products itself)
        ProjSeqParams q{};
        q.R = L.Palt; q.Q = L.P; q.dP = L.dPall; q.oact = L.oact;
        q.frames = frames; q.c_out = d.c_out; q.opix = L.opixels();
        q.arena_stride = arena_stride; q.p_stride = e.p_stride;
        if (bytes) {
            q.a_stride = (long long)L.opixels() * d.c_out;
            q.A0 = reinterpret_cast<int8_t*>(L.Aall); q.A = q.A0 + q.a_stride;
            q.act_fn = d.act; q.shift = d.shift; q.bn_scale = L.bn_scale; q.bn_shift = L.bn_shift;
            e.A0 = q.A0; e.A = q.A; e.a_stride = q.a_stride;
            if (L.bn_scale) launch_seq(project_seq_kernel<T_I32, true, true>, dim3(L.opixels()), dim3(256), 0, st, q);
            else launch_seq(project_seq_kernel<T_I32, true, false>, dim3(L.opixels()), dim3(256), 0, st, q);
        } else if (d.dtype == RRM_F32) launch_seq(project_seq_kernel<T_F32, false, false>, dim3(L.opixels()), dim3(256), 0, st, q);
        else launch_seq(project_seq_kernel<T_I32, false, false>, dim3(L.opixels()), dim3(256), 0, st, q);
    }
    const int blocks = out.pixels();                         // a CTA per output pixel
    int s = RRM_OK;
    if (bytes) {
        const int slices = ceil_div(ceil_div(out.cs >> 4, 8), 2) < 1 ? 1 : ceil_div(ceil_div(out.cs >> 4, 8), 2);
        const bool rd = e.readers.n > 0;
        if (d.pool_k == 2) { if (rd) launch_seq(epilogue_seq_pool8_kernel<2, true>, dim3(blocks, slices), dim3(256), 0, st, e); else launch_seq(epilogue_seq_pool8_kernel<2, false>, dim3(blocks, slices), dim3(256), 0, st, e); }
        else if (d.pool_k == 3) { if (rd) launch_seq(epilogue_seq_pool8_kernel<3, true>, dim3(blocks, slices), dim3(256), 0, st, e); else launch_seq(epilogue_seq_pool8_kernel<3, false>, dim3(blocks, slices), dim3(256), 0, st, e); }
        else s = RRM_ERR_UNSUPPORTED;
    }
    else if (d.dtype == RRM_F32) s = launch_epi_seq_t<T_F32, T_F32>(e, blocks, st);
    else if (out.dtype == T_I8) s = launch_epi_seq_t<T_I32, T_I8>(e, blocks, st);
    else if (out.dtype == T_BIN) s = launch_epi_seq_t<T_I32, T_BIN>(e, blocks, st);
    else s = launch_epi_seq_t<T_I32, T_I32>(e, blocks, st);
    RRM_TRY(s);
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

int seq_max_frames() { return SEQ_MAX_FRAMES; }

// Can delta chunks of this stack run layer by layer over all frames?  Buffers for SEQ_MAX_FRAMES frames: per tensor the delta
// rows (binary tensors: the new rows too; the last tensor: every frame's full rows), per layer the products.
int ensure_frame_batch(rrm_net* net)
{
    if (net->seq_ready) return RRM_OK;
    for (auto& L : net->layers) {
        if (L.d.res == 0) return RRM_ERR_UNSUPPORTED;       // (the input itself as a shortcut: the import keeps no per-frame rows of it)
        if (L.d.res > 0) net->tensors[L.d.res].shortcut_source = true;
    }
    const size_t G = SEQ_MAX_FRAMES;
    size_t need = 0;
    for (auto& T : net->tensors) need += T.bytes() * (G * ((T.dtype == T_BIN || T.shortcut_source) ? 2 : 1) + 1);
    need += net->tensors.back().bytes() * G;
    for (auto& L : net->layers) need += (size_t)L.opixels() * L.d.c_out * 4 * (G + 1);
    if (need > ((size_t)8 << 30)) return RRM_ERR_UNSUPPORTED;          // (a stack this large keeps the frame-pipelined form)
    auto alloc = [&](void** p, size_t bytes) -> int {
        if (*p) return RRM_OK;
        if (cudaMalloc(p, bytes ? bytes : 16) != cudaSuccess) { *p = nullptr; cudaGetLastError(); return RRM_ERR_ALLOC; }
        net->allocs.push_back(*p);
        return RRM_OK;
    };
    for (auto& T : net->tensors) {
        RRM_TRY(alloc(&T.Dall, T.bytes() * G));
        if (T.dtype == T_BIN || T.shortcut_source) RRM_TRY(alloc(&T.Xnall, T.bytes() * G));
        if (T.shortcut_source) RRM_TRY(alloc(&T.Xbefore, T.bytes()));
    }
    RRM_TRY(alloc(&net->tensors.back().Xfull, net->tensors.back().bytes() * G));
    for (auto& L : net->layers) {
        const size_t bytes = (size_t)L.opixels() * L.d.c_out * 4;
        RRM_TRY(alloc(&L.Palt, bytes));
        RRM_TRY(alloc(&L.dPall, bytes * G));
        // int8 outputs behind a 2x2 / 3x3 pool window, no shortcut, channels in whole groups of 16: f before the window as bytes
        const Tensor& out = net->tensors[(&L - &net->layers[0]) + 1];
        if (out.dtype == T_I8 && (L.d.pool_k == 2 || L.d.pool_k == 3) && L.d.res < 0 && L.d.c_out % 16 == 0 && L.d.dtype != RRM_F32)
            RRM_TRY(alloc(&L.Aall, (size_t)L.opixels() * L.d.c_out * (G + 1)));
    }
    net->seq_ready = true;
    return RRM_OK;
}

}  // namespace rrm
