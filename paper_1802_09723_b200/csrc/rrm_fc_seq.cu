// Delta-FC over a chunk of T consecutive frames in one launch (Algorithm 1, FC branch, with the
// frame loop moved inside the kernel).
//
// For a lone linear layer the deltas of all frames of a chunk are known up front:
//   dI_t = X_t - X_{t-1}   (X_{-1} = the stored snapshot),     dP_t = W dI_t   (Eq. 4),
//   P_t  = P_{t-1} + dP_t  (Eq. 5) is a running sum over t,    Y_t = f(P_t).
// So the T sparse products are independent and only the running sum is serial.  One launch,
// one CTA per (512-output slice, frame, stream):
//   1. the CTA scans X_t against X_{t-1} with 128-bit loads (all issued up front) and compacts the
//      non-zero delta entries (index, delta) into a list in shared memory: a 16-bit mask per
//      16-byte chunk, a warp prefix sum, one shared-memory atomic per warp to reserve list space
//      (the list is unordered; integer sums do not depend on the order, so results stay bit-exact);
//   2. each warp takes every 8th list entry and loads the 512-byte slice of that entry's weight
//      column (weights are stored transposed: one contiguous C_out-byte row per input) with one
//      fully coalesced 128-bit load per lane, many columns in flight, accumulating d_j * W[:, j];
//   3. the 8 warps' partial sums are added through shared memory into the slice of dP_t (scratch);
//   4. the CTA that finishes LAST for a given (stream, slice) - found with one atomic counter,
//      nobody waits - adds the T slices onto the stored projection in frame order, applies f and
//      writes Y_0 .. Y_{T-1}.
// Cost: the weight columns of the non-zero entries (HBM; frames of a chunk share columns through L2).
#include "rrm_common.cuh"
#include "rrm_dev.cuh"
#include <cstring>

namespace rrm {

constexpr int SQ_THREADS = 256;
constexpr int SQ_WARPS = SQ_THREADS / 32;
constexpr int SQ_TAIL = 16;                    // frames one thread of the closing sum holds (chunks of up to 2 * SQ_TAIL frames)
constexpr int SQ_PT = 4;                       // 16-byte chunks scanned per thread
constexpr int SQ_MAX_C_IN = 16 * SQ_PT * SQ_THREADS;   // 16384 (entry format: 14-bit index)
constexpr int SW_RING = 12;                    // weight-sparse form: records in flight per warp

struct FcSeqParams {
    const int8_t* x;         // [T][n][c_in] frames of the chunk
    const int8_t* xprev;     // [n][c_in] snapshot = frame before the chunk; nullptr: every entry active, d = x
    int8_t* xnext;           // [n][c_in] receives frame T-1, or nullptr
    const int8_t* Wt;        // [c_in][c_out]
    const int32_t* bias;     // non-null: frames are independent, P_t = bias + dP_t (dense evaluation)
    int32_t* P;              // [n][c_out] stored projection (chained mode: read and updated), may be nullptr with bias
    int32_t* dP;             // [T][n][c_out] scratch
    void* Y;                 // [T][n][c_out] int32 (shift < 0) or int8, or nullptr
    unsigned* counters;      // [n][slices], zero on entry, zero again on exit
    unsigned* stat;          // [T*n][2]: non-zero entries / active groups of 32 inputs per frame, or nullptr
    int T, n, c_in, c_out, shift, act;
    const uint32_t* Wsp;     // weight-sparse form: [c_in][slices] records of sp_stride words (map, then packed groups)
    int sp_stride;
};

// LANES: lanes of a warp that span one column slice (16 bytes each): the CTA owns OW = 16 * LANES
// outputs and a warp-wide load fetches 32 / LANES columns.  Narrow slices mean more CTAs and fewer
// list entries per lane (a shorter chain of dependent memory round trips); wide slices mean fewer
// redundant scans.  The host picks LANES from the size of the chunk.
// DEEP: 16 instead of 8 loads in flight per lane at 2 instead of 3 CTAs per SM; pays when the whole
// grid is resident at once (each CTA's chain of round trips is what the launch waits for).
// SW (LANES = 32 only): the weights are in the weight-sparse form (Sec. 3.5: EIE keeps the pruned weights of a
// compressed model in compressed columns).  A lane owns 16 outputs = 4 groups of four; the record of (input j, this
// slice) starts with a 128-bit map (bit 4 * lane + g: group g of that lane holds a non-zero weight) and the running
// word counts of the map's four words, followed (from byte 32 on) by the 4-byte words of the non-zero groups, in map order.  All lanes load the map (one 16-byte broadcast), find their
// word offset by counting the map bits below their own, and load only their non-zero groups.
template <int LANES, bool DEEP, bool SW>
__global__ void __launch_bounds__(SQ_THREADS, DEEP ? 2 : 3) fc_seq_kernel(FcSeqParams p)
{
    static_assert(!SW || LANES == 32, "the weight-sparse records are laid out for 512-output slices");
    constexpr int OW = 16 * LANES;                 // outputs per CTA
    constexpr int CPW = 32 / LANES;                // columns per warp-wide load
    constexpr int CPR = CPW * SQ_WARPS;            // columns per CTA-wide round
    constexpr int SQ_U = DEEP ? 16 : 8;            // rounds in flight (16-byte loads per lane)
    extern __shared__ __align__(16) unsigned char s_dyn[];
    int* s_red = reinterpret_cast<int*>(s_dyn);                                   // [SQ_WARPS][OW]
    uint32_t* s_list = reinterpret_cast<uint32_t*>(s_dyn + SQ_WARPS * OW * 4);     // [c_in] index | (delta + 256) << 16
    __shared__ int s_count, s_groups, s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slice = blockIdx.x;
    const int t = blockIdx.y / p.n, s = blockIdx.y - t * p.n;
    const int C = p.c_in, K = p.c_out;
    const int nchunks = C >> 4;
    const int slices = gridDim.x;
    const int width = min(OW, K - slice * OW);

    if (tid == 0) { s_count = 0; s_groups = 0; }
    // ---- 1. scan: chunk i*256 + tid for i < SQ_PT, all loads first
    const uint4* xt4 = reinterpret_cast<const uint4*>(p.x + ((size_t)t * p.n + s) * C);
    const uint4* xp4 = nullptr;
    if (p.xprev) xp4 = reinterpret_cast<const uint4*>(t > 0 ? p.x + ((size_t)(t - 1) * p.n + s) * C : p.xprev + (size_t)s * C);
    uint4 a[SQ_PT], b[SQ_PT];
    #pragma unroll
    for (int i = 0; i < SQ_PT; ++i) {
        const int chunk = i * SQ_THREADS + tid;
        a[i] = make_uint4(0, 0, 0, 0);
        b[i] = a[i];
        if (chunk < nchunks) {
            a[i] = __ldg(xt4 + chunk);
            if (xp4) b[i] = __ldg(xp4 + chunk);
        }
    }
    // while the frame is on its way: touch one line in every 2 MiB of the weights, so that the
    // address translations the gather will need are fetched now instead of on its first loads
    {
        const size_t wbytes = SW ? (size_t)C * slices * p.sp_stride * 4 : (size_t)C * K;
        const size_t off = (size_t)tid << 21;
        const char* wptr = SW ? reinterpret_cast<const char*>(p.Wsp) : reinterpret_cast<const char*>(p.Wt);
        if (off < wbytes) asm volatile("prefetch.global.L2 [%0];" ::"l"(wptr + off));
        // likewise the stored projection (or the bias), which only the closing sum reads
        const int32_t* pp = p.bias ? p.bias + slice * OW : p.P + (size_t)s * K + slice * OW;
        if (t == 0 && tid * 32 < width) asm volatile("prefetch.global.L2 [%0];" ::"l"(pp + tid * 32));
    }
    __syncthreads();                                         // s_count is initialised
    int groups = 0;
    #pragma unroll
    for (int i = 0; i < SQ_PT; ++i) {
        const int chunk = i * SQ_THREADS + tid;
        if (i * SQ_THREADS >= nchunks) break;                // uniform
        unsigned m = 0;
        if (chunk < nchunks)
            m = xp4 ? differing_bytes(a[i], b[i]) : 0xffffu;
        const int local = __popc(m);
        int incl = local;
        #pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const int wtot = __shfl_sync(0xffffffffu, incl, 31);
        if (wtot == 0) continue;                             // uniform inside the warp
        int base = 0;
        if (lane == 31) base = atomicAdd(&s_count, wtot);
        base = __shfl_sync(0xffffffffu, base, 31);
        // groups of 32 inputs = pairs of neighbouring chunks (an even/odd lane pair)
        const unsigned other = __shfl_xor_sync(0xffffffffu, m, 1);
        groups += ((lane & 1) == 0 && (m | other)) ? 1 : 0;
        if (m) {
            int off = base + incl - local;
            const unsigned aw[4] = {a[i].x, a[i].y, a[i].z, a[i].w}, bw[4] = {b[i].x, b[i].y, b[i].z, b[i].w};
            #pragma unroll
            for (int k = 0; k < 16; ++k) {
                if (m >> k & 1u) {
                    const int xa = (int)(int8_t)(aw[k >> 2] >> (8 * (k & 3)));
                    const int xb = (int)(int8_t)(bw[k >> 2] >> (8 * (k & 3)));
                    s_list[off++] = (uint32_t)(chunk * 16 + k) | (uint32_t)(xa - xb + 256) << 16;
                }
            }
        }
    }
    // the new snapshot is the chunk's last frame; the CTAs of slice 0 store it
    if (p.xnext && t == p.T - 1 && slice == 0) {
        #pragma unroll
        for (int i = 0; i < SQ_PT; ++i) {
            const int chunk = i * SQ_THREADS + tid;
            if (chunk < nchunks) reinterpret_cast<uint4*>(p.xnext + (size_t)s * C)[chunk] = a[i];
        }
    }
    if (p.stat && slice == 0) {
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) groups += __shfl_down_sync(0xffffffffu, groups, o);
        if (lane == 0 && groups) atomicAdd(&s_groups, groups);
    }
    __syncthreads();
    const int total = s_count;
    if (p.stat && slice == 0 && tid == 0) {
        p.stat[blockIdx.y * 2 + 0] = (unsigned)total;
        p.stat[blockIdx.y * 2 + 1] = (unsigned)s_groups;
    }

    // ---- 2. gather: LANES lanes x 16 bytes span the slice; SQ_U rounds of CPR columns in flight
    const int sub = lane % LANES, grp = warp * CPW + lane / LANES;
    const int o0 = slice * OW + sub * 16;
    int acc[16];
    #pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0;
    if (SW) {
        // Every warp streams the records of its list entries (entry warp, warp + 8, ...) through a ring of SW_RING slots
        // in shared memory with 16-byte asynchronous copies: one memory round trip per record, SW_RING records in flight.
        // A whole record (fixed stride: the longest record of the matrix) is fetched, map and packed groups together.
        const int stride_b = p.sp_stride * 4, pieces = stride_b >> 4;
        unsigned char* ringbuf = s_dyn + (size_t)SQ_WARPS * OW * 4 + (size_t)C * 4 + (size_t)warp * SW_RING * stride_b;
        const uint32_t ring_u32 = (uint32_t)__cvta_generic_to_shared(ringbuf);
        const int nib_shift = 4 * (lane & 7), nib_word = lane >> 3;
        const int mine_n = total > warp ? (total - warp + SQ_WARPS - 1) / SQ_WARPS : 0;
        auto issue = [&](int i) {
            if (i < mine_n) {
                const uint32_t ent = s_list[warp + i * SQ_WARPS];
                const unsigned char* src = reinterpret_cast<const unsigned char*>(p.Wsp + ((size_t)(ent & 0xffffu) * slices + slice) * p.sp_stride);
                for (int pc = lane; pc < pieces; pc += 32)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_u32 + (uint32_t)((i % SW_RING) * stride_b + pc * 16)), "l"(src + pc * 16) : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        for (int i = 0; i < SW_RING - 2; ++i) issue(i);
        // two records per turn: their decode chains (map -> offsets -> words -> products) overlap
        for (int i = 0; i < mine_n; i += 2) {
            issue(i + SW_RING - 2);                          // (refill the two slots read in the previous turn: every lane is past them)
            issue(i + SW_RING - 1);
            asm volatile("cp.async.wait_group %0;" ::"n"(SW_RING - 2) : "memory");
            __syncwarp();                                    // the pieces the other lanes copied are visible too
            uint32_t wg[2][4];
            int dl[2], dh[2];
            #pragma unroll
            for (int r = 0; r < 2; ++r) {
                const bool have = i + r < mine_n;            // (an odd tail: the second record is absent, all its words zero)
                const unsigned char* slot = ringbuf + ((i + r) % SW_RING) * stride_b;
                const uint4 map = have ? *reinterpret_cast<const uint4*>(slot) : make_uint4(0, 0, 0, 0);
                const uint32_t mine = nib_word == 0 ? map.x : (nib_word == 1 ? map.y : (nib_word == 2 ? map.z : map.w));
                const unsigned nib = (mine >> nib_shift) & 0xfu;
                // branch-free: a lane reads its (up to four) groups with predicated loads, absent groups are zero words
                // (the record carries the running counts of its map words, and the offsets inside a nibble are sums of
                // bits: one population count per record and lane - that pipe is the narrow one)
                const uint32_t cum = have ? reinterpret_cast<const uint32_t*>(slot)[4] : 0u;
                const int before = __popc(mine & ((1u << nib_shift) - 1u)) + (nib_word == 0 ? 0 : (int)((cum >> (8 * (nib_word - 1))) & 0xffu));
                const uint32_t* words = reinterpret_cast<const uint32_t*>(slot) + 8 + before;
                const unsigned b0 = nib & 1u, b01 = b0 + ((nib >> 1) & 1u), b012 = b01 + ((nib >> 2) & 1u);
                wg[r][0] = (nib & 1u) ? words[0] : 0u;
                wg[r][1] = (nib & 2u) ? words[b0] : 0u;
                wg[r][2] = (nib & 4u) ? words[b01] : 0u;
                wg[r][3] = (nib & 8u) ? words[b012] : 0u;
                const uint32_t ent = have ? s_list[warp + (i + r) * SQ_WARPS] : (256u << 16);
                const int d = (int)(ent >> 16) - 256;        // (the same for every lane: the branch below is uniform)
                dh[r] = (d >= -128 && d <= 127) ? 0 : d / 2;
                dl[r] = d - dh[r];
            }
            #pragma unroll
            for (int r = 0; r < 2; ++r) {
                #pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (half == 1 && dh[r] == 0) break;
                    const unsigned sel = (unsigned)(half ? dh[r] : dl[r]) & 0xffu;
                    const int s0 = (int)sel, s1 = (int)(sel << 8), s2 = (int)(sel << 16), s3 = (int)(sel << 24);
                    #pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        acc[g * 4 + 0] = __dp4a((int)wg[r][g], s0, acc[g * 4 + 0]);
                        acc[g * 4 + 1] = __dp4a((int)wg[r][g], s1, acc[g * 4 + 1]);
                        acc[g * 4 + 2] = __dp4a((int)wg[r][g], s2, acc[g * 4 + 2]);
                        acc[g * 4 + 3] = __dp4a((int)wg[r][g], s3, acc[g * 4 + 3]);
                    }
                }
            }
            __syncwarp();
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else if (o0 < K) {                                     // K is a multiple of 16
        // Two half-batches in flight alternately: while one half's columns are multiplied, the other half's loads
        // are already on their way (the memory system is never left idle behind the arithmetic).
        constexpr int HB = SQ_U / 2;                         // columns per half-batch and lane
        const int8_t* wbase = p.Wt + o0;
        uint32_t entA[HB], entB[HB];
        uint4 wA[HB], wB[HB];
        auto fetch = [&](int e, uint32_t (&ent)[HB], uint4 (&w)[HB]) {
            #pragma unroll
            for (int u = 0; u < HB; ++u) {
                const int eu = e + u * CPR;
                ent[u] = eu < total ? s_list[eu] : 0xffffffffu;
            }
            #pragma unroll
            for (int u = 0; u < HB; ++u)
                w[u] = ent[u] != 0xffffffffu
                           ? __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)(ent[u] & 0xffffu) * K))
                           : make_uint4(0, 0, 0, 0);
        };
        auto consume = [&](const uint32_t (&ent)[HB], const uint4 (&w)[HB]) {
            #pragma unroll
            for (int u = 0; u < HB; ++u)
                if (ent[u] != 0xffffffffu) fma16(acc, w[u], (int)(ent[u] >> 16) - 256);
        };
        constexpr int STEP = HB * CPR;                       // list entries one half-batch of the CTA covers
        fetch(grp, entA, wA);
        for (int e = grp; e < total; e += 2 * STEP) {
            fetch(e + STEP, entB, wB);
            consume(entA, wA);
            fetch(e + 2 * STEP, entA, wA);
            consume(entB, wB);
        }
    }
    // ---- 3. add the partial sums: the column groups of a warp by shuffles, the warps through shared memory
    #pragma unroll
    for (int i = 0; i < 16; ++i) {
        #pragma unroll
        for (int o = LANES; o < 32; o <<= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
    }
    if (lane < LANES) {
        #pragma unroll
        for (int i = 0; i < 16; i += 4)
            *reinterpret_cast<int4*>(&s_red[warp * OW + lane * 16 + i]) = make_int4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
    }
    __syncthreads();
    for (int o = tid; o < width; o += SQ_THREADS) {
        int v = 0;
        #pragma unroll
        for (int w = 0; w < SQ_WARPS; ++w) v += s_red[w * OW + o];
        p.dP[((size_t)t * p.n + s) * K + slice * OW + o] = v;
    }
    // ---- 4. whoever finishes last for this (stream, slice) runs the sum over the frames
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned old = atomicAdd(&p.counters[s * slices + slice], 1u);
        s_last = (old == (unsigned)(p.T - 1));
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // every thread owns 4 neighbouring outputs and a contiguous share of the frames: it sums its
    // share (all loads in flight), the shares are chained through shared memory, then it writes
    // its frames' outputs.  FS = threads per output group = frame shares.
    constexpr int OG = OW / 4;                                // output groups of 4
    constexpr int FS = SQ_THREADS / OG;                       // frame shares (2 for OW = 512 ... 8 for OW = 128)
    const int og = tid % OG, fs = tid / OG;
    const int per = (p.T + FS - 1) / FS;
    const int tb = fs * per, te = min(p.T, tb + per);
    const int o = slice * OW + og * 4;
    const bool live = og * 4 < width;                         // width is a multiple of 16
    const size_t stride = (size_t)p.n * K;
    const int32_t* dp = p.dP + (size_t)s * K + o;
    // the frames of this share stay in registers between the two steps (host guarantees per <= SQ_TAIL)
    int4 d[SQ_TAIL];
    int4 sum = make_int4(0, 0, 0, 0);
    #pragma unroll
    for (int u = 0; u < SQ_TAIL; ++u) {
        d[u] = (live && tb + u < te) ? __ldcg(reinterpret_cast<const int4*>(dp + (size_t)(tb + u) * stride)) : make_int4(0, 0, 0, 0);
    }
    #pragma unroll
    for (int u = 0; u < SQ_TAIL; ++u) { sum.x += d[u].x; sum.y += d[u].y; sum.z += d[u].z; sum.w += d[u].w; }
    int4* s_share = reinterpret_cast<int4*>(s_dyn);           // [FS][OG], reuses the reduction buffer
    __syncthreads();
    s_share[fs * OG + og] = sum;
    __syncthreads();
    if (!live) return;
    int4 v;
    if (p.bias) {
        v = *reinterpret_cast<const int4*>(p.bias + o);
    } else {
        v = *reinterpret_cast<const int4*>(p.P + (size_t)s * K + o);
        for (int f = 0; f < fs; ++f) {
            const int4 q = s_share[f * OG + og];
            v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w;
        }
    }
    const int4 bias4 = v;
    #pragma unroll
    for (int u = 0; u < SQ_TAIL; ++u) {
        if (tb + u < te) {
            if (p.bias) v = make_int4(bias4.x + d[u].x, bias4.y + d[u].y, bias4.z + d[u].z, bias4.w + d[u].w);
            else { v.x += d[u].x; v.y += d[u].y; v.z += d[u].z; v.w += d[u].w; }
            if (p.Y) {
                const size_t oi = ((size_t)(tb + u) * p.n + s) * K + o;
                if (p.shift < 0) {
                    *reinterpret_cast<int4*>(reinterpret_cast<int32_t*>(p.Y) + oi) = v;
                } else {
                    char4 q;
                    q.x = (signed char)fc_apply_f(v.x, p.shift, p.act); q.y = (signed char)fc_apply_f(v.y, p.shift, p.act);
                    q.z = (signed char)fc_apply_f(v.z, p.shift, p.act); q.w = (signed char)fc_apply_f(v.w, p.shift, p.act);
                    *reinterpret_cast<char4*>(reinterpret_cast<int8_t*>(p.Y) + oi) = q;
                }
            }
        }
    }
    // the share that holds the last frame stores the projection
    if (p.P && te == p.T && tb < te) *reinterpret_cast<int4*>(p.P + (size_t)s * K + o) = v;
    if (tid == 0) p.counters[s * slices + slice] = 0;
}

// Non-zero delta entries and active groups of 32 inputs of every (frame, stream) of a chunk: the
// delta + scan step alone, for chunks that are then evaluated densely.
__global__ void __launch_bounds__(SQ_THREADS) fc_count_kernel(const int8_t* __restrict__ x, const int8_t* __restrict__ xprev,
                                                            unsigned* stat, int n, int C)
{
    __shared__ int s_nnz, s_grp;
    const int tid = threadIdx.x, lane = tid & 31;
    const int t = blockIdx.x / n, s = blockIdx.x - t * n;
    if (tid == 0) { s_nnz = 0; s_grp = 0; }
    __syncthreads();
    const uint4* xt4 = reinterpret_cast<const uint4*>(x + ((size_t)t * n + s) * C);
    const uint4* xp4 = reinterpret_cast<const uint4*>(t > 0 ? x + ((size_t)(t - 1) * n + s) * C : xprev + (size_t)s * C);
    int nnz = 0, grp = 0;
    for (int base = 0; base < (C >> 4); base += SQ_THREADS) {     // same trip count for every thread: the shuffles below need whole warps
        const int chunk = base + tid;
        unsigned m = 0;
        if (chunk < (C >> 4)) {
            const uint4 a = __ldg(xt4 + chunk), b = __ldg(xp4 + chunk);
            m = differing_bytes(a, b);
        }
        nnz += __popc(m);
        const unsigned other = __shfl_xor_sync(0xffffffffu, m, 1);
        grp += ((lane & 1) == 0 && (m | other)) ? 1 : 0;
    }
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) { nnz += __shfl_down_sync(0xffffffffu, nnz, o); grp += __shfl_down_sync(0xffffffffu, grp, o); }
    if (lane == 0) { atomicAdd(&s_nnz, nnz); atomicAdd(&s_grp, grp); }
    __syncthreads();
    if (tid == 0) { stat[blockIdx.x * 2] = (unsigned)s_nnz; stat[blockIdx.x * 2 + 1] = (unsigned)s_grp; }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
// The switch between the column gather and the dense tensor-core evaluation of a chunk (W read once for all frames)
// is rrm_options.fc_dense_density (plain non-zero fraction of the previous chunk; measured break-even on fc6: ~7 %)
// and, for chunks of few rows (one launch that reads W once), rrm_options.fc_dense_rows (rows x non-zero fraction;
// measured break-even on fc6, 32 rows: 2.2 % non-zeros).

// Copies the chunk's counters to pinned host memory behind the work already on the stream.
static int seq_read_back(Layer& L, int rows, cudaStream_t st)
{
    if (L.seq_ev_pending) return RRM_OK;                     // an older copy is still in flight: keep it
    if (rows > L.seq_stat_host_cap) {
        if (L.seq_stat_host) cudaFreeHost(L.seq_stat_host);
        L.seq_stat_host = nullptr; L.seq_stat_host_cap = 0;
        if (cudaMallocHost(reinterpret_cast<void**>(&L.seq_stat_host), (size_t)rows * 2 * 4) != cudaSuccess) { cudaGetLastError(); return RRM_OK; }
        L.seq_stat_host_cap = rows;
    }
    if (!L.seq_ev && cudaEventCreateWithFlags(&L.seq_ev, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return RRM_OK; }
    RRM_CUDA_TRY(cudaMemcpyAsync(L.seq_stat_host, L.seq_stat, (size_t)rows * 2 * 4, cudaMemcpyDeviceToHost, st));
    RRM_CUDA_TRY(cudaEventRecord(L.seq_ev, st));
    L.seq_ev_pending = true;
    L.seq_pending_rows = rows;
    return RRM_OK;
}

int fc_dense_tc_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, int T, bool stateless, cudaStream_t st);

// (sp_stride > 0: the weight-sparse form adds every warp's ring of records)
static size_t seq_dyn_smem(int c_in, int lanes, int sp_stride = 0)
{
    return (size_t)SQ_WARPS * 16 * lanes * 4 + (size_t)c_in * 4 + (size_t)SQ_WARPS * SW_RING * sp_stride * 4;
}

static int seq_ensure(rrm_net* net, Layer& L, int T)
{
    if (T <= L.seq_cap) return RRM_OK;
    const int K = L.d.c_out, n = L.d.n;
    void* dP = nullptr;
    void* stat = nullptr;
    if (cudaMalloc(&dP, (size_t)T * n * K * 4) != cudaSuccess) { cudaGetLastError(); return RRM_ERR_ALLOC; }
    if (cudaMalloc(&stat, (size_t)T * n * 2 * 4) != cudaSuccess) { cudaFree(dP); cudaGetLastError(); return RRM_ERR_ALLOC; }
    if (L.seq_dP) {
        // growing: the smaller arrays may still be in use by a chunk in flight; after that they are freed
        cudaDeviceSynchronize();
        for (void* old : {static_cast<void*>(L.seq_dP), static_cast<void*>(L.seq_stat)}) {
            for (size_t i = 0; i < net->allocs.size(); ++i)
                if (net->allocs[i] == old) { net->allocs.erase(net->allocs.begin() + i); break; }
            cudaFree(old);
        }
    }
    net->allocs.push_back(dP);
    net->allocs.push_back(stat);
    L.seq_dP = reinterpret_cast<int32_t*>(dP);
    L.seq_stat = reinterpret_cast<unsigned*>(stat);
    L.seq_cap = T;
    return RRM_OK;
}

int fc_seq_create(rrm_net* net, Layer& L)
{
    const int K = L.d.c_out, n = L.d.n;
    const int slices = ceil_div(K, 16 * 8);                  // the narrowest slice the kernel is built for
    void* c = nullptr;
    if (cudaMalloc(&c, (size_t)n * slices * 4) != cudaSuccess) { cudaGetLastError(); return RRM_ERR_ALLOC; }
    net->allocs.push_back(c);
    RRM_CUDA_TRY(cudaMemset(c, 0, (size_t)n * slices * 4));
    L.seq_counters = reinterpret_cast<unsigned*>(c);
    RRM_CUDA_TRY(cudaFuncSetAttribute(fc_seq_kernel<32, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)seq_dyn_smem(SQ_MAX_C_IN, 32)));
    RRM_CUDA_TRY(cudaFuncSetAttribute(fc_seq_kernel<32, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)seq_dyn_smem(SQ_MAX_C_IN, 32)));
    RRM_CUDA_TRY(cudaFuncSetAttribute(fc_seq_kernel<16, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)seq_dyn_smem(SQ_MAX_C_IN, 16)));
    RRM_CUDA_TRY(cudaFuncSetAttribute(fc_seq_kernel<8, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)seq_dyn_smem(SQ_MAX_C_IN, 8)));
    // (weight-sparse form: up to 136 words per record, the stride of a matrix without zeros)
    RRM_CUDA_TRY(cudaFuncSetAttribute(fc_seq_kernel<32, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)seq_dyn_smem(SQ_MAX_C_IN, 32, 136)));
    RRM_CUDA_TRY(cudaFuncSetAttribute(fc_seq_kernel<32, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)seq_dyn_smem(SQ_MAX_C_IN, 32, 136)));
    return seq_ensure(net, L, 1);
}

bool fc_seq_supported(const Layer& L) { return L.fc_fused && L.d.c_in <= SQ_MAX_C_IN; }

// T frames of every stream in one launch.  dense: every entry is visited and frames are independent
// (P_t = b + W X_t); stateless: the RRM state (snapshot, stored projection) is left untouched.
int fc_seq_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, int T, bool dense, bool stateless, cudaStream_t st)
{
    const int C = L.d.c_in, K = L.d.c_out, n = L.d.n;
    if (T < 1) return RRM_ERR_INVALID_ARG;
    if ((long long)T * n > 65535) return RRM_ERR_CAPACITY;
    if (dense && stateless && L.tc_ready) return fc_dense_tc_run(net, L, X_dev, Y_dev, T, true, st);
    RRM_TRY(seq_ensure(net, L, T));
    FcSeqParams p;
    p.x = reinterpret_cast<const int8_t*>(X_dev);
    p.Wt = L.Wt;
    p.dP = L.seq_dP;
    p.Y = Y_dev;
    p.counters = L.seq_counters;
    p.T = T; p.n = n; p.c_in = C; p.c_out = K; p.shift = L.d.shift; p.act = L.d.act;
    p.Wsp = L.Wsp; p.sp_stride = L.sp_stride;
    if (dense) {
        p.xprev = nullptr;
        p.bias = reinterpret_cast<const int32_t*>(L.bias);
        p.stat = nullptr;
        if (stateless) { p.xnext = nullptr; p.P = nullptr; }
        else { p.xnext = L.xs[L.xs_cur ^ 1]; L.xs_cur ^= 1; p.P = reinterpret_cast<int32_t*>(L.P); }
    } else {
        // ---- which evaluation: the previous chunk's measured density decides (temporal coherence is the
        // method's premise).  Its counters were copied to pinned memory behind the chunk; they are used
        // once that copy has landed, and never waited for.
        if (L.seq_ev_pending && cudaEventQuery(L.seq_ev) == cudaSuccess) {
            unsigned long long nz = 0;
            for (int i = 0; i < L.seq_pending_rows; ++i) nz += L.seq_stat_host[2 * i];
            L.seq_density = (double)nz / ((double)L.seq_pending_rows * C);
            L.seq_ev_pending = false;
        }
        cudaGetLastError();                                  // cudaErrorNotReady from the query is not an error
        // (up to 1024 rows go through the streaming form, 256 rows per launch, each launch at the cost of reading W
        // once: it wins as soon as the rows' gathered columns add up to about that many bytes)
        const bool use_dense = L.tc_ready && L.d.variant == RRM_VARIANT_AUTO && (long long)T * n >= 8 &&
                               (fc_tc_usable(L, T * n) ? L.seq_density * T * n >= (double)net->opt.fc_dense_rows * fc_tc_launches(T * n)
                                                       : L.seq_density >= (double)net->opt.fc_dense_density);
        L.seq_last_T = T;
        L.seq_last_variant = use_dense ? RRM_VARIANT_DENSE : (L.Wsp ? RRM_VARIANT_SPARSE_W : RRM_VARIANT_GATHER);
        if (use_dense) {
            // the results are the same integers: P_t = b + W X_t for every frame, state := last frame
            if (fc_tc_usable(L, T * n)) {
                // few rows: one launch streams W once, and its idle warps count the delta entries meanwhile
                RRM_TRY(fc_tc_run(net, L, X_dev, Y_dev, T * n, false, L.seq_stat, st));
            } else {
                fc_count_kernel<<<T * n, SQ_THREADS, 0, st>>>(reinterpret_cast<const int8_t*>(X_dev), L.xs[L.xs_cur], L.seq_stat, n, C);
                RRM_TRY(fc_dense_tc_run(net, L, X_dev, Y_dev, T, false, st));
            }
            return seq_read_back(L, T * n, st);
        }
        p.xprev = L.xs[L.xs_cur];
        p.xnext = L.xs[L.xs_cur ^ 1];
        L.xs_cur ^= 1;
        p.bias = nullptr;
        p.P = reinterpret_cast<int32_t*>(L.P);
        p.stat = L.seq_stat;
    }
    // slice width: the widest (fewest redundant scans, one wave of CTAs with a short chain of dependent
    // round trips each), narrowed while the grid would leave a good part of the machine idle
    int lanes = L.Wsp ? 32 : L.seq_lanes;
    if (lanes == 0) {
        lanes = 32;
        while (lanes > 8 && (long long)ceil_div(K, 16 * lanes) * T * n < 200) lanes /= 2;
    }
    // the closing sum keeps SQ_TAIL frames per thread: longer chunks go out in pieces, each piece
    // taking the frame before it (still in X) as its "previous" frame
    const int piece_max = SQ_TAIL * (SQ_THREADS / (4 * lanes));
    const int8_t* snapshot = p.xprev;
    int8_t* const xnext = p.xnext;
    const size_t ybytes = (size_t)n * K * (L.d.shift < 0 ? 4 : 1);
    for (int t0 = 0; t0 < T; t0 += piece_max) {
        const int piece = T - t0 < piece_max ? T - t0 : piece_max;
        p.x = reinterpret_cast<const int8_t*>(X_dev) + (size_t)t0 * n * C;
        p.xprev = dense ? nullptr : (t0 == 0 ? snapshot : p.x - (size_t)n * C);
        p.xnext = t0 + piece == T ? xnext : nullptr;
        p.Y = Y_dev ? reinterpret_cast<char*>(Y_dev) + (size_t)t0 * ybytes : nullptr;
        p.stat = dense ? nullptr : L.seq_stat + (size_t)t0 * n * 2;
        p.T = piece;
        dim3 grid(ceil_div(K, 16 * lanes), piece * n);
        const size_t dyn = seq_dyn_smem(C, lanes, L.Wsp ? L.sp_stride : 0);
        if (L.Wsp && grid.x * grid.y <= 2 * 148) fc_seq_kernel<32, true, true><<<grid, SQ_THREADS, dyn, st>>>(p);
        else if (L.Wsp) fc_seq_kernel<32, false, true><<<grid, SQ_THREADS, dyn, st>>>(p);
        else if (lanes == 32 && grid.x * grid.y <= 2 * 148) fc_seq_kernel<32, true, false><<<grid, SQ_THREADS, dyn, st>>>(p);
        else if (lanes == 32) fc_seq_kernel<32, false, false><<<grid, SQ_THREADS, dyn, st>>>(p);
        else if (lanes == 16) fc_seq_kernel<16, false, false><<<grid, SQ_THREADS, dyn, st>>>(p);
        else fc_seq_kernel<8, false, false><<<grid, SQ_THREADS, dyn, st>>>(p);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    if (!dense) RRM_TRY(seq_read_back(L, T * n, st));
    return RRM_OK;
}

// ------------------------------------------------------------------------------------------------
// Dense evaluation of M = frames x streams input rows on the tensor cores: P = X W^T + b is the 1x1
// "convolution" of an M-pixel image with c_in channels, i.e. exactly what conv_tc_kernel computes from
// the [c_out][c_in] filters; W is read from HBM once for all rows.
// ------------------------------------------------------------------------------------------------
// Pstate (may be nullptr) receives the rows from `state_from` on: the projection of the last frame.
__global__ void fc_dense_finish_kernel(const int32_t* __restrict__ Pd, void* Y, int32_t* Pstate, long long state_from,
                                       long long total, int shift, int act)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int v = Pd[i];
    if (Pstate && i >= state_from) Pstate[i - state_from] = v;
    if (Y) {
        if (shift < 0) reinterpret_cast<int32_t*>(Y)[i] = v;
        else reinterpret_cast<int8_t*>(Y)[i] = (int8_t)fc_apply_f(v, shift, act);
    }
}

// stateless: Y only.  Otherwise the stored projection and the snapshot become those of the last frame.
int fc_dense_tc_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, int T, bool stateless, cudaStream_t st)
{
    const int C = L.d.c_in, K = L.d.c_out, n = L.d.n;
    // a few rows: one launch that streams W once and finishes the outputs itself
    if (fc_tc_usable(L, T * n)) return fc_tc_run(net, L, X_dev, Y_dev, T * n, stateless, nullptr, st);
    RRM_TRY(seq_ensure(net, L, T));
    Layer Lt = L;                                            // the M-row problem as a 1x1 convolution
    Lt.d.n = T * n; Lt.d.h = Lt.d.w = 1; Lt.oh = Lt.ow = 1;
    Lt.P = L.seq_dP;
    Tensor in;
    in.dtype = T_I8; in.n = T * n; in.c = C; in.h = in.w = 1; in.cs = C; in.unit_bytes = 1;
    in.X = const_cast<void*>(X_dev);
    RRM_TRY(launch_conv_tc(net, Lt, in, true, false, st));
    const long long total = (long long)T * n * K;
    fc_dense_finish_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(L.seq_dP, Y_dev, stateless ? nullptr : reinterpret_cast<int32_t*>(L.P),
                                                                           (long long)(T - 1) * n * K, total, L.d.shift, L.d.act);
    RRM_CUDA_TRY(cudaGetLastError());
    if (!stateless) {
        RRM_CUDA_TRY(cudaMemcpyAsync(L.xs[L.xs_cur ^ 1], reinterpret_cast<const int8_t*>(X_dev) + (size_t)(T - 1) * n * C, (size_t)n * C,
                                     cudaMemcpyDeviceToDevice, st));
        L.xs_cur ^= 1;
    }
    return RRM_OK;
}

// ------------------------------------------------------------------------------------------------
// Weight-sparse form: packs Wt[c_in][c_out] into records per (input, 512-output slice).  One warp per record; lane L
// owns outputs 16 L .. 16 L + 15 of the slice = 4 groups of four.  WRITE = false only finds the longest record.
// ------------------------------------------------------------------------------------------------
template <bool WRITE>
__global__ void __launch_bounds__(256) fc_sparse_w_pack_kernel(const int8_t* __restrict__ Wt, uint32_t* rec, int C, int K, int slices,
                                                               int stride, int* max_words, unsigned long long* total_words)
{
    const int lane = threadIdx.x & 31;
    const long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= (long long)C * slices) return;                  // uniform inside the warp
    const int j = (int)(r / slices), slice = (int)(r - (long long)j * slices);
    const int o = slice * 512 + lane * 16;
    uint4 w = make_uint4(0, 0, 0, 0);
    if (o < K) w = *reinterpret_cast<const uint4*>(Wt + (size_t)j * K + o);      // K is a multiple of 16
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
    unsigned nib = 0;
    #pragma unroll
    for (int g = 0; g < 4; ++g) if (ww[g]) nib |= 1u << g;
    const int cnt = __popc(nib);
    int incl = cnt;
    #pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    if (!WRITE) {
        if (lane == 0) { atomicMax(max_words, total); atomicAdd(total_words, (unsigned long long)total); }
        return;
    }
    uint32_t* out = rec + (size_t)r * stride;
    unsigned m = nib << (4 * (lane & 7));                    // the 8 lanes of a map word OR their nibbles together
    m |= __shfl_xor_sync(0xffffffffu, m, 1);
    m |= __shfl_xor_sync(0xffffffffu, m, 2);
    m |= __shfl_xor_sync(0xffffffffu, m, 4);
    if ((lane & 7) == 0) out[lane >> 3] = m;
    // word 4: the number of packed words before map word 1, 2 and 3 (one byte each); words 5-7 unused
    const int c0 = __shfl_sync(0xffffffffu, incl, 7), c1 = __shfl_sync(0xffffffffu, incl, 15), c2 = __shfl_sync(0xffffffffu, incl, 23);
    if (lane == 0) out[4] = (uint32_t)c0 | (uint32_t)c1 << 8 | (uint32_t)c2 << 16;
    int at = 8 + incl - cnt;
    #pragma unroll
    for (int g = 0; g < 4; ++g) if (nib >> g & 1u) out[at++] = ww[g];
}

int fc_sparse_w_create(rrm_net* net, Layer& L)
{
    const int C = L.d.c_in, K = L.d.c_out;
    const int slices = ceil_div(K, 512);
    const long long records = (long long)C * slices;
    int* d_max = nullptr;
    if (cudaMalloc(&d_max, 16) != cudaSuccess) { cudaGetLastError(); return RRM_ERR_ALLOC; }
    RRM_CUDA_TRY(cudaMemset(d_max, 0, 16));
    const unsigned blocks = (unsigned)((records + 7) / 8);
    fc_sparse_w_pack_kernel<false><<<blocks, 256>>>(L.Wt, nullptr, C, K, slices, 0, d_max, reinterpret_cast<unsigned long long*>(d_max + 2));
    int h[4] = {0, 0, 0, 0};
    const cudaError_t e = cudaMemcpy(h, d_max, 16, cudaMemcpyDeviceToHost);
    cudaFree(d_max);
    if (e != cudaSuccess) { cudaGetLastError(); return RRM_ERR_CUDA; }
    L.sp_stride = 8 + round_up(h[0] > 0 ? h[0] : 1, 4);      // 32-byte header, 16-byte aligned records
    std::memcpy(&L.sp_words, &h[2], 8);
    void* rec = nullptr;
    if (cudaMalloc(&rec, (size_t)records * L.sp_stride * 4) != cudaSuccess) { cudaGetLastError(); return RRM_ERR_ALLOC; }
    net->allocs.push_back(rec);
    RRM_CUDA_TRY(cudaMemset(rec, 0, (size_t)records * L.sp_stride * 4));
    fc_sparse_w_pack_kernel<true><<<blocks, 256>>>(L.Wt, reinterpret_cast<uint32_t*>(rec), C, K, slices, L.sp_stride, nullptr, nullptr);
    RRM_CUDA_TRY(cudaGetLastError());
    RRM_CUDA_TRY(cudaDeviceSynchronize());
    L.Wsp = reinterpret_cast<uint32_t*>(rec);
    if (getenv("RRM_DEBUG"))
        fprintf(stderr, "rrm: weight-sparse FC: %lld records of %d words, %lld packed weight words (%.1f %% of the dense bytes incl. maps)\n",
                records, L.sp_stride, L.sp_words, 100.0 * (L.sp_words * 4.0 + records * 32.0) / ((double)C * K));
    return RRM_OK;
}

// Sums the per-frame counters of the last chunk: non-zero delta entries and active groups of 32 inputs.
int fc_seq_stats(Layer& L, unsigned long long* nnz, unsigned long long* groups)
{
    const size_t cnt = (size_t)L.seq_last_T * L.d.n * 2;
    std::vector<unsigned> h(cnt);
    RRM_CUDA_TRY(cudaMemcpy(h.data(), L.seq_stat, cnt * 4, cudaMemcpyDeviceToHost));
    *nnz = 0; *groups = 0;
    for (size_t i = 0; i < cnt; i += 2) { *nnz += h[i]; *groups += h[i + 1]; }
    return RRM_OK;
}

}  // namespace rrm
