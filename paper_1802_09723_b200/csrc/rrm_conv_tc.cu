// Tensor-core variant of F*dI (and of the dense pass) for int8 and binary layers: an implicit GEMM
// over compacted projection pixels on the 5th-generation tensor cores (tcgen05.mma kind::i8, int32
// accumulators in tensor memory).
//
//   rows    M = 128 projection pixels per CTA: the compacted list of pixels that can change (delta)
//           or all pixels (dense);
//   columns N = 64 or 128 output channels per CTA;
//   depth   K = taps x input channels, cut into slabs of 128 bytes (4 MMA steps of 32 int8 each).
// A (activations) is gathered: each row of a slab is 128 contiguous bytes of one input pixel's delta
// row (zero when the pixel is outside the image or did not change), copied by four producer warps with
// asynchronous 16-byte copies into shared memory in the 128-byte-swizzled K-major layout the MMA reads.
// Binary layers expand their bit-packed rows on the way: delta = +2 / -2 / 0 per changed bit (dense: +1 / -1).
// B (filters) is packed once at create time as the exact shared-memory image of every (N tile, slab),
// so one bulk copy (cp.async.bulk, completion on an mbarrier) stages a slab.  One thread issues the
// MMAs; tcgen05.commit releases a stage when the tensor core has read it.  The K range can be split
// over CTAs (grid.z); every accumulator row leaves through shared memory as one bulk store or one bulk
// integer add-reduction onto the stored projection, which keeps the result exact in any order.
// (Pixel tile x tap) blocks with no changed input are skipped.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets ERRW_TIMEOUT in the net's error
// word and the CTA leaves through the common exit, which frees its tensor memory.
#include "rrm_common.cuh"
#include "rrm_rows.cuh"
#include "rrm_tc.cuh"
#include "rrm_dev.cuh"

namespace rrm {

constexpr int TC_SLAB = 128;                  // bytes of K per stage
constexpr int TC_STAGES = 3;
constexpr int TC_THREADS = 192;               // warps 0-3: A producers + epilogue, warp 4: MMA, warp 5: B loader
constexpr int TC_MAX_BN = 128;

struct TcParams {
    const void* A;            // int8: delta rows (delta) or values (dense); binary: changed bits (delta) / unused
    const void* Anew;         // binary: current sign bits
    const uint32_t* in_act;   // input activity bitmap (delta mode)
    const uint32_t* oact;     // projection pixels to update (delta mode)
    int* ocount;              // receives their number
    const int8_t* Wimg;       // [n_tiles][slabs][bn * 128] swizzled tile images
    const int32_t* bias;
    int32_t* P;               // [opixels][c_out]
    int* errw;
    int h, w, oh, ow, kw, taps, stride, pad, c_in, c_out, opixels;
    int row_units;            // int8: bytes per input pixel row (multiple of 32); binary: words per pixel
    int chunks_per_tap;       // 32-byte K chunks per tap (0 for the 4-bytes-per-pixel form)
    int kpp;                  // K bytes per tap: padded channels per pixel (int8) or 32 x words (binary)
    int slabs;                // total 128-byte slabs of K
    int bn;                   // 64 or 128
    int ksplit;               // gridDim.z
    unsigned wait_limit;      // polls of one bounded wait
    const uint32_t* count_bitmap;   // dense evaluation inside a delta step: the layer's update bitmap, whose set bits the
                                    // first CTA counts into *ocount (the measured activity); nullptr otherwise
    // several frames in one launch (delta only; gridDim.z = frames x ksplit): frame g reads its delta rows, new rows
    // and bitmaps, and writes its product, at these distances from frame 0's
    int frames;
    long long row_stride;     // bytes between the frames' sets of delta rows (and of new rows)
    long long arena_stride;   // bytes between the frames' arenas (bitmaps, counters)
    long long p_stride;       // elements between the frames' products
    int store;                // delta: the product is stored, not added (ksplit 1: every row written belongs to one CTA)
    // ceil(2^32 / d) for d = chunks_per_tap and d = kw: the K loop divides by them in every iteration of every role,
    // and its single-thread roles are bound by the length of their instruction chains (exact for the small operands here)
    unsigned magic_cpt, magic_kw;
};

// byte i of the result = bit i of the low nibble of x (0 or 1)
__device__ __forceinline__ uint32_t spread4(uint32_t x) { return ((x & 0xfu) * 0x00204081u) & 0x01010101u; }

// Dynamic shared memory: [stages][A 16 KB | B 16 KB] on a 1024-byte boundary, then barriers and row tables.
struct TcSmemTail {
    unsigned long long full[TC_STAGES], bfull[TC_STAGES], empty[TC_STAGES], done;   // A landed / B landed / stage free / all MMAs done
    uint32_t tmem_base;
    int fail;
    unsigned long long tap_mask[2];           // taps with a usable input under at least one row of this tile (up to 128 taps)
    uint32_t live[8];                         // bit r: slab s_begin + r has a usable tap (the first 256 slabs of the CTA's range)
    unsigned long long rmask[TC_M][2];        // per row: taps whose input pixel is inside the image (and changed, delta mode)
    int q[TC_M], pix0[TC_M];                  // projection pixel of the row; input pixel under tap (0,0) (may be outside)
};
constexpr size_t TC_STAGE_BYTES = (size_t)TC_M * TC_SLAB + (size_t)TC_MAX_BN * TC_SLAB;
constexpr size_t TC_SMEM_BYTES = 1024 + TC_STAGES * TC_STAGE_BYTES + sizeof(TcSmemTail);
constexpr int TC_LAG = 1;                     // a slab is handed to the tensor core when the next one has been issued (its copies
                                              // have landed by then); handing it over one slab later still, with the third stage's
                                              // copies in flight too, left the stage's MMAs too little time to commit before the
                                              // producers want the stage back (measured: 3-5 % slower steps)
constexpr int TC_ROW_WORDS = TC_MAX_BN + 4;   // epilogue row buffers: 16-byte aligned rows, staggered over the banks
static_assert((size_t)TC_M * TC_ROW_WORDS * 4 <= TC_STAGES * TC_STAGE_BYTES, "epilogue rows reuse the stage buffers");

template <bool BIN, bool DENSE>
__global__ void __launch_bounds__(TC_THREADS, 2) conv_tc_kernel(TcParams p)
{
    extern __shared__ unsigned char tc_smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, ntile = blockIdx.y;
    const int frame = (!DENSE && p.frames > 1) ? blockIdx.z / p.ksplit : 0, split = blockIdx.z - frame * p.ksplit;
    if (!DENSE && frame > 0) {
        p.A = reinterpret_cast<const char*>(p.A) + frame * p.row_stride;
        p.Anew = reinterpret_cast<const char*>(p.Anew) + frame * p.row_stride;
        p.in_act = reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(p.in_act) + frame * p.arena_stride);
        p.oact = reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(p.oact) + frame * p.arena_stride);
        p.ocount = reinterpret_cast<int*>(reinterpret_cast<char*>(p.ocount) + frame * p.arena_stride);
        p.P += frame * p.p_stride;
    }
    unsigned char* base = reinterpret_cast<unsigned char*>(((uintptr_t)tc_smem_raw + 1023) & ~(uintptr_t)1023);
    TcSmemTail* S = reinterpret_cast<TcSmemTail*>(base + TC_STAGES * TC_STAGE_BYTES);
    const uint32_t base_u32 = smem_u32(base);
    __shared__ int s_tmp[256 + 34];
    int count = p.opixels;
    pdl_launch_dependents();
    if (!DENSE) {
        pdl_wait();                                          // the update bitmap is the predecessors' work
        // this CTA's rows: the tile-th group of 128 set bits of the layer's update bitmap
        count = select_rows<TC_M>(p.oact, (p.opixels + 31) >> 5, tile, S->q, s_tmp);
        if (tile == 0 && ntile == 0 && split == 0 && tid == 0) *p.ocount = count;
        if (tile * TC_M >= count) return;                   // before anything is allocated
    }

    if (tid == 0) {
        for (int s = 0; s < TC_STAGES; ++s) {
            mbar_init(smem_u32(&S->full[s]), 128);          // 128 producer threads
            mbar_init(smem_u32(&S->bfull[s]), 1);           // the B loader's expect_tx (a barrier of its own, so that the
                                                            // loader can wait for its copies in flight on a give-up exit)
            mbar_init(smem_u32(&S->empty[s]), 1);           // one tcgen05.commit
        }
        mbar_init(smem_u32(&S->done), 1);
        S->fail = 0;
        S->tap_mask[0] = S->tap_mask[1] = 0ull;
        for (int i = 0; i < 8; ++i) S->live[i] = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {                                        // tensor memory for the accumulator tile
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&S->tmem_base)), "r"((uint32_t)TC_MAX_BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();                                        // tap_mask is zero before the rows add to it
    if (tid < TC_M) {
        // row -> projection pixel, and per tap: is its input pixel inside the image (and changed)?
        const int r = tile * TC_M + tid;
        const int q = DENSE ? (r < count ? r : -1) : S->q[tid];
        S->q[tid] = q;
        unsigned long long m0 = 0, m1 = 0;
        int pix0 = 0;
        if (q >= 0) {
            const int ox = q % p.ow, oy = (q / p.ow) % p.oh, ns = q / (p.ow * p.oh);
            const int y0 = oy * p.stride - p.pad, x0 = ox * p.stride - p.pad;
            pix0 = ns * p.h * p.w + y0 * p.w + x0;
            row_tap_masks<DENSE>(p.in_act, pix0, y0, x0, p.h, p.w, p.taps / p.kw, p.kw, m0, m1);
        }
        S->pix0[tid] = pix0;
        S->rmask[tid][0] = m0; S->rmask[tid][1] = m1;
        // OR over the warp first (32-bit halves), then one shared-memory atomic per warp and half
        const unsigned a0 = __reduce_or_sync(0xffffffffu, (unsigned)m0), a1 = __reduce_or_sync(0xffffffffu, (unsigned)(m0 >> 32));
        const unsigned a2 = __reduce_or_sync(0xffffffffu, (unsigned)m1), a3 = __reduce_or_sync(0xffffffffu, (unsigned)(m1 >> 32));
        if (lane == 0) {
            unsigned* tm = reinterpret_cast<unsigned*>(S->tap_mask);
            if (a0) atomicOr(tm + 0, a0);
            if (a1) atomicOr(tm + 1, a1);
            if (a2) atomicOr(tm + 2, a2);
            if (a3) atomicOr(tm + 3, a3);
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (DENSE) pdl_wait();                                   // barriers, tensor memory and row tables are set up; the inputs come next
    if (DENSE && p.count_bitmap && tile == 0 && ntile == 0 && split == 0) {
        // (uniform for the whole CTA) the layer's activity is still measured while it is evaluated densely
        int c = 0;
        for (int i = tid; i < ((p.opixels + 31) >> 5); i += TC_THREADS) c += __popc(__ldg(p.count_bitmap + i));
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if (lane == 0) s_tmp[warp] = c;
        __syncthreads();
        if (tid == 0) { int t = 0; for (int w = 0; w < TC_THREADS / 32; ++w) t += s_tmp[w]; *p.ocount = t; }
    }
    const uint32_t tmem = S->tmem_base;
    const unsigned long long tm0 = S->tap_mask[0], tm1 = S->tap_mask[1];

    // this CTA's share of the slabs; a slab none of whose taps is usable under any row is skipped
    const int per = (p.slabs + p.ksplit - 1) / p.ksplit;
    const int s_begin = split * per, s_end = min(p.slabs, s_begin + per);
    const int cpt = p.chunks_per_tap;
    auto slab_live = [&](int ks) -> bool {
        const int t_lo = (ks * TC_SLAB) / p.kpp, t_hi = min(p.taps - 1, (ks * TC_SLAB + TC_SLAB - 1) / p.kpp);
        for (int t = t_lo; t <= t_hi; ++t)
            if (t < 64 ? (tm0 >> t) & 1ull : (tm1 >> (t - 64)) & 1ull) return true;
        return false;
    };
    // which slabs are live is worked out once, by all threads, and kept as a bitmap: the roles' loops then find their
    // next slab with a shift instead of divisions (ranges beyond 256 slabs test the rest slab by slab)
    const int n_range = s_end - s_begin;
    for (int r = tid; r < min(n_range, 256); r += TC_THREADS)
        if (slab_live(s_begin + r)) atomicOr(&S->live[r >> 5], 1u << (r & 31));
    __syncthreads();
    auto next_live = [&](int ks) -> int {                   // first live slab >= ks, or s_end
        int r = ks - s_begin;
        while (r < min(n_range, 256)) {
            const uint32_t wbits = S->live[r >> 5] >> (r & 31);
            if (wbits) return s_begin + r + __ffs(wbits) - 1;
            r = (r | 31) + 1;
        }
        ks = s_begin + max(r, ks - s_begin);
        while (ks < s_end && !slab_live(ks)) ++ks;
        return min(ks, s_end);
    };
    auto div_cpt = [&](int x) -> int { return p.magic_cpt ? (int)__umulhi((unsigned)x, p.magic_cpt) : x; };   // (0: the divisor is 1)
    auto div_kw = [&](int x) -> int { return p.magic_kw ? (int)__umulhi((unsigned)x, p.magic_kw) : x; };
    const uint32_t tile_b_bytes = (uint32_t)p.bn * TC_SLAB;
    bool ok = true;
    int n_issued = 0;                                       // slabs that went through the pipeline (same in every role)

    if (warp < 4) {
        // ================= A producers: 8 lanes x 16 bytes = one 128-byte row; 4 rows per warp pass
        const int piece = lane & 7, rsub = lane >> 3;
        int it = 0;
        if (!BIN) {
            // int8 rows are copied as they are: asynchronous 16-byte copies (zero-filled where the input
            // pixel is unusable); a slab is handed to the tensor core TC_LAG slabs later, when its copies landed
            const unsigned char* Ab = reinterpret_cast<const unsigned char*>(p.A);
            // this thread's 8 rows stay the same for the whole K loop: their tap masks, source offsets and
            // shared-memory offsets live in registers, so a slab costs a few instructions per 16-byte copy
            unsigned long long rm0[8], rm1[8];
            int src_row[8];
            uint32_t dst_row[8];
            #pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = warp * 32 + i * 4 + rsub;
                rm0[i] = S->rmask[r][0]; rm1[i] = S->rmask[r][1];
                src_row[i] = S->pix0[r] * p.row_units;       // fits: a tensor holds fewer than 2^31 values
                dst_row[i] = (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u + (uint32_t)((piece ^ (r & 7)) << 4);
            }
            for (int ks = next_live(s_begin); ks < s_end; ks = next_live(ks + 1)) {
                const int stage = it % TC_STAGES;
                if (!mbar_wait(smem_u32(&S->empty[stage]), ((it / TC_STAGES) & 1) ^ 1, p.wait_limit)) { ok = false; break; }
                if (*(volatile int*)&S->fail) break;             // another role gave up: issue nothing more
                const uint32_t As = base_u32 + stage * (uint32_t)TC_STAGE_BYTES;
                if (p.kpp == 4) {
                    // first layers (up to 4 channels = 4 bytes per pixel): a 16-byte piece holds 4 taps, copied one by one;
                    // where a tap sits relative to the row's first pixel is the same for all 8 rows
                    int toff[4], tsh[4];
                    bool tok[4], thi[4];
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int tap = ks * (TC_SLAB / 4) + piece * 4 + j;
                        const int ky = div_kw(tap), kx = tap - ky * p.kw;
                        toff[j] = (ky * p.w + kx) * 4;
                        tok[j] = tap < p.taps; thi[j] = tap >= 64; tsh[j] = tap & 63;
                    }
                    #pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const bool use = tok[j] && (((thi[j] ? rm1[i] : rm0[i]) >> tsh[j]) & 1ull);
                            const unsigned char* src = use ? Ab + (src_row[i] + toff[j]) : Ab;
                            asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;"
                                         ::"r"(As + dst_row[i] + 4u * j), "l"(src), "r"(use ? 4u : 0u) : "memory");
                        }
                    }
                } else {
                const int kc = ks * 4 + (piece >> 1);       // this lane's 32-byte chunk of K
                const int tap = div_cpt(kc), cc = kc - tap * cpt;
                const int ky = div_kw(tap), kx = tap - ky * p.kw;
                const int slab_off = (ky * p.w + kx) * p.row_units + cc * 32 + (piece & 1) * 16;   // same for the 8 rows
                const bool tap_ok = tap < p.taps, hi = tap >= 64;
                const int sh = tap & 63;
                #pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const bool use = tap_ok && (((hi ? rm1[i] : rm0[i]) >> sh) & 1ull);
                    const unsigned char* src = use ? Ab + (src_row[i] + slab_off) : Ab;
                    cp_async16(As + dst_row[i], src, use ? 16u : 0u);
                }
                }
                cp_async_commit();
                if (it >= TC_LAG) {
                    cp_async_wait<TC_LAG>();                 // the copies of slab it - TC_LAG have landed
                    fence_async_smem();
                    mbar_arrive(smem_u32(&S->full[(it - TC_LAG) % TC_STAGES]));
                }
                ++it;
            }
            cp_async_wait<0>();
            fence_async_smem();
            if (ok) for (int j = max(0, it - TC_LAG); j < it; ++j) mbar_arrive(smem_u32(&S->full[j % TC_STAGES]));
        } else {
            // binary rows are expanded from bits to bytes on the way: the words of the next slab are
            // fetched into registers while the current slab is expanded and stored
            const uint32_t* Cu = reinterpret_cast<const uint32_t*>(p.A);
            const uint32_t* Nu = reinterpret_cast<const uint32_t*>(p.Anew);
            uint32_t nw[8], cw[8];
            unsigned long long bm0[8], bm1[8];               // per-row tap masks, word offsets and store offsets
            int bsrc[8];
            uint32_t bdst[8];
            #pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = warp * 32 + i * 4 + rsub;
                bm0[i] = S->rmask[r][0]; bm1[i] = S->rmask[r][1];
                bsrc[i] = S->pix0[r] * p.row_units;
                bdst[i] = (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u + (uint32_t)((piece ^ (r & 7)) << 4);
            }
            unsigned usemask = 0;
            int half_valid = 0;
            auto fetch = [&](int ks) {
                const int kc = ks * 4 + (piece >> 1);
                const int tap = div_cpt(kc), cc = kc - tap * cpt;
                const int ky = div_kw(tap), kx = tap - ky * p.kw;
                const int slab_off = (ky * p.w + kx) * p.row_units + cc;
                const bool tap_ok = tap < p.taps, hi = tap >= 64;
                const int sh = tap & 63;
                const int c_base = cc * 32 + (piece & 1) * 16;
                half_valid = c_base >= p.c_in ? 0 : (c_base + 16 > p.c_in ? (int)((1u << (p.c_in - c_base)) - 1u) : 0xffff);
                usemask = 0;
                #pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const bool use = tap_ok && (((hi ? bm1[i] : bm0[i]) >> sh) & 1ull);
                    nw[i] = 0; cw[i] = 0;
                    if (use) {
                        const int wi = bsrc[i] + slab_off;
                        nw[i] = Nu[wi];
                        if (!DENSE) cw[i] = Cu[wi];
                        usemask |= 1u << i;
                    }
                }
            };
            int ks = next_live(s_begin);
            if (ks < s_end) fetch(ks);
            while (ks < s_end) {
                // keep this slab's words, start fetching the next one
                uint32_t n_cur[8], c_cur[8];
                #pragma unroll
                for (int i = 0; i < 8; ++i) { n_cur[i] = nw[i]; c_cur[i] = cw[i]; }
                const unsigned use_cur = usemask;
                const uint32_t valid = (uint32_t)half_valid;
                const int ks_next = next_live(ks + 1);
                if (ks_next < s_end) fetch(ks_next);
                const int stage = it % TC_STAGES;
                if (!mbar_wait(smem_u32(&S->empty[stage]), ((it / TC_STAGES) & 1) ^ 1, p.wait_limit)) { ok = false; break; }
                unsigned char* As = base + stage * TC_STAGE_BYTES;
                const int shift = (piece & 1) * 16;
                #pragma unroll
                for (int i = 0; i < 8; ++i) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (use_cur >> i & 1u) {
                        const uint32_t nb = n_cur[i] >> shift;
                        uint32_t pos, neg;                 // channels that contribute +1 / -1 (dense) or +2 / -2 (delta)
                        if (DENSE) { pos = nb & valid; neg = ~nb & valid; }
                        else { const uint32_t ch = (c_cur[i] >> shift) & valid; pos = ch & nb; neg = ch & ~nb; }
                        const uint32_t pm = DENSE ? 0x01u : 0x02u, nm = DENSE ? 0xffu : 0xfeu;
                        v.x = spread4(pos) * pm + spread4(neg) * nm;
                        v.y = spread4(pos >> 4) * pm + spread4(neg >> 4) * nm;
                        v.z = spread4(pos >> 8) * pm + spread4(neg >> 8) * nm;
                        v.w = spread4(pos >> 12) * pm + spread4(neg >> 12) * nm;
                    }
                    *reinterpret_cast<uint4*>(As + bdst[i]) = v;
                }
                fence_async_smem();                          // generic-proxy stores -> visible to the tensor core
                mbar_arrive(smem_u32(&S->full[stage]));
                ++it;
                ks = ks_next;
            }
        }
        n_issued = it;
    } else if (warp == 5) {
        // ================= B loader: one bulk copy per slab
        if (lane == 0) {
            int it = 0;
            for (int ks = next_live(s_begin); ks < s_end; ks = next_live(ks + 1)) {
                const int stage = it % TC_STAGES;
                if (!mbar_wait(smem_u32(&S->empty[stage]), ((it / TC_STAGES) & 1) ^ 1, p.wait_limit)) { ok = false; break; }
                if (*(volatile int*)&S->fail) break;
                const uint32_t bar = smem_u32(&S->bfull[stage]);
                mbar_arrive_expect_tx(bar, tile_b_bytes);
                bulk_copy_g2s(base_u32 + stage * (uint32_t)TC_STAGE_BYTES + TC_M * TC_SLAB,
                              p.Wimg + ((size_t)ntile * p.slabs + ks) * tile_b_bytes, tile_b_bytes, bar);
                ++it;
            }
            n_issued = it;
        }
    } else {
        // ================= MMA issuer
        if (lane == 0) {
            const uint32_t idesc = tc_instr_desc(p.bn);
            int it = 0;
            for (int ks = next_live(s_begin); ks < s_end; ks = next_live(ks + 1)) {
                const int stage = it % TC_STAGES;
                if (!mbar_wait(smem_u32(&S->full[stage]), (it / TC_STAGES) & 1, p.wait_limit) ||
                    !mbar_wait(smem_u32(&S->bfull[stage]), (it / TC_STAGES) & 1, p.wait_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_addr = base_u32 + stage * (uint32_t)TC_STAGE_BYTES;
                const uint64_t adesc = tc_smem_desc(a_addr), bdesc = tc_smem_desc(a_addr + TC_M * TC_SLAB);
                #pragma unroll
                for (int j = 0; j < 4; ++j)                  // 32 bytes of K per MMA: +2 in 16-byte address units
                    tc_mma_i8(tmem, adesc + 2 * j, bdesc + 2 * j, idesc, (it > 0 || j > 0) ? 1u : 0u);
                tc_commit(smem_u32(&S->empty[stage]));       // stage is free once these MMAs have read it
                ++it;
            }
            if (ok) tc_commit(smem_u32(&S->done));          // all MMAs of this CTA have completed
            else if (it > 0) {
                // giving up with MMAs issued: they must have completed before the tensor memory is freed
                *(volatile int*)&S->fail = 1;               // (before the commit below: the epilogue warps must not take
                __threadfence_block();                      // the completed barrier for a finished tile)
                tc_commit(smem_u32(&S->done));
                mbar_wait(smem_u32(&S->done), 0, WAIT_LIMIT_DEFAULT);
            }
        }
    }
    if (!ok) { *(volatile int*)&S->fail = 1; atomicOr(p.errw, ERRW_TIMEOUT); }

    // ================= epilogue: each of the 128 threads of warps 0-3 owns one accumulator row.  It copies
    // the row from tensor memory into shared memory (the stage buffers are free now) and hands it to the
    // copy engine as ONE bulk operation on the row's c_out-contiguous slice of the projection: a bulk
    // store for a dense pass that owns its outputs, a bulk integer add-reduction otherwise (exact in any
    // order).  Channel counts that are not a multiple of 4 take the element-wise path.
    if (warp < 4) {
        ok = __all_sync(0xffffffffu, ok);                   // the tensor-memory loads below need the whole warp
        const bool have = n_issued > 0;                     // identical for all producer threads
        if (ok && have && !mbar_wait(smem_u32(&S->done), 0, p.wait_limit)) { ok = false; *(volatile int*)&S->fail = 1; atomicOr(p.errw, ERRW_TIMEOUT); }
        asm volatile("bar.sync 1, 128;" ::: "memory");      // the four warps agree: nobody stores results of a tile that gave up
        ok = ok && *(volatile int*)&S->fail == 0;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        const bool atomic = p.ksplit > 1;
        const int n0 = ntile * p.bn;
        const int r = warp * 32 + lane;
        const int q = S->q[r];
        const int ncols = min(p.bn, p.c_out - n0);
        const bool bulk = (p.c_out & 3) == 0;
        int* row = reinterpret_cast<int*>(base) + r * TC_ROW_WORDS;
        if (ok && (have || DENSE || p.store)) {             // (a stored product is written even if it is all zero)
            for (int c0 = 0; c0 < p.bn; c0 += 32) {
                uint32_t v[32];
                if (have) {
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                        : "r"(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                } else {
                    #pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0;
                }
                if (q < 0) continue;
                if (bulk) {
                    #pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        int4 o = make_int4((int)v[j], (int)v[j + 1], (int)v[j + 2], (int)v[j + 3]);
                        if (DENSE && split == 0 && p.bias && c0 + j < ncols) {   // split 0 carries the bias
                            const int4 bb = *reinterpret_cast<const int4*>(p.bias + n0 + c0 + j);
                            o.x += bb.x; o.y += bb.y; o.z += bb.z; o.w += bb.w;
                        }
                        *reinterpret_cast<int4*>(row + c0 + j) = o;
                    }
                } else {
                    #pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int co = n0 + c0 + j;
                        if (co >= p.c_out) break;
                        const int val = (int)v[j];
                        int32_t* dst = p.P + (size_t)q * p.c_out + co;
                        if (DENSE) {
                            const int b = (split == 0 && p.bias) ? p.bias[co] : 0;
                            if (atomic) atomicAdd(dst, val + b); else *dst = val + b;
                        } else if (p.store) {
                            *dst = val;
                        } else if (val != 0) {
                            atomicAdd(dst, val);
                        }
                    }
                }
            }
            if (bulk && q >= 0) {
                fence_async_smem();                          // this thread's row -> visible to the copy engine
                int32_t* dst = p.P + (size_t)q * p.c_out + n0;
                const uint32_t bytes = (uint32_t)ncols * 4u;
                if ((DENSE && !atomic) || (!DENSE && p.store))
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                 ::"l"(dst), "r"(smem_u32(row)), "r"(bytes) : "memory");
                else                                         // with a split K of a dense pass the projection was zeroed beforehand
                    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.s32 [%0], [%1], %2;"
                                 ::"l"(dst), "r"(smem_u32(row)), "r"(bytes) : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the row buffer may be released
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5 && lane == 0 && S->fail) {
        // a role gave up: the bulk copies this thread may still have in flight must land before the CTA's shared
        // memory goes away (at most one per stage; a phase that completed long ago returns at once)
        for (int j = max(0, n_issued - TC_STAGES); j < n_issued; ++j)
            mbar_wait(smem_u32(&S->bfull[j % TC_STAGES]), (j / TC_STAGES) & 1, WAIT_LIMIT_DEFAULT);
    }
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TC_MAX_BN) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// Filter image: for every (N tile, slab) the [bn rows][128 bytes] tile exactly as the MMA wants it in
// shared memory (K-major, 128-byte swizzle).  K index = tap * kpp + channel, kpp = padded channels per pixel.
// ------------------------------------------------------------------------------------------------
__global__ void pack_weights_tc_kernel(const int8_t* W, int8_t* img, int c_in, int c_out, int taps, int kpp,
                                       int slabs, int bn, int n_tiles)
{
    const size_t total = (size_t)n_tiles * slabs * bn * TC_SLAB;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int kb = (int)(idx % TC_SLAB);
    const int n = (int)((idx / TC_SLAB) % bn);
    const int ks = (int)((idx / ((size_t)TC_SLAB * bn)) % slabs);
    const int nt = (int)(idx / ((size_t)TC_SLAB * bn * slabs));
    const int k = ks * TC_SLAB + kb;
    const int tap = k / kpp, c = k - tap * kpp;
    const int co = nt * bn + n;
    int8_t v = 0;
    if (tap < taps && c < c_in && co < c_out) v = W[((size_t)co * c_in + c) * taps + tap];
    const size_t off = (size_t)(n >> 3) * 1024 + (size_t)(n & 7) * 128 + (size_t)(((kb >> 4) ^ (n & 7)) << 4) + (kb & 15);
    img[((size_t)nt * slabs + ks) * bn * TC_SLAB + off] = v;
}

__global__ void zero_projection_kernel(int32_t* P, long long total)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();                                              // the predecessor may still read the projection
    if (i < total) P[i] = 0;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
int zero_projection(void* P, long long words, cudaStream_t st)
{
    launch_seq(zero_projection_kernel, dim3((unsigned)((words + 255) / 256)), dim3(256), 0, st, reinterpret_cast<int32_t*>(P), words);
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

bool conv_tc_eligible(const rrm_net* net, const Layer& L)
{
    const rrm_layer_desc& d = L.d;
    const Tensor& in = net->tensors[d.src];
    if (d.dtype == RRM_I8) { if (in.dtype != T_I8 || (in.cs % 32 != 0 && in.cs != 4)) return false; }
    else if (d.dtype == RRM_BIN) { if (in.dtype != T_BIN) return false; }
    else return false;
    if (d.kh * d.kw > 128) return false;
    return true;
}

int conv_tc_create(rrm_net* net, Layer& L, const void* W_dev)
{
    const rrm_layer_desc& d = L.d;
    const Tensor& in = net->tensors[d.src];
    const int taps = d.kh * d.kw;
    L.tc_kpp = d.dtype == RRM_I8 ? in.cs : in.cs * 32;       // K bytes per tap
    L.tc_bn = d.c_out <= 64 ? 64 : 128;
    L.tc_ntiles = ceil_div(d.c_out, L.tc_bn);
    L.tc_slabs = ceil_div(taps * L.tc_kpp, TC_SLAB);
    const size_t bytes = (size_t)L.tc_ntiles * L.tc_slabs * L.tc_bn * TC_SLAB;
    void* img = nullptr;
    if (cudaMalloc(&img, bytes) != cudaSuccess) { cudaGetLastError(); return RRM_ERR_ALLOC; }
    net->allocs.push_back(img);
    L.tc_Wimg = reinterpret_cast<int8_t*>(img);
    pack_weights_tc_kernel<<<(unsigned)((bytes + 255) / 256), 256>>>(reinterpret_cast<const int8_t*>(W_dev), L.tc_Wimg,
                                                                      d.c_in, d.c_out, taps, L.tc_kpp, L.tc_slabs, L.tc_bn,
                                                                      L.tc_ntiles);
    RRM_CUDA_TRY(cudaGetLastError());
    // (the attribute belongs to the current device's copy of the function: set at every create, it is cheap)
    RRM_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
    RRM_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
    RRM_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
    RRM_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
    L.tc_ready = true;
    return RRM_OK;
}

// F*dI (dense: F*X + b) on the tensor cores; P is updated in place (dense: overwritten).  P_dst (delta only): the
// product is added there instead of onto the stored projection.
// frames > 1 (delta only): that many frames in one launch; the tensor's delta rows and new rows, the bound arena and
// P_dst are frame 0's, the other frames' lie the tensor's size / arena_stride bytes and one projection further each;
// K is not split and the products are stored.
int launch_conv_tc(rrm_net* net, Layer& L, const Tensor& in, bool dense, bool stateless, cudaStream_t st,
                   const uint32_t* count_bitmap, void* P_dst, int frames, long long arena_stride)
{
    const rrm_layer_desc& d = L.d;
    TcParams p{};
    const bool bin = d.dtype == RRM_BIN;
    const void* X = stateless ? in.X2 : in.X;
    p.A = bin ? in.D : (dense ? X : in.D);
    p.Anew = (!dense && !stateless && in.Xn_cur) ? in.Xn_cur : X;    // (pipelined chunk: this frame's copy of the new rows)
    p.in_act = in.act; p.oact = L.oact; p.ocount = L.ocount;
    p.Wimg = L.tc_Wimg; p.bias = reinterpret_cast<const int32_t*>(L.bias);
    p.P = reinterpret_cast<int32_t*>(P_dst && !dense ? P_dst : (stateless ? L.P2 : L.P));
    p.errw = net->errw;
    p.h = d.h; p.w = d.w; p.oh = L.oh; p.ow = L.ow; p.kw = d.kw; p.taps = d.kh * d.kw; p.stride = d.stride; p.pad = d.pad;
    p.c_in = d.c_in; p.c_out = d.c_out; p.opixels = L.opixels();
    p.row_units = bin ? in.cs : in.cs;                       // int8: bytes per pixel; binary: words per pixel
    p.chunks_per_tap = L.tc_kpp / 32;
    p.kpp = L.tc_kpp;
    p.slabs = L.tc_slabs; p.bn = L.tc_bn;
    p.wait_limit = net->opt.wait_limit;
    p.count_bitmap = count_bitmap;
    const bool batched = frames > 1 && !dense;
    p.frames = batched ? frames : 1;
    p.row_stride = (long long)in.bytes(); p.arena_stride = arena_stride; p.p_stride = (long long)L.opixels() * d.c_out;
    p.store = batched ? 1 : 0;
    p.magic_cpt = p.chunks_per_tap > 1 ? (unsigned)(((1ull << 32) + p.chunks_per_tap - 1) / p.chunks_per_tap) : 0u;
    p.magic_kw = p.kw > 1 ? (unsigned)(((1ull << 32) + p.kw - 1) / p.kw) : 0u;
    const int m_tiles = ceil_div(L.opixels(), TC_M);
    // split K towards the point where a CTA's slabs all fit in its pipeline at once
    // (its gather is then one round trip instead of a chain of them) - but no further than one wave of the
    // machine needs: once the tiles alone fill it, a tile owned by one CTA saves the adds of shared tiles
    // (measured: for one frame at a time one CTA per SM is enough, more shares only add reductions; inside a chunk
    // graph, where the layers of several frames run side by side, half of that gives the best frames per second)
    const int wave = net->many_in_flight ? 74 : 148;
    int ksplit = 1;
    const int ks_max = ceil_div(L.tc_slabs, TC_STAGES);
    const long long tiles = (long long)m_tiles * L.tc_ntiles;
    while (!batched && ksplit < ks_max && tiles * ksplit < wave) ++ksplit;
    ksplit = ceil_div(L.tc_slabs, ceil_div(L.tc_slabs, ksplit));   // no empty shares
    p.ksplit = ksplit;
    if (dense && ksplit > 1) {
        const long long tot = (long long)L.opixels() * d.c_out;
        launch_seq(zero_projection_kernel, dim3((unsigned)((tot + 255) / 256)), dim3(256), 0, st, p.P, tot);
    }
    dim3 grid(m_tiles, L.tc_ntiles, ksplit * p.frames);
    if (bin) {
        if (dense) launch_seq(conv_tc_kernel<true, true>, dim3(grid), dim3(TC_THREADS), TC_SMEM_BYTES, st, p);
        else launch_seq(conv_tc_kernel<true, false>, dim3(grid), dim3(TC_THREADS), TC_SMEM_BYTES, st, p);
    } else {
        if (dense) launch_seq(conv_tc_kernel<false, true>, dim3(grid), dim3(TC_THREADS), TC_SMEM_BYTES, st, p);
        else launch_seq(conv_tc_kernel<false, false>, dim3(grid), dim3(TC_THREADS), TC_SMEM_BYTES, st, p);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

}  // namespace rrm
