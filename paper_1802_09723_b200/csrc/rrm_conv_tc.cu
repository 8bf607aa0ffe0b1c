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
// 128-bit loads into shared memory in the 128-byte-swizzled K-major layout the MMA reads.  Binary
// layers expand their bit-packed rows on the way: delta = +2 / -2 / 0 per changed bit (dense: +1 / -1).
// B (filters) is packed once at create time as the exact shared-memory image of every (N tile, slab),
// so one bulk copy (cp.async.bulk, completion on an mbarrier) stages a slab.  One thread issues the
// MMAs; tcgen05.commit releases a stage when the tensor core has read it.  The K range can be split
// over CTAs (grid.z); partial sums are then added onto the stored projection with integer atomics,
// which keeps the result exact.  (Pixel tile x tap) blocks with no changed input are skipped.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets ERRW_TIMEOUT in the net's error
// word and the CTA leaves through the common exit, which frees its tensor memory.
#include "rrm_common.cuh"

namespace rrm {

constexpr int TC_M = 128;
constexpr int TC_SLAB = 128;                  // bytes of K per stage
constexpr int TC_STAGES = 4;
constexpr int TC_THREADS = 192;               // warps 0-3: A producers + epilogue, warp 4: MMA, warp 5: B loader
constexpr int TC_MAX_BN = 128;
constexpr unsigned TC_SPIN_LIMIT = 1u << 20;

struct TcParams {
    const void* A;            // int8: delta rows (delta) or values (dense); binary: changed bits (delta) / unused
    const void* Anew;         // binary: current sign bits
    const uint32_t* in_act;   // input activity bitmap (delta mode)
    const int* olist;         // compacted projection pixels (delta mode)
    const int* ocount;
    const int8_t* Wimg;       // [n_tiles][slabs][bn * 128] swizzled tile images
    const int32_t* bias;
    int32_t* P;               // [opixels][c_out]
    int* errw;
    int h, w, oh, ow, kw, taps, stride, pad, c_in, c_out, opixels;
    int row_units;            // int8: bytes per input pixel row (multiple of 32); binary: words per pixel
    int chunks_per_tap;       // 32-byte K chunks per tap
    int slabs;                // total 128-byte slabs of K
    int bn;                   // 64 or 128
    int ksplit;               // gridDim.z
};

// ---- raw PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (unsigned i = 0; i < TC_SPIN_LIMIT; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, rows 128 bytes apart, 8-row groups 1024
// bytes apart (the tile starts on a 1024-byte boundary).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);            // start address, 16-byte units
    d |= (uint64_t)1 << 16;                             // leading byte offset (unused with swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                             // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                             // 128-byte swizzle
    return d;
}
// Instruction descriptor: int8 x int8 -> int32, both operands K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t tc_instr_desc(int bn)
{
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// byte i of the result = bit i of the low nibble of x (0 or 1)
__device__ __forceinline__ uint32_t spread4(uint32_t x) { return ((x & 0xfu) * 0x00204081u) & 0x01010101u; }

// Dynamic shared memory: [stages][A 16 KB | B 16 KB] on a 1024-byte boundary, then barriers and row tables.
struct TcSmemTail {
    unsigned long long full[TC_STAGES], empty[TC_STAGES], done;
    uint32_t tmem_base;
    int fail;
    unsigned long long tap_mask[2];           // taps with at least one changed input under this tile (up to 128 taps)
    int q[TC_M], nbase[TC_M], iy0[TC_M], ix0[TC_M];
};
constexpr size_t TC_STAGE_BYTES = (size_t)TC_M * TC_SLAB + (size_t)TC_MAX_BN * TC_SLAB;
constexpr size_t TC_SMEM_BYTES = 1024 + TC_STAGES * TC_STAGE_BYTES + sizeof(TcSmemTail);

template <bool BIN, bool DENSE>
__global__ void __launch_bounds__(TC_THREADS, 1) conv_tc_kernel(TcParams p)
{
    extern __shared__ unsigned char tc_smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, ntile = blockIdx.y, split = blockIdx.z;
    int count = p.opixels;
    if (!DENSE) {
        count = *p.ocount;
        if (tile * TC_M >= count) return;                   // before anything is allocated
    }
    unsigned char* base = reinterpret_cast<unsigned char*>(((uintptr_t)tc_smem_raw + 1023) & ~(uintptr_t)1023);
    TcSmemTail* S = reinterpret_cast<TcSmemTail*>(base + TC_STAGES * TC_STAGE_BYTES);
    const uint32_t base_u32 = smem_u32(base);

    if (tid == 0) {
        for (int s = 0; s < TC_STAGES; ++s) {
            mbar_init(smem_u32(&S->full[s]), 128 + 1);      // 128 producer threads + the B loader's expect_tx
            mbar_init(smem_u32(&S->empty[s]), 1);           // one tcgen05.commit
        }
        mbar_init(smem_u32(&S->done), 1);
        S->fail = 0;
        S->tap_mask[0] = S->tap_mask[1] = DENSE ? ~0ull : 0ull;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < TC_M) {
        const int r = tile * TC_M + tid;
        int q = -1;
        if (r < count) q = DENSE ? r : p.olist[r];
        S->q[tid] = q;
        if (q >= 0) {
            const int ox = q % p.ow, oy = (q / p.ow) % p.oh, ns = q / (p.ow * p.oh);
            S->nbase[tid] = ns * p.h * p.w;
            S->iy0[tid] = oy * p.stride - p.pad;
            S->ix0[tid] = ox * p.stride - p.pad;
        } else {
            S->nbase[tid] = 0; S->iy0[tid] = -(1 << 20); S->ix0[tid] = -(1 << 20);
        }
    }
    if (warp == 4) {                                        // tensor memory for the accumulator tile
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&S->tmem_base)), "r"((uint32_t)TC_MAX_BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = S->tmem_base;

    // taps that see a changed input pixel under any row of this tile
    if (!DENSE && tid < TC_M && S->q[tid] >= 0) {
        const int nb = S->nbase[tid], y0 = S->iy0[tid], x0 = S->ix0[tid];
        unsigned long long m0 = 0, m1 = 0;
        for (int t = 0; t < p.taps; ++t) {
            const int iy = y0 + t / p.kw, ix = x0 + t % p.kw;
            if (iy < 0 || iy >= p.h || ix < 0 || ix >= p.w) continue;
            const int pix = nb + iy * p.w + ix;
            if ((p.in_act[pix >> 5] >> (pix & 31)) & 1u) { if (t < 64) m0 |= 1ull << t; else m1 |= 1ull << (t - 64); }
        }
        if (m0) atomicOr(&S->tap_mask[0], m0);
        if (m1) atomicOr(&S->tap_mask[1], m1);
    }
    __syncthreads();
    const unsigned long long tm0 = S->tap_mask[0], tm1 = S->tap_mask[1];

    // this CTA's share of the slabs
    const int per = (p.slabs + p.ksplit - 1) / p.ksplit;
    const int s_begin = split * per, s_end = min(p.slabs, s_begin + per);
    const int cpt = p.chunks_per_tap;
    auto slab_live = [&](int ks) -> bool {                  // any tap of the slab's 4 chunks changed?
        const int t_lo = (ks * 4) / cpt, t_hi = min(p.taps - 1, (ks * 4 + 3) / cpt);
        for (int t = t_lo; t <= t_hi; ++t)
            if (t < 64 ? (tm0 >> t) & 1ull : (tm1 >> (t - 64)) & 1ull) return true;
        return false;
    };
    const uint32_t tile_b_bytes = (uint32_t)p.bn * TC_SLAB;
    bool ok = true;
    int n_issued = 0;                                       // slabs that went through the pipeline (same in every role)

    if (warp < 4) {
        // ================= A producers: 8 lanes x 16 bytes = one 128-byte row; 4 rows per warp pass
        const int piece = lane & 7, rsub = lane >> 3;
        const uint32_t* Au = reinterpret_cast<const uint32_t*>(p.A);
        const uint32_t* Nu = reinterpret_cast<const uint32_t*>(p.Anew);
        int it = 0;
        for (int ks = s_begin; ks < s_end; ++ks) {
            if (!slab_live(ks)) continue;
            const int stage = it % TC_STAGES;
            if (ok && !mbar_wait(smem_u32(&S->empty[stage]), ((it / TC_STAGES) & 1) ^ 1)) ok = false;
            if (!ok) break;
            unsigned char* As = base + stage * TC_STAGE_BYTES;
            const int kc = ks * 4 + (piece >> 1);           // this lane's 32-byte chunk of K
            const int tap = kc / cpt, cc = kc - tap * cpt;
            const int ky = tap / p.kw, kx = tap - ky * p.kw;
            const bool tap_ok = tap < p.taps;
            #pragma unroll 4
            for (int i = 0; i < 8; ++i) {
                const int r = warp * 32 + i * 4 + rsub;
                uint4 v = make_uint4(0, 0, 0, 0);
                const int iy = S->iy0[r] + ky, ix = S->ix0[r] + kx;
                if (tap_ok && iy >= 0 && iy < p.h && ix >= 0 && ix < p.w) {
                    const int pix = S->nbase[r] + iy * p.w + ix;
                    if (DENSE || ((p.in_act[pix >> 5] >> (pix & 31)) & 1u)) {
                        if (!BIN) {
                            v = *reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(p.A) +
                                                                (size_t)pix * p.row_units + cc * 32 + (piece & 1) * 16);
                        } else {
                            // 16 channels of word cc: bits -> bytes
                            const uint32_t nw = Nu[(size_t)pix * p.row_units + cc] >> ((piece & 1) * 16);
                            uint32_t valid = 0xffffu;
                            const int c_base = cc * 32 + (piece & 1) * 16;
                            if (c_base + 16 > p.c_in) valid = c_base >= p.c_in ? 0u : ((1u << (p.c_in - c_base)) - 1u);
                            uint32_t pos, neg;                 // channels that contribute +1 / -1 (dense) or +2 / -2 (delta)
                            if (DENSE) { pos = nw & valid; neg = ~nw & valid; }
                            else {
                                const uint32_t ch = (Au[(size_t)pix * p.row_units + cc] >> ((piece & 1) * 16)) & valid;
                                pos = ch & nw; neg = ch & ~nw;
                            }
                            const uint32_t pm = DENSE ? 0x01u : 0x02u, nm = DENSE ? 0xffu : 0xfeu;
                            v.x = spread4(pos) * pm + spread4(neg) * nm;
                            v.y = spread4(pos >> 4) * pm + spread4(neg >> 4) * nm;
                            v.z = spread4(pos >> 8) * pm + spread4(neg >> 8) * nm;
                            v.w = spread4(pos >> 12) * pm + spread4(neg >> 12) * nm;
                        }
                    }
                }
                const uint32_t off = (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u + (uint32_t)((piece ^ (r & 7)) << 4);
                *reinterpret_cast<uint4*>(As + off) = v;
            }
            fence_async_smem();                              // generic-proxy stores -> visible to the tensor core
            mbar_arrive(smem_u32(&S->full[stage]));
            ++it;
        }
        n_issued = it;
    } else if (warp == 5) {
        // ================= B loader: one bulk copy per slab
        if (lane == 0) {
            int it = 0;
            for (int ks = s_begin; ks < s_end; ++ks) {
                if (!slab_live(ks)) continue;
                const int stage = it % TC_STAGES;
                if (!mbar_wait(smem_u32(&S->empty[stage]), ((it / TC_STAGES) & 1) ^ 1)) { ok = false; break; }
                const uint32_t bar = smem_u32(&S->full[stage]);
                mbar_arrive_expect_tx(bar, tile_b_bytes);
                bulk_copy_g2s(base_u32 + stage * (uint32_t)TC_STAGE_BYTES + TC_M * TC_SLAB,
                              p.Wimg + ((size_t)ntile * p.slabs + ks) * tile_b_bytes, tile_b_bytes, bar);
                ++it;
            }
        }
    } else {
        // ================= MMA issuer
        if (lane == 0) {
            const uint32_t idesc = tc_instr_desc(p.bn);
            int it = 0;
            for (int ks = s_begin; ks < s_end; ++ks) {
                if (!slab_live(ks)) continue;
                const int stage = it % TC_STAGES;
                if (!mbar_wait(smem_u32(&S->full[stage]), (it / TC_STAGES) & 1)) { ok = false; break; }
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
            n_issued = it;
        }
    }
    if (!ok) { S->fail = 1; atomicOr(p.errw, ERRW_TIMEOUT); }

    // ================= epilogue: warps 0-3 read their 32 accumulator rows and update the projection
    if (warp < 4) {
        ok = __all_sync(0xffffffffu, ok);                   // the tensor-memory loads below need the whole warp
        bool have = n_issued > 0;                           // identical for all producer threads
        if (ok && have && !mbar_wait(smem_u32(&S->done), 0)) { ok = false; S->fail = 1; atomicOr(p.errw, ERRW_TIMEOUT); }
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        const int r = warp * 32 + lane;
        const int q = S->q[r];
        const bool atomic = p.ksplit > 1;
        const int n0 = ntile * p.bn;
        if (ok && (have || DENSE)) {
            for (int c0 = 0; c0 < p.bn; c0 += 16) {
                uint32_t v[16];
                if (have) {
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                        : "r"(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                } else {
                    #pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0;
                }
                if (q < 0) continue;
                int32_t* Pq = p.P + (size_t)q * p.c_out + n0 + c0;
                #pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int co = n0 + c0 + j;
                    if (co >= p.c_out) break;
                    const int val = (int)v[j];
                    if (DENSE) {
                        // split 0 carries the bias; with a split K the projection was zeroed beforehand
                        const int b = (split == 0 && p.bias) ? p.bias[co] : 0;
                        if (atomic) atomicAdd(Pq + j, val + b); else Pq[j] = val + b;
                    } else if (val != 0) {
                        if (atomic) atomicAdd(Pq + j, val); else Pq[j] += val;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
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
    if (i < total) P[i] = 0;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
bool conv_tc_eligible(const rrm_net* net, const Layer& L)
{
    const rrm_layer_desc& d = L.d;
    const Tensor& in = net->tensors[d.src];
    if (d.dtype == RRM_I8) { if (in.dtype != T_I8 || in.cs % 32 != 0) return false; }
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
    static bool attr_done = false;
    if (!attr_done) {
        RRM_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
        RRM_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
        RRM_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
        RRM_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
        attr_done = true;
    }
    L.tc_ready = true;
    return RRM_OK;
}

// F*dI (dense: F*X + b) on the tensor cores; P is updated in place (dense: overwritten).
int launch_conv_tc(rrm_net* net, Layer& L, const Tensor& in, bool dense, bool stateless, cudaStream_t st)
{
    const rrm_layer_desc& d = L.d;
    TcParams p;
    const bool bin = d.dtype == RRM_BIN;
    const void* X = stateless ? in.X2 : in.X;
    p.A = bin ? in.D : (dense ? X : in.D);
    p.Anew = X;
    p.in_act = in.act; p.olist = L.olist; p.ocount = L.ocount;
    p.Wimg = L.tc_Wimg; p.bias = reinterpret_cast<const int32_t*>(L.bias);
    p.P = reinterpret_cast<int32_t*>(stateless ? L.P2 : L.P);
    p.errw = net->errw;
    p.h = d.h; p.w = d.w; p.oh = L.oh; p.ow = L.ow; p.kw = d.kw; p.taps = d.kh * d.kw; p.stride = d.stride; p.pad = d.pad;
    p.c_in = d.c_in; p.c_out = d.c_out; p.opixels = L.opixels();
    p.row_units = bin ? in.cs : in.cs;                       // int8: bytes per pixel; binary: words per pixel
    p.chunks_per_tap = L.tc_kpp / 32;
    p.slabs = L.tc_slabs; p.bn = L.tc_bn;
    const int m_tiles = ceil_div(L.opixels(), TC_M);
    // split K until the grid covers the machine (a split needs at least 2 slabs to be worth a CTA)
    int ksplit = 1;
    while (m_tiles * L.tc_ntiles * ksplit < 148 && ksplit * 2 <= L.tc_slabs / 2) ksplit *= 2;
    p.ksplit = ksplit;
    if (dense && ksplit > 1) {
        const long long tot = (long long)L.opixels() * d.c_out;
        zero_projection_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(p.P, tot);
    }
    dim3 grid(m_tiles, L.tc_ntiles, ksplit);
    if (bin) {
        if (dense) conv_tc_kernel<true, true><<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(p);
        else conv_tc_kernel<true, false><<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(p);
    } else {
        if (dense) conv_tc_kernel<false, true><<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(p);
        else conv_tc_kernel<false, false><<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(p);
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

}  // namespace rrm
