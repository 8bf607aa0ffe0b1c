// Dense evaluation of an int8 FC layer for a few input rows (frames x streams) in ONE launch:
// P[row][o] = b[o] + sum_j W[o][j] X[row][j]  (Eq. 3), on the 5th-generation tensor cores.
//
// The weights are the M operand: a CTA owns 128 outputs and a share of K and streams its slice of W
// through a deep ring of stages.  A stage holds one 128-byte slab of K: 16 KB of W, filled by one bulk
// copy of the pre-swizzled tile image the tensor-core convolution already keeps, and the same slab of
// the input rows (the N operand, 16 to 256 rows), which the copy engine takes straight from the
// caller's [rows][c_in] array through a tensor map that applies the 128-byte swizzle and zero-fills
// rows and channels past the end.  With W read exactly once the launch is bound by HBM: c_out x c_in bytes.
// The int32 accumulators leave tensor memory transposed (thread = output, register = row), so for every
// row a warp touches 32 consecutive outputs.  With K split over CTAs the partial sums are added into a
// zeroed scratch array; the CTA that arrives last at a tile's counter adds the bias, applies f, writes
// the outputs and the stored projection, and leaves scratch and counter zeroed for the next launch.
//
// Every mbarrier wait is bounded; a wait that runs out sets ERRW_TIMEOUT and the CTA still takes part
// in the arrival protocol and frees its tensor memory.
#include <cuda.h>
#include "rrm_common.cuh"
#include "rrm_tc.cuh"
#include "rrm_dev.cuh"

namespace rrm {

constexpr int FT_THREADS = 192;               // warps 0-3: snapshot, then epilogue; warp 4: MMA; warp 5: loader
constexpr int FT_SLAB = 128;                  // bytes of K per stage
constexpr int FT_A_BYTES = TC_M * FT_SLAB;    // the W part of a stage
constexpr int FT_MAX_STAGES = 12;
constexpr int FT_MAX_ROWS = 256;              // input rows of one launch (the N of one MMA, and the accumulator's columns)
constexpr int FT_MAX_LAUNCHES = 4;            // more rows than this many launches hold go to the convolution kernel
constexpr size_t FT_SMEM_BUDGET = 220 * 1024;

struct FtSmemTail {
    unsigned long long full[FT_MAX_STAGES], empty[FT_MAX_STAGES], done;
    uint32_t tmem_base;
    int last;
    int cnt_nnz, cnt_grp;     // per-row counters of the delta scan
};

struct FtParams {
    const int8_t* Wimg;       // [m_tiles][slabs][128 x 128] swizzled tile images
    const int8_t* X;          // [rows][c_in]
    const int32_t* bias;
    int32_t* acc;             // [rows][m_tiles * 128] partial sums (split K only); zero between launches
    unsigned* arrive;         // [m_tiles]; zero between launches
    void* Y;                  // [rows][c_out] int32 (shift < 0) or int8; may be null
    int32_t* Pstate;          // receives the rows from state_from on; may be null
    int8_t* snap;             // receives X of the rows from state_from on; may be null
    unsigned* stat;           // [rows][2]: non-zero delta entries and active groups of 32 inputs per row; may be null
    const int8_t* xprev;      // the n rows before this launch's first row (the delta of row r is against row r - n)
    int n;                    // streams
    int* errw;
    int rows, c_in, c_out, slabs, per, ksplit, bn, stages, tmem_cols, state_from, shift, act;
    unsigned wait_limit;      // polls of one bounded wait
};

__device__ __forceinline__ void ft_finish(const FtParams& p, int row, int o, int v)
{
    if (p.bias) v += p.bias[o];
    const size_t i = (size_t)row * p.c_out + o;
    if (p.Pstate && row >= p.state_from) p.Pstate[i - (size_t)p.state_from * p.c_out] = v;
    if (p.Y) {
        if (p.shift < 0) reinterpret_cast<int32_t*>(p.Y)[i] = v;
        else reinterpret_cast<int8_t*>(p.Y)[i] = (int8_t)fc_apply_f(v, p.shift, p.act);
    }
}

// four consecutive outputs of one row: bias, stored projection, output through f
__device__ __forceinline__ void ft_finish4(const FtParams& p, int row, int oo, int4 w)
{
    if (p.bias) { const int4 b = *reinterpret_cast<const int4*>(p.bias + oo); w.x += b.x; w.y += b.y; w.z += b.z; w.w += b.w; }
    const size_t at = (size_t)row * p.c_out + oo;
    if (p.Pstate && row >= p.state_from) *reinterpret_cast<int4*>(p.Pstate + at - (size_t)p.state_from * p.c_out) = w;
    if (p.Y) {
        if (p.shift < 0) *reinterpret_cast<int4*>(reinterpret_cast<int32_t*>(p.Y) + at) = w;
        else {
            char4 q;
            q.x = (signed char)fc_apply_f(w.x, p.shift, p.act); q.y = (signed char)fc_apply_f(w.y, p.shift, p.act);
            q.z = (signed char)fc_apply_f(w.z, p.shift, p.act); q.w = (signed char)fc_apply_f(w.w, p.shift, p.act);
            *reinterpret_cast<char4*>(reinterpret_cast<int8_t*>(p.Y) + at) = q;
        }
    }
}

// CLUSTER: the CTAs that share an output block (the K shares) form one thread-block cluster and add their
// partial sums through distributed shared memory; otherwise through the scratch array in global memory.
template <bool CLUSTER>
__global__ void __launch_bounds__(FT_THREADS, 1) fc_tc_kernel(FtParams p, const __grid_constant__ CUtensorMap tmapX)
{
    extern __shared__ unsigned char ft_smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mtile = blockIdx.x, split = blockIdx.y;
    unsigned char* base = reinterpret_cast<unsigned char*>(((uintptr_t)ft_smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t base_u32 = smem_u32(base);
    const int s_begin = split * p.per, s_end = min(p.slabs, s_begin + p.per), mine = s_end - s_begin;
    const uint32_t b_bytes = (uint32_t)p.bn * FT_SLAB;                          // the input rows' part of a stage
    const uint32_t stage_bytes = FT_A_BYTES + b_bytes;
    FtSmemTail* S = reinterpret_cast<FtSmemTail*>(base + (size_t)p.stages * stage_bytes);

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&S->full[s]), 1);            // the loader's expect_tx
            mbar_init(smem_u32(&S->empty[s]), 1);           // one tcgen05.commit
        }
        mbar_init(smem_u32(&S->done), 1);
        S->last = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&S->tmem_base)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = S->tmem_base;
    bool ok = true;
    int n_loaded = 0;                                        // loader: stages issued

    if (warp < 4) {
        // ================= the CTAs of the first output block refresh the input snapshot (their K share of the state rows)
        if (p.snap && mtile == 0) {
            const int k_lo = s_begin * FT_SLAB, k_hi = min(p.c_in, s_end * FT_SLAB), w16 = (k_hi - k_lo) >> 4;
            for (int i = tid; i < (p.rows - p.state_from) * w16; i += 128) {
                const int r = i / w16, k = k_lo + (i - r * w16) * 16;
                *reinterpret_cast<int4*>(p.snap + (size_t)r * p.c_in + k) =
                    *reinterpret_cast<const int4*>(p.X + (size_t)(p.state_from + r) * p.c_in + k);
            }
        }
        // ================= while W streams: the delta scan's counters (Alg. 1: dI = I_t - I_{t-1}), one row per CTA and turn
        if (p.stat) {
            const int ncta = gridDim.x * gridDim.y, c16 = p.c_in >> 4;
            for (int row = split * gridDim.x + mtile; row < p.rows; row += ncta) {
                const uint4* xt4 = reinterpret_cast<const uint4*>(p.X + (size_t)row * p.c_in);
                const uint4* xp4 = reinterpret_cast<const uint4*>(row >= p.n ? p.X + (size_t)(row - p.n) * p.c_in
                                                                               : p.xprev + (size_t)row * p.c_in);
                if (tid == 0) { S->cnt_nnz = 0; S->cnt_grp = 0; }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                int nnz = 0, grp = 0;
                for (int b0 = 0; b0 < c16; b0 += 128) {      // same trip count for every thread: the shuffles need whole warps
                    const int chunk = b0 + tid;
                    unsigned m = 0;
                    if (chunk < c16) {
                        const uint4 a = __ldg(xt4 + chunk), b = __ldg(xp4 + chunk);
                        m = differing_bytes(a, b);
                    }
                    nnz += __popc(m);
                    const unsigned other = __shfl_xor_sync(0xffffffffu, m, 1);
                    grp += ((lane & 1) == 0 && (m | other)) ? 1 : 0;
                }
                #pragma unroll
                for (int o = 16; o > 0; o >>= 1) { nnz += __shfl_down_sync(0xffffffffu, nnz, o); grp += __shfl_down_sync(0xffffffffu, grp, o); }
                if (lane == 0) { atomicAdd(&S->cnt_nnz, nnz); atomicAdd(&S->cnt_grp, grp); }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (tid == 0) { p.stat[row * 2] = (unsigned)S->cnt_nnz; p.stat[row * 2 + 1] = (unsigned)S->cnt_grp; }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
        }
    } else if (warp == 5) {
        // ================= loader: per slab one 16 KB bulk copy of W and one tensor copy of the input rows
        if (lane == 0) {
            const int8_t* src = p.Wimg + ((size_t)mtile * p.slabs + s_begin) * FT_A_BYTES;
            for (int it = 0; it < mine; ++it) {
                const int stage = it % p.stages;
                if (!mbar_wait(smem_u32(&S->empty[stage]), ((it / p.stages) & 1) ^ 1, p.wait_limit)) { ok = false; break; }
                const uint32_t bar = smem_u32(&S->full[stage]);
                const uint32_t dst = base_u32 + (uint32_t)stage * stage_bytes;
                mbar_arrive_expect_tx(bar, stage_bytes);
                asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                             ::"r"(dst + FT_A_BYTES), "l"(&tmapX), "r"((s_begin + it) * FT_SLAB), "r"(0), "r"(bar) : "memory");
                bulk_copy_g2s(dst, src + (size_t)it * FT_A_BYTES, FT_A_BYTES, bar);
                n_loaded = it + 1;
            }
        }
    } else {
        // ================= MMA issuer
        if (lane == 0) {
            const uint32_t idesc = tc_instr_desc(p.bn);
            for (int it = 0; it < mine; ++it) {
                const int stage = it % p.stages;
                if (!mbar_wait(smem_u32(&S->full[stage]), (it / p.stages) & 1, p.wait_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_addr = base_u32 + (uint32_t)stage * stage_bytes;
                const uint64_t adesc = tc_smem_desc(a_addr), bdesc = tc_smem_desc(a_addr + FT_A_BYTES);
                #pragma unroll
                for (int j = 0; j < 4; ++j)                  // 32 bytes of K per MMA: +2 in 16-byte address units
                    tc_mma_i8(tmem, adesc + 2 * j, bdesc + 2 * j, idesc, (it > 0 || j > 0) ? 1u : 0u);
                tc_commit(smem_u32(&S->empty[stage]));
                n_loaded = it + 1;                           // (here: MMA groups issued)
            }
            if (ok) tc_commit(smem_u32(&S->done));
            else {
                // giving up: flagged first, so that the epilogue warps do not take the barrier for a finished tile;
                // MMAs already issued must have completed before the tensor memory is freed
                *(volatile int*)&S->last = -1;
                __threadfence_block();
                if (n_loaded > 0) {
                    tc_commit(smem_u32(&S->done));
                    mbar_wait(smem_u32(&S->done), 0, WAIT_LIMIT_DEFAULT);
                }
            }
        }
    }
    if (!ok) atomicOr(p.errw, ERRW_TIMEOUT);

    // ================= epilogue: thread = output (tensor-memory lane), register j = input row
    const int o = mtile * TC_M + (warp & 3) * 32 + lane;     // (only warps 0-3 use it)
    int* red = reinterpret_cast<int*>(base);                 // [rows][128] partial sums; the ring is free by then
    if (warp < 4) {
        ok = __all_sync(0xffffffffu, ok);
        if (ok && !mbar_wait(smem_u32(&S->done), 0, p.wait_limit)) { ok = false; atomicOr(p.errw, ERRW_TIMEOUT); }
        ok = ok && *(volatile int*)&S->last != -1;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        if (ok) {
            for (int c0 = 0; c0 < p.bn; c0 += 32) {
                uint32_t v[32];
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
                #pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int row = c0 + j;
                    if (row >= p.rows) break;
                    if (p.ksplit == 1) { if (o < p.c_out) ft_finish(p, row, o, (int)v[j]); }
                    else if (CLUSTER) red[row * TC_M + (warp & 3) * 32 + lane] = (int)v[j];
                    else atomicAdd(p.acc + (size_t)row * (gridDim.x * TC_M) + o, (int)v[j]);
                }
            }
        }
        if (!CLUSTER) __threadfence();                       // the partial sums are out before the arrival below
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5 && lane == 0 && (!ok || S->last == -1)) {
        // a role gave up: the loader's copies still in flight must land before the CTA's shared memory goes away
        for (int j = max(0, n_loaded - p.stages); j < n_loaded; ++j)
            mbar_wait(smem_u32(&S->full[j % p.stages]), (j / p.stages) & 1, WAIT_LIMIT_DEFAULT);
    }
    if (warp == 4)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)p.tmem_cols) : "memory");
    if (p.ksplit == 1) return;

    if (CLUSTER) {
        // ================= every CTA of the cluster closes its share of the rows: row r belongs to rank r mod ksplit
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        uint32_t rank;
        asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
        const int my_rows = (p.rows - (int)rank + p.ksplit - 1) / p.ksplit;
        const uint32_t red_u32 = smem_u32(red);
        for (int i = tid; i < my_rows * (TC_M / 4); i += FT_THREADS) {
            const int row = (int)rank + (i / (TC_M / 4)) * p.ksplit, o4 = (i % (TC_M / 4)) * 4;
            int4 w = make_int4(0, 0, 0, 0);
            for (int c = 0; c < p.ksplit; ++c) {
                uint32_t remote;
                int4 t;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(red_u32 + (uint32_t)(row * TC_M + o4) * 4u), "r"(c));
                asm volatile("ld.shared::cluster.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(t.x), "=r"(t.y), "=r"(t.z), "=r"(t.w) : "r"(remote) : "memory");
                w.x += t.x; w.y += t.y; w.z += t.z; w.w += t.w;
            }
            const int oo = mtile * TC_M + o4;
            if (oo < p.c_out) ft_finish4(p, row, oo, w);
        }
        // nobody leaves while its shared memory may still be read
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        return;
    }

    // ================= the last CTA of this output block closes it
    if (tid == 0) S->last = atomicAdd(p.arrive + mtile, 1u) == (unsigned)p.ksplit - 1u;   // (overwrites a give-up mark)
    __syncthreads();
    if (!S->last) return;
    __threadfence();
    // (c_out is a multiple of 16 here, so a group of 4 outputs is inside or outside as a whole; the loads of
    // a batch are all issued before the first store, which the compiler cannot do across possible aliases)
    const int ld = gridDim.x * TC_M;
    const int total4 = p.rows * (TC_M / 4);
    constexpr int FB = 6;
    for (int i0 = tid; i0 < total4; i0 += FT_THREADS * FB) {
        int4 v[FB];
        #pragma unroll
        for (int u = 0; u < FB; ++u) {
            const int i = i0 + u * FT_THREADS;
            if (i < total4) v[u] = __ldcg(reinterpret_cast<const int4*>(p.acc + (size_t)(i / (TC_M / 4)) * ld + mtile * TC_M + (i % (TC_M / 4)) * 4));
        }
        #pragma unroll
        for (int u = 0; u < FB; ++u) {
            const int i = i0 + u * FT_THREADS;
            if (i >= total4) continue;
            const int row = i / (TC_M / 4), oo = mtile * TC_M + (i % (TC_M / 4)) * 4;
            *reinterpret_cast<int4*>(p.acc + (size_t)row * ld + oo) = make_int4(0, 0, 0, 0);
            if (oo < p.c_out) ft_finish4(p, row, oo, v[u]);
        }
    }
    if (tid == 0) p.arrive[mtile] = 0;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct FtPlan { int ksplit, per; };

static FtPlan ft_plan(const Layer& L)
{
    FtPlan f;
    int ks = 148 / L.tc_ntiles;
    ks = ks < 1 ? 1 : (ks > L.tc_slabs ? L.tc_slabs : ks);
    f.per = ceil_div(L.tc_slabs, ks);
    f.ksplit = ceil_div(L.tc_slabs, f.per);
    return f;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (the library does not link the driver)
typedef CUresult (*ft_encode_t)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static ft_encode_t ft_encoder()
{
    static ft_encode_t fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            f = nullptr;
        }
        return reinterpret_cast<ft_encode_t>(f);
    }();
    return fn;
}

static void ft_cluster_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* at, int tiles, int ksplit, size_t dyn, cudaStream_t st)
{
    cfg.gridDim = dim3(tiles, ksplit);
    cfg.blockDim = dim3(FT_THREADS);
    cfg.dynamicSmemBytes = dyn;
    cfg.stream = st;
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = ksplit; at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
}

int fc_tc_launches(int rows) { return ceil_div(rows, FT_MAX_ROWS); }

bool fc_tc_usable(const Layer& L, int rows)
{
    return L.tc_ready && L.tc_bn == TC_M && L.ft_acc && rows <= FT_MAX_LAUNCHES * FT_MAX_ROWS && L.d.c_in % 16 == 0;
}

int fc_tc_create(rrm_net* net, Layer& L)
{
    if (!L.tc_ready || L.tc_bn != TC_M || !ft_encoder()) return RRM_OK;
    const size_t acc_bytes = (size_t)FT_MAX_ROWS * L.tc_ntiles * TC_M * 4, arr_bytes = (size_t)L.tc_ntiles * 4;
    void* a = nullptr;
    if (cudaMalloc(&a, acc_bytes + arr_bytes) != cudaSuccess) { cudaGetLastError(); return RRM_ERR_ALLOC; }
    net->allocs.push_back(a);
    RRM_CUDA_TRY(cudaMemset(a, 0, acc_bytes + arr_bytes));
    L.ft_acc = reinterpret_cast<int32_t*>(a);
    L.ft_arrive = reinterpret_cast<unsigned*>(reinterpret_cast<char*>(a) + acc_bytes);
    RRM_CUDA_TRY(cudaFuncSetAttribute(fc_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(FT_SMEM_BUDGET + 2048)));
    RRM_CUDA_TRY(cudaFuncSetAttribute(fc_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(FT_SMEM_BUDGET + 2048)));
    // the K shares of an output block as one cluster, when all clusters of the grid can be resident at once
    const FtPlan f = ft_plan(L);
    L.ft_cluster = false;
    if (f.ksplit > 1 && f.ksplit <= 8) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        ft_cluster_config(cfg, at, L.tc_ntiles, f.ksplit, FT_SMEM_BUDGET + 2048, nullptr);
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, fc_tc_kernel<true>, &cfg) == cudaSuccess) L.ft_cluster = clusters >= L.tc_ntiles;
        else cudaGetLastError();
        if (getenv("RRM_DEBUG")) fprintf(stderr, "rrm: few-row FC: %d tiles x %d K shares, %d clusters can be resident -> %s\n", L.tc_ntiles, f.ksplit, clusters, L.ft_cluster ? "cluster" : "global scratch");
    }
    return RRM_OK;
}

// rows = frames x streams, frame-major.  stateless: Y only.  Otherwise the stored projection and the
// input snapshot become those of the last frame (the last n rows).  stat (may be null, not with stateless)
// receives per row the counters of the delta against the row n before it (the snapshot for the first n).
int fc_tc_run(rrm_net* net, Layer& L, const void* X_dev, void* Y_dev, int rows, bool stateless, unsigned* stat, cudaStream_t st)
{
    const int C = L.d.c_in, K = L.d.c_out, n = L.d.n;
    if (reinterpret_cast<uintptr_t>(X_dev) & 15) return RRM_ERR_INVALID_ARG;    // the copy engine wants 16-byte aligned rows
    const FtPlan f = ft_plan(L);
    FtParams p;
    p.Wimg = L.tc_Wimg;
    p.bias = reinterpret_cast<const int32_t*>(L.bias);
    p.acc = L.ft_acc; p.arrive = L.ft_arrive;
    p.errw = net->errw;
    p.c_in = C; p.c_out = K; p.slabs = L.tc_slabs; p.per = f.per; p.ksplit = f.ksplit;
    p.shift = L.d.shift; p.act = L.d.act;
    p.wait_limit = net->opt.wait_limit;
    const size_t ybytes = (size_t)K * (L.d.shift < 0 ? 4 : 1);
    const int state_row = rows - n;                          // first row of the last frame
    const int8_t* old_snap = L.xs[L.xs_cur];
    p.n = n;
    if (!stateless) L.xs_cur ^= 1;
    // even pieces rather than full ones and a remainder (every launch streams W again, from L2 when it fits)
    const int pieces = ceil_div(rows, FT_MAX_ROWS);
    const int piece_max = ceil_div(rows, pieces);
    for (int r0 = 0; r0 < rows; r0 += piece_max) {
        const int piece = rows - r0 < piece_max ? rows - r0 : piece_max;
        p.rows = piece;
        p.bn = (piece + 15) & ~15;
        p.tmem_cols = p.bn <= 32 ? 32 : (p.bn <= 64 ? 64 : (p.bn <= 128 ? 128 : 256));
        const size_t stage_bytes = (size_t)FT_A_BYTES + (size_t)p.bn * FT_SLAB;
        const int stages = (int)(FT_SMEM_BUDGET / stage_bytes);
        p.stages = stages > FT_MAX_STAGES ? FT_MAX_STAGES : stages;
        p.X = reinterpret_cast<const int8_t*>(X_dev) + (size_t)r0 * C;
        p.Y = Y_dev ? reinterpret_cast<char*>(Y_dev) + (size_t)r0 * ybytes : nullptr;
        // rows of the last frame inside this piece update the state
        const bool has_state = !stateless && r0 + piece > state_row;
        p.state_from = has_state ? (state_row > r0 ? state_row - r0 : 0) : piece;
        const int state_off = has_state ? (r0 + p.state_from) - state_row : 0;     // stream index of the first state row
        p.Pstate = has_state ? reinterpret_cast<int32_t*>(L.P) + (size_t)state_off * K : nullptr;
        p.snap = has_state ? L.xs[L.xs_cur] + (size_t)state_off * C : nullptr;
        p.stat = stat && !stateless ? stat + (size_t)r0 * 2 : nullptr;
        p.xprev = r0 == 0 ? old_snap : reinterpret_cast<const int8_t*>(X_dev) + (size_t)(r0 - n) * C;
        // the piece's rows as a 2-D byte tensor [rows][c_in]; a box is one slab of all rows, swizzled on the way in
        CUtensorMap tm;
        const cuuint64_t dims[2] = {(cuuint64_t)C, (cuuint64_t)piece};
        const cuuint64_t strides[1] = {(cuuint64_t)C};
        const cuuint32_t box[2] = {(cuuint32_t)FT_SLAB, (cuuint32_t)p.bn};
        const cuuint32_t es[2] = {1, 1};
        if (ft_encoder()(&tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(p.X), dims, strides, box, es,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return RRM_ERR_CUDA;
        const size_t dyn = 1024 + (size_t)p.stages * stage_bytes + sizeof(FtSmemTail);
        if (L.ft_cluster) {
            cudaLaunchConfig_t cfg = {};
            cudaLaunchAttribute at[1];
            ft_cluster_config(cfg, at, L.tc_ntiles, f.ksplit, dyn, st);
            RRM_CUDA_TRY(cudaLaunchKernelEx(&cfg, fc_tc_kernel<true>, p, tm));
        } else {
            fc_tc_kernel<false><<<dim3(L.tc_ntiles, f.ksplit), FT_THREADS, dyn, st>>>(p, tm);
        }
    }
    RRM_CUDA_TRY(cudaGetLastError());
    return RRM_OK;
}

}  // namespace rrm
