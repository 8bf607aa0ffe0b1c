// Measured peak rates of the plain ALU pipes that bound the CUDA-core kernels of the library (the fp32,
// tiny-channel int8 and binary forms of conv_gemm_kernel, the column products of the delta-FC kernels):
// register-only loops of independent FFMA, dp4a and popc chains on every SM, timed with CUDA events.
// The roofline of an ALU-bound kernel is quoted against these figures instead of unit counts x clock.
#include "rrm_common.cuh"

namespace rrm {

constexpr int PROBE_THREADS = 256;
constexpr int PROBE_CHAINS = 8;               // independent dependency chains per thread
constexpr int PROBE_ITERS = 1024;             // loop trips; each does PROBE_CHAINS x 4 operations per thread

// KIND 0: fp32 fused multiply-add; 1: dp4a (four int8 multiply-accumulates); 2: popc of a 32-bit word and an add
// (32 one-bit multiply-accumulates, the inner operation of the binary convolution).
template <int KIND>
__global__ void __launch_bounds__(PROBE_THREADS) alu_probe_kernel(unsigned seed, unsigned* sink)
{
    float f[PROBE_CHAINS];
    int a[PROBE_CHAINS];
    const unsigned t = blockIdx.x * blockDim.x + threadIdx.x;
    #pragma unroll
    for (int c = 0; c < PROBE_CHAINS; ++c) { f[c] = (float)(t + c) * 1e-9f; a[c] = (int)(t * 2654435761u + c + seed); }
    const float m = 1.0f + (float)seed * 1e-12f, d = (float)seed * 1e-20f;
    const int w = (int)(seed | 0x01010101u);
    for (int i = 0; i < PROBE_ITERS; ++i) {
        #pragma unroll
        for (int u = 0; u < 4; ++u) {
            #pragma unroll
            for (int c = 0; c < PROBE_CHAINS; ++c) {
                if (KIND == 0) f[c] = fmaf(f[c], m, d);
                else if (KIND == 1) a[c] = __dp4a(a[c], w, a[c]);
                else a[c] += __popc((unsigned)a[c] ^ (unsigned)w);
            }
        }
    }
    unsigned r = 0;
    #pragma unroll
    for (int c = 0; c < PROBE_CHAINS; ++c) r += (KIND == 0) ? __float_as_uint(f[c]) : (unsigned)a[c];
    if (r == 0x9e3779b9u && seed == 0xffffffffu) *sink = r;        // never true for the seeds used: keeps the chains alive
}

template <int KIND>
static int probe_run(double* ops_per_s)
{
    int dev = 0, sms = 0;
    RRM_CUDA_TRY(cudaGetDevice(&dev));
    RRM_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    unsigned* sink = nullptr;
    RRM_CUDA_TRY(cudaMalloc(&sink, 4));
    cudaEvent_t e0, e1;
    RRM_CUDA_TRY(cudaEventCreate(&e0));
    RRM_CUDA_TRY(cudaEventCreate(&e1));
    const int blocks = sms * 8;                               // 8 x 256 threads = every warp slot of an SM
    double best = 0.0;
    for (int rep = 0; rep < 4; ++rep) {                       // the first repetitions also serve as warm-up
        cudaEventRecord(e0);
        alu_probe_kernel<KIND><<<blocks, PROBE_THREADS>>>(17u + rep, sink);
        cudaEventRecord(e1);
        if (cudaEventSynchronize(e1) != cudaSuccess) break;
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double ops = (double)blocks * PROBE_THREADS * PROBE_ITERS * 4.0 * PROBE_CHAINS;
        if (ms > 0.f && ops / (ms * 1e-3) > best) best = ops / (ms * 1e-3);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(sink);
    RRM_CUDA_TRY(cudaGetLastError());
    *ops_per_s = best;
    return RRM_OK;
}

}  // namespace rrm

extern "C" int rrm_measure_alu_peak(int kind, double* macs_per_s)
{
    if (!macs_per_s || kind < 0 || kind > 2) return RRM_ERR_INVALID_ARG;
    double ops = 0.0;
    int s;
    if (kind == 0) s = rrm::probe_run<0>(&ops);
    else if (kind == 1) s = rrm::probe_run<1>(&ops);
    else s = rrm::probe_run<2>(&ops);
    if (s != RRM_OK) return s;
    *macs_per_s = ops * (kind == 0 ? 1.0 : (kind == 1 ? 4.0 : 32.0));
    return RRM_OK;
}
