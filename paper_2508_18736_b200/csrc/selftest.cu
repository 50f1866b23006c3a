// Diagnostics of the library that touch no cache contents:
//   siso_selftest_wait_timeout  lets the bounded mbarrier wait of the tensor-core kernels run out on purpose, on a
//                               barrier that nothing will ever arrive on and with nothing in flight, so that the
//                               path "wait gives up -> SISO_ERR_TIMEOUT in the status word -> normal return" can be
//                               exercised without disturbing a real sweep;
//   siso_measure_fp32_fma       the FP32 FMA rate the CUDA cores of this device sustain, the roof that the
//                               CUDA-core sweeps are measured against.
#include "umma_pair.cuh"

namespace siso {
namespace {

// One warp.  Thread 0 initialises a barrier that expects one arrival, nobody arrives, and the wait shared with the
// sweep kernels (umma2::mbar_wait) polls it `limit` times.  What follows is what those kernels do when a wait
// gives up: first error wins in the status word, then a normal return.  polls_out receives the outcome for the
// caller to see (1 = the wait gave up, 0 = it returned as if the barrier had completed).
__global__ void wait_timeout_kernel(int *status, uint32_t limit, int *gave_up_out) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        umma2::mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool done = umma2::mbar_wait(&bar, 0, &abort_flag, limit);
        if (!done) set_status(status, SISO_ERR_TIMEOUT);
        if (gave_up_out) *gave_up_out = done ? 0 : 1;
    }
}

constexpr int FMA_THREADS = 256;
constexpr int FMA_CHAINS = 8;
constexpr int FMA_INNER = 64;

// FMA_CHAINS independent dependency chains per thread keep the FP32 pipes full; the result is written so that the
// loop cannot be removed.
__global__ void __launch_bounds__(FMA_THREADS) fp32_fma_kernel(float *sink, int outer, float a, float b) {
    float x[FMA_CHAINS];
#pragma unroll
    for (int i = 0; i < FMA_CHAINS; ++i) x[i] = static_cast<float>(threadIdx.x + i);
    for (int o = 0; o < outer; ++o) {
#pragma unroll
        for (int r = 0; r < FMA_INNER; ++r) {
#pragma unroll
            for (int i = 0; i < FMA_CHAINS; ++i) x[i] = fmaf(x[i], a, b);
        }
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < FMA_CHAINS; ++i) s += x[i];
    if (s == 12345.678f) sink[0] = s;      // practically never true; keeps the chains alive
}

}  // namespace
}  // namespace siso

using namespace siso;

extern "C" siso_status_t siso_selftest_wait_timeout(siso_cache_t *c, uint32_t poll_limit, int32_t *d_gave_up, void *stream) {
    Cache *cc = reinterpret_cast<Cache *>(c);
    if (!cc || poll_limit < 1 || poll_limit > (1u << 20)) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(cc->device));
    wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(cc->status, poll_limit, d_gave_up);
    SISO_LAUNCHED(cc);
    return SISO_OK;
}

extern "C" siso_status_t siso_measure_fp32_fma(siso_cache_t *c, double *h_tflops, void *stream) {
    Cache *cc = reinterpret_cast<Cache *>(c);
    if (!cc || !h_tflops) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(cc->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Scratch scr;
    SISO_TRY(scratch_reserve(cc, 256, s, &scr));
    float *sink = scr.take<float>(1);
    const int grid = cc->sm_count * 8, outer = 512;
    cudaEvent_t e0, e1;
    SISO_CUDA(cudaEventCreate(&e0));
    SISO_CUDA(cudaEventCreate(&e1));
    double best_ms = 1e30;
    siso_status_t st = SISO_OK;
    for (int rep = 0; rep < 4 && st == SISO_OK; ++rep) {      // the first repetition warms up
        cudaEventRecord(e0, s);
        fp32_fma_kernel<<<grid, FMA_THREADS, 0, s>>>(sink, outer, 0.999f, 0.001f);
        cc->launches += 1;
        cudaEventRecord(e1, s);
        st = check_cuda(cudaEventSynchronize(e1), "fp32 fma probe");
        float ms = 0.f;
        if (st == SISO_OK) st = check_cuda(cudaEventElapsedTime(&ms, e0, e1), "fp32 fma probe");
        if (rep > 0 && ms > 0.f && ms < best_ms) best_ms = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (st != SISO_OK) return st;
    const double flop = 2.0 * grid * FMA_THREADS * static_cast<double>(outer) * FMA_INNER * FMA_CHAINS;
    *h_tflops = flop / (best_ms * 1e-3) / 1e12;
    return SISO_OK;
}
