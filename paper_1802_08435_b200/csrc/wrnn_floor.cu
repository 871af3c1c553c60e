// Exchange-floor measurement: the latency of one chip-wide all-gather of K tagged fp32 values through L2,
// in an otherwise empty persistent kernel with the same CTA shape as the resident sampling kernel.
// Section 2.1 names the synchronisation between multiprocessors as the overhead that remains once the
// weights are resident; this is that cost on the device at hand, measured rather than assumed.  The
// batch-1 roofline of the benchmark is "weight bytes / shared-memory bandwidth + 2 x this".
#include "wrnn_internal.h"

namespace wrnn {

__global__ void exchange_floor_kernel(unsigned long long *slots, int K, int U, int iters, int *err)
{
    __shared__ float sh[2048];
    float acc = 0.f;
    for (int it = 0; it < iters; ++it) {
        unsigned long long *buf = slots + (size_t)(it & 1) * K;
        const unsigned tag = (unsigned)(it + 1);
        if (threadIdx.x < U) {
            const unsigned long long v = ((unsigned long long)tag << 32) | __float_as_uint(acc + (float)threadIdx.x);
            asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(buf + blockIdx.x * U + threadIdx.x), "l"(v) : "memory");
        }
        bool bad = false;
        for (int i = threadIdx.x; i < K; i += blockDim.x) {
            unsigned long long v;
            unsigned n = 0;
            while (true) {
                asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(buf + i) : "memory");
                if ((unsigned)(v >> 32) == tag) break;
                if (++n > (1u << 22)) { bad = true; break; }       // bounded: give up instead of hanging
            }
            sh[i & 2047] = __uint_as_float((unsigned)v);
        }
        if (__syncthreads_or(bad)) { if (threadIdx.x == 0) *err = 1; return; }
        acc = sh[(threadIdx.x * 7) % (K < 2048 ? K : 2048)] * 1e-9f;
        __syncthreads();
    }
}

}  // namespace wrnn

using namespace wrnn;

extern "C" int wrnn_measure_exchange_floor(int32_t n_ctas, int32_t n_threads, int32_t K, int32_t iters, float *ns_per_exchange)
{
    if (n_ctas < 1 || n_threads < 32 || n_threads > 1024 || K < n_ctas || K % n_ctas != 0 || K > 65536 || iters < 1 || !ns_per_exchange)
        return WRNN_ERR_INVALID_ARG;
    int U = K / n_ctas;
    if (U > n_threads) return WRNN_ERR_INVALID_ARG;
    unsigned long long *slots = nullptr;
    int *err = nullptr;
    if (cudaMalloc((void **)&slots, (size_t)2 * K * 8) != cudaSuccess || cudaMalloc((void **)&err, 4) != cudaSuccess) {
        cudaGetLastError(); cudaFree(slots); return WRNN_ERR_NOMEM;
    }
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    int rc = WRNN_OK;
    float ms = 0.f;
    for (int rep = 0; rep < 2 && rc == WRNN_OK; ++rep) {             // first repetition warms up
        cudaMemset(slots, 0, (size_t)2 * K * 8);
        cudaMemset(err, 0, 4);
        void *args[] = {(void *)&slots, (void *)&K, (void *)&U, (void *)&iters, (void *)&err};
        cudaEventRecord(e0, 0);
        if (cudaLaunchCooperativeKernel((void *)exchange_floor_kernel, dim3(n_ctas), dim3(n_threads), args, 0, 0) != cudaSuccess) {
            cudaGetLastError(); rc = WRNN_ERR_CUDA; break;
        }
        ++g_launches;
        cudaEventRecord(e1, 0);
        if (cudaEventSynchronize(e1) != cudaSuccess) { rc = WRNN_ERR_CUDA; break; }
        cudaEventElapsedTime(&ms, e0, e1);
        int herr = 0;
        cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
        if (herr) rc = WRNN_ERR_TIMEOUT;
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    cudaFree(slots); cudaFree(err);
    if (rc == WRNN_OK) *ns_per_exchange = ms * 1e6f / (float)iters;
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded waits: two CTAs, the first waits at the grid barrier for an arrival that never comes
// (the second returns at once), gives up after limit_ns, records where, and returns; the context stays usable.
namespace wrnn {
__global__ void bounded_wait_selftest_kernel(unsigned long long *counter, DevStatus *status, unsigned long long limit_ns)
{
    if (blockIdx.x != 0) return;
    GridBarrier bar{counter, status, 0ull, limit_ns};
    bar.sync(7, 3);
}
}  // namespace wrnn

extern "C" int wrnn_selftest_bounded_wait(int64_t limit_ns, int32_t *code, int32_t *cta, int32_t *step, int32_t *phase, float *waited_ms)
{
    if (limit_ns < 1000 || limit_ns > 1000000000ll || !code) return WRNN_ERR_INVALID_ARG;
    unsigned long long *counter = nullptr;
    wrnn::DevStatus *status = nullptr;
    if (cudaMalloc((void **)&counter, 8) != cudaSuccess || cudaMalloc((void **)&status, sizeof(wrnn::DevStatus)) != cudaSuccess) {
        cudaGetLastError(); cudaFree(counter); return WRNN_ERR_NOMEM;
    }
    cudaMemset(counter, 0, 8);
    cudaMemset(status, 0, sizeof(wrnn::DevStatus));
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    cudaEventRecord(e0, 0);
    wrnn::bounded_wait_selftest_kernel<<<2, 64>>>(counter, status, (unsigned long long)limit_ns);
    ++wrnn::g_launches;
    cudaEventRecord(e1, 0);
    int rc = cudaEventSynchronize(e1) == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
    float ms = 0.f;
    wrnn::DevStatus h = {0, 0, 0, 0};
    if (rc == WRNN_OK) {
        cudaEventElapsedTime(&ms, e0, e1);
        if (cudaMemcpy(&h, status, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) rc = WRNN_ERR_CUDA;
    }
    *code = h.code;
    if (cta) *cta = h.cta;
    if (step) *step = h.step;
    if (phase) *phase = h.phase;
    if (waited_ms) *waited_ms = ms;
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    cudaFree(counter); cudaFree(status);
    cudaGetLastError();
    return rc;
}

