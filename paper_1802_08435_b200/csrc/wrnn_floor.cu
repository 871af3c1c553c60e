// Exchange-floor measurement: the latency of one chip-wide all-gather of K tagged fp32 values through L2,
// in an otherwise empty persistent kernel with the same CTA shape as the resident sampling kernel.
// Section 2.1 names the synchronisation between multiprocessors as the overhead that remains once the
// weights are resident; this is that cost on the device at hand, measured rather than assumed.  The
// batch-1 roofline of the benchmark is "weight bytes / shared-memory bandwidth + 2 x this".
#include "wrnn_internal.h"

namespace wrnn {

// gap: cycles between a CTA's own publication and its first poll (0 = poll at once).  A poll that reaches L2 before the
// words do costs a whole round trip before the same thread can look again, and early polls load the L2 slices the
// publishing stores have to get through; the sampling kernels hold their pollers back the same way.
__global__ void exchange_floor_kernel(unsigned long long *slots, int K, int U, int iters, int gap, int *err)
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
        if (gap > 0) { const long long c0 = clock64(); while (clock64() - c0 < gap) { } }
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
    float ms = 0.f, best_ms = 0.f;
    // repetition 0 warms up; 1: pollers start at once; 2: pollers held back (the protocol of the sampling kernels); the
    // smaller of the two is reported
    for (int rep = 0; rep < 3 && rc == WRNN_OK; ++rep) {
        int gap = rep == 2 ? 150 : 0;
        cudaMemset(slots, 0, (size_t)2 * K * 8);
        cudaMemset(err, 0, 4);
        void *args[] = {(void *)&slots, (void *)&K, (void *)&U, (void *)&iters, (void *)&gap, (void *)&err};
        cudaEventRecord(e0, 0);
        if (cudaLaunchCooperativeKernel((void *)exchange_floor_kernel, dim3(n_ctas), dim3(n_threads), args, 0, 0) != cudaSuccess) {
            cudaGetLastError(); rc = WRNN_ERR_CUDA; break;
        }
        ++g_launches;
        cudaEventRecord(e1, 0);
        if (cudaEventSynchronize(e1) != cudaSuccess) { rc = WRNN_ERR_CUDA; break; }
        cudaEventElapsedTime(&ms, e0, e1);
        if (rep == 1 || (rep == 2 && ms < best_ms)) best_ms = ms;
        int herr = 0;
        cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
        if (herr) rc = WRNN_ERR_TIMEOUT;
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    cudaFree(slots); cudaFree(err);
    if (rc == WRNN_OK) *ns_per_exchange = best_ms * 1e6f / (float)iters;
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

// ---------------------------------------------------------------------------------------------
// Shared-memory stream rate: every SM reads a resident buffer of the size the sampling kernels keep their weights in,
// over and over, with 16-byte loads from all its threads (what the resident kernels' product phases do with their
// weight shards, minus the arithmetic).  The aggregate rate is the measured counterpart of the nominal
// SMs x 128 B/clk x clock that bounds "every resident weight read once per step" (Section 2.1: the weights stay on chip).
namespace wrnn {
__global__ void smem_stream_kernel(int bytes, int iters, unsigned *sink)
{
    extern __shared__ uint4 sbuf[];
    const int n16 = bytes / 16;
    for (int i = threadIdx.x; i < n16; i += blockDim.x) sbuf[i] = make_uint4(i, i + 1, i + 2, i + 3);
    __syncthreads();
    unsigned a0 = 0, a1 = 0, a2 = 0, a3 = 0;
    const unsigned base = (unsigned)__cvta_generic_to_shared(sbuf);
    for (int it = 0; it < iters; ++it) {
        // four independent loads per pass keep the load/store unit busy; consecutive lanes read consecutive 16-byte pieces
        int i = threadIdx.x;
        for (; i + 3 * (int)blockDim.x < n16; i += 4 * blockDim.x) {
            uint4 v0, v1, v2, v3;
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v0.x), "=r"(v0.y), "=r"(v0.z), "=r"(v0.w) : "r"(base + 16u * i));
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v1.x), "=r"(v1.y), "=r"(v1.z), "=r"(v1.w) : "r"(base + 16u * (i + blockDim.x)));
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v2.x), "=r"(v2.y), "=r"(v2.z), "=r"(v2.w) : "r"(base + 16u * (i + 2 * blockDim.x)));
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v3.x), "=r"(v3.y), "=r"(v3.z), "=r"(v3.w) : "r"(base + 16u * (i + 3 * blockDim.x)));
            a0 ^= v0.x ^ v1.y ^ v2.z ^ v3.w; a1 ^= v0.y ^ v1.z ^ v2.w ^ v3.x;
            a2 ^= v0.z ^ v1.w ^ v2.x ^ v3.y; a3 ^= v0.w ^ v1.x ^ v2.y ^ v3.z;
        }
        for (; i < n16; i += blockDim.x) {
            uint4 v;
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(base + 16u * i));
            a0 ^= v.x; a1 ^= v.y; a2 ^= v.z; a3 ^= v.w;
        }
    }
    if ((a0 ^ a1 ^ a2 ^ a3) == 0x9e3779b9u && iters < 0) sink[blockIdx.x] = a0;       // keeps the loads alive; never taken
}
}  // namespace wrnn

extern "C" int wrnn_measure_smem_stream(int32_t n_ctas, int32_t n_threads, int32_t bytes_per_cta, int32_t iters, float *gb_per_s)
{
    if (n_ctas < 1 || n_threads < 32 || n_threads > 1024 || n_threads % 32 != 0 || bytes_per_cta < 1024 || bytes_per_cta % 16 != 0 ||
        bytes_per_cta > 227 * 1024 || iters < 1 || !gb_per_s)
        return WRNN_ERR_INVALID_ARG;
    if (cudaFuncSetAttribute(wrnn::smem_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes_per_cta) != cudaSuccess) {
        cudaGetLastError();
        return WRNN_ERR_UNSUPPORTED;
    }
    unsigned *sink = nullptr;
    if (cudaMalloc((void **)&sink, (size_t)n_ctas * 4) != cudaSuccess) { cudaGetLastError(); return WRNN_ERR_NOMEM; }
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    int rc = WRNN_OK;
    float ms = 0.f;
    for (int rep = 0; rep < 2 && rc == WRNN_OK; ++rep) {             // first repetition warms up
        cudaEventRecord(e0, 0);
        wrnn::smem_stream_kernel<<<n_ctas, n_threads, bytes_per_cta>>>(bytes_per_cta, iters, sink);
        if (cudaGetLastError() != cudaSuccess) { rc = WRNN_ERR_CUDA; break; }
        ++wrnn::g_launches;
        cudaEventRecord(e1, 0);
        if (cudaEventSynchronize(e1) != cudaSuccess) { rc = WRNN_ERR_CUDA; break; }
        cudaEventElapsedTime(&ms, e0, e1);
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    cudaFree(sink);
    if (rc == WRNN_OK) *gb_per_s = (float)((double)n_ctas * bytes_per_cta * iters / (ms * 1e-3) / 1e9);
    return rc;
}
