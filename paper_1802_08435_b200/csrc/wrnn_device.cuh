// Device-side helpers shared by the WaveRNN kernels: counter-based uniforms,
// gate non-linearities, warp reductions, the 256-way softmax draw and bounded
// grid-wide waits.  sm_100a only.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace wrnn {

constexpr unsigned FULL = 0xffffffffu;

// Status word written by a kernel that gave up on a bounded wait: {code, cta, step, phase}.
struct DevStatus { int code; int cta; int step; int phase; };
constexpr int DEV_OK = 0;
constexpr int DEV_TIMEOUT = 5;      // == WRNN_ERR_TIMEOUT
constexpr int DEV_CHECK = 6;        // == WRNN_ERR_CHECK: the checked build found an index outside its array or a clobbered guard

// ------------------------------------------------------------------ Philox4x32-10
// Counter-based generator of Salmon et al. (SC'11).  One call per (row, step, head).
__device__ __forceinline__ uint32_t philox_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0;
}

// Uniform in [0,1), a multiple of 2^-24, keyed by (seed, global row id, absolute step, head).
__device__ __forceinline__ float uniform24(uint64_t seed, uint32_t row, uint64_t step, uint32_t head)
{
    const uint32_t w = philox_word0((uint32_t)step, head, row, (uint32_t)(step >> 32),
                                    (uint32_t)seed, (uint32_t)(seed >> 32));
    return (float)(w >> 8) * (1.0f / 16777216.0f);
}

// ------------------------------------------------------------------ scalar maths
// 8-bit value scaled to [-1, 1] (paragraph after Eq. 2): 0 -> -1, 255 -> +1.
__device__ __forceinline__ float scale8(int v) { return (float)v * (1.0f / 127.5f) - 1.0f; }

// Accurate forms (expf / tanhf, not the .approx instructions): the parity bound on
// gates is 1e-4 relative and the drawn index depends on them.
__device__ __forceinline__ float sigmoidf_acc(float x) { return 1.0f / (1.0f + expf(-x)); }

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// ------------------------------------------------------------------ warp reductions
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(FULL, v, o));
    return v;
}

// Reduce N per-lane partial sums (N a power of two <= 32) across the warp so that
// every lane l ends up with the total of element (l & (N-1)) in v[0].
// N-1 + log2(32/N) shuffles instead of 5 N.
template <int N>
__device__ __forceinline__ float warp_reduce_scatter(float (&v)[N], int lane)
{
#pragma unroll
    for (int off = N / 2; off >= 1; off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < off; ++i) {
            const float send = upper ? v[i] : v[i + off];
            const float keep = upper ? v[i + off] : v[i];
            v[i] = keep + __shfl_xor_sync(FULL, send, off);
        }
    }
    float r = v[0];
#pragma unroll
    for (int off = N; off < 32; off <<= 1) r += __shfl_xor_sync(FULL, r, off);
    return r;
}

// ------------------------------------------------------------------ softmax + inverse-CDF draw
// One warp, 256 logits, lane l holds logits [8l, 8l+8).  Returns (on every lane) the
// smallest k whose running sum of exp(l_k - max) exceeds u * total; 255 if none does.
__device__ __forceinline__ int warp_softmax_draw(const float (&l)[8], float u, int lane)
{
    float m = l[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) m = fmaxf(m, l[i]);
    m = warp_max(m);
    float w[8], s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) { w[i] = expf(l[i] - m); s += w[i]; }
    // inclusive scan of the per-lane sums
    float inc = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += t;
    }
    const float total = __shfl_sync(FULL, inc, 31);
    const float thr = u * total;
    float run = inc - s;                 // exclusive prefix of this lane
    int pick = 256;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        run += w[i];
        if (pick == 256 && run > thr) pick = 8 * lane + i;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) pick = min(pick, __shfl_xor_sync(FULL, pick, o));
    return pick == 256 ? 255 : pick;
}

// Latency-lean variant for the single-stream kernel, where this sits on the per-step critical path:
// one integer redux for the max and for the pick instead of ten shuffles, exp through ex2.approx
// (relative error about 2^-21 on arguments in [-88, 0], far inside the 1e-5 CDF margin that index
// parity allows).  Same contract as warp_softmax_draw.
__device__ __forceinline__ int float_order_key(float x)
{
    const int i = __float_as_int(x);
    return i ^ ((i >> 31) & 0x7fffffff);          // signed-integer order == float order
}
// SCAN = false: exclusive prefix and grand total of the lane sums by one five-step butterfly (no broadcast after the scan;
// the shorter chain where the drawing warp is alone on the critical path: the lean single-stream kernel).  SCAN = true: an
// inclusive shuffle-up scan and a broadcast of the last lane's total (fewer instructions; faster where several warps draw
// at once or other warps compete for issue slots: measured per kernel).  The two orders of summation differ in rounding only.
template <bool SCAN>
__device__ __forceinline__ int warp_softmax_draw_impl(const float (&l)[8], float u, int lane)
{
    // (pairwise trees instead of chains: this sits on the critical path of every half-step)
    float m = fmaxf(fmaxf(fmaxf(l[0], l[1]), fmaxf(l[2], l[3])), fmaxf(fmaxf(l[4], l[5]), fmaxf(l[6], l[7])));
    const int km = __reduce_max_sync(FULL, float_order_key(m));
    m = __int_as_float(km ^ ((km >> 31) & 0x7fffffff));
    float w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = __expf(l[i] - m);
    // running sums inside the lane: p[i] = w[0] + ... + w[i]
    const float p1 = w[0] + w[1], p3 = p1 + (w[2] + w[3]), p5 = p3 + (w[4] + w[5]), p7 = p5 + (w[6] + w[7]);
    const float p0 = w[0], p2 = p1 + w[2], p4 = p3 + w[4], p6 = p5 + w[6];
    // butterfly over the lanes: after step o every lane holds the total of its block of 2 o lanes and, in `run`, the sum of
    // the lanes of that block below itself -- the exclusive prefix and the grand total in five shuffles, no broadcast after
    float tot = p7, run = 0.f;
    if (SCAN) {
        float inc = p7;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(FULL, inc, o);
            if (lane >= o) inc += t;
        }
        tot = __shfl_sync(FULL, inc, 31);
        run = inc - p7;                  // exclusive prefix of this lane
    } else {
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float other = __shfl_xor_sync(FULL, tot, o);
            if (lane & o) run += other;
            tot += other;
        }
    }
    const float thr = u * tot;
    int pick = 256;                      // last assignment wins: the smallest qualifying index
    if (run + p7 > thr) pick = 8 * lane + 7;
    if (run + p6 > thr) pick = 8 * lane + 6;
    if (run + p5 > thr) pick = 8 * lane + 5;
    if (run + p4 > thr) pick = 8 * lane + 4;
    if (run + p3 > thr) pick = 8 * lane + 3;
    if (run + p2 > thr) pick = 8 * lane + 2;
    if (run + p1 > thr) pick = 8 * lane + 1;
    if (run + p0 > thr) pick = 8 * lane;
    pick = __reduce_min_sync(FULL, pick);
    return pick == 256 ? 255 : pick;
}
__device__ __forceinline__ int warp_softmax_draw_fast(const float (&l)[8], float u, int lane) { return warp_softmax_draw_impl<false>(l, u, lane); }
__device__ __forceinline__ int warp_softmax_draw_scan(const float (&l)[8], float u, int lane) { return warp_softmax_draw_impl<true>(l, u, lane); }

// Four softmaxes of 16 in one warp (the 4-bit heads of the Fused Subscale WaveRNN 2x): lane l holds logits 2 l, 2 l + 1 of
// 64, lanes [8 k, 8 k + 8) form softmax k and share the uniform u.  Returns, on every lane, the index its group drew
// (same rule as warp_softmax_draw: smallest k whose running sum exceeds u * total, 15 if none).
__device__ __forceinline__ int group16_softmax_draw(float l0, float l1, float u, int lane)
{
    float m = fmaxf(l0, l1);
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) m = fmaxf(m, __shfl_xor_sync(FULL, m, o));
    const float w0 = __expf(l0 - m), w1 = __expf(l1 - m);
    const float s = w0 + w1;
    float inc = s;
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
        const float t = __shfl_up_sync(FULL, inc, o, 8);
        if ((lane & 7) >= o) inc += t;
    }
    const float thr = u * __shfl_sync(FULL, inc, 7, 8);
    const float run = inc - s;           // exclusive prefix of this lane inside its group
    int pick = 16;
    if (inc > thr) pick = 2 * (lane & 7) + 1;
    if (run + w0 > thr) pick = 2 * (lane & 7);
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) pick = min(pick, __shfl_xor_sync(FULL, pick, o));
    return pick == 16 ? 15 : pick;
}
__device__ __forceinline__ float scale4(int v) { return (float)v * (1.0f / 7.5f) - 1.0f; }

// sigmoid / tanh through ex2.approx and the fast reciprocal: absolute error about 1e-7 .. 3e-7.
__device__ __forceinline__ float sigmoidf_fast(float x) { return __fdividef(1.0f, 1.0f + __expf(-x)); }
__device__ __forceinline__ float tanhf_fast(float x)
{
    // 1 - 2 / (1 + e^{2x}): one ex2, one rcp; saturates to +-1 through e^{2x} = inf / 0 (the argument is clamped so that
    // the reciprocal never sees inf)
    const float e = __expf(2.0f * fminf(x, 40.0f));
    return 1.0f - __fdividef(2.0f, 1.0f + e);
}

// ------------------------------------------------------------------ memory-order helpers
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed_s32(const int *p)
{
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Grid-wide barrier on a monotonically increasing arrival counter.  Every CTA of the
// (co-resident, cooperative) grid calls it the same number of times; `epoch` counts the
// calls.  The wait is bounded: after `limit_ns` the CTA records where it gave up, raises
// the abort word every other CTA also polls, and the call returns false so that the
// kernel can return instead of hanging.
struct GridBarrier {
    unsigned long long *counter;     // zeroed before launch
    DevStatus *status;               // zeroed before launch
    unsigned long long epoch;
    unsigned long long limit_ns;

    __device__ __forceinline__ bool sync(int step, int phase)
    {
        __shared__ int s_ok;
        __syncthreads();
        if (threadIdx.x == 0) {
            ++epoch;
            const unsigned long long target = epoch * (unsigned long long)gridDim.x;
            __threadfence();
            atomicAdd(counter, 1ull);
            int ok = 1;
            unsigned long long t0 = 0;
            unsigned spins = 0;
            while (ld_acquire_u64(counter) < target) {
                if ((++spins & 1023u) == 0) {
                    if (ld_relaxed_s32(&status->code) != DEV_OK) { ok = 0; break; }
                    const unsigned long long now = globaltimer_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > limit_ns) {
                        if (atomicCAS(&status->code, DEV_OK, DEV_TIMEOUT) == DEV_OK) {
                            status->cta = blockIdx.x; status->step = step; status->phase = phase;
                        }
                        ok = 0;
                        break;
                    }
                }
            }
            s_ok = ok;
        }
        __syncthreads();
        return s_ok != 0;
    }
};

}  // namespace wrnn
