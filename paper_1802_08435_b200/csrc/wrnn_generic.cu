// Generic WaveRNN step kernel: one persistent cooperative kernel per call, weights streamed
// from global memory (L2-resident) every step, every matrix held as 4x4 block rows, any H,
// any batch, dense or block-sparse, fp32 or bf16 storage.  This is the bring-up and
// cross-check path; the shared-memory-resident kernels are the fast ones.
//
// Per step (Eq. 2 in the order of Fig. 1), phases separated by grid-wide barriers:
//   A  a = R h_{t-1} for all 3H rows; coarse gates -> y_c; fine rows keep their a
//   B  q_c = relu(O1 y_c + b1)          C  l_c = O2 q_c + b2         D  draw c_t
//   E  fine gates (now with c_t) -> y_f
//   F  q_f = relu(O3 y_f + b3)          G  l_f = O4 q_f + b4         H  draw f_t, emit sample
#include <algorithm>
#include <cstdio>

#include "wrnn_internal.h"

namespace wrnn {

struct GenericParams {
    int H, Hh, G, batch;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    int row_lag;                 // > 0: row b of the call is row_lag steps behind row b - 1 (staggered subscale rows); its
                                 // conditioning then holds one frame per step of the call
    long long out_pitch;         // samples between the rows of `out`
    BsrDev R, O1, O2, O3, O4;
    const float *I, *b1, *b2, *b3, *b4, *g;
    float *h0, *h1, *a_fine, *q, *logits;
    uint8_t *c_cur, *c_prev, *f_prev;
    const float *h_in; float *h_out;
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;
    uint8_t *c_out, *f_out;
    int16_t *out;
    float *dbg_gates, *dbg_h, *dbg_logits;
    unsigned long long *bar;
    DevStatus *status;
    unsigned long long limit_ns;
    int skip_cta; long long skip_step;      // self-test: this CTA withholds what it publishes at this step (-1: none)
};

template <typename WT> __device__ __forceinline__ void load_block(const void *vals, int i, float (&w)[16]);

template <> __device__ __forceinline__ void load_block<float>(const void *vals, int i, float (&w)[16])
{
    const float4 *p = reinterpret_cast<const float4 *>(vals) + 4 * (size_t)i;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const float4 v = __ldg(p + r);
        w[4 * r] = v.x; w[4 * r + 1] = v.y; w[4 * r + 2] = v.z; w[4 * r + 3] = v.w;
    }
}
template <> __device__ __forceinline__ void load_block<uint16_t>(const void *vals, int i, float (&w)[16])
{
    const uint4 *p = reinterpret_cast<const uint4 *>(vals) + 2 * (size_t)i;
#pragma unroll
    for (int hlf = 0; hlf < 2; ++hlf) {
        const uint4 v = __ldg(p + hlf);
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) { w[8 * hlf + 2 * k] = bf16lo(u[k]); w[8 * hlf + 2 * k + 1] = bf16hi(u[k]); }
    }
}

// acc[r * TB + b] += sum over the kept blocks of block row br of W[4 br + r][:] . x[b][:]
// (lanes stride over the blocks; the caller reduces across lanes).  x was written by other
// CTAs in an earlier phase, hence the L1-bypassing loads.
template <typename WT, int TB>
__device__ __forceinline__ void blockrow_dot(const BsrDev &M, int br, const float *x, int ldx, int nb,
                                             int lane, float (&acc)[4 * TB])
{
    const int beg = __ldg(M.row_ptr + br), end = __ldg(M.row_ptr + br + 1);
    for (int i = beg + lane; i < end; i += 32) {
        float w[16];
        load_block<WT>(M.vals, i, w);
        const int bc = __ldg(M.col + i);
#pragma unroll
        for (int b = 0; b < TB; ++b) {
            if (b < nb) {
                const float4 xv = __ldcg(reinterpret_cast<const float4 *>(x + (size_t)b * ldx + 4 * bc));
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    float s = acc[r * TB + b];
                    s = fmaf(w[4 * r], xv.x, s);
                    s = fmaf(w[4 * r + 1], xv.y, s);
                    s = fmaf(w[4 * r + 2], xv.z, s);
                    s = fmaf(w[4 * r + 3], xv.w, s);
                    acc[r * TB + b] = s;
                }
            }
        }
    }
}

template <typename WT, int TB>
__device__ __forceinline__ float blockrow_total(const BsrDev &M, int br, const float *x, int ldx, int nb, int lane)
{
    float acc[4 * TB];
#pragma unroll
    for (int i = 0; i < 4 * TB; ++i) acc[i] = 0.f;
    blockrow_dot<WT, TB>(M, br, x, ldx, nb, lane, acc);
    return warp_reduce_scatter<4 * TB>(acc, lane);
}

__device__ __forceinline__ long long frame_of(const GenericParams &p, long long s, int gb)
{
    if (p.row_lag > 0) return s;
    return ((p.step0 + s) * p.row_stride + (long long)(p.stream0 + (unsigned)gb) * p.row_offset_mul) / p.hop;
}

// Gate evaluation of one state unit (Eq. 2).  a* = (R h)[row]; x2 is used on fine rows only.
__device__ __forceinline__ float gate_unit(const GenericParams &p, int j, int gb, long long s, float au, float ar,
                                           float ae, float hprev, float x0, float x1, float x2, bool fine)
{
    const int H = p.H;
    const float *g = p.g + ((size_t)gb * p.n_frames + (size_t)frame_of(p, s, gb)) * p.G;
    const float *Iu = p.I + 3 * (size_t)j, *Ir = p.I + 3 * (size_t)(H + j), *Ie = p.I + 3 * (size_t)(2 * H + j);
    float pu = au + fmaf(Iu[0], x0, fmaf(Iu[1], x1, g[j]));
    float pr = ar + fmaf(Ir[0], x0, fmaf(Ir[1], x1, g[H + j]));
    float pe = fmaf(Ie[0], x0, fmaf(Ie[1], x1, g[2 * H + j]));
    if (fine) { pu = fmaf(Iu[2], x2, pu); pr = fmaf(Ir[2], x2, pr); pe = fmaf(Ie[2], x2, pe); }
    const float u = sigmoidf_acc(pu);
    const float r = sigmoidf_acc(pr);
    const float e = tanhf(fmaf(r, ae, pe));
    const float hn = fmaf(u, hprev, (1.0f - u) * e);
    if (p.dbg_gates) {
        float *d = p.dbg_gates + ((size_t)s * p.batch + gb) * p.G;
        d[j] = u; d[H + j] = r; d[2 * H + j] = e;
    }
    if (p.dbg_h) p.dbg_h[((size_t)s * p.batch + gb) * H + j] = hn;
    return hn;
}

template <typename WT, int TB>
__global__ void __launch_bounds__(512, 1) generic_step_kernel(const GenericParams p)
{
    const int lane = threadIdx.x & 31;
    const int warps_per_cta = blockDim.x >> 5;
    const int gw = blockIdx.x * warps_per_cta + (threadIdx.x >> 5);
    const int nw = gridDim.x * warps_per_cta;
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x;
    const int nthreads = gridDim.x * blockDim.x;
    const int H = p.H, Hh = p.Hh, B = p.batch;
    const int ntiles = (B + TB - 1) / TB;
    constexpr int N = 4 * TB;

    GridBarrier bar{p.bar, p.status, 0ull, p.limit_ns};

    float *hc = p.h0, *hn = p.h1;
    for (int i = gtid; i < B * H; i += nthreads) hc[i] = p.h_in ? p.h_in[i] : 0.f;
    for (int i = gtid; i < B; i += nthreads) {
        p.c_prev[i] = p.c_in ? p.c_in[i] : (uint8_t)128;
        p.f_prev[i] = p.f_in ? p.f_in[i] : (uint8_t)0;
    }
    if (!bar.sync(-1, 0)) return;

    for (long long s = 0; s < p.n_steps; ++s) {
        if ((int)blockIdx.x == p.skip_cta && s == p.skip_step) return;      // self-test: this CTA's arrivals go missing
        // ---- A: recurrent product for all gates; coarse gates finish here
        for (int item = gw; item < (H / 4) * ntiles; item += nw) {
            const int ug = item / ntiles, b0 = (item % ntiles) * TB, nb = min(TB, B - b0);
            const float *x = hc + (size_t)b0 * H;
            const float au = blockrow_total<WT, TB>(p.R, ug, x, H, nb, lane);
            const float ar = blockrow_total<WT, TB>(p.R, H / 4 + ug, x, H, nb, lane);
            const float ae = blockrow_total<WT, TB>(p.R, 2 * (H / 4) + ug, x, H, nb, lane);
            const int r = (lane & (N - 1)) / TB, b = (lane & (N - 1)) % TB;
            if (lane < N && b < nb) {
                const int j = 4 * ug + r, gb = b0 + b;
                if (j < Hh) {
                    const float x0 = scale8(__ldcg(p.c_prev + gb)), x1 = scale8(__ldcg(p.f_prev + gb));
                    hn[(size_t)gb * H + j] = gate_unit(p, j, gb, s, au, ar, ae, __ldcg(hc + (size_t)gb * H + j), x0, x1, 0.f, false);
                } else {
                    float *af = p.a_fine + (size_t)gb * 3 * Hh + (j - Hh);
                    af[0] = au; af[Hh] = ar; af[2 * Hh] = ae;
                }
            }
        }
        if (!bar.sync((int)s, 1)) return;

        for (int head = 0; head < 2; ++head) {
            const BsrDev &Oa = head ? p.O3 : p.O1, &Ob = head ? p.O4 : p.O2;
            const float *ba = head ? p.b3 : p.b1, *bb = head ? p.b4 : p.b2;
            if (head == 1) {
                // ---- E: fine gates, one thread per (row, fine unit)
                for (int i = gtid; i < B * Hh; i += nthreads) {
                    const int gb = i / Hh, jf = i % Hh, j = Hh + jf;
                    const float *af = p.a_fine + (size_t)gb * 3 * Hh + jf;
                    const float x0 = scale8(__ldcg(p.c_prev + gb)), x1 = scale8(__ldcg(p.f_prev + gb));
                    const float x2 = scale8(__ldcg(p.c_cur + gb));
                    hn[(size_t)gb * H + j] = gate_unit(p, j, gb, s, __ldcg(af), __ldcg(af + Hh), __ldcg(af + 2 * Hh),
                                                       __ldcg(hc + (size_t)gb * H + j), x0, x1, x2, true);
                }
                if (!bar.sync((int)s, 5)) return;
            }
            // ---- B / F: hidden layer of the head on its half of the new state
            for (int item = gw; item < (Hh / 4) * ntiles; item += nw) {
                const int br = item / ntiles, b0 = (item % ntiles) * TB, nb = min(TB, B - b0);
                const float v = blockrow_total<WT, TB>(Oa, br, hn + (size_t)b0 * H + head * Hh, H, nb, lane);
                const int r = (lane & (N - 1)) / TB, b = (lane & (N - 1)) % TB;
                if (lane < N && b < nb) {
                    const int row = 4 * br + r;
                    p.q[(size_t)(b0 + b) * Hh + row] = fmaxf(v + (ba ? ba[row] : 0.f), 0.f);
                }
            }
            if (!bar.sync((int)s, head ? 6 : 2)) return;
            // ---- C / G: logits
            for (int item = gw; item < 64 * ntiles; item += nw) {
                const int br = item / ntiles, b0 = (item % ntiles) * TB, nb = min(TB, B - b0);
                const float v = blockrow_total<WT, TB>(Ob, br, p.q + (size_t)b0 * Hh, Hh, nb, lane);
                const int r = (lane & (N - 1)) / TB, b = (lane & (N - 1)) % TB;
                if (lane < N && b < nb) {
                    const int row = 4 * br + r;
                    const float l = v + (bb ? bb[row] : 0.f);
                    p.logits[(size_t)(b0 + b) * 256 + row] = l;
                    if (p.dbg_logits) p.dbg_logits[(((size_t)s * B + b0 + b) * 2 + head) * 256 + row] = l;
                }
            }
            if (!bar.sync((int)s, head ? 7 : 3)) return;
            // ---- D / H: softmax + inverse-CDF draw, one warp per row
            for (int gb = gw; gb < B; gb += nw) {
                float l[8];
                const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(p.logits + (size_t)gb * 256 + 8 * lane));
                const float4 v1 = __ldcg(reinterpret_cast<const float4 *>(p.logits + (size_t)gb * 256 + 8 * lane + 4));
                l[0] = v0.x; l[1] = v0.y; l[2] = v0.z; l[3] = v0.w; l[4] = v1.x; l[5] = v1.y; l[6] = v1.z; l[7] = v1.w;
                const float u = uniform24(p.seed, p.stream0 + (unsigned)gb, (unsigned long long)(p.step0 + s - (long long)gb * p.row_lag), head);
                int idx = warp_softmax_draw(l, u, lane);
                if (lane == 0) {
                    const size_t o = (size_t)gb * p.n_steps + s;
                    if (head == 0) {
                        if (p.c_out) p.c_out[o] = (uint8_t)idx;
                        if (p.c_forced) idx = p.c_forced[o];
                        p.c_cur[gb] = (uint8_t)idx;
                    } else {
                        if (p.f_out) p.f_out[o] = (uint8_t)idx;
                        if (p.f_forced) idx = p.f_forced[o];
                        const int c = p.c_cur[gb];
                        if (p.out) p.out[(size_t)gb * p.out_pitch + s] = (int16_t)(256 * c + idx - 32768);
                        p.c_prev[gb] = (uint8_t)c;
                        p.f_prev[gb] = (uint8_t)idx;
                    }
                }
            }
            if (!bar.sync((int)s, head ? 8 : 4)) return;
        }
        float *t = hc; hc = hn; hn = t;
    }

    if (p.h_out) for (int i = gtid; i < B * H; i += nthreads) p.h_out[i] = __ldcg(hc + i);
    for (int i = gtid; i < B; i += nthreads) {
        if (p.c_st_out) p.c_st_out[i] = __ldcg(p.c_prev + i);
        if (p.f_st_out) p.f_st_out[i] = __ldcg(p.f_prev + i);
    }
}

// ---------------------------------------------------------------------------------------------
// Prologue: g[b][k][row] = W_cond[row][:] . frame[b][k][:] + b_gate[row]   (the per-step
// conditioning vector; one frame is held for `hop` samples).

__global__ void cond_project_kernel(const float *__restrict__ cond, const float *__restrict__ W_condT,
                                    const float *__restrict__ b_gate, float *__restrict__ g, int G, int D,
                                    long long n_pairs)
{
    // blockIdx.y strides over the (row of the batch, frame) pairs, so no grid dimension limits their number
    extern __shared__ float fr[];
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    for (long long kb = blockIdx.y; kb < n_pairs; kb += gridDim.y) {
        const float *f = cond + (size_t)kb * D;
        __syncthreads();
        for (int d = threadIdx.x; d < D; d += blockDim.x) fr[d] = f[d];
        __syncthreads();
        if (row < G) {
            float acc = 0.f;
            for (int d = 0; d < D; ++d) acc = fmaf(W_condT[(size_t)d * G + row], fr[d], acc);
            g[(size_t)kb * G + row] = acc + (b_gate ? b_gate[row] : 0.f);
        }
    }
}

__global__ void cond_bias_only_kernel(const float *__restrict__ b_gate, float *__restrict__ g, int G, int batch)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < G * batch) g[i] = b_gate ? b_gate[i % G] : 0.f;
}

int cond_project(wrnn_model *m, const float *cond, int batch, int n_frames, cudaStream_t s)
{
    const int G = 3 * m->H;
    if (m->cond_dim == 0) {
        cond_bias_only_kernel<<<(G * batch + 255) / 256, 256, 0, s>>>(m->b_gate, m->g, G, batch);
    } else {
        const long long n_pairs = (long long)batch * n_frames;
        dim3 grid((G + 255) / 256, (unsigned)std::min<long long>(n_pairs, 65535));
        cond_project_kernel<<<grid, 256, m->cond_dim * sizeof(float), s>>>(cond, m->W_condT, m->b_gate, m->g, G,
                                                                           m->cond_dim, n_pairs);
    }
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Subscale fold / unfold (Eq. 4): sub[s][i] = x[B i + s].

__global__ void fold_kernel(const int16_t *__restrict__ src, int16_t *__restrict__ dst, long long n, int B, int unfold)
{
    const long long len = n / B;
    for (long long o = blockIdx.x * (long long)blockDim.x + threadIdx.x; o < n; o += (long long)gridDim.x * blockDim.x) {
        if (unfold) { const long long i = o / B; const int s = (int)(o % B); dst[o] = src[(long long)s * len + i]; }
        else        { const int s = (int)(o / len); const long long i = o % len; dst[o] = src[(long long)B * i + s]; }
    }
}

int fold_launch(const int16_t *x, long long n_total, int B, int16_t *sub, bool unfold, cudaStream_t s)
{
    if (n_total == 0) return WRNN_OK;
    const int blocks = (int)((n_total + 255) / 256 > 1184 ? 1184 : (n_total + 255) / 256);
    fold_kernel<<<blocks, 256, 0, s>>>(x, sub, n_total, B, unfold ? 1 : 0);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
}

// Conditioning of staggered subscale rows (Section 4.1: sub-tensor r sees the future of sub-tensors z < r up to F
// positions; one masked convolution stands in for the paper's network):
//     v[b][c][k] = frame_r[(B (p + c) + r) div hop][k] + relu(bias[k] + sum_{delta=1..r} sum_{d=0..F} V[delta-1][d][k] x(hist[r-delta][p+c+d]))
// for row r = r_lo + b of the call, whose first position is p = p_lo - b * lag; x(u) = u / 32768; positions >= L give 0.
__global__ void subscale_cond_kernel(const int16_t *__restrict__ hist, const float *__restrict__ frames, const float *__restrict__ V,
                                     const float *__restrict__ bias, float *__restrict__ v, int B, long long L, int F, int D,
                                     int n_frames, int hop, int r_lo, long long p_lo, int lag, int n_steps)
{
    // one block per (row, step): threadIdx.x = output channel (strided), threadIdx.y = one of four slices of the (earlier
    // row, offset) pairs; the slices meet in shared memory
    extern __shared__ float cpart[];                 // [4][D]
    const int b = blockIdx.y, c = blockIdx.x, r = r_lo + b;
    const long long pos = p_lo - (long long)b * lag + c;
    const int n_pairs = r * (F + 1);
    for (int k = threadIdx.x; k < D; k += blockDim.x) {
        float acc = 0.f;
        for (int j = threadIdx.y; j < n_pairs; j += blockDim.y) {
            const int delta = j / (F + 1) + 1, d = j - (delta - 1) * (F + 1);
            if (pos + d < L)
                acc = fmaf(V[((size_t)(delta - 1) * (F + 1) + d) * D + k], (float)hist[(size_t)(r - delta) * L + pos + d] * (1.0f / 32768.0f), acc);
        }
        cpart[threadIdx.y * D + k] = acc;
    }
    __syncthreads();
    if (threadIdx.y == 0)
        for (int k = threadIdx.x; k < D; k += blockDim.x) {
            const float acc = bias[k] + ((cpart[k] + cpart[D + k]) + (cpart[2 * D + k] + cpart[3 * D + k]));
            const long long fr = ((long long)B * pos + r) / hop;
            v[((size_t)b * n_steps + c) * D + k] = frames[((size_t)r * n_frames + fr) * D + k] + fmaxf(acc, 0.f);
        }
}

int subscale_cond_launch(const int16_t *hist, const float *frames, const float *V, const float *bias, float *v, int B, long long L, int F,
                         int D, int n_frames, int hop, int r_lo, int n_rows, long long p_lo, int lag, int n_steps, cudaStream_t s)
{
    if (n_rows <= 0 || n_steps <= 0) return WRNN_OK;
    if (n_rows > 65535) return WRNN_ERR_UNSUPPORTED;                                  // grid.y
    const size_t smem = (size_t)4 * D * sizeof(float);
    if (smem > 48 * 1024 && cudaFuncSetAttribute(subscale_cond_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return WRNN_ERR_UNSUPPORTED;
    }
    subscale_cond_kernel<<<dim3(n_steps, n_rows), dim3(64, 4), (size_t)4 * D * sizeof(float), s>>>(hist, frames, V, bias, v, B, L, F, D, n_frames, hop, r_lo, p_lo, lag, n_steps);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
}

// The two streams of the fused subscale variant back in the original order: u[2 i] = a_i, u[2 i + 1] = the sample part B
// emitted two steps later (Section 4.4 with F = 2).
__global__ void fs2_unfold_kernel(const int16_t *__restrict__ ab, long long n, int16_t *__restrict__ u)
{
    for (long long o = blockIdx.x * (long long)blockDim.x + threadIdx.x; o < 2 * (n - 2); o += (long long)gridDim.x * blockDim.x)
        u[o] = (o & 1) ? ab[n + (o >> 1) + 2] : ab[o >> 1];
}

int fs2_unfold_launch(const int16_t *ab, long long n, int16_t *u, cudaStream_t s)
{
    if (n <= 2) return WRNN_OK;
    const long long tot = 2 * (n - 2);
    const int blocks = (int)((tot + 255) / 256 > 1184 ? 1184 : (tot + 255) / 256);
    fs2_unfold_kernel<<<blocks, 256, 0, s>>>(ab, n, u);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------

static void *generic_kernel_ptr(int dtype, int tb)
{
    if (dtype == WRNN_F32) return tb == 1 ? (void *)generic_step_kernel<float, 1> : (void *)generic_step_kernel<float, 8>;
    return tb == 1 ? (void *)generic_step_kernel<uint16_t, 1> : (void *)generic_step_kernel<uint16_t, 8>;
}

int generic_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem)
{
    (void)batch;
    if (n_ctas) *n_ctas = m->n_sms;
    if (n_threads) *n_threads = 512;
    if (smem) *smem = 0;
    return WRNN_OK;
}

int generic_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    GenericParams p;
    p.H = m->H; p.Hh = m->H / 2; p.G = 3 * m->H; p.batch = a.batch;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.R = m->R; p.O1 = m->O1; p.O2 = m->O2; p.O3 = m->O3; p.O4 = m->O4;
    p.I = m->I; p.b1 = m->b1; p.b2 = m->b2; p.b3 = m->b3; p.b4 = m->b4; p.g = m->g;
    p.h0 = m->hbuf[0]; p.h1 = m->hbuf[1]; p.a_fine = m->a_fine; p.q = m->q; p.logits = m->logits;
    p.c_cur = m->c_cur; p.c_prev = m->c_prev; p.f_prev = m->f_prev;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in;
    p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.row_lag = a.row_lag; p.out_pitch = a.out_pitch ? a.out_pitch : a.n_steps;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.bar = m->bar; p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;

    if (cudaMemsetAsync(m->bar, 0, sizeof(unsigned long long), s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    void *fn = generic_kernel_ptr(m->dtype, a.batch == 1 ? 1 : 8);
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, 512, 0) != cudaSuccess || per_sm < 1) {
        m->err = "generic kernel does not fit one CTA per SM";
        return WRNN_ERR_UNSUPPORTED;
    }
    void *args[] = {(void *)&p};
    const cudaError_t e = cudaLaunchCooperativeKernel(fn, dim3(m->n_sms), dim3(512), args, 0, s);
    if (e != cudaSuccess) {
        m->err = std::string("cooperative launch failed: ") + cudaGetErrorString(e);
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    return WRNN_OK;
}

// ---------------------------------------------------------------------------------------------
// Sampling without any allocation.  Everything the generic step kernel needs besides the model's
// weights and the caller's buffers -- projected conditioning, the two state buffers, the head
// exchange buffers, the per-row sample bytes and the grid-barrier counter -- is carved out of one
// fixed array in device memory that belongs to the library image.  Every device that loads the
// library holds these 8 MiB until the process exits.
constexpr size_t kStaticScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code the array's name is only a handle for the symbol, not a device address; the address
// is looked up once per device (with that device current) and cached.
constexpr int kMaxDevices = 64;
static void *g_static_scratch_addr[kMaxDevices];
static std::atomic<int> g_static_scratch_ready[kMaxDevices];

static int static_scratch_base(int device, unsigned char **base, std::string *err)
{
    if (device < 0 || device >= kMaxDevices) { *err = "device index out of range for the static scratch table"; return WRNN_ERR_UNSUPPORTED; }
    if (!g_static_scratch_ready[device].load(std::memory_order_acquire)) {
        void *ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            *err = std::string("cudaGetSymbolAddress(static scratch) failed: ") + cudaGetErrorString(e);
            cudaGetLastError();
            return WRNN_ERR_CUDA;
        }
        g_static_scratch_addr[device] = ptr;         // racing first calls store the same value
        g_static_scratch_ready[device].store(1, std::memory_order_release);
    }
    *base = static_cast<unsigned char *>(g_static_scratch_addr[device]);
    return WRNN_OK;
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Called by wrnn_create (which allocates anyway) with the model's device current: looks the address up ahead of time, so
// that with lazily loaded modules the load of the image that holds the array does not fall into a sampling call.
void noalloc_warm(int device)
{
    unsigned char *base = nullptr;
    std::string err;
    (void)static_scratch_base(device, &base, &err);
}

}  // namespace wrnn

using namespace wrnn;

extern "C" int wrnn_sample_noalloc(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch, uint64_t seed,
                                   const wrnn_state *st, int16_t *out, void *cuda_stream)
{
    StepArgs a;
    int rc = check_step(m, cond, n_steps, batch, st, &a);
    if (rc != WRNN_OK) return rc;
    if (n_steps == 0) return WRNN_OK;
    if (!out) { m->err = "out is NULL"; return WRNN_ERR_INVALID_ARG; }
    a.seed = seed; a.out = out;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaSetDevice(m->device) != cudaSuccess) { m->err = "cudaSetDevice failed"; return WRNN_ERR_CUDA; }

    // carve the fixed array; refuse sizes it cannot hold
    const size_t B = (size_t)batch, H = (size_t)m->H, Hh = H / 2, G = 3 * H;
    const size_t nf = m->cond_dim ? (size_t)a.n_frames : 1;
    size_t off = 0;
    const size_t o_bar = off;    off += 256;
    const size_t o_bytes = off;  off += align256(3 * B);
    const size_t o_h0 = off;     off += align256(B * H * 4);
    const size_t o_h1 = off;     off += align256(B * H * 4);
    const size_t o_af = off;     off += align256(B * 3 * Hh * 4);
    const size_t o_q = off;      off += align256(B * Hh * 4);
    const size_t o_l = off;      off += align256(B * 256 * 4);
    const size_t o_g = off;      off += align256(B * nf * G * 4);
    if (off > kStaticScratchBytes) {
        char buf[200];
        std::snprintf(buf, sizeof(buf), "wrnn_sample_noalloc: batch %d x %zu frames x 3H = %zu needs %zu bytes of scratch, the fixed array holds %zu",
                      batch, nf, G, off, kStaticScratchBytes);
        m->err = buf;
        return WRNN_ERR_UNSUPPORTED;
    }
    unsigned char *base = nullptr;
    rc = static_scratch_base(m->device, &base, &m->err);
    if (rc != WRNN_OK) return rc;
    float *g = reinterpret_cast<float *>(base + o_g);

    // conditioning projection into the fixed array
    if (m->cond_dim == 0) {
        cond_bias_only_kernel<<<(unsigned)((G * B + 255) / 256), 256, 0, s>>>(m->b_gate, g, (int)G, batch);
    } else {
        const long long n_pairs = (long long)(B * nf);
        dim3 grid((unsigned)((G + 255) / 256), (unsigned)std::min<long long>(n_pairs, 65535));
        cond_project_kernel<<<grid, 256, m->cond_dim * sizeof(float), s>>>(a.cond, m->W_condT, m->b_gate, g, (int)G, m->cond_dim, n_pairs);
    }
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) { m->err = "conditioning projection launch failed"; return WRNN_ERR_CUDA; }

    GenericParams p;
    p.H = m->H; p.Hh = m->H / 2; p.G = 3 * m->H; p.batch = batch;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = (int)nf;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.R = m->R; p.O1 = m->O1; p.O2 = m->O2; p.O3 = m->O3; p.O4 = m->O4;
    p.I = m->I; p.b1 = m->b1; p.b2 = m->b2; p.b3 = m->b3; p.b4 = m->b4; p.g = g;
    p.h0 = reinterpret_cast<float *>(base + o_h0); p.h1 = reinterpret_cast<float *>(base + o_h1);
    p.a_fine = reinterpret_cast<float *>(base + o_af); p.q = reinterpret_cast<float *>(base + o_q);
    p.logits = reinterpret_cast<float *>(base + o_l);
    p.c_cur = base + o_bytes; p.c_prev = base + o_bytes + B; p.f_prev = base + o_bytes + 2 * B;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in;
    p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = nullptr; p.f_forced = nullptr; p.c_out = nullptr; p.f_out = nullptr; p.out = a.out;
    p.row_lag = 0; p.out_pitch = a.n_steps;
    p.dbg_gates = nullptr; p.dbg_h = nullptr; p.dbg_logits = nullptr;
    p.bar = reinterpret_cast<unsigned long long *>(base + o_bar);
    p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;

    // the array keeps the previous call's contents: the arrival counter must start at zero; the state and
    // sample bytes are (re)initialised by the kernel itself before use
    if (cudaMemsetAsync(base + o_bar, 0, 256, s) != cudaSuccess) { m->err = "memset failed"; return WRNN_ERR_CUDA; }
    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) { m->err = "memset failed"; return WRNN_ERR_CUDA; }
    void *fn = generic_kernel_ptr(m->dtype, batch == 1 ? 1 : 8);
    void *args[] = {(void *)&p};
    const cudaError_t e = cudaLaunchCooperativeKernel(fn, dim3(m->n_sms), dim3(512), args, 0, s);
    if (e != cudaSuccess) {
        m->err = std::string("cooperative launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    return WRNN_OK;
}
