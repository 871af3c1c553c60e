// The conditioning network of the Subscale WaveRNN (Sections 4.1 and 5.3 of the paper): a masked dilated 1-D CNN with
// relus through which the WaveRNN that generates sub-tensor s sees the FUTURE context of the sub-tensors z < s -- ten
// layers, kernels of size 3, 384 convolution channels, 768 residual channels, five stages of increasing dilation, a
// future horizon of 128 positions.  The paper prints no equations for it; the reading built here:
//     X[i][z]    = u_{B i + z} / 32768 for z < s, 0 otherwise                              (block input, masked to earlier rows)
//     x_0[i]     = W_in X[i] + b_in
//     a_l[i]     = relu(b_conv[l] + sum_{t = 0..taps-1} W_conv[l][t] x_l[i + t d_l])       (connections reach forward only)
//     x_{l+1}[i] = x_l[i] + W_res[l] a_l[i] + b_res[l]
//     v_s[i]     = frame_s[(B i + s) div hop] + W_out relu(x_last[i]) + b_out
// with the zero vector at positions at or beyond the row length in every layer, and bf16-rounded matrices.
//
// A chunk of positions is a chain of matrix products over (positions x channels), so it runs on the fifth-generation
// tensor cores: one CTA per tile of 128 positions x BN output channels; the activations (M side) enter as bf16 high and
// low parts of their fp32 values (two MMAs into the same TMEM accumulator, operand error 2^-17), the weights (N side)
// as bf16; operands come in by TMA (128-byte swizzle) through a ring of mbarriers, a dilated tap being nothing but a
// row offset of the activation box; one thread issues tcgen05.mma, four warps drain the accumulator with tcgen05.ld and
// apply bias / relu / residual.  The residual stream is kept in fp32 beside its bf16 parts.  Every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>
#include <new>

#include "wrnn_internal.h"
#include "wrnn_tc.cuh"

struct wrnn_subscale_net {
    int B = 0, n_layers = 0, taps = 0, conv_ch = 0, res_ch = 0, cond_dim = 0, reach = 0, device = 0;
    std::vector<int> dilation;
    __nv_bfloat16 *Wc = nullptr;      // [layers][taps][conv_ch][res_ch]
    __nv_bfloat16 *Wr = nullptr;      // [layers][res_ch][conv_ch]
    __nv_bfloat16 *Wo = nullptr;      // [64][res_ch] (rows >= cond_dim zero)
    float *W_in = nullptr, *b_in = nullptr, *b_conv = nullptr, *b_res = nullptr, *b_out = nullptr;
    // activations of one call: n_seg row segments of n_alloc positions each
    int n_seg = 0, n_alloc = 0;
    float *xf = nullptr;                              // [n_seg * n_alloc][res_ch] fp32 residual stream
    __nv_bfloat16 *xh = nullptr, *xl = nullptr;       // its bf16 high / low parts (relu'd after the last layer)
    __nv_bfloat16 *ah = nullptr, *al = nullptr;       // [n_seg * n_alloc][conv_ch] convolution outputs
    CUtensorMap tmWc, tmWr, tmWo, tmXh, tmXl, tmAh, tmAl;
    wrnn::DevStatus *status = nullptr;
    std::string err;
};

namespace wrnn {

constexpr int SN_BM = 128;           // positions per tile (the M side: one TMEM lane per position)
constexpr int SN_THREADS = 192;      // warp 0: TMA producer, warp 1: MMA issuer, warps 2..5: epilogue
enum { SN_CONV = 0, SN_RES = 1, SN_OUT = 2 };

struct SubnetGemmParams {
    int n_kb_tap;                    // 64-wide k-blocks per tap
    int taps, dil;                   // taps of this product and their distance in positions (1 tap for RES / OUT)
    int w_row0, w_tap_rows;          // first row of this layer in the weight tensor, rows between taps
    int n_alloc;                     // positions per row segment of the activation tensors
    int n_pos;                       // positions of a segment this product must write ([0, n_pos))
    int C_out;                       // channels of the output tensor (row pitch)
    const float *bias;               // [C_out] of this layer
    // positions: segment b holds row r_lo + b from position p_lo - b * lag on; positions >= L hold zeros
    int r_lo; long long p_lo; int lag; long long L;
    float *xf; __nv_bfloat16 *oh, *ol;      // RES: fp32 stream (in/out) and its parts; CONV: oh / ol = convolution outputs
    int relu_parts;                          // RES: the parts hold relu(x) (after the last layer: operand of the output product)
    // OUT
    float *v; int n_steps, cond_dim; const float *frames; int n_frames, hop, Bsub;
    const float *b_out;
    DevStatus *status;
    unsigned long long limit_ns;
};

template <int BN, int MODE, int STAGES>
__global__ void __launch_bounds__(SN_THREADS, 1) subnet_gemm_kernel(const __grid_constant__ CUtensorMap tmAh, const __grid_constant__ CUtensorMap tmAl,
                                                                    const __grid_constant__ CUtensorMap tmW, const SubnetGemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nt = blockIdx.x, mt = blockIdx.y, seg = blockIdx.z;
    constexpr uint32_t A_BYTES = SN_BM * TC_BK * 2, W_BYTES = BN * TC_BK * 2, STAGE_BYTES = 2 * A_BYTES + W_BYTES;
    constexpr int TMEM_COLS = BN <= 64 ? 64 : BN <= 128 ? 128 : 256;
    __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES], done;
    __shared__ uint32_t tmem_slot;
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t ring0 = smem_u32(ring);

    if (tid == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(smem_u32(&full[i]), 1); mbar_init(smem_u32(&empty[i]), 1); }
        mbar_init(smem_u32(&done), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    // Programmatic dependent launch: the next product of the chain may be scheduled now (its CTAs set up their barriers and
    // TMEM on SMs that this grid has left or never used); nothing of the previous product is read before it has completed.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const int nkb = p.taps * p.n_kb_tap;
    const int arow0 = seg * p.n_alloc + mt * SN_BM;          // first activation row (position) of this tile
    bool ok = true;
    if (warp == 0 && lane == 0) {
        for (int kb = 0; kb < nkb; ++kb) {
            const int st = kb % STAGES, ph = (kb / STAGES) & 1;
            if (!mbar_wait(smem_u32(&empty[st]), ph ^ 1, p.limit_ns)) { ok = false; break; }
            const int tap = kb / p.n_kb_tap, kc = (kb - tap * p.n_kb_tap) * TC_BK;
            const uint32_t fb = smem_u32(&full[st]), base = ring0 + st * STAGE_BYTES;
            mbar_expect_tx(fb, STAGE_BYTES);
            tma_load_2d(base, &tmAh, fb, kc, arow0 + tap * p.dil);
            tma_load_2d(base + A_BYTES, &tmAl, fb, kc, arow0 + tap * p.dil);
            tma_load_2d(base + 2 * A_BYTES, &tmW, fb, kc, p.w_row0 + tap * p.w_tap_rows + nt * BN);
        }
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = umma_idesc_bf16(SN_BM, BN);
        for (int kb = 0; kb < nkb; ++kb) {
            const int st = kb % STAGES, ph = (kb / STAGES) & 1;
            if (!mbar_wait(smem_u32(&full[st]), ph, p.limit_ns)) { ok = false; break; }
            tc_fence_after();
            const uint32_t base = ring0 + st * STAGE_BYTES;
            const uint64_t dh = umma_desc_sw128(base), dl = umma_desc_sw128(base + A_BYTES), dw = umma_desc_sw128(base + 2 * A_BYTES);
#pragma unroll
            for (int k = 0; k < TC_BK / 16; ++k) {             // 32 bytes along K per MMA inside the swizzle atom
                umma_bf16(tmem, dh + 2 * k, dw + 2 * k, idesc, (kb | k) ? 1u : 0u);
                umma_bf16(tmem, dl + 2 * k, dw + 2 * k, idesc, 1u);
            }
            umma_commit(smem_u32(&empty[st]));
        }
        if (ok) umma_commit(smem_u32(&done));
    } else if (warp >= 2) {
        if (mbar_wait(smem_u32(&done), 0, p.limit_ns)) {
            tc_fence_after();
            const int q = warp & 3;                             // TMEM lane quadrant this warp may read
            const int j = mt * SN_BM + 32 * q + lane;           // position inside the segment
            const long long pos = p.p_lo - (long long)seg * p.lag + j;
            const bool live = j < p.n_pos;                      // positions beyond are never read by a valid output
            const bool inside = pos < p.L;                      // at or beyond the row length every layer holds zeros
            const size_t row = (size_t)seg * p.n_alloc + j;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                float acc[32];
                tmem_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)c0, acc);
                tmem_wait_ld();
                const int ch = nt * BN + c0;
                if (MODE == SN_OUT) {
                    if (live && j < p.n_steps) {
                        const int r = p.r_lo + seg;
                        const long long fr = ((long long)p.Bsub * pos + r) / p.hop;
                        const float *f = p.frames + ((size_t)r * p.n_frames + fr) * p.cond_dim;
                        float *dst = p.v + ((size_t)seg * p.n_steps + j) * p.cond_dim;
                        for (int c = 0; c < 32; ++c)
                            if (ch + c < p.cond_dim) dst[ch + c] = f[ch + c] + (acc[c] + p.b_out[ch + c]);
                    }
                } else if (live) {
                    uint32_t hi[16], lo[16];
                    if (MODE == SN_RES) {
                        float4 *xf4 = reinterpret_cast<float4 *>(p.xf + row * p.C_out + ch);
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const float4 b = __ldg(reinterpret_cast<const float4 *>(p.bias + ch + c));
                            float4 x = xf4[c / 4];
                            x.x = inside ? x.x + (acc[c] + b.x) : 0.f; x.y = inside ? x.y + (acc[c + 1] + b.y) : 0.f;
                            x.z = inside ? x.z + (acc[c + 2] + b.z) : 0.f; x.w = inside ? x.w + (acc[c + 3] + b.w) : 0.f;
                            xf4[c / 4] = x;
                            acc[c] = x.x; acc[c + 1] = x.y; acc[c + 2] = x.z; acc[c + 3] = x.w;
                        }
                        if (p.relu_parts) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) acc[c] = fmaxf(acc[c], 0.f);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const float4 b = __ldg(reinterpret_cast<const float4 *>(p.bias + ch + c));
                            acc[c] = inside ? fmaxf(acc[c] + b.x, 0.f) : 0.f; acc[c + 1] = inside ? fmaxf(acc[c + 1] + b.y, 0.f) : 0.f;
                            acc[c + 2] = inside ? fmaxf(acc[c + 2] + b.z, 0.f) : 0.f; acc[c + 3] = inside ? fmaxf(acc[c + 3] + b.w, 0.f) : 0.f;
                        }
                    }
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const __nv_bfloat16 h0 = __float2bfloat16_rn(acc[c]), h1 = __float2bfloat16_rn(acc[c + 1]);
                        const __nv_bfloat16 l0 = __float2bfloat16_rn(acc[c] - __bfloat162float(h0)), l1 = __float2bfloat16_rn(acc[c + 1] - __bfloat162float(h1));
                        hi[c / 2] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                        lo[c / 2] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
                    }
                    uint4 *dh = reinterpret_cast<uint4 *>(p.oh + row * p.C_out + ch), *dl = reinterpret_cast<uint4 *>(p.ol + row * p.C_out + ch);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        dh[c] = make_uint4(hi[4 * c], hi[4 * c + 1], hi[4 * c + 2], hi[4 * c + 3]);
                        dl[c] = make_uint4(lo[4 * c], lo[4 * c + 1], lo[4 * c + 2], lo[4 * c + 3]);
                    }
                }
            }
            tc_fence_before();
        } else ok = false;
    }
    if (!ok && atomicCAS(&p.status->code, DEV_OK, DEV_TIMEOUT) == DEV_OK) { p.status->cta = blockIdx.x; p.status->step = blockIdx.y; p.status->phase = 20 + MODE; }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// x_0 = W_in X + b_in for the positions [0, n_pos) of every segment, fp32 and bf16 parts (N1, N2 of the reading above)
__global__ void subnet_input_kernel(const int16_t *__restrict__ hist, const float *__restrict__ W_in, const float *__restrict__ b_in, int Bsub,
                                    long long L, int C, int r_lo, long long p_lo, int lag, int n_alloc, int n_pos, float *__restrict__ xf,
                                    __nv_bfloat16 *__restrict__ xh, __nv_bfloat16 *__restrict__ xl)
{
    const int seg = blockIdx.y, j = blockIdx.x, r = r_lo + seg;
    const long long pos = p_lo - (long long)seg * lag + j;
    if (j >= n_pos) return;
    __shared__ float X[64];
    if ((int)threadIdx.x < Bsub) X[threadIdx.x] = ((int)threadIdx.x < r && pos < L) ? (float)hist[(size_t)threadIdx.x * L + pos] * (1.0f / 32768.0f) : 0.f;
    __syncthreads();
    const size_t row = (size_t)seg * n_alloc + j;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        float v = 0.f;
        if (pos < L) {
            v = b_in[c];
            for (int z = 0; z < r; ++z) v = fmaf(W_in[(size_t)c * Bsub + z], X[z], v);
        }
        xf[row * C + c] = v;
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        xh[row * C + c] = h;
        xl[row * C + c] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

static float round_bf16_host(float v)
{
    uint32_t b;
    std::memcpy(&b, &v, 4);
    b += 0x7fffu + ((b >> 16) & 1u);
    b &= 0xffff0000u;
    float r;
    std::memcpy(&r, &b, 4);
    return r;
}

static bool upload_bf16(__nv_bfloat16 **dst, const float *src, size_t n, size_t n_alloc)
{
    std::vector<uint16_t> h(n_alloc, 0);
    for (size_t i = 0; i < n; ++i) {
        const float r = round_bf16_host(src[i]);
        uint32_t b;
        std::memcpy(&b, &r, 4);
        h[i] = (uint16_t)(b >> 16);
    }
    return cudaMalloc((void **)dst, n_alloc * 2) == cudaSuccess && cudaMemcpy(*dst, h.data(), n_alloc * 2, cudaMemcpyHostToDevice) == cudaSuccess;
}

static bool upload_f32(float **dst, const float *src, size_t n)
{
    return cudaMalloc((void **)dst, n * 4) == cudaSuccess && cudaMemcpy(*dst, src, n * 4, cudaMemcpyHostToDevice) == cudaSuccess;
}

static void free_acts(wrnn_subscale_net *n)
{
    cudaFree(n->xf); cudaFree(n->xh); cudaFree(n->xl); cudaFree(n->ah); cudaFree(n->al);
    n->xf = nullptr; n->xh = n->xl = n->ah = n->al = nullptr; n->n_seg = n->n_alloc = 0;
}

// activation tensors for n_seg segments of n_pos positions (grown on demand; synchronises when it grows)
static int ensure_acts(wrnn_subscale_net *n, int n_seg, int n_pos)
{
    const int n_alloc = ((n_pos + SN_BM - 1) / SN_BM) * SN_BM + SN_BM;       // tiles are whole, taps may reach one tile further
    if (n_seg <= n->n_seg && n_alloc <= n->n_alloc) return WRNN_OK;
    cudaDeviceSynchronize();
    free_acts(n);
    const size_t rows = (size_t)n_seg * n_alloc;
    if (cudaMalloc((void **)&n->xf, rows * n->res_ch * 4) != cudaSuccess || cudaMalloc((void **)&n->xh, rows * n->res_ch * 2) != cudaSuccess ||
        cudaMalloc((void **)&n->xl, rows * n->res_ch * 2) != cudaSuccess || cudaMalloc((void **)&n->ah, rows * n->conv_ch * 2) != cudaSuccess ||
        cudaMalloc((void **)&n->al, rows * n->conv_ch * 2) != cudaSuccess) {
        cudaGetLastError(); free_acts(n); n->err = "activation buffers of the conditioning network do not fit"; return WRNN_ERR_NOMEM;
    }
    cudaMemset(n->xh, 0, rows * n->res_ch * 2); cudaMemset(n->xl, 0, rows * n->res_ch * 2);
    cudaMemset(n->ah, 0, rows * n->conv_ch * 2); cudaMemset(n->al, 0, rows * n->conv_ch * 2);
    cudaMemset(n->xf, 0, rows * n->res_ch * 4);
    if (!make_map(&n->tmXh, n->xh, (long long)rows, n->res_ch, SN_BM) || !make_map(&n->tmXl, n->xl, (long long)rows, n->res_ch, SN_BM) ||
        !make_map(&n->tmAh, n->ah, (long long)rows, n->conv_ch, SN_BM) || !make_map(&n->tmAl, n->al, (long long)rows, n->conv_ch, SN_BM)) {
        free_acts(n); n->err = "tensor map encoding failed"; return WRNN_ERR_CUDA;
    }
    n->n_seg = n_seg; n->n_alloc = n_alloc;
    return WRNN_OK;
}

constexpr int SN_BN_CONV = 96, SN_BN_RES = 96, SN_BN_OUT = 64;
constexpr int SN_ST_CONV = 4, SN_ST_RES = 4, SN_ST_OUT = 4;
// launch with programmatic stream serialization: the kernel may start while its predecessor in the stream drains (it waits for
// the predecessor's completion itself, with griddepcontrol.wait, before it reads anything)
template <typename K>
static void pdl_launch(K kernel, dim3 grid, int smem, cudaStream_t s, const CUtensorMap &a, const CUtensorMap &b, const CUtensorMap &w, const SubnetGemmParams &p)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(SN_THREADS); cfg.dynamicSmemBytes = (size_t)smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, a, b, w, p);
}

template <int BN, int ST> constexpr int sn_smem() { return ST * (2 * SN_BM * TC_BK * 2 + BN * TC_BK * 2) + 1024; }

// The whole network for the segments of one call: v[seg][n_steps][cond_dim] (the conditioning vectors the stepping call
// of these rows consumes).  Segment b is row r_lo + b from position p_lo - b * lag on.
int subnet_run(wrnn_subscale_net *n, const int16_t *hist, const float *frames, int n_frames, int hop, long long L, int r_lo, int n_rows,
               long long p_lo, int lag, int n_steps, float *v, unsigned long long limit_ns, cudaStream_t s)
{
    if (n_rows <= 0 || n_steps <= 0) return WRNN_OK;
    const int n0 = n_steps + n->reach;                       // positions of x_0 a segment needs
    int rc = ensure_acts(n, n_rows, n0);
    if (rc != WRNN_OK) return rc;
    if (cudaMemsetAsync(n->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    subnet_input_kernel<<<dim3(n0, n_rows), 256, 0, s>>>(hist, n->W_in, n->b_in, n->B, L, n->res_ch, r_lo, p_lo, lag, n->n_alloc, n0, n->xf, n->xh, n->xl);
    ++g_launches;
    SubnetGemmParams p;
    std::memset(&p, 0, sizeof(p));
    p.n_alloc = n->n_alloc; p.r_lo = r_lo; p.p_lo = p_lo; p.lag = lag; p.L = L; p.status = n->status; p.limit_ns = limit_ns;
    int need = n0;                                           // positions of x_l still needed
    for (int l = 0; l < n->n_layers; ++l) {
        const int d = n->dilation[l];
        need -= (n->taps - 1) * d;                           // positions of a_l and x_{l+1}
        const int mtiles = (need + SN_BM - 1) / SN_BM;
        // a_l = relu(conv): K = taps x res_ch, N = conv_ch
        p.n_kb_tap = n->res_ch / TC_BK; p.taps = n->taps; p.dil = d; p.w_row0 = l * n->taps * n->conv_ch; p.w_tap_rows = n->conv_ch;
        p.n_pos = need; p.C_out = n->conv_ch; p.bias = n->b_conv + (size_t)l * n->conv_ch; p.oh = n->ah; p.ol = n->al; p.xf = nullptr; p.relu_parts = 0;
        pdl_launch(subnet_gemm_kernel<SN_BN_CONV, SN_CONV, SN_ST_CONV>, dim3(n->conv_ch / SN_BN_CONV, mtiles, n_rows), sn_smem<SN_BN_CONV, SN_ST_CONV>(), s,
                   n->tmXh, n->tmXl, n->tmWc, p);
        // x_{l+1} = x_l + W_res a_l + b_res: K = conv_ch, N = res_ch
        p.n_kb_tap = n->conv_ch / TC_BK; p.taps = 1; p.dil = 0; p.w_row0 = l * n->res_ch; p.w_tap_rows = 0;
        p.C_out = n->res_ch; p.bias = n->b_res + (size_t)l * n->res_ch; p.oh = n->xh; p.ol = n->xl; p.xf = n->xf; p.relu_parts = l == n->n_layers - 1;
        pdl_launch(subnet_gemm_kernel<SN_BN_RES, SN_RES, SN_ST_RES>, dim3(n->res_ch / SN_BN_RES, mtiles, n_rows), sn_smem<SN_BN_RES, SN_ST_RES>(), s,
                   n->tmAh, n->tmAl, n->tmWr, p);
        g_launches += 2;
    }
    // v = frames + W_out relu(x_last) + b_out
    p.n_kb_tap = n->res_ch / TC_BK; p.taps = 1; p.dil = 0; p.w_row0 = 0; p.w_tap_rows = 0; p.n_pos = n_steps; p.C_out = 0; p.bias = nullptr;
    p.v = v; p.n_steps = n_steps; p.cond_dim = n->cond_dim; p.frames = frames; p.n_frames = n_frames; p.hop = hop; p.Bsub = n->B; p.b_out = n->b_out;
    pdl_launch(subnet_gemm_kernel<SN_BN_OUT, SN_OUT, SN_ST_OUT>, dim3(1, (n_steps + SN_BM - 1) / SN_BM, n_rows), sn_smem<SN_BN_OUT, SN_ST_OUT>(), s,
               n->tmXh, n->tmXl, n->tmWo, p);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) { n->err = "conditioning network launch failed"; return WRNN_ERR_CUDA; }
    return WRNN_OK;
}

int subnet_reach(const wrnn_subscale_net *n) { return n->reach; }
int subnet_B(const wrnn_subscale_net *n) { return n->B; }
int subnet_cond_dim(const wrnn_subscale_net *n) { return n->cond_dim; }
int subnet_status(wrnn_subscale_net *n)
{
    DevStatus st;
    if (cudaMemcpy(&st, n->status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) return WRNN_ERR_CUDA;
    return st.code == DEV_OK ? WRNN_OK : WRNN_ERR_TIMEOUT;
}

}  // namespace wrnn

using namespace wrnn;

extern "C" int wrnn_subscale_net_create(const wrnn_subscale_net_params *q, wrnn_subscale_net **out)
{
    if (out) *out = nullptr;
    if (!q || !out || !q->dilation || !q->W_in || !q->b_in || !q->W_conv || !q->b_conv || !q->W_res || !q->b_res || !q->W_out || !q->b_out)
        return WRNN_ERR_INVALID_ARG;
    if (q->B < 1 || q->B > 64 || q->n_layers < 1 || q->n_layers > 64 || q->taps < 1 || q->taps > 8 || q->cond_dim < 1 || q->cond_dim > 64)
        return WRNN_ERR_INVALID_ARG;
    // the tensor-core tiling: whole 64-wide k-blocks and whole channel tiles
    if (q->conv_ch < SN_BN_CONV || q->conv_ch % SN_BN_CONV || q->res_ch < SN_BN_RES || q->res_ch % SN_BN_RES) return WRNN_ERR_UNSUPPORTED;
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { cudaGetLastError(); return WRNN_ERR_CUDA; }
    if (prop.major != 10) return WRNN_ERR_UNSUPPORTED;
    wrnn_subscale_net *n = new (std::nothrow) wrnn_subscale_net();
    if (!n) return WRNN_ERR_NOMEM;
    n->B = q->B; n->n_layers = q->n_layers; n->taps = q->taps; n->conv_ch = q->conv_ch; n->res_ch = q->res_ch; n->cond_dim = q->cond_dim; n->device = dev;
    n->dilation.assign(q->dilation, q->dilation + q->n_layers);
    n->reach = 0;
    for (int d : n->dilation) {
        if (d < 1 || d > SN_BM / 2) { delete n; return WRNN_ERR_INVALID_ARG; }
        n->reach += (q->taps - 1) * d;
    }
    const size_t nc = (size_t)q->n_layers * q->taps * q->conv_ch * q->res_ch, nr = (size_t)q->n_layers * q->res_ch * q->conv_ch;
    std::vector<float> win((size_t)q->res_ch * q->B);
    for (size_t i = 0; i < win.size(); ++i) win[i] = round_bf16_host(q->W_in[i]);
    bool ok = upload_bf16(&n->Wc, q->W_conv, nc, nc) && upload_bf16(&n->Wr, q->W_res, nr, nr) &&
              upload_bf16(&n->Wo, q->W_out, (size_t)q->cond_dim * q->res_ch, (size_t)64 * q->res_ch) &&
              upload_f32(&n->W_in, win.data(), win.size()) && upload_f32(&n->b_in, q->b_in, q->res_ch) &&
              upload_f32(&n->b_conv, q->b_conv, (size_t)q->n_layers * q->conv_ch) && upload_f32(&n->b_res, q->b_res, (size_t)q->n_layers * q->res_ch) &&
              upload_f32(&n->b_out, q->b_out, q->cond_dim) && cudaMalloc((void **)&n->status, sizeof(DevStatus)) == cudaSuccess &&
              cudaMemset(n->status, 0, sizeof(DevStatus)) == cudaSuccess;
    ok = ok && make_map(&n->tmWc, n->Wc, (long long)q->n_layers * q->taps * q->conv_ch, q->res_ch, SN_BN_CONV) &&
         make_map(&n->tmWr, n->Wr, (long long)q->n_layers * q->res_ch, q->conv_ch, SN_BN_RES) && make_map(&n->tmWo, n->Wo, 64, q->res_ch, SN_BN_OUT);
    ok = ok && cudaFuncSetAttribute(subnet_gemm_kernel<SN_BN_CONV, SN_CONV, SN_ST_CONV>, cudaFuncAttributeMaxDynamicSharedMemorySize, sn_smem<SN_BN_CONV, SN_ST_CONV>()) == cudaSuccess &&
         cudaFuncSetAttribute(subnet_gemm_kernel<SN_BN_RES, SN_RES, SN_ST_RES>, cudaFuncAttributeMaxDynamicSharedMemorySize, sn_smem<SN_BN_RES, SN_ST_RES>()) == cudaSuccess &&
         cudaFuncSetAttribute(subnet_gemm_kernel<SN_BN_OUT, SN_OUT, SN_ST_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, sn_smem<SN_BN_OUT, SN_ST_OUT>()) == cudaSuccess;
    if (!ok) { cudaGetLastError(); wrnn_subscale_net_destroy(n); return WRNN_ERR_NOMEM; }
    *out = n;
    return WRNN_OK;
}

extern "C" void wrnn_subscale_net_destroy(wrnn_subscale_net *n)
{
    if (!n) return;
    cudaSetDevice(n->device);
    cudaDeviceSynchronize();
    free_acts(n);
    cudaFree(n->Wc); cudaFree(n->Wr); cudaFree(n->Wo); cudaFree(n->W_in); cudaFree(n->b_in); cudaFree(n->b_conv); cudaFree(n->b_res);
    cudaFree(n->b_out); cudaFree(n->status);
    cudaGetLastError();
    delete n;
}

extern "C" int wrnn_subscale_net_conditioning(wrnn_subscale_net *n, const int16_t *hist, const float *frames, int32_t n_frames, int32_t hop,
                                              int32_t row, int64_t L, float *v, void *cuda_stream)
{
    if (!n || !hist || !frames || !v || hop < 1 || row < 0 || row >= n->B || L < 1 || L > (1ll << 24)) return WRNN_ERR_INVALID_ARG;
    if (((long long)n->B * (L - 1) + row) / hop >= n_frames) return WRNN_ERR_INVALID_ARG;
    if (cudaSetDevice(n->device) != cudaSuccess) return WRNN_ERR_CUDA;
    return subnet_run(n, hist, frames, n_frames, hop, L, row, 1, 0, 0, (int)L, v, 2000000000ull, (cudaStream_t)cuda_stream);
}

extern "C" int wrnn_subscale_net_status(wrnn_subscale_net *n) { return n ? subnet_status(n) : WRNN_ERR_INVALID_ARG; }
