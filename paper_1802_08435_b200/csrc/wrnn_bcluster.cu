// Cluster-partitioned multi-row kernel (dense bf16 models, 2 or more rows advancing in lock step: the folded
// sub-tensors of Section 4 and the batched form of Section 2's sampling step).
//
// The rows of a batch are independent streams, so the batch is cut into groups of up to 64 rows and each group
// is given to one thread-block cluster of 16 CTAs.  Nothing ever crosses a cluster: the nine phases of a step
// (Fig. 1, Eq. 2) are separated by hardware cluster barriers instead of grid-wide ones, and clusters drift
// freely against one another.  Inside a cluster the weight rows are dealt out in chunks of eight rows:
//
//   A    a = R h_{t-1}                 CTA c holds the (u, r, e) rows of hidden-unit chunks c, c+16, c+32, ...
//   Gc   coarse gates -> y_c           in the epilogue of A, straight from the TMEM accumulator
//   O1   q_c = relu(O1 y_c + b1)       chunks c, c+16, ... of the hidden layer
//   O2   l_c = O2 q_c + b2             logits 16 c .. 16 c + 15
//   Sc   draw c_t                      one warp per row, rows c, c+16, ... of the group
//   Gf   fine gates -> y_f             the fine columns of A's accumulator, still in TMEM, now that c_t is known
//   O3, O4, Sf                         the fine head, then the sample 256 c_t + f_t - 32768
//
// Every contraction runs on the fifth-generation tensor cores.  The activations are the M side: the rows of a
// group are stacked as a 128-row operand whose lane quadrant q holds the bf16 high parts of rows 16 q .. 16 q + 15
// in lanes 0-15 and the low parts (x - bf16(x)) in lanes 16-31, so that one tcgen05.mma (M = 128, N = the CTA's
// weight rows, K = 16) yields both partial products and the epilogue adds them with one shuffle.  The weights are
// the N side, streamed every step from L2 (they are shared by all clusters) by TMA with the 128-byte swizzle,
// together with the activation tile, through an mbarrier ring; accumulators live in TMEM (A: columns 0-255,
// kept until Gf; O1 / O3: 256-287; O2 / O4: 320-335).  The fp32 hidden state of a (row, chunk) pair never
// leaves the registers of the thread that owns it; only its bf16 high / low split is written out (to L2, in the
// operand layout) for the next contractions.  Every mbarrier wait is bounded; a CTA whose wait ran out records
// it, skips its remaining work and keeps arriving at the cluster barriers so that the launch drains cleanly.
#include <cuda_bf16.h>

#include <cstdlib>
#include <cstring>

#include "wrnn_internal.h"
#include "wrnn_tc.cuh"

namespace wrnn {

constexpr int BC_CS = 16;             // CTAs per cluster
constexpr int BC_THREADS = 512;
constexpr int BC_MAX_STAGES = 8;
constexpr int BC_SLACK = 16384;       // the 128-row A operand may read this far past a short activation tile
constexpr int BC_MROWS = 128;         // rows of the activation arrays reserved per cluster
constexpr int BC_GROUP = 64;          // most rows of a batch one cluster takes
constexpr int BC_COL_A = 0, BC_COL_O1 = 256, BC_COL_O2 = 320, BC_TMEM_COLS = 512;

struct BcPack {
    int H = 0, NCH = 0, NRp = 0, NOC = 0, NO1 = 0;
    __nv_bfloat16 *Wr = nullptr, *O1p = nullptr, *O2p = nullptr, *O3p = nullptr, *O4p = nullptr;   // [16][rows per CTA][K]
    float4 *Ip = nullptr;                                   // [16][3][64]: I of the CTA's gate rows
    __nv_bfloat16 *act[2] = {nullptr, nullptr};             // [clusters * 128][H]   stacked high / low state
    __nv_bfloat16 *q = nullptr;                             // [clusters * 128][H/2] stacked hidden layer
    float *logits = nullptr;                                // [max rows][256]
    uint8_t *c_cur = nullptr, *c_prev = nullptr, *f_prev = nullptr;
    CUtensorMap tmWr, tmO1, tmO2, tmO3, tmO4;
    int max_clusters = 0, max_dyn_smem = 0;
    int64_t weight_bytes = 0;
};

struct BcParams {
    int H, Hh, G, batch, RB, MR, NCH, NRp, NO1, n_stages, stage_bytes;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    const float4 *Ip;
    const float *b1, *b2, *b3, *b4, *g;
    __nv_bfloat16 *act0, *act1, *q;
    float *logits;
    uint8_t *c_cur, *c_prev, *f_prev;
    const float *h_in; float *h_out;
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;
    uint8_t *c_out, *f_out;
    int16_t *out;
    float *dbg_gates, *dbg_h, *dbg_logits;
    DevStatus *status;
    alignas(64) CUtensorMap tmWr;
    alignas(64) CUtensorMap tmO1;
    alignas(64) CUtensorMap tmO2;
    alignas(64) CUtensorMap tmO3;
    alignas(64) CUtensorMap tmO4;
    alignas(64) CUtensorMap tmAct[2];
    alignas(64) CUtensorMap tmQ;
};

// all threads of all CTAs of the cluster; orders global-memory and TMEM traffic across it
__device__ __forceinline__ void cluster_barrier()
{
    tc_fence_before();
    asm volatile("barrier.cluster.arrive.release;\nbarrier.cluster.wait.acquire;" ::: "memory");
    tc_fence_after();
}

__device__ __forceinline__ uint4 pack8_bf16(const __nv_bfloat16 (&v)[8])
{
    uint4 o;
    o.x = (uint32_t)__bfloat16_as_ushort(v[0]) | ((uint32_t)__bfloat16_as_ushort(v[1]) << 16);
    o.y = (uint32_t)__bfloat16_as_ushort(v[2]) | ((uint32_t)__bfloat16_as_ushort(v[3]) << 16);
    o.z = (uint32_t)__bfloat16_as_ushort(v[4]) | ((uint32_t)__bfloat16_as_ushort(v[5]) << 16);
    o.w = (uint32_t)__bfloat16_as_ushort(v[6]) | ((uint32_t)__bfloat16_as_ushort(v[7]) << 16);
    return o;
}

// Eight values -> their bf16 high parts at `hi` and low parts at `lo` (16-byte stores).
__device__ __forceinline__ void store_split8(__nv_bfloat16 *hi, __nv_bfloat16 *lo, const float (&x)[8])
{
    __nv_bfloat16 h[8], l[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        h[e] = __float2bfloat16_rn(x[e]);
        l[e] = __float2bfloat16_rn(x[e] - __bfloat162float(h[e]));
    }
    *reinterpret_cast<uint4 *>(hi) = pack8_bf16(h);
    *reinterpret_cast<uint4 *>(lo) = pack8_bf16(l);
}

#ifdef WRNN_PROFILE_BC
__device__ long long g_bcprof[32];
#define CSTAMP(i) do { if (blockIdx.x == 0 && threadIdx.x == 96) { const long long n_ = clock64(); g_bcprof[i] += n_ - bt_; bt_ = n_; } } while (0)
#else
#define CSTAMP(i) do { } while (0)
#endif

__global__ void __launch_bounds__(BC_THREADS, 1) bcluster_step_kernel(const __grid_constant__ BcParams p)
{
#ifdef WRNN_PROFILE_BC
    long long bt_ = clock64();
#endif
    extern __shared__ __align__(16) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t s_full[BC_MAX_STAGES], s_empty[BC_MAX_STAGES], s_done;
    __shared__ uint32_t s_tmem;
    __shared__ int s_failed;
    __shared__ float4 s_I[3 * 64];                  // [gate][unit of this CTA] -> (I0, I1, I2, -)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned crank;
    asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
    const int cl = blockIdx.x / BC_CS;
    const int row0 = cl * p.RB;
    const int nrows = min(p.RB, p.batch - row0);
    if (nrows <= 0) return;                         // the same for every CTA of the cluster
    const int H = p.H, Hh = p.Hh, NCH = p.NCH;

    // ---- fixed roles of this thread
    const int qd = warp & 3, slot = warp >> 2, half = lane >> 4, lr = lane & 15;
    const int nQ = (nrows + 15) >> 4;               // lane quadrants in use
    const int bl = 16 * qd + lr;                    // row of the group this lane serves in the epilogues
    const bool rowv = bl < nrows;
    const int gb = row0 + bl;                       // its row of the batch
    const int ci = 2 * slot + half;                 // gate chunk of this thread (8 hidden units)
    const int gch = (int)crank + BC_CS * ci;
    const bool chv = ci < NCH && gch < H / 8;
    const bool ch_coarse = gch < Hh / 8;
    const int unit0 = 8 * gch;
    const size_t arow_hi = (size_t)cl * BC_MROWS + 32 * qd + lr, arow_lo = arow_hi + 16;
    // warp-uniform: does either chunk of this warp belong to the coarse / fine half
    const int gch_a = (int)crank + BC_CS * (2 * slot), gch_b = gch_a + BC_CS;
    const bool va = 2 * slot < NCH && gch_a < H / 8, vb = 2 * slot + 1 < NCH && gch_b < H / 8;
    const bool warp_coarse = (va && gch_a < Hh / 8) || (vb && gch_b < Hh / 8);
    const bool warp_fine = (va && gch_a >= Hh / 8) || (vb && gch_b >= Hh / 8);
    // hidden-layer chunk (8 outputs of O1 / O3) of this warp
    const int och = (int)crank + BC_CS * slot;
    const bool ochv = och < Hh / 8;

    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t ring0 = smem_u32(ring);
    const uint32_t done_bar = smem_u32(&s_done);
    volatile int *failed = &s_failed;

    if (tid == 0) {
        for (int i = 0; i < BC_MAX_STAGES; ++i) { mbar_init(smem_u32(&s_full[i]), 2); mbar_init(smem_u32(&s_empty[i]), 1); }
        mbar_init(done_bar, 1);
        s_failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(BC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    for (int i = tid; i < 3 * 64; i += BC_THREADS) s_I[i] = p.Ip[(size_t)crank * 3 * 64 + i];
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;

    auto fail = [&](int step, int phase) {
        *failed = 1;
        if (atomicCAS(&p.status->code, DEV_OK, DEV_TIMEOUT) == DEV_OK) { p.status->cta = blockIdx.x; p.status->step = step; p.status->phase = phase; }
    };

    // ---- initial state: fp32 in registers, stacked high / low image in buffer 0 (other rows of the image stay zero)
    float hreg[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) hreg[e] = (rowv && chv && p.h_in) ? p.h_in[(size_t)gb * H + unit0 + e] : 0.f;
    if (rowv && chv && qd < nQ) store_split8(p.act0 + arow_hi * H + unit0, p.act0 + arow_lo * H + unit0, hreg);
    if (tid < 4) {
        const int r = (int)crank + BC_CS * tid;
        if (r < nrows) {
            p.c_prev[row0 + r] = p.c_in ? p.c_in[row0 + r] : (uint8_t)128;
            p.f_prev[row0 + r] = p.f_in ? p.f_in[row0 + r] : (uint8_t)0;
        }
    }
    fence_proxy_async();
    cluster_barrier();

    // ring position of the three role threads (they walk the same sequence of k-blocks) and parity of `done`
    int rst = 0;
    uint32_t rph = 0, dph = 0;
    const uint32_t abytes = (uint32_t)p.MR * 128u;

    // One contraction: D[128 x n_w] (TMEM column dcol) = activations[cluster rows, columns ax ..] . W[rows wy ..]^T over nkb
    // k-blocks of 64.  warp 0 / lane 0 loads the activation tiles, warp 2 / lane 0 the weight tiles, warp 1 / lane 0
    // issues the MMAs; every thread returns once the accumulator is complete.
    auto gemm = [&](const CUtensorMap *tmA, int ax, const CUtensorMap *tmW, int wy, int nkb, int n_w, uint32_t dcol, int step, int phase) {
        if (lane == 0 && warp < 3 && !*failed) {
            if (warp == 1) {
                const uint32_t idesc = umma_idesc_bf16(128, n_w);
                bool ok = true;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(smem_u32(&s_full[rst]), rph)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t base = ring0 + (uint32_t)rst * (uint32_t)p.stage_bytes;
                    const uint64_t da = umma_desc_sw128(base), db = umma_desc_sw128(base + abytes);
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k) umma_bf16(tmem + dcol, da + 2 * k, db + 2 * k, idesc, (kb | k) ? 1u : 0u);
                    umma_commit(smem_u32(&s_empty[rst]));
                    if (++rst == p.n_stages) { rst = 0; rph ^= 1; }
                }
                if (ok) umma_commit(done_bar);
                else fail(step, phase);
            } else {
                const bool is_act = warp == 0;
                const uint32_t bytes = is_act ? abytes : (uint32_t)n_w * 128u;
                const CUtensorMap *tm = is_act ? tmA : tmW;
                const int x0 = is_act ? ax : 0, y = is_act ? cl * BC_MROWS : wy;
                const uint32_t off = is_act ? 0u : abytes;
                fence_proxy_async();               // earlier generic-proxy writes of the activations, by this and (through the barrier) other CTAs
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(smem_u32(&s_empty[rst]), rph ^ 1)) { fail(step, phase); break; }
                    const uint32_t fb = smem_u32(&s_full[rst]);
                    mbar_expect_tx(fb, bytes);
                    tma_load_2d(ring0 + (uint32_t)rst * (uint32_t)p.stage_bytes + off, tm, fb, x0 + kb * TC_BK, y);
                    if (++rst == p.n_stages) { rst = 0; rph ^= 1; }
                }
            }
        }
        __syncwarp();
        if (!*failed && !mbar_wait(done_bar, dph)) fail(step, phase);
        dph ^= 1;
        tc_fence_after();
    };

    // Gates of Eq. 2 for the chunks of one half (coarse: x2 = 0; fine: x2 = c_t), from the accumulator of phase A.
    auto gates = [&](bool coarse, long long s, float x0, float x1, float x2, const float *grow, __nv_bfloat16 *anext) {
        if (qd >= nQ || !(coarse ? warp_coarse : warp_fine)) return;
        // columns of gate g of chunk i: 8 NCH g + 8 i; both chunks of the warp are read by all lanes
        float a[3][8], b[3][8];
        const uint32_t t0 = tmem + ((uint32_t)(32 * qd) << 16) + BC_COL_A + 16 * slot;
#pragma unroll
        for (int g = 0; g < 3; ++g) { tmem_ld8(t0 + 8 * NCH * g, a[g]); tmem_ld8(t0 + 8 * NCH * g + 8, b[g]); }
        tmem_wait_ld();
        // lanes 0-15 hold the high-part products of a row, lanes 16-31 the low-part ones: the lower half-warp takes
        // chunk a, the upper chunk b, each adding the other half's partial
        float acc[3][8];
#pragma unroll
        for (int g = 0; g < 3; ++g)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float send = half ? a[g][e] : b[g][e];
                const float recv = __shfl_xor_sync(0xffffffffu, send, 16);
                acc[g][e] = (half ? b[g][e] : a[g][e]) + recv;
            }
        if (!(rowv && chv && ch_coarse == coarse)) return;
        float gu[8], gr[8], ge[8];
        {
            const float4 *g4 = reinterpret_cast<const float4 *>(grow + unit0);
            const float4 u0 = __ldg(g4), u1 = __ldg(g4 + 1);
            const float4 *r4 = reinterpret_cast<const float4 *>(grow + H + unit0);
            const float4 r0 = __ldg(r4), r1 = __ldg(r4 + 1);
            const float4 *e4 = reinterpret_cast<const float4 *>(grow + 2 * H + unit0);
            const float4 e0 = __ldg(e4), e1 = __ldg(e4 + 1);
            gu[0] = u0.x; gu[1] = u0.y; gu[2] = u0.z; gu[3] = u0.w; gu[4] = u1.x; gu[5] = u1.y; gu[6] = u1.z; gu[7] = u1.w;
            gr[0] = r0.x; gr[1] = r0.y; gr[2] = r0.z; gr[3] = r0.w; gr[4] = r1.x; gr[5] = r1.y; gr[6] = r1.z; gr[7] = r1.w;
            ge[0] = e0.x; ge[1] = e0.y; ge[2] = e0.z; ge[3] = e0.w; ge[4] = e1.x; ge[5] = e1.y; ge[6] = e1.z; ge[7] = e1.w;
        }
        float uu[8], rr[8], ee[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float4 Iu = s_I[8 * ci + e], Ir = s_I[64 + 8 * ci + e], Ie = s_I[128 + 8 * ci + e];
            const float pu = acc[0][e] + fmaf(Iu.x, x0, fmaf(Iu.y, x1, fmaf(Iu.z, x2, gu[e])));
            const float pr = acc[1][e] + fmaf(Ir.x, x0, fmaf(Ir.y, x1, fmaf(Ir.z, x2, gr[e])));
            const float pe = fmaf(Ie.x, x0, fmaf(Ie.y, x1, fmaf(Ie.z, x2, ge[e])));
            uu[e] = sigmoidf_acc(pu);
            rr[e] = sigmoidf_acc(pr);
            ee[e] = tanhf(fmaf(rr[e], acc[2][e], pe));
            hreg[e] = fmaf(uu[e], hreg[e], (1.0f - uu[e]) * ee[e]);
        }
        store_split8(anext + arow_hi * H + unit0, anext + arow_lo * H + unit0, hreg);
        if (p.dbg_gates) {
            float *d = p.dbg_gates + ((size_t)s * p.batch + gb) * p.G + unit0;
#pragma unroll
            for (int e = 0; e < 8; ++e) { d[e] = uu[e]; d[H + e] = rr[e]; d[2 * H + e] = ee[e]; }
        }
        if (p.dbg_h) {
            float *d = p.dbg_h + ((size_t)s * p.batch + gb) * H + unit0;
#pragma unroll
            for (int e = 0; e < 8; ++e) d[e] = hreg[e];
        }
    };

    for (long long s = 0; s < p.n_steps; ++s) {
        __nv_bfloat16 *anext = (s & 1) ? p.act0 : p.act1;
        const int cur = (int)(s & 1);
        // inputs of the gates that do not depend on this step's contractions
        float x0 = 0.f, x1 = 0.f;
        const float *grow = p.g;
        if (rowv) {
            x0 = scale8(__ldcg(p.c_prev + gb));
            x1 = scale8(__ldcg(p.f_prev + gb));
            const long long frame = ((p.step0 + s) * p.row_stride + (long long)(p.stream0 + (unsigned)gb) * p.row_offset_mul) / p.hop;
            grow = p.g + ((size_t)gb * p.n_frames + (size_t)frame) * p.G;
        }
        // ---- A + Gc
        CSTAMP(0);
        gemm(&p.tmAct[cur], 0, &p.tmWr, (int)crank * p.NRp, H / TC_BK, p.NRp, BC_COL_A, (int)s, 1);
        CSTAMP(1);
        gates(true, s, x0, x1, 0.f, grow, anext);
        fence_proxy_async();
        CSTAMP(2);
        cluster_barrier();
        CSTAMP(3);

        for (int head = 0; head < 2; ++head) {
            const float *ba = head ? p.b3 : p.b1, *bb = head ? p.b4 : p.b2;
            // ---- O1 / O3: hidden layer on this half of the new state
            gemm(&p.tmAct[cur ^ 1], head * Hh, head ? &p.tmO3 : &p.tmO1, (int)crank * p.NO1, Hh / TC_BK, p.NO1, BC_COL_O1, (int)s, 2 + 4 * head);
            CSTAMP(4 + 8 * head);
            if (qd < nQ && 8 * slot < p.NO1) {
                float v[8];
                tmem_ld8(tmem + ((uint32_t)(32 * qd) << 16) + BC_COL_O1 + 8 * slot, v);
                tmem_wait_ld();
                float x[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float t = v[e] + __shfl_xor_sync(0xffffffffu, v[e], 16);
                    x[e] = ochv ? fmaxf(t + (ba ? __ldg(ba + 8 * och + e) : 0.f), 0.f) : 0.f;
                }
                if (rowv && ochv) {
                    // both half-warps hold the sums: the lower writes the high parts, the upper the low parts
                    __nv_bfloat16 o[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const __nv_bfloat16 hi = __float2bfloat16_rn(x[e]);
                        o[e] = half ? __float2bfloat16_rn(x[e] - __bfloat162float(hi)) : hi;
                    }
                    *reinterpret_cast<uint4 *>(p.q + (half ? arow_lo : arow_hi) * Hh + 8 * och) = pack8_bf16(o);
                }
            }
            fence_proxy_async();
            CSTAMP(5 + 8 * head);
            cluster_barrier();
            CSTAMP(6 + 8 * head);
            // ---- O2 / O4: logits 16 crank .. + 15
            gemm(&p.tmQ, 0, head ? &p.tmO4 : &p.tmO2, (int)crank * 16, Hh / TC_BK, 16, BC_COL_O2, (int)s, 3 + 4 * head);
            CSTAMP(7 + 8 * head);
            if (qd < nQ && slot < 2) {
                float v[8];
                tmem_ld8(tmem + ((uint32_t)(32 * qd) << 16) + BC_COL_O2 + 8 * slot, v);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] += __shfl_xor_sync(0xffffffffu, v[e], 16);
                if (rowv) {
                    const int r0 = 16 * (int)crank + 8 * slot + 4 * half;      // four logits per lane
                    float4 o;
                    o.x = (half ? v[4] : v[0]) + (bb ? __ldg(bb + r0 + 0) : 0.f);
                    o.y = (half ? v[5] : v[1]) + (bb ? __ldg(bb + r0 + 1) : 0.f);
                    o.z = (half ? v[6] : v[2]) + (bb ? __ldg(bb + r0 + 2) : 0.f);
                    o.w = (half ? v[7] : v[3]) + (bb ? __ldg(bb + r0 + 3) : 0.f);
                    *reinterpret_cast<float4 *>(p.logits + (size_t)gb * 256 + r0) = o;
                    if (p.dbg_logits) *reinterpret_cast<float4 *>(p.dbg_logits + (((size_t)s * p.batch + gb) * 2 + head) * 256 + r0) = o;
                }
            }
            CSTAMP(8 + 8 * head);
            cluster_barrier();
            CSTAMP(9 + 8 * head);
            // ---- Sc / Sf: softmax + inverse-CDF draw, one warp per row
            if (warp < 4) {
                const int r = (int)crank + BC_CS * warp;
                if (r < nrows) {
                    const int sb = row0 + r;
                    float l[8];
                    const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(p.logits + (size_t)sb * 256 + 8 * lane));
                    const float4 v1 = __ldcg(reinterpret_cast<const float4 *>(p.logits + (size_t)sb * 256 + 8 * lane + 4));
                    l[0] = v0.x; l[1] = v0.y; l[2] = v0.z; l[3] = v0.w; l[4] = v1.x; l[5] = v1.y; l[6] = v1.z; l[7] = v1.w;
                    const float u = uniform24(p.seed, p.stream0 + (unsigned)sb, (unsigned long long)(p.step0 + s), head);
                    int idx = warp_softmax_draw(l, u, lane);
                    const size_t o = (size_t)sb * p.n_steps + s;
                    if (lane == 0) {
                        if (head == 0) {
                            if (p.c_out) p.c_out[o] = (uint8_t)idx;
                            if (p.c_forced) idx = p.c_forced[o];
                            p.c_cur[sb] = (uint8_t)idx;
                        } else {
                            if (p.f_out) p.f_out[o] = (uint8_t)idx;
                            if (p.f_forced) idx = p.f_forced[o];
                            const int c = __ldcg(p.c_cur + sb);
                            if (p.out) p.out[o] = (int16_t)(256 * c + idx - 32768);
                            p.c_prev[sb] = (uint8_t)c;
                            p.f_prev[sb] = (uint8_t)idx;
                        }
                    }
                }
            }
            CSTAMP(10 + 8 * head);
            cluster_barrier();
            CSTAMP(11 + 8 * head);
            if (head == 0) {
                // ---- Gf: fine gates, now that c_t is known (it reaches only these rows, Section 2)
                const float x2 = rowv ? scale8(__ldcg(p.c_cur + gb)) : 0.f;
                gates(false, s, x0, x1, x2, grow, anext);
                fence_proxy_async();
                CSTAMP(20);
                cluster_barrier();
                CSTAMP(21);
            }
        }
    }

    if (p.h_out && rowv && chv && qd < nQ) {
#pragma unroll
        for (int e = 0; e < 8; ++e) p.h_out[(size_t)gb * H + unit0 + e] = hreg[e];
    }
    if (tid < 4) {
        const int r = (int)crank + BC_CS * tid;
        if (r < nrows) {
            if (p.c_st_out) p.c_st_out[row0 + r] = __ldcg(p.c_prev + row0 + r);
            if (p.f_st_out) p.f_st_out[row0 + r] = __ldcg(p.f_prev + row0 + r);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(BC_TMEM_COLS) : "memory");
    cluster_barrier();      // no CTA leaves while a peer may still be inside a cluster barrier sequence
}

// ---------------------------------------------------------------------------------------------
static int round_up(int x, int m) { return (x + m - 1) / m * m; }

// rows of a dense matrix (bf16 bits, `cols` wide) dealt out in chunks of 8 rows: CTA c gets chunks c, c + 16, ... of each
// of the `gates` row blocks of `rows_per_gate` rows, laid out [c][gate][chunk slot][8] and padded with zero rows to rp rows
static std::vector<uint16_t> deal_rows(const std::vector<uint16_t> &dense, int cols, int gates, int rows_per_gate, int nch, int rp)
{
    std::vector<uint16_t> out((size_t)BC_CS * rp * cols, 0);
    for (int c = 0; c < BC_CS; ++c)
        for (int g = 0; g < gates; ++g)
            for (int i = 0; i < nch; ++i) {
                const int ch = c + BC_CS * i;
                if (ch >= rows_per_gate / 8) continue;
                for (int e = 0; e < 8; ++e)
                    std::memcpy(&out[((size_t)c * rp + (size_t)g * 8 * nch + 8 * i + e) * cols],
                                &dense[((size_t)g * rows_per_gate + 8 * ch + e) * cols], (size_t)cols * 2);
            }
    return out;
}

int bcluster_supported(const wrnn_model *m, int batch, std::string *why)
{
    if (!m->bcluster) { if (why) *why = "model was not packed for the cluster-partitioned kernel"; return WRNN_ERR_UNSUPPORTED; }
    if (batch < 2) { if (why) *why = "cluster-partitioned kernel needs at least two rows"; return WRNN_ERR_UNSUPPORTED; }
    if (batch > m->bcluster->max_clusters * BC_GROUP) { if (why) *why = "batch exceeds 64 rows per co-resident cluster"; return WRNN_ERR_UNSUPPORTED; }
    return WRNN_OK;
}

static void bc_geometry(const BcPack &k, int batch, int *n_cl, int *RB, int *MR, int *stage_bytes, int *n_stages, int *smem)
{
    int ncl = (batch + 15) / 16;
    if (ncl > k.max_clusters) ncl = k.max_clusters;
    const int rb = (batch + ncl - 1) / ncl;
    *n_cl = (batch + rb - 1) / rb;
    *RB = rb;
    *MR = 32 * ((rb + 15) / 16);
    *stage_bytes = (*MR + k.NRp) * 128;
    int ns = (k.max_dyn_smem - 1024 - BC_SLACK) / *stage_bytes;
    if (ns > BC_MAX_STAGES) ns = BC_MAX_STAGES;
    *n_stages = ns;
    *smem = ns * *stage_bytes + 1024 + BC_SLACK;
}

int bcluster_prepare(wrnn_model *m)
{
    if (m->dtype != WRNN_BF16 || m->sparse) { m->err = "cluster-partitioned kernel takes dense bf16 models"; return WRNN_ERR_UNSUPPORTED; }
    if (m->H % 128 != 0 || m->H > 1024) { m->err = "cluster-partitioned kernel needs H to be a multiple of 128, at most 1024"; return WRNN_ERR_UNSUPPORTED; }
    if (m->max_batch < 2) { m->err = "max_batch < 2"; return WRNN_ERR_UNSUPPORTED; }
    if (!encode_tiled_fn()) { m->err = "driver has no tensor-map encoder"; return WRNN_ERR_UNSUPPORTED; }
    BcPack *k = new BcPack();
    m->bcluster = k;
    const int H = m->H, Hh = H / 2;
    k->H = H;
    k->NCH = (H / 8 + BC_CS - 1) / BC_CS;
    k->NRp = round_up(24 * k->NCH, 16);
    k->NOC = (Hh / 8 + BC_CS - 1) / BC_CS;
    k->NO1 = round_up(8 * k->NOC, 16);
    auto failed = [&](const char *msg, int rc) {
        cudaGetLastError();
        bcluster_destroy(m);
        m->err = msg;
        return rc;
    };

    // how many clusters of this shape the device keeps resident
    int dev_smem = 0;
    cudaDeviceGetAttribute(&dev_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, m->device);
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, bcluster_step_kernel) != cudaSuccess) return failed("cluster-partitioned kernel image missing", WRNN_ERR_CUDA);
    k->max_dyn_smem = dev_smem - (int)fa.sharedSizeBytes;
    if (cudaFuncSetAttribute(bcluster_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, k->max_dyn_smem) != cudaSuccess ||
        cudaFuncSetAttribute(bcluster_step_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
        return failed("cluster-partitioned kernel attributes rejected", WRNN_ERR_UNSUPPORTED);
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(BC_CS); cfg.blockDim = dim3(BC_THREADS); cfg.dynamicSmemBytes = (size_t)k->max_dyn_smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = BC_CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, bcluster_step_kernel, &cfg) != cudaSuccess || n < 1)
            return failed("device cannot co-schedule a 16-CTA cluster of this size", WRNN_ERR_UNSUPPORTED);
        k->max_clusters = n;
    }
    if (m->max_batch > k->max_clusters * BC_GROUP) return failed("max_batch exceeds 64 rows per co-resident cluster", WRNN_ERR_UNSUPPORTED);
    {
        int ncl, rb, mr, sb, ns, smem;
        bc_geometry(*k, m->max_batch, &ncl, &rb, &mr, &sb, &ns, &smem);
        if (ns < 2) return failed("shared memory too small for the tile ring", WRNN_ERR_UNSUPPORTED);
    }

    auto up = [&](const std::vector<uint16_t> &v, __nv_bfloat16 **dst) {
        k->weight_bytes += (int64_t)v.size() * 2;
        return cudaMalloc((void **)dst, v.size() * 2) == cudaSuccess && cudaMemcpy(*dst, v.data(), v.size() * 2, cudaMemcpyHostToDevice) == cudaSuccess;
    };
    bool ok = up(deal_rows(dense_bf16_bits(m->hR), H, 3, H, k->NCH, k->NRp), &k->Wr) &&
              up(deal_rows(dense_bf16_bits(m->hO1), Hh, 1, Hh, k->NOC, k->NO1), &k->O1p) &&
              up(deal_rows(dense_bf16_bits(m->hO3), Hh, 1, Hh, k->NOC, k->NO1), &k->O3p) &&
              up(dense_bf16_bits(m->hO2), &k->O2p) && up(dense_bf16_bits(m->hO4), &k->O4p);
    {
        std::vector<float4> Ih((size_t)BC_CS * 3 * 64, make_float4(0.f, 0.f, 0.f, 0.f));
        for (int c = 0; c < BC_CS; ++c)
            for (int g = 0; g < 3; ++g)
                for (int i = 0; i < k->NCH; ++i) {
                    const int ch = c + BC_CS * i;
                    if (ch >= H / 8) continue;
                    for (int e = 0; e < 8; ++e) {
                        const float *src = &m->hI[(size_t)(g * H + 8 * ch + e) * 3];
                        Ih[((size_t)c * 3 + g) * 64 + 8 * i + e] = make_float4(src[0], src[1], src[2], 0.f);
                    }
                }
        ok = ok && cudaMalloc((void **)&k->Ip, Ih.size() * sizeof(float4)) == cudaSuccess &&
             cudaMemcpy(k->Ip, Ih.data(), Ih.size() * sizeof(float4), cudaMemcpyHostToDevice) == cudaSuccess;
    }
    const size_t arows = (size_t)k->max_clusters * BC_MROWS, mb = (size_t)m->max_batch;
    ok = ok && cudaMalloc((void **)&k->act[0], arows * H * 2) == cudaSuccess && cudaMalloc((void **)&k->act[1], arows * H * 2) == cudaSuccess &&
         cudaMalloc((void **)&k->q, arows * Hh * 2) == cudaSuccess && cudaMalloc((void **)&k->logits, mb * 256 * 4) == cudaSuccess &&
         cudaMalloc((void **)&k->c_cur, mb) == cudaSuccess && cudaMalloc((void **)&k->c_prev, mb) == cudaSuccess &&
         cudaMalloc((void **)&k->f_prev, mb) == cudaSuccess;
    ok = ok && make_map(&k->tmWr, k->Wr, (long long)BC_CS * k->NRp, H, k->NRp) && make_map(&k->tmO1, k->O1p, (long long)BC_CS * k->NO1, Hh, k->NO1) &&
         make_map(&k->tmO3, k->O3p, (long long)BC_CS * k->NO1, Hh, k->NO1) && make_map(&k->tmO2, k->O2p, 256, Hh, 16) &&
         make_map(&k->tmO4, k->O4p, 256, Hh, 16);
    if (!ok) return failed("device allocation for the cluster-partitioned kernel failed", WRNN_ERR_NOMEM);
    return WRNN_OK;
}

void bcluster_destroy(wrnn_model *m)
{
    BcPack *k = m->bcluster;
    if (!k) return;
    cudaFree(k->Wr); cudaFree(k->O1p); cudaFree(k->O2p); cudaFree(k->O3p); cudaFree(k->O4p); cudaFree(k->Ip);
    cudaFree(k->act[0]); cudaFree(k->act[1]); cudaFree(k->q); cudaFree(k->logits);
    cudaFree(k->c_cur); cudaFree(k->c_prev); cudaFree(k->f_prev);
    delete k;
    m->bcluster = nullptr;
}

int bcluster_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes)
{
    const BcPack &k = *m->bcluster;
    int ncl, rb, mr, sb, ns, sm;
    bc_geometry(k, batch, &ncl, &rb, &mr, &sb, &ns, &sm);
    if (n_ctas) *n_ctas = ncl * BC_CS;
    if (n_threads) *n_threads = BC_THREADS;
    if (smem) *smem = sm;
    if (weight_bytes) *weight_bytes = k.weight_bytes;
    return WRNN_OK;
}

int bcluster_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    BcPack &k = *m->bcluster;
    BcParams p;
    std::memset(&p, 0, sizeof(p));
    int ncl, smem;
    bc_geometry(k, a.batch, &ncl, &p.RB, &p.MR, &p.stage_bytes, &p.n_stages, &smem);
    p.H = m->H; p.Hh = m->H / 2; p.G = 3 * m->H; p.batch = a.batch;
    p.NCH = k.NCH; p.NRp = k.NRp; p.NO1 = k.NO1;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.Ip = k.Ip; p.b1 = m->b1; p.b2 = m->b2; p.b3 = m->b3; p.b4 = m->b4; p.g = m->g;
    p.act0 = k.act[0]; p.act1 = k.act[1]; p.q = k.q; p.logits = k.logits;
    p.c_cur = k.c_cur; p.c_prev = k.c_prev; p.f_prev = k.f_prev;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in; p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.status = m->status;
    p.tmWr = k.tmWr; p.tmO1 = k.tmO1; p.tmO2 = k.tmO2; p.tmO3 = k.tmO3; p.tmO4 = k.tmO4;
    const long long arows = (long long)k.max_clusters * BC_MROWS;
    if (!make_map(&p.tmAct[0], k.act[0], arows, m->H, p.MR) || !make_map(&p.tmAct[1], k.act[1], arows, m->H, p.MR) ||
        !make_map(&p.tmQ, k.q, arows, m->H / 2, p.MR)) {
        m->err = "tensor-map encoding failed";
        return WRNN_ERR_CUDA;
    }
    // rows of the stacked images that no thread writes must read as zero
    if (cudaMemsetAsync(k.act[0], 0, (size_t)arows * m->H * 2, s) != cudaSuccess || cudaMemsetAsync(k.act[1], 0, (size_t)arows * m->H * 2, s) != cudaSuccess ||
        cudaMemsetAsync(k.q, 0, (size_t)arows * (m->H / 2) * 2, s) != cudaSuccess || cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess)
        return WRNN_ERR_CUDA;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ncl * BC_CS); cfg.blockDim = dim3(BC_THREADS); cfg.dynamicSmemBytes = (size_t)smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = BC_CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, bcluster_step_kernel, p);
    if (e != cudaSuccess) {
        m->err = std::string("cluster-partitioned kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    return WRNN_OK;
}

}  // namespace wrnn

#ifdef WRNN_PROFILE_BC
extern "C" int wrnn_debug_bc_prof(long long *out32, int reset)
{
    if (reset) { long long z[32] = {0}; return cudaMemcpyToSymbol(wrnn::g_bcprof, z, sizeof(z)) == cudaSuccess ? 0 : 4; }
    return cudaMemcpyFromSymbol(out32, wrnn::g_bcprof, 32 * sizeof(long long)) == cudaSuccess ? 0 : 4;
}
#endif
