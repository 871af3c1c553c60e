// Batched WaveRNN step kernel (Section 4: many rows advance in lock-step with shared weights, so every
// product of Eq. 2 becomes a matrix-matrix contraction): dense bf16 weights, 2 <= batch rows.
//
// One persistent cooperative kernel per call.  Every contraction W[M x K] . X^T[K x B] runs on the tensor
// pipe as m16n8k16 bf16 MMAs with the weights as the A operand (pre-packed in fragment order in global
// memory, read once per stream block and step from L2) and the activations as the B operand: each fp32
// activation is carried as two bf16 (hi + lo, relative error 2^-17) in a fragment-ordered "image" that the
// producing phase writes and the consuming phase stages in shared memory once per CTA.  Accumulation is fp32.
//
// CTAs are arranged as (stream block of 8 NT rows) x (group of 16-row weight tiles); a warp owns one weight
// tile against the CTA's stream block.  Phases of a step, separated by bounded grid barriers:
//   A   a = R h_{t-1}                         (all 3H rows)
//   Gc  coarse gates -> y_c                   (element-wise)
//   O1  q_c = relu(O1 y_c + b1)      O2  l_c = O2 q_c + b2
//   Sc  draw c_t (one warp per row)           Gf  fine gates -> y_f (element-wise)
//   O3  q_f = relu(O3 y_f + b3)      O4  l_f = O4 q_f + b4
//   Sf  draw f_t, emit the sample
//
// With 16 or more rows, phase A -- the [B x H] . [H x 3H] recurrent contraction, 79 % of the flops -- runs on the
// fifth-generation tensor cores instead: one CTA per (128 rows of R) x (block of BN rows of the batch), the weight
// tile and the hi / lo activation tiles brought in by TMA (128-byte swizzle, three-stage mbarrier ring), one
// elected thread issuing tcgen05.mma (M = 128, N = BN, K = 16, bf16 -> fp32) into a TMEM accumulator, and four
// warps reading it back with tcgen05.ld for the epilogue.  Every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include <cstdlib>
#include <cstring>

#include "wrnn_internal.h"
#include "wrnn_tc.cuh"

namespace wrnn {

struct BatchedPack {
    int H = 0, NKT_R = 0, NKT_H = 0;          // k-tiles of R (H/16) and of the head matrices (H/32)
    uint4 *Rf = nullptr, *O1f = nullptr, *O2f = nullptr, *O3f = nullptr, *O4f = nullptr;   // fragment-packed weights
    int max_bp = 0;                            // max batch rounded up to 8
    __nv_bfloat16 *himg[2] = {nullptr, nullptr};   // state images [Bp/8][2][H/16][32][4]
    __nv_bfloat16 *qimg = nullptr;                 // hidden-layer image [Bp/8][2][H/32][32][4]
    float *hf32[2] = {nullptr, nullptr};           // fp32 state [Bp][H]
    float *a_buf = nullptr;                        // [Bp][3H]
    float *logits = nullptr;                       // [Bp][256]
    uint8_t *c_cur = nullptr, *c_prev = nullptr, *f_prev = nullptr;
    unsigned long long *bar = nullptr;
    int64_t weight_bytes = 0;
    // tcgen05 path of phase A: plain row-major bf16 copies (K-major operands for TMA) and their tensor maps
    bool tc = false;
    int tc_rows = 0;                               // rows of the hrm arrays (max batch rounded up to 64)
    __nv_bfloat16 *Rrm = nullptr;                  // [3H][H]
    __nv_bfloat16 *hrm[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};   // [buffer][part] -> [tc_rows][H]
    CUtensorMap tmR, tmH64[2][2], tmH16[2][2];     // box 64 x 128 (R), 64 x 64 and 64 x 16 (activations)
};

struct BatchedParams {
    int H, Hh, G, batch, Bp, NKT_R, NKT_H;
    int NSB, NMG;                               // stream blocks, CTAs per stream block
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    const uint4 *Rf, *O1f, *O2f, *O3f, *O4f;
    const float *I, *b1, *b2, *b3, *b4, *g;
    __nv_bfloat16 *himg0, *himg1, *qimg;
    float *hf0, *hf1, *a_buf, *logits;
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
    int tc;                                     // phase A on tcgen05
    __nv_bfloat16 *hrm[2][2];                   // [buffer][part] row-major hi / lo state
    alignas(64) CUtensorMap tmR;
    alignas(64) CUtensorMap tmH[2][2];
};

// bf16 index of (row b, element k, part) inside an activation image with nkt k-tiles:
// [b / 8][part][k / 16][lane = 4 (b % 8) + t][e], the B fragment of lane (group b % 8, t) for that k-tile.
__device__ __forceinline__ size_t img_index(int b, int k, int part, int nkt)
{
    const int c = k & 15, t = (c & 7) >> 1, e = 2 * (c >> 3) + (c & 1);
    return ((((size_t)(b >> 3) * 2 + part) * nkt + (k >> 4)) * 32 + 4 * (b & 7) + t) * 4 + e;
}
__device__ __forceinline__ void img_store(__nv_bfloat16 *img, int b, int k, int nkt, float x)
{
    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
    const __nv_bfloat16 lo = __float2bfloat16_rn(x - __bfloat162float(hi));
    img[img_index(b, k, 0, nkt)] = hi;
    img[img_index(b, k, 1, nkt)] = lo;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint4 &a, const uint2 &b)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y));
}

// Copy the image slice of one stream block (NT n8-tiles, both parts, k-tiles [kt0, kt0 + nk)) into shared
// memory as [ntl][part][nk][32] uint2, with asynchronous 16-byte copies that bypass L1 (the image was written
// by other CTAs in an earlier phase) so that the whole slice costs about one L2 round trip.
template <int NT>
__device__ __forceinline__ void stage_image(uint2 *sB, const __nv_bfloat16 *img, int sb, int nkt_img, int kt0, int nk)
{
    const uint4 *src = reinterpret_cast<const uint4 *>(img);
    const int per = nk * 16;                    // uint4 per (ntl, part)
    const unsigned sbase = (unsigned)__cvta_generic_to_shared(sB);
    for (int np = 0; np < NT * 2; ++np) {       // np = ntl * 2 + part
        const uint4 *g = src + (((size_t)(sb * NT) * 2 + np) * nkt_img + kt0) * 16;
        for (int r = threadIdx.x; r < per; r += blockDim.x)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sbase + (unsigned)(np * per + r) * 16u), "l"(g + r) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// One 16-row weight tile (A fragments in global memory, nk k-tiles, nk a multiple of 4) against the staged
// stream block.  The k loop runs in chunks of four k-tiles of straight-line code; the A fragments of the next
// DEPTH chunks are already in flight (L2 latency), with the prefetch index clamped instead of branched.
// acc[ntl][0..3]: rows g / g+8 of the tile, rows (streams) 8 ntl + 2t, 2t+1 of the block.
template <int NT>
__device__ __forceinline__ void tile_gemm(const uint4 *Af, int nk, const uint2 *sB, int lane, float (&acc)[NT][4])
{
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[n][i] = 0.f;
    constexpr int KC = 4;
    constexpr int DEPTH = NT >= 4 ? 2 : 4;
    const int nchunks = nk / KC;
    uint4 a[DEPTH][KC];
    const uint4 *ap = Af + lane;
#pragma unroll
    for (int d = 0; d < DEPTH; ++d) {
        const int c = min(d, nchunks - 1);
#pragma unroll
        for (int i = 0; i < KC; ++i) a[d][i] = __ldg(ap + (size_t)(c * KC + i) * 32);
    }
    for (int c0 = 0; c0 < nchunks; c0 += DEPTH) {
#pragma unroll
        for (int d = 0; d < DEPTH; ++d) {
            const int c = c0 + d;
            if (c < nchunks) {
                uint4 av[KC];
#pragma unroll
                for (int i = 0; i < KC; ++i) av[i] = a[d][i];
                const int cn = min(c + DEPTH, nchunks - 1);
#pragma unroll
                for (int i = 0; i < KC; ++i) a[d][i] = __ldg(ap + (size_t)(cn * KC + i) * 32);
#pragma unroll
                for (int i = 0; i < KC; ++i) {
                    const int kt = c * KC + i;
                    uint2 bhi[NT], blo[NT];
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        bhi[n] = sB[((n * 2 + 0) * nk + kt) * 32 + lane];
                        blo[n] = sB[((n * 2 + 1) * nk + kt) * 32 + lane];
                    }
#pragma unroll
                    for (int n = 0; n < NT; ++n) mma_bf16(acc[n], av[i], bhi[n]);
#pragma unroll
                    for (int n = 0; n < NT; ++n) mma_bf16(acc[n], av[i], blo[n]);
                }
            }
        }
    }
}

// ---- tcgen05 phase A (16 or more rows): tile and ring geometry
constexpr int TC_STAGES = 3, TC_BM = 128;

__device__ __forceinline__ long long frame_of_b(const BatchedParams &p, long long s, int gb)
{
    return ((p.step0 + s) * p.row_stride + (long long)(p.stream0 + (unsigned)gb) * p.row_offset_mul) / p.hop;
}

// Gates of Eq. 2 for one (row, unit); writes the fp32 state, its image and the optional dumps.
__device__ __forceinline__ void gate_unit_b(const BatchedParams &p, int j, int gb, long long s, const float *hcur, float *hnext,
                                            __nv_bfloat16 *img_next, __nv_bfloat16 *hrm_hi, __nv_bfloat16 *hrm_lo, float x0, float x1,
                                            float x2)
{
    const int H = p.H;
    const float *a = p.a_buf + (size_t)gb * p.G;
    const float *g = p.g + ((size_t)gb * p.n_frames + (size_t)frame_of_b(p, s, gb)) * p.G;
    const float *Iu = p.I + 3 * (size_t)j, *Ir = p.I + 3 * (size_t)(H + j), *Ie = p.I + 3 * (size_t)(2 * H + j);
    const float pu = __ldcg(a + j) + fmaf(Iu[0], x0, fmaf(Iu[1], x1, fmaf(Iu[2], x2, g[j])));
    const float pr = __ldcg(a + H + j) + fmaf(Ir[0], x0, fmaf(Ir[1], x1, fmaf(Ir[2], x2, g[H + j])));
    const float pe = fmaf(Ie[0], x0, fmaf(Ie[1], x1, fmaf(Ie[2], x2, g[2 * H + j])));
    const float u = sigmoidf_acc(pu), r = sigmoidf_acc(pr);
    const float e = tanhf(fmaf(r, __ldcg(a + 2 * H + j), pe));
    const float hn = fmaf(u, __ldcg(hcur + (size_t)gb * H + j), (1.0f - u) * e);
    hnext[(size_t)gb * H + j] = hn;
    img_store(img_next, gb, j, p.NKT_R, hn);
    if (hrm_hi) {
        const __nv_bfloat16 hi = __float2bfloat16_rn(hn);
        hrm_hi[(size_t)gb * H + j] = hi;
        hrm_lo[(size_t)gb * H + j] = __float2bfloat16_rn(hn - __bfloat162float(hi));
    }
    if (p.dbg_gates) { float *d = p.dbg_gates + ((size_t)s * p.batch + gb) * p.G; d[j] = u; d[H + j] = r; d[2 * H + j] = e; }
    if (p.dbg_h) p.dbg_h[((size_t)s * p.batch + gb) * H + j] = hn;
}

#ifdef WRNN_PROFILE_BATCHED
__device__ long long g_bprof[32];
#define BSTAMP(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) { const long long n_ = clock64(); g_bprof[i] += n_ - bt_; bt_ = n_; } } while (0)
#define BROLE_BEGIN() long long rt_ = clock64(), ra_ = 0, rb_ = 0
#define BROLE_A() do { const long long n_ = clock64(); ra_ += n_ - rt_; rt_ = n_; } while (0)
#define BROLE_B() do { const long long n_ = clock64(); rb_ += n_ - rt_; rt_ = n_; } while (0)
#define BROLE_FLUSH(i) do { if (blockIdx.x == 0) { g_bprof[i] += ra_; g_bprof[i + 1] += rb_; } } while (0)
#else
#define BSTAMP(i) do { } while (0)
#define BROLE_BEGIN() do { } while (0)
#define BROLE_A() do { } while (0)
#define BROLE_B() do { } while (0)
#define BROLE_FLUSH(i) do { } while (0)
#endif

// BN: rows of the batch per tcgen05 tile of phase A (0: phase A stays on mma.sync).
template <int NT, int BN>
__global__ void __launch_bounds__(512, 1) batched_step_kernel(const __grid_constant__ BatchedParams p)
{
#ifdef WRNN_PROFILE_BATCHED
    long long bt_ = clock64();
#endif
    extern __shared__ __align__(16) uint8_t smem_raw[];
    uint2 *sB = reinterpret_cast<uint2 *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int gw = blockIdx.x * nwarps + warp, nw = gridDim.x * nwarps;
    const int gtid = blockIdx.x * blockDim.x + tid, nthreads = gridDim.x * blockDim.x;
    const int H = p.H, Hh = p.Hh, B = p.batch, Bp = p.Bp;
    const int g4 = lane >> 2, t4 = lane & 3;
    const bool active = blockIdx.x < p.NSB * p.NMG;
    const int sb = blockIdx.x % p.NSB, mg = blockIdx.x / p.NSB;
    const bool tc = BN > 0 && p.tc != 0;

    GridBarrier bar{p.bar, p.status, 0ull, p.limit_ns};
    bool failed = false;

    // ---- tcgen05 set-up: mbarrier ring, TMEM accumulator of BN fp32 columns (allocated by warp 1, freed at exit)
    __shared__ __align__(8) uint64_t tc_full[TC_STAGES], tc_empty[TC_STAGES], tc_done;
    __shared__ uint32_t tc_slot;
    uint32_t tmem_base = 0;
    unsigned tc_kb = 0, tc_tasks = 0;            // running k-block and task counters (mbarrier phases)
    constexpr int TMEM_COLS = BN >= 64 ? 64 : 32;
    if (tc) {
        if (tid == 0) {
            for (int i = 0; i < TC_STAGES; ++i) { mbar_init(smem_u32(&tc_full[i]), 1); mbar_init(smem_u32(&tc_empty[i]), 1); }
            mbar_init(smem_u32(&tc_done), 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        if (warp == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tc_slot)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        tmem_base = tc_slot;
    }

    float *hc = p.hf0, *hn = p.hf1;
    __nv_bfloat16 *ic = p.himg0, *in = p.himg1;
    int cur = 0;                                  // buffer of the row-major hi / lo state that holds h_{t-1}
    // initial state: fp32 and images (rows beyond the batch stay zero)
    for (int i = gtid; i < Bp * H; i += nthreads) {
        const int b = i / H, j = i - b * H;
        const float x = (b < B && p.h_in) ? p.h_in[i] : 0.f;
        hc[i] = x;
        img_store(ic, b, j, p.NKT_R, x);
        img_store(in, b, j, p.NKT_R, 0.f);
        if (tc) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(x);
            p.hrm[0][0][i] = hi; p.hrm[0][1][i] = __float2bfloat16_rn(x - __bfloat162float(hi));
            p.hrm[1][0][i] = __float2bfloat16_rn(0.f); p.hrm[1][1][i] = __float2bfloat16_rn(0.f);
        }
    }
    for (int i = gtid; i < Bp * Hh; i += nthreads) img_store(p.qimg, i / Hh, i % Hh, p.NKT_H, 0.f);
    for (int i = gtid; i < B; i += nthreads) {
        p.c_prev[i] = p.c_in ? p.c_in[i] : (uint8_t)128;
        p.f_prev[i] = p.f_in ? p.f_in[i] : (uint8_t)0;
    }
    if (tc) asm volatile("fence.proxy.async.global;" ::: "memory");     // generic-proxy writes before TMA reads
    if (!bar.sync(-1, 0)) failed = true;

    // Generic contraction phase: rows [0, n_mt * 16) of a fragment-packed matrix with nk k-tiles against the
    // image slice [kt0, kt0 + nk) of `img`; `epi(row, stream, value)` consumes the results.
    auto contraction = [&](const uint4 *Wf, int n_mt, int nk, const __nv_bfloat16 *img, int nkt_img, int kt0, auto epi) {
        if (active) {
            stage_image<NT>(sB, img, sb, nkt_img, kt0, nk);
            __syncthreads();
            for (int mt = mg + warp * p.NMG; mt < n_mt; mt += p.NMG * nwarps) {
                float acc[NT][4];
                tile_gemm<NT>(Wf + (size_t)mt * nk * 32, nk, sB, lane, acc);
#pragma unroll
                for (int n = 0; n < NT; ++n) {
                    const int s0 = (sb * NT + n) * 8 + 2 * t4;
                    const int r0 = 16 * mt + g4;
                    if (s0 < B) { epi(r0, s0, acc[n][0]); epi(r0 + 8, s0, acc[n][2]); }
                    if (s0 + 1 < B) { epi(r0, s0 + 1, acc[n][1]); epi(r0 + 8, s0 + 1, acc[n][3]); }
                }
            }
            __syncthreads();      // the staged image is reused by the next phase
        }
    };

    // Phase A on tcgen05: CTA (mtile, nblk) computes a[nblk * BN .. + BN][mtile * 128 .. + 128] = R tile . (h_hi + h_lo)^T.
    // warp 0 / lane 0 feeds the TMA ring, warp 1 / lane 0 issues the MMAs, warps 4..7 drain the TMEM accumulator.
    auto phase_a_tc = [&]() {
        const int n_mt = (3 * H) / TC_BM, n_nb = (Bp + BN - 1) / (BN > 0 ? BN : 1), nkb = H / TC_BK;
        const bool mine = (int)blockIdx.x < n_mt * n_nb;
        if (mine) {
            const int mtile = blockIdx.x % n_mt, nblk = blockIdx.x / n_mt;
            uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
            constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2, B_BYTES = (BN > 0 ? BN : 1) * TC_BK * 2, STAGE_BYTES = A_BYTES + 2 * B_BYTES;
            const uint32_t ring0 = smem_u32(ring);
            bool ok = true;
            if (warp == 0 && lane == 0) {
                asm volatile("fence.proxy.async;" ::: "memory");         // earlier generic-proxy use of this shared memory and of h
                BROLE_BEGIN();
                for (int kb = 0; kb < nkb; ++kb) {
                    const unsigned it = tc_kb + kb, st = it % TC_STAGES, ph = (it / TC_STAGES) & 1;
                    BROLE_A();
                    if (!mbar_wait(smem_u32(&tc_empty[st]), ph ^ 1)) { ok = false; break; }
                    BROLE_B();
                    const uint32_t fb = smem_u32(&tc_full[st]), base = ring0 + st * STAGE_BYTES;
                    mbar_expect_tx(fb, STAGE_BYTES);
                    tma_load_2d(base, &p.tmR, fb, kb * TC_BK, mtile * TC_BM);
                    tma_load_2d(base + A_BYTES, &p.tmH[cur][0], fb, kb * TC_BK, nblk * BN);
                    tma_load_2d(base + A_BYTES + B_BYTES, &p.tmH[cur][1], fb, kb * TC_BK, nblk * BN);
                }
                BROLE_A(); BROLE_FLUSH(18);
            } else if (warp == 1 && lane == 0) {
                // instruction descriptor: D fp32, A / B bf16, both K-major, N = BN, M = 128
                const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
                BROLE_BEGIN();
                for (int kb = 0; kb < nkb; ++kb) {
                    const unsigned it = tc_kb + kb, st = it % TC_STAGES, ph = (it / TC_STAGES) & 1;
                    BROLE_A();
                    if (!mbar_wait(smem_u32(&tc_full[st]), ph)) { ok = false; break; }
                    BROLE_B();
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t base = ring0 + st * STAGE_BYTES;
                    const uint64_t da = umma_desc_sw128(base), dhi = umma_desc_sw128(base + A_BYTES), dlo = umma_desc_sw128(base + A_BYTES + B_BYTES);
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k) {                 // 32 bytes along K per MMA inside the swizzle atom
                        umma_bf16(tmem_base, da + 2 * k, dhi + 2 * k, idesc, (kb | k) ? 1u : 0u);
                        umma_bf16(tmem_base, da + 2 * k, dlo + 2 * k, idesc, 1u);
                    }
                    umma_commit(smem_u32(&tc_empty[st]));
                }
                if (ok) umma_commit(smem_u32(&tc_done));
                BROLE_A(); BROLE_FLUSH(20);
            } else if (warp >= 4 && warp < 8) {
                BROLE_BEGIN();
                if (mbar_wait(smem_u32(&tc_done), tc_tasks & 1)) {
                    BROLE_A();
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const int sub = warp & 3;
                    const int row = mtile * TC_BM + sub * 32 + lane;
#pragma unroll
                    for (int c0 = 0; c0 < BN; c0 += 16) {
                        uint32_t r[16];
                        tmem_ld16(tmem_base + ((uint32_t)(sub * 32) << 16) + c0, r);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int b = nblk * BN + c0 + c;
                            if (b < B) p.a_buf[(size_t)b * p.G + row] = __uint_as_float(r[c]);
                        }
                    }
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    BROLE_B(); if (tid == 128) BROLE_FLUSH(22);
                } else ok = false;
            }
            if (!ok && atomicCAS(&p.status->code, DEV_OK, DEV_TIMEOUT) == DEV_OK) { p.status->cta = blockIdx.x; p.status->step = -2; p.status->phase = 1; }
            tc_kb += nkb; ++tc_tasks;
        }
        __syncthreads();
    };

    for (long long s = 0; s < p.n_steps && !failed; ++s) {
        if ((int)blockIdx.x == p.skip_cta && s == p.skip_step) { failed = true; break; }      // self-test: this CTA's arrivals go missing
        __nv_bfloat16 *nhi = tc ? p.hrm[cur ^ 1][0] : nullptr, *nlo = tc ? p.hrm[cur ^ 1][1] : nullptr;
        // ---- A: a = R h_{t-1}
        BSTAMP(31);
        if (tc) phase_a_tc();
        else contraction(p.Rf, 3 * H / 16, p.NKT_R, ic, p.NKT_R, 0, [&](int row, int b, float v) { p.a_buf[(size_t)b * p.G + row] = v; });
        BSTAMP(0);
        if (!bar.sync((int)s, 1)) { failed = true; break; }
        BSTAMP(1);
        // ---- Gc: coarse gates
        for (int i = gtid; i < B * Hh; i += nthreads) {
            const int gb = i / Hh, j = i - gb * Hh;
            gate_unit_b(p, j, gb, s, hc, hn, in, nhi, nlo, scale8(__ldcg(p.c_prev + gb)), scale8(__ldcg(p.f_prev + gb)), 0.f);
        }
        BSTAMP(2);
        if (!bar.sync((int)s, 2)) { failed = true; break; }
        BSTAMP(3);

        for (int head = 0; head < 2 && !failed; ++head) {
            const uint4 *Oa = head ? p.O3f : p.O1f, *Ob = head ? p.O4f : p.O2f;
            const float *ba = head ? p.b3 : p.b1, *bb = head ? p.b4 : p.b2;
            // ---- O1 / O3: hidden layer on this half of the new state (k-tiles [head * H/32, +H/32) of its image)
            contraction(Oa, Hh / 16, p.NKT_H, in, p.NKT_R, head * p.NKT_H, [&](int row, int b, float v) {
                img_store(p.qimg, b, row, p.NKT_H, fmaxf(v + (ba ? ba[row] : 0.f), 0.f));
            });
            BSTAMP(4 + 8 * head);
            if (!bar.sync((int)s, 3 + 4 * head)) { failed = true; break; }
            BSTAMP(5 + 8 * head);
            // ---- O2 / O4: logits
            contraction(Ob, 16, p.NKT_H, p.qimg, p.NKT_H, 0, [&](int row, int b, float v) {
                const float l = v + (bb ? bb[row] : 0.f);
                p.logits[(size_t)b * 256 + row] = l;
                if (p.dbg_logits) p.dbg_logits[(((size_t)s * B + b) * 2 + head) * 256 + row] = l;
            });
            BSTAMP(6 + 8 * head);
            if (!bar.sync((int)s, 4 + 4 * head)) { failed = true; break; }
            BSTAMP(7 + 8 * head);
            // ---- Sc / Sf: softmax + inverse-CDF draw, one warp per row
            for (int gb = gw; gb < B; gb += nw) {
                float l[8];
                const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(p.logits + (size_t)gb * 256 + 8 * lane));
                const float4 v1 = __ldcg(reinterpret_cast<const float4 *>(p.logits + (size_t)gb * 256 + 8 * lane + 4));
                l[0] = v0.x; l[1] = v0.y; l[2] = v0.z; l[3] = v0.w; l[4] = v1.x; l[5] = v1.y; l[6] = v1.z; l[7] = v1.w;
                const float u = uniform24(p.seed, p.stream0 + (unsigned)gb, (unsigned long long)(p.step0 + s), head);
                int idx = warp_softmax_draw(l, u, lane);
                const size_t o = (size_t)gb * p.n_steps + s;
                if (lane == 0) {
                    if (head == 0) {
                        if (p.c_out) p.c_out[o] = (uint8_t)idx;
                        if (p.c_forced) idx = p.c_forced[o];
                        p.c_cur[gb] = (uint8_t)idx;
                    } else {
                        if (p.f_out) p.f_out[o] = (uint8_t)idx;
                        if (p.f_forced) idx = p.f_forced[o];
                        const int c = __ldcg(p.c_cur + gb);
                        if (p.out) p.out[o] = (int16_t)(256 * c + idx - 32768);
                        p.c_prev[gb] = (uint8_t)c;
                        p.f_prev[gb] = (uint8_t)idx;
                    }
                }
            }
            BSTAMP(8 + 8 * head);
            if (!bar.sync((int)s, 5 + 4 * head)) { failed = true; break; }
            BSTAMP(9 + 8 * head);
            if (head == 0) {
                // ---- Gf: fine gates, now that c_t is known (it reaches only these rows, Section 2)
                for (int i = gtid; i < B * Hh; i += nthreads) {
                    const int gb = i / Hh, j = Hh + (i - gb * Hh);
                    gate_unit_b(p, j, gb, s, hc, hn, in, nhi, nlo, scale8(__ldcg(p.c_prev + gb)), scale8(__ldcg(p.f_prev + gb)),
                                scale8(__ldcg(p.c_cur + gb)));
                }
                if (tc) asm volatile("fence.proxy.async.global;" ::: "memory");
                BSTAMP(10);
                if (!bar.sync((int)s, 6)) { failed = true; break; }
                BSTAMP(11);
            }
        }
        { float *t = hc; hc = hn; hn = t; }
        { __nv_bfloat16 *t = ic; ic = in; in = t; }
        cur ^= 1;
    }

    if (!failed) {
        if (p.h_out) for (int i = gtid; i < B * H; i += nthreads) p.h_out[i] = __ldcg(hc + i);
        for (int i = gtid; i < B; i += nthreads) {
            if (p.c_st_out) p.c_st_out[i] = __ldcg(p.c_prev + i);
            if (p.f_st_out) p.f_st_out[i] = __ldcg(p.f_prev + i);
        }
    }
    if (tc) {
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
static uint16_t bf16_bits_b(float rounded)
{
    uint32_t b;
    std::memcpy(&b, &rounded, 4);
    return (uint16_t)(b >> 16);
}

// host block rows (values already rounded) -> dense row-major bf16 bits
std::vector<uint16_t> dense_bf16_bits(const BsrHost &M)
{
    const int rows = M.rows4 * 4, cols = M.cols4 * 4;
    std::vector<uint16_t> dense((size_t)rows * cols, 0);
    for (int br = 0; br < M.rows4; ++br)
        for (int i = M.row_ptr[br]; i < M.row_ptr[br + 1]; ++i)
            for (int r = 0; r < 4; ++r)
                for (int c = 0; c < 4; ++c)
                    dense[(size_t)(4 * br + r) * cols + 4 * M.col[i] + c] = bf16_bits_b(M.vals[(size_t)i * 16 + 4 * r + c]);
    return dense;
}

// dense matrix -> A fragments [rows/16][cols/16][32 lanes][8 bf16]
static std::vector<uint16_t> pack_fragments(const BsrHost &M)
{
    const int rows = M.rows4 * 4, cols = M.cols4 * 4, nmt = rows / 16, nkt = cols / 16;
    const std::vector<uint16_t> dense = dense_bf16_bits(M);
    std::vector<uint16_t> out((size_t)nmt * nkt * 256);
    for (int mt = 0; mt < nmt; ++mt)
        for (int kt = 0; kt < nkt; ++kt)
            for (int lane = 0; lane < 32; ++lane) {
                const int g = lane >> 2, t = lane & 3;
                uint16_t *o = out.data() + (((size_t)mt * nkt + kt) * 32 + lane) * 8;
                const int rsel[4] = {g, g + 8, g, g + 8}, csel[4] = {2 * t, 2 * t, 2 * t + 8, 2 * t + 8};
                for (int q = 0; q < 4; ++q)
                    for (int j = 0; j < 2; ++j) o[2 * q + j] = dense[(size_t)(16 * mt + rsel[q]) * cols + 16 * kt + csel[q] + j];
            }
    return out;
}

static int bn_for(int nt) { return nt == 4 ? 64 : (nt == 2 ? 16 : 0); }
static size_t smem_for(int nt, int nkt_r)
{
    const size_t img = (size_t)nt * 2 * nkt_r * 32 * 8;
    const size_t ring = bn_for(nt) ? (size_t)TC_STAGES * (TC_BM * TC_BK * 2 + 2 * bn_for(nt) * TC_BK * 2) + 1024 : 0;
    return img > ring ? img : ring;
}

static int nt_for(int batch) { return batch <= 8 ? 1 : (batch <= 16 ? 2 : 4); }

static void *batched_fn(int nt)
{
    return nt == 1 ? (void *)batched_step_kernel<1, 0> : nt == 2 ? (void *)batched_step_kernel<2, 16> : (void *)batched_step_kernel<4, 64>;
}

int batched_supported(const wrnn_model *m, int batch, std::string *why)
{
    if (!m->batched) { if (why) *why = "model was not packed for the batched kernel"; return WRNN_ERR_UNSUPPORTED; }
    if (batch < 2) { if (why) *why = "batched kernel needs at least two rows"; return WRNN_ERR_UNSUPPORTED; }
    return WRNN_OK;
}

int batched_prepare(wrnn_model *m)
{
    if (m->dtype != WRNN_BF16 || m->sparse) { m->err = "batched kernel takes dense bf16 models"; return WRNN_ERR_UNSUPPORTED; }
    if (m->H % 128 != 0) { m->err = "batched kernel needs H to be a multiple of 128 (k-tiles in chunks of four)"; return WRNN_ERR_UNSUPPORTED; }
    if (m->max_batch < 2) { m->err = "max_batch < 2"; return WRNN_ERR_UNSUPPORTED; }
    BatchedPack *k = new BatchedPack();
    const int H = m->H, Hh = H / 2;
    k->H = H; k->NKT_R = H / 16; k->NKT_H = Hh / 16;
    k->max_bp = (m->max_batch + 7) / 8 * 8;
    if (nt_for(m->max_batch) == 4) k->max_bp = (m->max_batch + 31) / 32 * 32;
    else if (nt_for(m->max_batch) == 2) k->max_bp = 16;
    const size_t Bp = (size_t)k->max_bp;
    auto up = [&](const BsrHost &M, uint4 **dst) {
        std::vector<uint16_t> f = pack_fragments(M);
        k->weight_bytes += (int64_t)f.size() * 2;
        return cudaMalloc((void **)dst, f.size() * 2) == cudaSuccess &&
               cudaMemcpy(*dst, f.data(), f.size() * 2, cudaMemcpyHostToDevice) == cudaSuccess;
    };
    bool ok = up(m->hR, &k->Rf) && up(m->hO1, &k->O1f) && up(m->hO2, &k->O2f) && up(m->hO3, &k->O3f) && up(m->hO4, &k->O4f);
    ok = ok && cudaMalloc((void **)&k->himg[0], Bp * H * 4) == cudaSuccess && cudaMalloc((void **)&k->himg[1], Bp * H * 4) == cudaSuccess &&
         cudaMalloc((void **)&k->qimg, Bp * Hh * 4) == cudaSuccess &&
         cudaMalloc((void **)&k->hf32[0], Bp * H * 4) == cudaSuccess && cudaMalloc((void **)&k->hf32[1], Bp * H * 4) == cudaSuccess &&
         cudaMalloc((void **)&k->a_buf, Bp * 3 * H * 4) == cudaSuccess && cudaMalloc((void **)&k->logits, Bp * 256 * 4) == cudaSuccess &&
         cudaMalloc((void **)&k->c_cur, Bp) == cudaSuccess && cudaMalloc((void **)&k->c_prev, Bp) == cudaSuccess &&
         cudaMalloc((void **)&k->f_prev, Bp) == cudaSuccess && cudaMalloc((void **)&k->bar, 256) == cudaSuccess;
    // tcgen05 phase A: row-major R, row-major hi / lo state (rows beyond the padded batch stay zero), tensor maps
    const int nt_max = nt_for(m->max_batch);
    if (ok && nt_max >= 2 && !std::getenv("WRNN_BATCHED_NO_TC") && encode_tiled_fn()) {
        k->tc_rows = (k->max_bp + 63) / 64 * 64;
        const std::vector<uint16_t> Rd = dense_bf16_bits(m->hR);
        bool t = cudaMalloc((void **)&k->Rrm, Rd.size() * 2) == cudaSuccess &&
                 cudaMemcpy(k->Rrm, Rd.data(), Rd.size() * 2, cudaMemcpyHostToDevice) == cudaSuccess;
        for (int b = 0; b < 2 && t; ++b)
            for (int q = 0; q < 2 && t; ++q)
                t = cudaMalloc((void **)&k->hrm[b][q], (size_t)k->tc_rows * H * 2) == cudaSuccess &&
                    cudaMemset(k->hrm[b][q], 0, (size_t)k->tc_rows * H * 2) == cudaSuccess;
        t = t && make_map(&k->tmR, k->Rrm, 3 * H, H, TC_BM);
        for (int b = 0; b < 2 && t; ++b)
            for (int q = 0; q < 2 && t; ++q)
                t = make_map(&k->tmH64[b][q], k->hrm[b][q], k->tc_rows, H, 64) && make_map(&k->tmH16[b][q], k->hrm[b][q], k->tc_rows, H, 16);
        if (t) { k->tc = true; k->weight_bytes += (int64_t)Rd.size() * 2; }
        else ok = false;
    }
    for (int nt : {1, 2, 4}) {
        const size_t smem = smem_for(nt, k->NKT_R);
        if (ok && cudaFuncSetAttribute(batched_fn(nt), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) ok = false;
    }
    m->batched = k;
    if (!ok) {
        cudaGetLastError();
        batched_destroy(m);
        m->err = "device allocation for the batched kernel failed";
        return WRNN_ERR_NOMEM;
    }
    return WRNN_OK;
}

void batched_destroy(wrnn_model *m)
{
    BatchedPack *k = m->batched;
    if (!k) return;
    cudaFree(k->Rf); cudaFree(k->O1f); cudaFree(k->O2f); cudaFree(k->O3f); cudaFree(k->O4f);
    cudaFree(k->himg[0]); cudaFree(k->himg[1]); cudaFree(k->qimg); cudaFree(k->hf32[0]); cudaFree(k->hf32[1]);
    cudaFree(k->a_buf); cudaFree(k->logits); cudaFree(k->c_cur); cudaFree(k->c_prev); cudaFree(k->f_prev); cudaFree(k->bar);
    cudaFree(k->Rrm);
    for (int b = 0; b < 2; ++b)
        for (int q = 0; q < 2; ++q) cudaFree(k->hrm[b][q]);
    delete k;
    m->batched = nullptr;
}

int batched_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes)
{
    const BatchedPack &k = *m->batched;
    const int nt = nt_for(batch);
    if (n_ctas) *n_ctas = m->n_sms;
    if (n_threads) *n_threads = 512;
    if (smem) *smem = (int)smem_for(nt, k.NKT_R);
    if (weight_bytes) *weight_bytes = k.weight_bytes;
    return WRNN_OK;
}

int batched_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    const BatchedPack &k = *m->batched;
    const int nt = nt_for(a.batch);
    BatchedParams p;
    std::memset(&p, 0, sizeof(p));
    p.H = m->H; p.Hh = m->H / 2; p.G = 3 * m->H; p.batch = a.batch;
    p.Bp = (a.batch + 8 * nt - 1) / (8 * nt) * (8 * nt);
    p.NKT_R = k.NKT_R; p.NKT_H = k.NKT_H;
    p.NSB = p.Bp / (8 * nt);
    p.NMG = m->n_sms / p.NSB;
    if (p.NMG < 1) { m->err = "batch too large for the batched kernel on this device"; return WRNN_ERR_UNSUPPORTED; }
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.Rf = k.Rf; p.O1f = k.O1f; p.O2f = k.O2f; p.O3f = k.O3f; p.O4f = k.O4f;
    p.I = m->I; p.b1 = m->b1; p.b2 = m->b2; p.b3 = m->b3; p.b4 = m->b4; p.g = m->g;
    p.himg0 = k.himg[0]; p.himg1 = k.himg[1]; p.qimg = k.qimg; p.hf0 = k.hf32[0]; p.hf1 = k.hf32[1];
    p.a_buf = k.a_buf; p.logits = k.logits; p.c_cur = k.c_cur; p.c_prev = k.c_prev; p.f_prev = k.f_prev;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in; p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.bar = k.bar; p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;
    // tcgen05 phase A: one CTA per (128 rows of R) x (BN rows of the batch); falls back to mma.sync when the grid is too small
    const int bn = bn_for(nt);
    if (k.tc && bn && (3 * m->H / TC_BM) * ((p.Bp + bn - 1) / bn) <= m->n_sms) {
        p.tc = 1;
        p.tmR = k.tmR;
        for (int b = 0; b < 2; ++b)
            for (int q = 0; q < 2; ++q) { p.hrm[b][q] = k.hrm[b][q]; p.tmH[b][q] = bn == 64 ? k.tmH64[b][q] : k.tmH16[b][q]; }
    }

    if (cudaMemsetAsync(k.bar, 0, sizeof(unsigned long long), s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    void *args[] = {(void *)&p};
    const size_t smem = smem_for(nt, k.NKT_R);
    const cudaError_t e = cudaLaunchCooperativeKernel(batched_fn(nt), dim3(m->n_sms), dim3(512), args, smem, s);
    if (e != cudaSuccess) {
        m->err = std::string("batched kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    return WRNN_OK;
}

}  // namespace wrnn

#ifdef WRNN_PROFILE_BATCHED
extern "C" int wrnn_debug_batched_prof(long long *out32, int reset)
{
    if (reset) { long long z[32] = {0}; return cudaMemcpyToSymbol(wrnn::g_bprof, z, sizeof(z)) == cudaSuccess ? 0 : 4; }
    return cudaMemcpyFromSymbol(out32, wrnn::g_bprof, 32 * sizeof(long long)) == cudaSuccess ? 0 : 4;
}
#endif
