// Shared-memory-resident persistent sampling kernel for 2 to 16 streams that advance in lock step (the rows of a
// subscale fold, Section 4 of the paper, or a small batch, Section 5.1), dense bf16 weights, H = 896.
//
// Same machine as the single-stream resident kernel: 7 clusters x 16 CTAs, every weight in shared memory for the
// whole call, two chip-wide exchanges of the state halves per step through tagged L2 slots (Fig. 1's order).  What
// changes with several streams:
//   * the recurrent matrix is sharded over all 112 CTAs as before (four state units of each half per CTA), and every
//     CTA multiplies its rows with the state of ALL streams: the B operand of an m16n8k16 MMA holds four streams
//     (columns 2 j, 2 j + 1 = the bf16 high and low parts of stream j's fp32 vector), so 16 streams are four column
//     groups;
//   * the output heads are still held once per cluster, but cluster c serves only the streams of column group c
//     (streams 4 c .. 4 c + 3) or, with up to seven streams, stream c alone (its state half is kept a second time as a
//     column group of its own): one MMA column group per head, as for a single stream.  The logits go to the cluster's
//     first CTA, which draws;
//   * the gates of a stream are computed in the cluster that draws it (every CTA of the cluster takes 28 state units of
//     each half), so the drawn symbol only crosses distributed shared memory; the rows of R h they need are published
//     by the CTAs that own those rows of R as tagged L2 words, once per step, half a step or more before they are used;
//   * the recurrent products of a half step are not needed before the gates at its end, so twelve warps compute them
//     while the other four wait for the logits, draw and broadcast: they are off the critical path.
// Every wait is bounded; a CTA that gives up records where and all CTAs leave through the final cluster barrier.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>

#include "wrnn_cluster.cuh"
#include "wrnn_internal.h"

namespace cg = cooperative_groups;

namespace wrnn {

namespace {
constexpr int MK = 448;              // H / 2
constexpr int MKP = 14;              // pairs of k-tiles
constexpr int MUC = 4;               // state units of each half per CTA
constexpr int MNR = 6 * MUC;         // rows of R per CTA
constexpr int MHR = 28;              // hidden-layer rows per CTA
constexpr int MLR = 16;              // logits rows per CTA
constexpr int MCS = 16;              // CTAs per cluster
constexpr int MNC = 7;               // clusters
constexpr int MAXS = 16;             // streams per launch
constexpr int TILE_U4 = 28 * 32;     // uint4 per 16-row tile of A fragments
constexpr int IMG_U4 = MKP * 32;     // uint4 per column-group image of a vector
constexpr int P0S = 136;             // floats per stream of the head partial sums (8 slots x 16 rows + 8 so that the streams hit different banks)
constexpr int PR_FLOATS = 1664;      // partial sums of the recurrent rows
}  // namespace

struct ResMultiPack {
    size_t blob_bytes = 0, w_bytes = 0;
    uint8_t *d_blob = nullptr;               // [112][blob_bytes]
    unsigned long long *d_slots = nullptr;   // [2 halves][2 parities][16 streams][K] (value, tag)
    unsigned long long *d_aslots = nullptr;  // [2 parities][16 streams][2 halves x 3 gates x K] (R h value, tag)
    long long *d_prof = nullptr;             // [16]
    int smem_bytes = 0;
    int64_t weight_bytes_per_step = 0;
};

struct MultiParams {
    int H, NS;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul, row_lag;
    long long out_pitch;
    const uint8_t *blob; unsigned long long blob_bytes, w_bytes;
    const float *g;                          // [NS][n_frames][3H]
    unsigned long long *slots, *aslots;
    const float *I;                          // [3H][3] input weights (fp32, masked column zeroed)
    const float *h_in; float *h_out;
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;
    uint8_t *c_out, *f_out;
    int16_t *out;
    float *dbg_gates, *dbg_h, *dbg_logits;
    DevStatus *status;
    unsigned long long limit_ns;
    int skip_cta; long long skip_step;      // self-test: this CTA withholds what it publishes at this step (-1: none)
    long long *prof;
    unsigned flag_mode;                      // bit 0 / 1: with one / several column groups the gather waits for this CTA's own publication first
};

// Position (in bf16 units) of element i of column `col` in a column-group image: [k-tile pair][8 columns][4 t][2 k-tiles][4 bf16],
// the four bf16 of (k-tile, column, t) being elements 2t, 2t+1, 2t+8, 2t+9 of the k-tile: one 16-byte load per lane
// brings the B fragments of two k-tiles and a warp's loads are one contiguous 512-byte run.
__device__ __forceinline__ int mimg_pos(int i, int col)
{
    const int c = i & 15, kt = i >> 4;
    const int t = (c & 7) >> 1, j = c & 1, hi = c >> 3;
    return ((((((kt >> 1) * 8 + col) * 4 + t) << 1) + (kt & 1)) << 2) + 2 * hi + j;
}
// two adjacent elements (j even) of stream st: high and low bf16 parts, one 32-bit store each
__device__ __forceinline__ void mimg_store_pair(uint4 *img, int st, int j, float x0, float x1)
{
    const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
    const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0)), l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
    unsigned *s32 = reinterpret_cast<unsigned *>(img + (st >> 2) * IMG_U4);
    const int col = 2 * (st & 3);
    s32[mimg_pos(j, col) >> 1] = (unsigned)__bfloat16_as_ushort(h0) | ((unsigned)__bfloat16_as_ushort(h1) << 16);
    s32[mimg_pos(j, col + 1) >> 1] = (unsigned)__bfloat16_as_ushort(l0) | ((unsigned)__bfloat16_as_ushort(l1) << 16);
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint4 &a, unsigned b0, unsigned b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void named_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int n) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory"); }

// MODE 0: plain sampling (no forced symbols, no dumps, no stamps, no self-test predicate); MODE 1: the instantiation that
// wrnn_selftest_lost_word runs (one CTA withholds one publication); MODE 2: the one with the phase stamps of wrnn_phase_profile
// (and with forced symbols and dumps, like mode 1); MODE 4: stamp code without forced symbols and dumps
template <int MODE>
__global__ void __launch_bounds__(512, 1) resident_multi_kernel(const MultiParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int cta = blockIdx.x, cl = cta / MCS;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = p.H, NS = p.NS, NG = (NS + 3) >> 2;
    // streams whose heads this cluster holds: up to seven streams, one per cluster (the exchanges inside a cluster are
    // those of a single stream); more streams, the four of column group cl
    const bool spread = NS <= MNC;
    const int own_n = spread ? (cl < NS ? 1 : 0) : min(4, max(0, NS - 4 * cl));
    constexpr int K = MK;

    // ---- shared memory carve-up (must match resmulti_smem_bytes)
    const uint4 *wMA = reinterpret_cast<const uint4 *>(smem);                  // 4 tiles: [R x coarse columns (24 rows) ; O1 (28 rows)]
    const uint4 *wMB = wMA + 4 * TILE_U4;                                      // 4 tiles: [R x fine columns ; O3]
    const uint4 *wO2 = wMB + 4 * TILE_U4;
    const uint4 *wO4 = wO2 + TILE_U4;
    const float *sI = reinterpret_cast<const float *>(smem + p.w_bytes);       // [24][3]
    const float *sb1 = sI + MNR * 3, *sb3 = sb1 + MHR, *sb2 = sb3 + MHR, *sb4 = sb2 + MLR;
    float *a_part = reinterpret_cast<float *>(smem + p.blob_bytes);            // [16][24] R[:, :K] y_c
    float *sIg = a_part + MAXS * MNR;                                          // [2 halves][3 gates][28 units][3] input weights of the gate threads' units
    float *part_R = sIg + 2 * 3 * MHR * 3 + 8;                                       // [streams][2 tiles x slots][16] (+8 per stream)
    float *part0 = part_R + PR_FLOATS;                                         // [4 streams][8 slots][16] (+8 per stream)
    float *part1 = part0 + 4 * P0S;                                            // the same for the logits (its writers do not wait for the readers of part0)
    uint4 *spl = reinterpret_cast<uint4 *>(part1 + 4 * P0S);                   // [4 column groups] images of the state half
    uint4 *splQ = spl + 4 * IMG_U4;                                            // the hidden layers of the own streams, split by their senders (layout below)
    uint4 *splOwn = splQ + IMG_U4;                                             // up to seven streams: the own stream's state half as a column group of its own
    uint4 *lbuf = splOwn + IMG_U4;                                             // [2 parities][4 streams][128] {v, tag, v, tag}
    __shared__ __align__(8) unsigned long long xbar[2];
    __shared__ __align__(8) unsigned long long s_sym[8];   // [2 parities][4 own streams] (symbol, tag) from the drawing CTA
    __shared__ long long s_pub;                 // the last half step whose state values this CTA's gate threads have published

    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.blob + (size_t)cta * p.blob_bytes);
        uint4 *dst = reinterpret_cast<uint4 *>(smem);
        for (size_t i = tid; i < p.blob_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
        for (int i = tid; i < 1024; i += blockDim.x) lbuf[i] = make_uint4(0, 0, 0, 0);
        for (int i = tid; i < 6 * IMG_U4; i += blockDim.x) spl[i] = make_uint4(0, 0, 0, 0);  // spl, splQ and splOwn are adjacent
        for (int i = tid; i < MAXS * MNR + 2 * 3 * MHR * 3 + 8 + PR_FLOATS + 8 * P0S; i += blockDim.x) a_part[i] = 0.f;
        if (tid == 0) {
            for (int i = 0; i < 2; ++i) mbar_init_cluster(smem_addr(&xbar[i]), 1);
            mbar_fence_init();
            s_pub = -1;
        }
        if (tid < 8) s_sym[tid] = 0;
    }
    __syncthreads();
    for (int i = tid; i < 2 * 3 * MHR * 3; i += blockDim.x) {
        const int c = i % 3, gq = (i / 3) % MHR, hg = i / (3 * MHR);          // hg = half * 3 + gate
        sIg[i] = p.I[((size_t)(hg % 3) * H + (hg / 3) * K + MHR * rank + gq) * 3 + c];
    }
    __syncthreads();
    cluster.sync();

    Waiter wt{p.status, p.limit_ns};
    bool my_bad = false;
    const int g4 = lane >> 2, t4 = lane & 3;
    constexpr bool HOOK = MODE == 1, PROF = MODE == 2 || MODE == 4, DBG = MODE == 1 || MODE == 2;
    const bool prof_on = PROF && p.prof != nullptr && cta == 0 && warp == 0;
    __shared__ long long s_prof[16];
    if (tid < 16) s_prof[tid] = 0;
    __syncthreads();
    long long prof_t = clock64();
#define STAMP(i) do { if (PROF && prof_on) { const long long now_ = clock64(); if (lane == 0) s_prof[i] += now_ - prof_t; prof_t = now_; } } while (0)

    // ---- roles
    const int ws = warp;                                  // drawing warps 0..3: own stream ws
    const bool drawer = warp < 4 && ws < own_n && rank == 0;   // the cluster's first CTA draws for its streams
    const int d_st = spread ? cl : 4 * cl + ws;           // the stream a drawing warp serves
    // recurrent products: warps 7..15 (warps 0..6 hold the logits MMAs of the head chain); with four column groups also
    // warps 4..6, after their logits MMAs (measured: 10.47 against 10.52 us per 16-row lock-step; 7.81 against 8.09 at 4 rows)
    const int RW0 = NG >= 4 ? 4 : 7, NRW = 16 - RW0;
    const int rw = warp - RW0, ridx = tid - 128;          // warps 4..15: sums of the products, then the gates
    // gate threads: the state units 28 rank .. + 27 of both halves, for every own stream of the cluster
    const bool gater = warp >= 4 && ridx < own_n * MHR;
    const int gl = ridx / MHR, gq = ridx % MHR;           // (own stream, unit of this CTA's share) of a gate thread
    const int gst = (spread ? cl : 4 * cl) + gl, gj = MHR * rank + gq;
    const int r_cg = rw >= 0 ? rw % NG : 0, r_j = rw >= 0 ? rw / NG : 0;
    const int nsl = (NRW + NG - 1) / NG, PS = 2 * nsl * 16 + 8;
    const int r_nw = (NRW - r_cg + NG - 1) / NG;                               // warps that share column group r_cg
    const int s_st = ridx >= 0 ? ridx / MNR : 0, s_row = ridx >= 0 ? ridx - s_st * MNR : 0;      // (stream, row) a thread sums
    const int s_nw = (NRW - (s_st >> 2) + NG - 1) / NG;

    // recurrent rows (tiles 0, 1 of Mx) times all streams: warp rw takes column group r_cg, k-tile pairs r_j, r_j + nw, ..
    auto r_products = [&](const uint4 *Mx) {
        const int nw = r_nw;
        float acc[2][2][4];
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int k = 0; k < 4; ++k) acc[n][i][k] = 0.f;
        const uint4 *bimg = spl + r_cg * IMG_U4 + g4 * 4 + t4;
#pragma unroll 2
        for (int kp = r_j; kp < MKP; kp += nw) {
            const uint4 bv = bimg[kp * 32];
            uint4 av[2][2];
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int i = 0; i < 2; ++i) av[n][i] = Mx[n * TILE_U4 + (2 * kp + i) * 32 + lane];
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                mma16816(acc[n][0], av[n][0], bv.x, bv.y);
                mma16816(acc[n][1], av[n][1], bv.z, bv.w);
            }
        }
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            float *d = part_R + (4 * r_cg + t4) * PS + (n * nsl + r_j) * 16;
            d[g4] = (acc[n][0][0] + acc[n][1][0]) + (acc[n][0][1] + acc[n][1][1]);
            d[g4 + 8] = (acc[n][0][2] + acc[n][1][2]) + (acc[n][0][3] + acc[n][1][3]);
        }
    };
    // sums of the K-split partials; a completed row of R h (tag: the step whose gates use it, + 1) goes to the cluster
    // that computes the gates of its stream
    auto r_sums = [&](bool completes, long long s_use) {
        if (ridx < NS * MNR) {
            const int st = s_st, row = s_row, nw = s_nw;
            const float *s = part_R + st * PS + ((row >> 4) * nsl) * 16 + (row & 15);
            float v = 0.f;
            for (int j = 0; j < nw; ++j) v += s[j * 16];
            if (completes) {
                const int hg = row / MUC, u = row % MUC;                         // hg = half * 3 + gate
                st_relaxed_u64(p.aslots + ((size_t)(s_use & 1) * NS + st) * (6 * K) + hg * K + cta * MUC + u,
                               ((unsigned long long)(unsigned)(s_use + 1) << 32) | __float_as_uint(a_part[ridx] + v));
            } else a_part[ridx] = v;
        }
    };
    auto fill_image = [&](int part) {
        for (int idx = tid; idx < NS * K / 2; idx += blockDim.x) {
            const int st = (2 * idx) / K, j = 2 * idx - st * K;
            const float x0 = p.h_in ? p.h_in[(size_t)st * H + part * K + j] : 0.f, x1 = p.h_in ? p.h_in[(size_t)st * H + part * K + j + 1] : 0.f;
            mimg_store_pair(spl, st, j, x0, x1);
        }
    };

    // ---- prologue: R h of the initial state
    fill_image(0);
    __syncthreads();
    if (warp >= 4) { if (warp >= RW0) r_products(wMA); named_sync(1, 384); r_sums(false, 0); }
    __syncthreads();
    fill_image(1);
    __syncthreads();
    if (warp >= 4) { if (warp >= RW0) r_products(wMB); named_sync(1, 384); r_sums(true, 0); }
    __syncthreads();

    // state of a gate thread: its unit of both halves of its stream, and the stream's last symbols
    int c_prev = 128, f_prev = 0;
    float hC = 0.f, hF = 0.f;
    if (gater) {
        c_prev = p.c_in ? p.c_in[gst] : 128; f_prev = p.f_in ? p.f_in[gst] : 0;
        if (p.h_in) { hC = p.h_in[(size_t)gst * H + gj]; hF = p.h_in[(size_t)gst * H + K + gj]; }
    }
    if (drawer) { c_prev = p.c_in ? p.c_in[d_st] : 128; f_prev = p.f_in ? p.f_in[d_st] : 0; }

    struct GatePre { float pu, pr, pe, ae, ku, kr, ke; };
    // the three rows of R h of this thread's unit (published by the CTA that owns those rows of R)
    auto load_a = [&](int half_g, long long s_use, float (&av)[3]) {
        const unsigned long long *src = p.aslots + ((size_t)(s_use & 1) * NS + gst) * (6 * K) + (half_g * 3) * K + gj;
        const unsigned atag = (unsigned)(s_use + 1);
        unsigned long long v[3], t0 = 0; unsigned cnt = 0;
        while (true) {
#pragma unroll
            for (int gate = 0; gate < 3; ++gate) v[gate] = ld_relaxed_u64(src + gate * K);
            if ((unsigned)(v[0] >> 32) == atag && (unsigned)(v[1] >> 32) == atag && (unsigned)(v[2] >> 32) == atag) break;
            if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s_use, 9)) { my_bad = true; break; }
        }
#pragma unroll
        for (int gate = 0; gate < 3; ++gate) av[gate] = __uint_as_float((unsigned)v[gate]);
    };
    auto gates_prepare = [&](int half_g, const float (&gv)[3], const float (&av)[3]) {
        GatePre q;
        const float x0 = scale8(c_prev), x1 = scale8(f_prev);
        const float *Iu = sIg + ((half_g * 3 + 0) * MHR + gq) * 3, *Ir = sIg + ((half_g * 3 + 1) * MHR + gq) * 3, *Ie = sIg + ((half_g * 3 + 2) * MHR + gq) * 3;
        q.pu = av[0] + fmaf(Iu[0], x0, half_g ? fmaf(Iu[1], x1, gv[0]) : gv[0]);
        q.pr = av[1] + fmaf(Ir[0], x0, half_g ? fmaf(Ir[1], x1, gv[1]) : gv[1]);
        q.pe = fmaf(Ie[0], x0, half_g ? fmaf(Ie[1], x1, gv[2]) : gv[2]);
        q.ae = av[2];
        q.ku = half_g ? Iu[2] : Iu[1]; q.kr = half_g ? Ir[2] : Ir[1]; q.ke = half_g ? Ie[2] : Ie[1];
        return q;
    };
    const int skip_at = (HOOK && cta == p.skip_cta) ? (int)p.skip_step : -1;      // self-test: the step at which this CTA withholds its publication
    auto gates_and_publish = [&](int half_g, long long s, int drawn, const GatePre &q) {
        const float xk = scale8(drawn);
        const float u = sigmoidf_fast(fmaf(q.ku, xk, q.pu)), r = sigmoidf_fast(fmaf(q.kr, xk, q.pr));
        const float e = tanhf_fast(fmaf(r, q.ae, fmaf(q.ke, xk, q.pe)));
        const float hn = fmaf(u, half_g ? hF : hC, (1.0f - u) * e);
        if (half_g) hF = hn; else hC = hn;
        const int jj = (half_g ? K : 0) + gj;
        // published as the operand the 112 readers need: bf16 high and low parts, split once here
        const __nv_bfloat16 hh = __float2bfloat16_rn(hn), hl = __float2bfloat16_rn(hn - __bfloat162float(hh));
        if (!HOOK || (int)s != skip_at)
            st_relaxed_u64(p.slots + ((size_t)((half_g ? 2 : 0) + (s & 1)) * NS + gst) * K + gj,
                           ((unsigned long long)(unsigned)(s + 1) << 32) | (unsigned)__bfloat16_as_ushort(hh) | ((unsigned)__bfloat16_as_ushort(hl) << 16));
        if (DBG && p.dbg_gates) { float *d = p.dbg_gates + ((size_t)s * NS + gst) * 3 * H; d[jj] = u; d[H + jj] = r; d[2 * H + jj] = e; }
        if (DBG && p.dbg_h) p.dbg_h[((size_t)s * NS + gst) * H + jj] = hn;
    };
    auto load_g = [&](int half_g, long long s, float (&gv)[3]) {
        const long long fr = p.row_lag > 0 ? s : ((p.step0 + s) * p.row_stride + (long long)(p.stream0 + (unsigned)gst) * p.row_offset_mul) / p.hop;
        const float *g = p.g + ((size_t)gst * p.n_frames + fr) * 3 * H + (half_g ? K : 0) + gj;
#pragma unroll
        for (int gate = 0; gate < 3; ++gate) gv[gate] = __ldg(g + gate * H);
    };
    if (gater) {
        float gv[3], av[3];
        load_g(0, 0, gv);
        load_a(0, 0, av);
        if (!my_bad) gates_and_publish(0, 0, f_prev, gates_prepare(0, gv, av));
    }
    if (warp == 4) { __syncwarp(); if (lane == 0) *(volatile long long *)&s_pub = 0; }

    // send addresses: one peer per warp
    const int q_st = lane / 7, q_quad = lane % 7;             // hidden layer: lanes [0, 28): stream, four rows
    const int l_st = lane >> 3, l_ll = lane & 7;              // logits: stream, two rows
    unsigned q_snd[2], l_snd[2], q_bar[2], q_off = 0;        // (a sending warp serves CTAs warp, warp + 4, warp + 8, warp + 12 of the cluster)
#pragma unroll
    for (int par2 = 0; par2 < 2; ++par2) {
        const unsigned peer = (unsigned)warp;
        {
            // The hidden layer travels already split: a lane's four rows j0 .. j0 + 3 (j0 a multiple of 4) of one stream are
            // four 32-bit words -- (high parts of j0, j0+1), (high of j0+2, j0+3), (low of j0, j0+1), (low of j0+2, j0+3) --
            // stored as one 16-byte piece of the receivers' image [k-tile pair][t / 2][k-tile & 1][upper half of the k-tile]
            // [stream][part][t & 1], from which a B fragment is four words 16 words apart.
            const int j0 = rank * MHR + 4 * q_quad, kt = j0 >> 4, c = j0 & 15;
            const int w = (((((kt >> 1) * 2 + ((c & 7) >> 2)) * 2 + (kt & 1)) * 2 + (c >> 3)) * 4 + (q_st < 4 ? q_st : 0)) * 4;
            q_snd[par2] = map_to_rank(smem_addr(reinterpret_cast<unsigned *>(splQ) + w), peer);
        }
        l_snd[par2] = map_to_rank(smem_addr(lbuf + (size_t)(par2 * 4 + l_st) * 128 + (rank * MLR) / 2 + l_ll), 0u);
        q_bar[par2] = map_to_rank(smem_addr(&xbar[par2]), peer);
        q_off = q_snd[par2] - map_to_rank(smem_addr(reinterpret_cast<unsigned *>(splQ)), peer);
    }
    auto wait_arrival = [&](int which, unsigned use, int step, int phase) {
        const unsigned bar = smem_addr(&xbar[which]);
        unsigned long long t0 = 0; unsigned cnt = 0;
        while (!mbar_try_parity(bar, use & 1u))
            if ((++cnt & 1023u) == 0 && wt.expired(t0, step, phase)) return false;
        return true;
    };

    const long long T = p.n_steps;
    constexpr int NPT = (MAXS * K / 2 + 511) / 512;          // slot pairs per thread in the chip-wide gather
#pragma unroll 1
    for (long long n = 1; n <= 2 * T; ++n) {
        const int half = (int)(n & 1);
        const long long s = n >> 1;
        const bool last = n == 2 * T;
        const unsigned tag = (unsigned)n, par = (unsigned)((n - 1) & 1);
        const uint4 *M = half ? wMA : wMB, *L = half ? wO2 : wO4;
        const float *bh = half ? sb1 : sb3, *bl = half ? sb2 : sb4;
        const unsigned use = (unsigned)((n - 1) >> 1);
        if (tid == 0 && own_n > 0) mbar_arrive_expect(smem_addr(&xbar[par]), (unsigned)(own_n * K * 4));
        float gv[3] = {0.f, 0.f, 0.f}, u01 = 0.f;
        int forced = -1;
        if (gater && !last) load_g(half, s, gv);
        if (drawer) {
            const long long t = half ? s : s - 1;
            const long long o = (long long)d_st * T + t;
            if (DBG) {
                if (half) { if (p.c_forced) forced = p.c_forced[o]; }
                else      { if (p.f_forced) forced = p.f_forced[o]; }
            }
            u01 = uniform24(p.seed, p.stream0 + (unsigned)d_st, (unsigned long long)(p.step0 + t - (long long)d_st * p.row_lag), half ? 0u : 1u);
        }

        // ---- 1. the state halves of all streams from the whole chip: all loads first, then the checks
        {
            const unsigned long long *slots = p.slots + (size_t)(half ? (s & 1) : 2 + ((s - 1) & 1)) * NS * K;
            const unsigned ytag = (unsigned)(half ? s + 1 : s);
            const int total = NS * K / 2;
            // every CTA sweeps the slots from a start of its own, so that the 112 readers do not visit the same L2 lines at the same time
            const int rot = NG > 1 ? (cta * total) / (MNC * MCS) : 0;
            unsigned long long v0[NPT], v1[NPT];
            int at[NPT];
#pragma unroll
            for (int q = 0; q < NPT; ++q) {
                const int lin = tid + q * 512;
                at[q] = lin + rot < total ? lin + rot : lin + rot - total;
                v0[q] = v1[q] = 0;
            }
            // a pair goes into the image as soon as it is there
            auto put = [&](int q) {
                const int idx = at[q];
                const int st = (2 * idx) / K, j = 2 * idx - st * K;
                const unsigned x0 = (unsigned)v0[q], x1 = (unsigned)v1[q];       // (high | low << 16) of elements j, j + 1
                const unsigned w_hi = (x0 & 0xffffu) | (x1 << 16), w_lo = (x0 >> 16) | (x1 & 0xffff0000u);
                const int col = 2 * (st & 3);
                unsigned *s32 = reinterpret_cast<unsigned *>(spl + (st >> 2) * IMG_U4);
                s32[mimg_pos(j, col) >> 1] = w_hi; s32[mimg_pos(j, col + 1) >> 1] = w_lo;
                if (spread && st == cl) {
                    unsigned *o32 = reinterpret_cast<unsigned *>(splOwn);
                    o32[mimg_pos(j, 0) >> 1] = w_hi; o32[mimg_pos(j, 1) >> 1] = w_lo;
                }
            };
            unsigned pending = 0;
#pragma unroll
            for (int q = 0; q < NPT; ++q) if (tid + q * 512 < total) pending |= 1u << q;
            {
                unsigned long long t0 = 0; unsigned cnt = 0;
                if (own_n > 0 && (p.flag_mode & (NG == 1 ? 1u : 2u))) {
                    // few streams: nobody polls L2 before this CTA's own gate threads have published (the others do so at
                    // about the same time), so the publishing stores do not queue behind polls
                    while (*(volatile long long *)&s_pub < n - 1)
                        if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
                }
                if (NG > 1 && (pending & 1u) && !my_bad) {
                    // many streams: the first pair alone until it is there, so that the wait does not multiply the polling traffic
                    while (true) {
                        asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v0[0]), "=l"(v1[0]) : "l"(slots + 2 * at[0]) : "memory");
                        if ((unsigned)(v0[0] >> 32) == ytag && (unsigned)(v1[0] >> 32) == ytag) break;
                        if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
                    }
                    pending &= ~1u;
                }
                // then all pairs of the thread together, round after round, so that their round trips overlap
#pragma unroll
                for (int q = 0; q < NPT; ++q)
                    if (pending & (1u << q))
                        asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v0[q]), "=l"(v1[q]) : "l"(slots + 2 * at[q]) : "memory");
                if (NG > 1 && tid < total && !my_bad) put(0);
                while (pending && !my_bad) {
#pragma unroll
                    for (int q = 0; q < NPT; ++q)
                        if ((pending & (1u << q)) && (unsigned)(v0[q] >> 32) == ytag && (unsigned)(v1[q] >> 32) == ytag) { pending &= ~(1u << q); put(q); }
                    if (!pending) break;
                    if ((++cnt & 1023u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
#pragma unroll
                    for (int q = 0; q < NPT; ++q)
                        if (pending & (1u << q))
                            asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v0[q]), "=l"(v1[q]) : "l"(slots + 2 * at[q]) : "memory");
                }
            }
            if (__syncthreads_or(my_bad)) break;
        }
        STAMP(0 + 6 * half);

        // ---- 2. hidden layers of the own streams (tiles 2, 3 of M times column group cl), sent to the cluster
        if (own_n > 0) {
            if (warp < 8) {
                const int tsel = warp & 1, sp = warp >> 1;
                const int p0 = (MKP * sp) / 4, p1 = (MKP * (sp + 1)) / 4;
                float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                const uint4 *bimg = (spread ? splOwn : spl + cl * IMG_U4) + g4 * 4 + t4;
                const uint4 *A = M + (2 + tsel) * TILE_U4 + lane;
                // three or four k-tile pairs: all fragment loads first, then the MMAs back to back
                uint4 bv[4], a0[4], a1[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int kp = p0 + i < p1 ? p0 + i : p0;           // (a fourth pair that is not there repeats the first; its products are dropped)
                    bv[i] = bimg[kp * 32]; a0[i] = A[(2 * kp) * 32]; a1[i] = A[(2 * kp + 1) * 32];
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (p0 + i < p1) {
                        mma16816(acc[0], a0[i], bv[i].x, bv[i].y);
                        mma16816(acc[1], a1[i], bv[i].z, bv[i].w);
                    }
                float *d = part0 + t4 * P0S + (tsel * 4 + sp) * 16;
                d[g4] = (acc[0][0] + acc[1][0]) + (acc[0][1] + acc[1][1]);
                d[g4 + 8] = (acc[0][2] + acc[1][2]) + (acc[0][3] + acc[1][3]);
            }
            __syncthreads();
            STAMP(12 + half);
            // warps 0..3 send, each to four CTAs of the cluster; the others go straight on
            if (warp < 4 && lane < 28 && q_st < own_n) {
                const int r0 = 4 * q_quad;
                const float *pt = part0 + q_st * P0S + ((r0 >> 4) * 4) * 16 + (r0 & 15);
                float4 v = *reinterpret_cast<const float4 *>(bh + r0);
#pragma unroll
                for (int sp = 0; sp < 4; ++sp) {
                    const float4 a = *reinterpret_cast<const float4 *>(pt + sp * 16);
                    v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
                }
                v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f);
                const __nv_bfloat16 hx = __float2bfloat16_rn(v.x), hy = __float2bfloat16_rn(v.y), hz = __float2bfloat16_rn(v.z), hw = __float2bfloat16_rn(v.w);
                const __nv_bfloat16 lx = __float2bfloat16_rn(v.x - __bfloat162float(hx)), ly = __float2bfloat16_rn(v.y - __bfloat162float(hy));
                const __nv_bfloat16 lz = __float2bfloat16_rn(v.z - __bfloat162float(hz)), lw = __float2bfloat16_rn(v.w - __bfloat162float(hw));
                auto pk = [](__nv_bfloat16 a, __nv_bfloat16 b) { return __uint_as_float((unsigned)__bfloat16_as_ushort(a) | ((unsigned)__bfloat16_as_ushort(b) << 16)); };
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const unsigned peer = (unsigned)(warp + 4 * k);
                    st_async_v4(map_to_rank(smem_addr(reinterpret_cast<unsigned *>(splQ)), peer) + q_off, pk(hx, hy), pk(hz, hw), pk(lx, ly), pk(lz, lw),
                                map_to_rank(smem_addr(&xbar[par]), peer));
                }
            }
            STAMP(1 + 6 * half);

        }
        // ---- 3. the cluster's hidden layers -> logits rows of this CTA: warps 0..6 only; the others start the
        // recurrent products (4b) while the hidden layers are in flight, so that R h reaches the gate threads early
        if (own_n > 0 && warp < 7) {
            if (!wait_arrival(par, use, (int)s, 2 + 4 * half)) my_bad = true;
            STAMP(2 + 6 * half);
            {
                float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                const unsigned *bimg = reinterpret_cast<const unsigned *>(splQ) + (t4 >> 1) * 64 + (g4 >> 1) * 4 + (g4 & 1) * 2 + (t4 & 1);
                const uint4 *A = L + lane;
#pragma unroll
                for (int kp = 2 * warp; kp < 2 * warp + 2; ++kp) {
                    const unsigned *b = bimg + kp * 128;
                    const unsigned b00 = b[0], b01 = b[16], b10 = b[32], b11 = b[48];
                    const uint4 a0 = A[(2 * kp) * 32], a1 = A[(2 * kp + 1) * 32];
                    mma16816(acc[0], a0, b00, b01);
                    mma16816(acc[1], a1, b10, b11);
                }
                float *d = part1 + t4 * P0S + warp * 16;
                d[g4] = (acc[0][0] + acc[1][0]) + (acc[0][1] + acc[1][1]);
                d[g4 + 8] = (acc[0][2] + acc[1][2]) + (acc[0][3] + acc[1][3]);
            }
            named_sync(3, 224);
            STAMP(14 + half);
            if (warp == 0 && l_st < own_n) {            // the logits go to the drawing CTA only
                const int r0 = 2 * l_ll;
                const float *pt = part1 + l_st * P0S + r0;
                float v0 = bl[r0], v1 = bl[r0 + 1];
#pragma unroll
                for (int sp = 0; sp < 7; ++sp) { const float2 a = *reinterpret_cast<const float2 *>(pt + sp * 16); v0 += a.x; v1 += a.y; }
                st_cluster_ll(l_snd[par], v0, v1, tag);
            }
            STAMP(3 + 6 * half);
        }

        if (warp < 4) {
            // ---- 4a. drawing warps: the 256 logits of their stream -> draw -> the symbol to every CTA's gate threads
            if (drawer) {
                float l[8];
                {
                    const unsigned a = smem_addr(lbuf + (size_t)(par * 4 + ws) * 128 + 4 * lane);
                    uint4 v0, v1, v2, v3;
                    unsigned long long t0 = 0; unsigned cnt = 0;
                    while (true) {
                        v0 = ld_shared_volatile_v4(a); v1 = ld_shared_volatile_v4(a + 16);
                        v2 = ld_shared_volatile_v4(a + 32); v3 = ld_shared_volatile_v4(a + 48);
                        const bool ok = v0.y == tag && v0.w == tag && v1.y == tag && v1.w == tag && v2.y == tag && v2.w == tag && v3.y == tag && v3.w == tag;
                        if (ok) break;
                        if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 3 + 4 * half)) { my_bad = true; break; }
                    }
                    l[0] = __uint_as_float(v0.x); l[1] = __uint_as_float(v0.z); l[2] = __uint_as_float(v1.x); l[3] = __uint_as_float(v1.z);
                    l[4] = __uint_as_float(v2.x); l[5] = __uint_as_float(v2.z); l[6] = __uint_as_float(v3.x); l[7] = __uint_as_float(v3.z);
                }
                my_bad = __any_sync(FULL, my_bad);
                STAMP(4 + 6 * half);
                const int drawn = warp_softmax_draw_fast(l, u01, lane);
                const int fed = (DBG && forced >= 0) ? forced : drawn;
                {
                    // the symbol to the gate threads of the cluster's 16 CTAs
                    if (lane < MCS && !my_bad) {
                        const unsigned dst = map_to_rank(smem_addr(&s_sym[(n & 1) * 4 + ws]), (unsigned)lane);
                        asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(dst), "l"(((unsigned long long)tag << 32) | (unsigned)fed) : "memory");
                    }
                    const long long t = half ? s : s - 1;
                    if (DBG && p.dbg_logits) {
                        float *d = p.dbg_logits + (((size_t)t * NS + d_st) * 2 + (half ? 0 : 1)) * 256 + 8 * lane;
#pragma unroll
                        for (int k = 0; k < 8; ++k) d[k] = l[k];
                    }
                    if (lane == 0) {
                        const long long o = (long long)d_st * T + t;
                        if (half) { if (p.c_out) p.c_out[o] = (uint8_t)drawn; }
                        else      { if (p.f_out) p.f_out[o] = (uint8_t)drawn; }
                        if (!half && p.out) p.out[(long long)d_st * p.out_pitch + t] = (int16_t)(256 * c_prev + fed - 32768);
                    }
                }
                if (half) c_prev = fed; else f_prev = fed;
            }
            named_sync(2, 512);                       // the image of this half is free once the recurrent products are done
            STAMP(5 + 6 * half);
        } else {
            // ---- 4b. recurrent rows times all streams, then the gates of the other half of the state
            if (warp >= RW0) r_products(M);
            named_arrive(2, 512);
            named_sync(1, 384);
            r_sums(!half, s);
            if (gater && !last) {
                float av[3];
                load_a(half, s, av);
                const GatePre gp = gates_prepare(half, gv, av);
                const volatile unsigned long long *sp = &s_sym[(n & 1) * 4 + gl];
                unsigned long long v, t0 = 0; unsigned cnt = 0;
                while (true) {
                    v = *sp;
                    if ((unsigned)(v >> 32) == tag) break;
                    if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 4 + 4 * half)) { my_bad = true; break; }
                }
                const int fed = (int)(v & 0xffffu);
                if (!my_bad) gates_and_publish(half, s, fed, gp);
                if (half) c_prev = fed; else f_prev = fed;
            }
            if (warp == 4 && !last) { __syncwarp(); if (lane == 0 && !my_bad) *(volatile long long *)&s_pub = n; }
        }
    }
    if (prof_on && lane == 0) for (int i = 0; i < 16; ++i) p.prof[i] = s_prof[i];
#undef STAMP

    const int any_bad = __syncthreads_or(my_bad);
    if (!any_bad) {
        if (gater && p.h_out) { p.h_out[(size_t)gst * H + gj] = hC; p.h_out[(size_t)gst * H + K + gj] = hF; }
        if (drawer && lane == 0) {
            if (p.c_st_out) p.c_st_out[d_st] = (uint8_t)c_prev;
            if (p.f_st_out) p.f_st_out[d_st] = (uint8_t)f_prev;
        }
    }
    cluster.sync();
}

// ---------------------------------------------------------------------------------------------
static int resmulti_smem_bytes(const ResMultiPack &k)
{
    size_t b = k.blob_bytes;
    b += (size_t)MAXS * MNR * 4 + (size_t)(2 * 3 * MHR * 3 + 8) * 4;   // a_part, the gate threads' input weights
    b += (size_t)PR_FLOATS * 4 + (size_t)8 * P0S * 4;
    b += (size_t)6 * IMG_U4 * 16;                   // four column-group images, the hidden-layer image, the own streams' image
    b += (size_t)1024 * 16;                         // lbuf
    return (int)b;
}

static void multi_fill_launch(const ResMultiPack &k, cudaLaunchConfig_t *cfg, cudaLaunchAttribute *at, cudaStream_t s, bool coop)
{
    std::memset(cfg, 0, sizeof(*cfg));
    cfg->gridDim = dim3(MNC * MCS);
    cfg->blockDim = dim3(512);
    cfg->dynamicSmemBytes = k.smem_bytes;
    cfg->stream = s;
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = MCS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative;
    at[1].val.cooperative = 1;
    cfg->attrs = at;
    cfg->numAttrs = coop ? 2 : 1;
}

int resmulti_prepare(wrnn_model *m)
{
    const int H = m->H, K = MK;
    if (m->dtype != WRNN_BF16 || m->sparse || m->variant != 0 || H != 2 * MK || m->max_batch < 2 || m->n_sms < MNC * MCS) {
        m->err = "multi-stream resident kernel: dense bf16 H = 896 models with max_batch >= 2 only";
        return WRNN_ERR_UNSUPPORTED;
    }
    ResMultiPack k;
    k.w_bytes = (size_t)10 * 16 * K * 2;
    k.blob_bytes = k.w_bytes + ((size_t)(MNR * 3 + 2 * MHR + 2 * MLR) * 4 + 15) / 16 * 16;
    k.smem_bytes = resmulti_smem_bytes(k);
    cudaDeviceProp prop;
    cudaGetDeviceProperties(&prop, m->device);
    if ((size_t)k.smem_bytes > prop.sharedMemPerBlockOptin ||
        cudaFuncSetAttribute(resident_multi_kernel<0>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
        cudaFuncSetAttribute(resident_multi_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem_bytes) != cudaSuccess ||
        cudaFuncSetAttribute(resident_multi_kernel<1>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
        cudaFuncSetAttribute(resident_multi_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem_bytes) != cudaSuccess ||
        cudaFuncSetAttribute(resident_multi_kernel<2>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
        cudaFuncSetAttribute(resident_multi_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem_bytes) != cudaSuccess ||
        cudaFuncSetAttribute(resident_multi_kernel<4>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
        cudaFuncSetAttribute(resident_multi_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem_bytes) != cudaSuccess) {
        cudaGetLastError();
        m->err = "multi-stream resident kernel does not fit in shared memory";
        return WRNN_ERR_UNSUPPORTED;
    }
    {
        cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
        multi_fill_launch(k, &cfg, at, 0, false);
        int max_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&max_clusters, resident_multi_kernel<0>, &cfg) != cudaSuccess || max_clusters < MNC) {
            cudaGetLastError();
            m->err = "not enough co-resident clusters for the multi-stream resident kernel";
            return WRNN_ERR_UNSUPPORTED;
        }
    }

    // ---- per-CTA blobs: A fragments of [R rows ; hidden-layer rows] for both halves, logits rows, small fp32 parameters
    const std::vector<uint16_t> dR = dense_bf16_bits(m->hR), dO1 = dense_bf16_bits(m->hO1), dO2 = dense_bf16_bits(m->hO2),
                                dO3 = dense_bf16_bits(m->hO3), dO4 = dense_bf16_bits(m->hO4);
    const std::vector<uint16_t> *Oa[2] = {&dO1, &dO3}, *Ob[2] = {&dO2, &dO4};
    const int NCTA = MNC * MCS;
    std::vector<uint8_t> blob((size_t)NCTA * k.blob_bytes, 0);
    std::vector<const uint16_t *> rows(16);
    const std::vector<uint16_t> zero_row(K, 0);
    // rows[16] (K bf16 each) -> A fragments [K / 16][32 lanes][8]: lane (g, t) holds (row g, k 2t..2t+1), (row g + 8, same),
    // (row g, k 2t+8..9), (row g + 8, same)
    auto pack_tile = [&](uint16_t *dst) {
        for (int kt = 0; kt < K / 16; ++kt)
            for (int lane = 0; lane < 32; ++lane) {
                const int g = lane >> 2, t = lane & 3;
                uint16_t *o = dst + ((size_t)kt * 32 + lane) * 8;
                const int rsel[4] = {g, g + 8, g, g + 8};
                const int csel[4] = {2 * t, 2 * t, 2 * t + 8, 2 * t + 8};
                for (int q = 0; q < 4; ++q)
                    for (int j = 0; j < 2; ++j) o[2 * q + j] = rows[rsel[q]][16 * kt + csel[q] + j];
            }
    };
    for (int cta = 0; cta < NCTA; ++cta) {
        const int rank = cta % MCS;
        uint8_t *base = blob.data() + (size_t)cta * k.blob_bytes;
        uint16_t *w = reinterpret_cast<uint16_t *>(base);
        float *sm = reinterpret_cast<float *>(base + k.w_bytes);
        const size_t tile_elems = (size_t)16 * K;
        // R row rr = (half * 3 + gate) * UC + u  ->  matrix row gate * H + half * K + cta * UC + u
        auto r_row = [&](int rr) { return ((rr / MUC) % 3) * H + (rr / (3 * MUC)) * K + cta * MUC + rr % MUC; };
        for (int part = 0; part < 2; ++part)
            for (int mt = 0; mt < 4; ++mt) {
                for (int r = 0; r < 16; ++r) {
                    const int row = 16 * (mt & 1) + r;
                    if (mt < 2) rows[r] = row < MNR ? dR.data() + (size_t)r_row(row) * H + part * K : zero_row.data();
                    else rows[r] = row < MHR ? Oa[part]->data() + (size_t)(rank * MHR + row) * K : zero_row.data();
                }
                pack_tile(w + ((size_t)part * 4 + mt) * tile_elems);
            }
        for (int h = 0; h < 2; ++h) {
            for (int r = 0; r < 16; ++r) rows[r] = Ob[h]->data() + (size_t)(rank * MLR + r) * K;
            pack_tile(w + ((size_t)8 + h) * tile_elems);
        }
        for (int rr = 0; rr < MNR; ++rr)
            for (int c = 0; c < 3; ++c) sm[rr * 3 + c] = m->hI[(size_t)r_row(rr) * 3 + c];
        float *b = sm + MNR * 3;
        for (int r = 0; r < MHR; ++r) { b[r] = m->hb1[rank * MHR + r]; b[MHR + r] = m->hb3[rank * MHR + r]; }
        b += 2 * MHR;
        for (int r = 0; r < MLR; ++r) { b[r] = m->hb2[rank * MLR + r]; b[MLR + r] = m->hb4[rank * MLR + r]; }
    }
    ResMultiPack *pk = new ResMultiPack(k);
    const bool ok = cudaMalloc((void **)&pk->d_blob, blob.size()) == cudaSuccess &&
                    cudaMemcpy(pk->d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice) == cudaSuccess &&
                    cudaMalloc((void **)&pk->d_slots, (size_t)4 * MAXS * K * 8) == cudaSuccess &&
                    cudaMalloc((void **)&pk->d_aslots, (size_t)2 * MAXS * 6 * K * 8) == cudaSuccess &&
                    cudaMalloc((void **)&pk->d_prof, 16 * sizeof(long long)) == cudaSuccess &&
                    cudaMemset(pk->d_prof, 0, 16 * sizeof(long long)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        cudaFree(pk->d_blob); cudaFree(pk->d_slots); cudaFree(pk->d_aslots); cudaFree(pk->d_prof);
        delete pk;
        m->err = "device allocation for the multi-stream resident kernel failed";
        return WRNN_ERR_NOMEM;
    }
    pk->weight_bytes_per_step = (int64_t)NCTA * (int64_t)k.w_bytes;
    m->resmulti = pk;
    return WRNN_OK;
}

void resmulti_destroy(wrnn_model *m)
{
    if (!m->resmulti) return;
    cudaFree(m->resmulti->d_blob);
    cudaFree(m->resmulti->d_slots);
    cudaFree(m->resmulti->d_aslots);
    cudaFree(m->resmulti->d_prof);
    delete m->resmulti;
    m->resmulti = nullptr;
}

int resmulti_supported(const wrnn_model *m, int batch)
{
    return m->resmulti && batch >= 2 && batch <= MAXS ? WRNN_OK : WRNN_ERR_UNSUPPORTED;
}

int resmulti_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes)
{
    (void)batch;
    const ResMultiPack &k = *m->resmulti;
    if (n_ctas) *n_ctas = MNC * MCS;
    if (n_threads) *n_threads = 512;
    if (smem) *smem = k.smem_bytes;
    if (weight_bytes) *weight_bytes = k.weight_bytes_per_step;
    return WRNN_OK;
}

int resmulti_phase_cycles(const wrnn_model *m, long long *out16)
{
    if (!m->resmulti) return WRNN_ERR_UNSUPPORTED;
    return cudaMemcpy(out16, m->resmulti->d_prof, 16 * sizeof(long long), cudaMemcpyDeviceToHost) == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
}

int resmulti_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    static const int MODE0_MAX_ROWS = [] { const char *e = getenv("WRNN_MULTI_MODE0_ROWS"); return e ? atoi(e) : 4; }();
    const ResMultiPack &k = *m->resmulti;
    MultiParams p;
    std::memset(&p, 0, sizeof(p));
    p.H = m->H; p.NS = a.batch;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.row_lag = a.row_lag; p.out_pitch = a.out_pitch ? a.out_pitch : a.n_steps;
    p.blob = k.d_blob; p.blob_bytes = k.blob_bytes; p.w_bytes = k.w_bytes;
    p.g = m->g; p.slots = k.d_slots; p.aslots = k.d_aslots; p.I = m->I;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in; p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;
    p.prof = m->prof_enabled ? k.d_prof : nullptr;     // phase stamps cost the stamped warp some 50 cycles each: off unless asked for
    { const char *d = getenv("WRNN_MULTI_FLAG"); p.flag_mode = d ? (unsigned)atoi(d) : 1u; }    // diagnostic: A/B of the gather protocol

    if (cudaMemsetAsync(k.d_slots, 0, (size_t)4 * MAXS * MK * 8, s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(k.d_aslots, 0, (size_t)2 * MAXS * 6 * MK * 8, s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
    multi_fill_launch(k, &cfg, at, s, coop_launch_allowed());
    // Plain sampling of up to four rows runs the instantiation without stamps, forced symbols and dumps (mode 0); above four
    // rows the one that carries the (unexecuted) stamp code but no forced symbols or dumps (mode 4) is the fastest: 16 rows 9.52 us
    // per lock-step against 9.55 with everything compiled in and 9.95 with nothing, 4 rows 7.21 against 6.97 (same call,
    // alternating): the compiler orders the half-step differently around the clock reads.
    const bool teacher = p.c_forced || p.f_forced || p.dbg_gates || p.dbg_h || p.dbg_logits;
    const int mode = m->dbg_skip_cta >= 0 ? 1 : (p.prof || teacher) ? 2 : a.batch > MODE0_MAX_ROWS ? 4 : 0;
    const cudaError_t e = mode == 1 ? cudaLaunchKernelEx(&cfg, resident_multi_kernel<1>, p)
                          : mode == 2 ? cudaLaunchKernelEx(&cfg, resident_multi_kernel<2>, p)
                          : mode == 4 ? cudaLaunchKernelEx(&cfg, resident_multi_kernel<4>, p)
                                      : cudaLaunchKernelEx(&cfg, resident_multi_kernel<0>, p);
    if (e != cudaSuccess) {
        m->err = std::string("multi-stream resident kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    m->prof_multi = true;
    return WRNN_OK;
}

}  // namespace wrnn
