// Shared-memory-resident persistent sampling kernel for one stream (batch 1), dense bf16 weights.
//
// The whole utterance is one cooperative launch of NC clusters x CS CTAs (Section 2.1 of the paper:
// one persistent operation, parameters loaded on-chip once).  Weights never leave shared memory:
//   * every CTA owns UC coarse and UC fine state units, i.e. 6 UC rows of R (gates u, r, e), split
//     into the columns that multiply y_c and the columns that multiply y_f;
//   * both output heads are replicated once per cluster and row-sharded over its CS CTAs
//     (O1/O3: Hh/CS rows each, O2/O4: 256/CS rows each), so the drawn c_t / f_t are produced
//     inside every cluster (bit-identically) and never have to be broadcast across the chip.
// Per step there are exactly two chip-wide exchanges through L2 -- y_c(t) before the coarse head and
// y_f(t) before the fine head (Fig. 1's order) -- each an all-gather of (value, step-tag) words so
// that arrival of the data is the signal.  Inside a cluster the logits travel through distributed
// shared memory the same way (one warp consumes them), the hidden layer by asynchronous stores that
// complete an mbarrier at the receiver (every warp of the CTA consumes it: nobody polls).  The fine head
// of step t overlaps the recurrent product of step t+1 (f_t is only needed by the coarse gates of t+1).
//
// Mat-vec products run on the tensor pipe as m16n8k16 bf16 MMAs: the weights sit in shared memory
// in A-fragment order (one 16-byte load per lane per 16x16 tile), and the fp32 input vector is split
// exactly into three bf16 vectors (hi + mid + lo) that occupy three of the eight B columns, so the
// fp32 state is not rounded on its way in; accumulation is fp32.
//
// Every wait is bounded; a CTA that gives up records where and all CTAs leave through the final
// cluster barrier.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>

#include "wrnn_cluster.cuh"
#include "wrnn_internal.h"

namespace cg = cooperative_groups;

namespace wrnn {

struct ResidentPack {
    int NC = 0, CS = 0, NCTA = 0, UC = 0, HR = 0, LR = 0, K = 0, NKT = 0, NMT = 0, NLT = 0, NW = 0, KSH = 0, KSL = 0;
    int n_rrows = 0;                 // 6 UC
    bool fused = false;              // Fused Subscale WaveRNN 2x: 12 input columns, 64 logits per head
    int pair_smem = 0;               // dynamic shared memory of the two-stream kernel; 0 = not available
    unsigned long long *d_slots2 = nullptr;  // [2 halves][2 parities][2 streams][K] (value, tag)
    size_t blob_bytes = 0;           // per CTA: bf16 weight fragments then fp32 small parameters
    size_t w_bytes = 0;              // bf16 part of the blob
    uint8_t *d_blob = nullptr;       // [NCTA][blob_bytes]
    unsigned long long *d_slots = nullptr;   // [2 halves][2 parities][K] (value, tag)
    int smem_bytes = 0;
    int64_t weight_bytes_per_step = 0;
    long long *d_prof = nullptr;     // [16] phase cycle totals of the last call (diagnostic)
};

struct ResidentParams {
    int H, K, NKT, NMT, NLT, UC, HR, LR, CS, n_rrows;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    long long frame_shift;                   // subtracted from the frame index (a call whose conditioning starts at its first step)
    const uint8_t *blob; unsigned long long blob_bytes, w_bytes;
    const float *g;                          // [n_frames][3H]
    unsigned long long *slots;               // [2][2][K]
    const float *h_in; float *h_out;
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;
    uint8_t *c_out, *f_out;
    int16_t *out;
    // the fused variant's 16-bit counterparts of the byte arrays above (part A = the coarse half, part B = the fine half)
    const uint16_t *a_in, *b_in; uint16_t *a_st_out, *b_st_out;
    const uint16_t *a_forced, *b_forced;
    uint16_t *a_out, *b_out;
    float *dbg_gates, *dbg_h, *dbg_logits;
    DevStatus *status;
    unsigned long long limit_ns;
    int skip_cta; long long skip_step;      // self-test: this CTA withholds what it publishes at this step (-1: none)
    long long *prof;                         // optional [16] per-phase cycle totals of CTA 0, warp 0
};

// KSH / KSL: K-splits per hidden / logits tile; NKH / NKL: k-tiles per split (KSH * NKH = KSL * NKL = K / 16).
// FUSED: the Fused Subscale WaveRNN 2x.  The same cell and schedule; the coarse half of the state is part A (sub-tensor
// 0), the fine half part B (sub-tensor 1, which sees the sample of part A inside the step: future horizon 2); each head
// has 64 logits = four softmaxes of 4 bits, every input is a group of four nibbles instead of one byte, and the
// symbols (c, f) below are the 16-bit samples (a, b).
template <int KSH, int NKH, int KSL, int NKL, bool FUSED>
__global__ void __launch_bounds__(512, 1) resident_dense_kernel(const ResidentParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int cta = blockIdx.x;                       // global CTA index = owner index of state units
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = p.K, NKT = p.NKT, NMT = p.NMT, NLT = p.NLT, UC = p.UC, HR = p.HR, LR = p.LR, CS = p.CS, H = p.H;
    const int NR = p.n_rrows;                          // 6 UC
    constexpr int NP = FUSED ? 4 : 1;                  // scalars per symbol: four nibbles, or one byte
    constexpr int NIN = 3 * NP;                        // columns of I*: previous c, previous f, this step's c

    // ---- shared memory carve-up (must match resident_smem_bytes)
    const size_t tile_u4 = (size_t)NKT * 32;                                   // uint4 per 16-row tile
    const uint4 *wMA = reinterpret_cast<const uint4 *>(smem);                  // [NMT] tiles: rows [O1 ; R x coarse cols]
    const uint4 *wMB = wMA + (size_t)NMT * tile_u4;                            // [NMT] tiles: rows [O3 ; R x fine cols]
    const uint4 *wO2 = wMB + (size_t)NMT * tile_u4;                            // [NLT] tiles
    const uint4 *wO4 = wO2 + (size_t)NLT * tile_u4;
    const float *sI = reinterpret_cast<const float *>(smem + p.w_bytes);       // [NR][NIN]
    const float *sb1 = sI + NR * NIN, *sb3 = sb1 + HR, *sb2 = sb3 + HR, *sb4 = sb2 + LR;
    float *vecC = reinterpret_cast<float *>(smem + p.blob_bytes);              // [K] y_c (fp32, natural order)
    float *vecF = vecC + K;                                                    // [K] y_f
    float *a_part = vecF + K;                                                  // [NR] R[:, :Hh] y_c
    float *a_full = a_part + NR;                                               // [NR] R h
    float *part = a_full + NR + ((2 * NR) % 4 ? 4 - (2 * NR) % 4 : 0);         // [tiles x K-splits][16] partial sums
    __nv_bfloat16 *splC = reinterpret_cast<__nv_bfloat16 *>(part + 512);       // split images, 4 K bf16 each
    __nv_bfloat16 *splF = splC + 4 * K;
    __nv_bfloat16 *splQ = splF + 4 * K;
    float *qbuf = reinterpret_cast<float *>(splQ + 4 * K);                    // [2][K] hidden layer of the cluster
    uint4 *lbuf = reinterpret_cast<uint4 *>(qbuf + 2 * K);                     // [2][128] logits of the cluster: {v, tag, v, tag}
    __shared__ __align__(8) unsigned long long xbar[2];                        // arrival barriers of qbuf[0], qbuf[1]

    // ---- one-time load of this CTA's weights
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.blob + (size_t)cta * p.blob_bytes);
        uint4 *dst = reinterpret_cast<uint4 *>(smem);
        for (size_t i = tid; i < p.blob_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
        for (int i = tid; i < 2 * K + 1024; i += blockDim.x) qbuf[i] = 0.f;             // qbuf and lbuf are adjacent
        if (tid == 0) {
            for (int i = 0; i < 2; ++i) mbar_init_cluster(smem_addr(&xbar[i]), 1);
            mbar_fence_init();
        }
        for (int i = tid; i < 12 * K / 8; i += blockDim.x) reinterpret_cast<uint4 *>(splC)[i] = make_uint4(0, 0, 0, 0);
        __syncthreads();
        for (int i = tid; i < K; i += blockDim.x) {
            const float c = p.h_in ? p.h_in[i] : 0.f, f = p.h_in ? p.h_in[K + i] : 0.f;
            vecC[i] = c; vecF[i] = f;
            store_split2(splC, i, c);
            store_split2(splF, i, f);
        }
    }
    __syncthreads();
    cluster.sync();     // peers' exchange buffers are zeroed before anyone writes into them

    Waiter wt{p.status, p.limit_ns};
    bool my_bad = false;      // this thread gave up on a wait; made CTA-uniform by __syncthreads_or
    // optional phase timing (CTA 0, warp 0): cycles spent up to each stamp since the previous one
    const bool prof_on = p.prof != nullptr && cta == 0 && warp == 0;
    __shared__ long long s_prof[16];
    if (tid < 16) s_prof[tid] = 0;
    __syncthreads();
    long long prof_t = clock64();
#define STAMP(i) do { if (prof_on) { const long long now_ = clock64(); if (lane == 0) s_prof[i] += now_ - prof_t; prof_t = now_; } } while (0)

    const bool writer = (cta == 0);
    const int g4 = lane >> 2;

    // warp 0 keeps the stream's scalar state
    int c_prev, f_prev;
    if (FUSED) { c_prev = p.a_in ? p.a_in[0] : 0x8000; f_prev = p.b_in ? p.b_in[0] : 0x8000; }
    else { c_prev = p.c_in ? p.c_in[0] : 128; f_prev = p.f_in ? p.f_in[0] : 0; }
    // scalar k of a symbol as the network sees it
    auto xin = [](int v, int k) { return FUSED ? scale4((v >> (12 - 4 * k)) & 15) : scale8(v); };
    float hC = 0.f, hF = 0.f;
    if (warp == 0 && lane < UC) { hC = vecC[cta * UC + lane]; hF = vecF[cta * UC + lane]; }

    // Fixed roles: in the hidden phase warp w takes K-split (w % KSH) of the tile pair (w / KSH), one load of the vector
    // fragments serving both tiles; in the logits phase K-split (w % KSL) of tile (w / KSL).  Each leaves 16 partial row
    // sums per tile in part[tile * K-splits + split].
    const int h_pair = warp / KSH, h_ks = warp % KSH, h_kt0 = h_ks * NKH;
    const int l_tile = warp / KSL, l_ks = warp % KSL, l_kt0 = l_ks * NKL;
    const bool h_on = warp < (NMT / 2) * KSH, l_on = warp < NLT * KSL;
    const bool h_fin = warp < NMT;
    auto hidden_products = [&](const uint4 *Mx, const __nv_bfloat16 *sp) {
        float lo[2], hi[2];
        mma_tiles<NKH, 2>(Mx + (size_t)(2 * h_pair) * tile_u4, tile_u4, h_kt0, sp, lane, lo, hi);
        if ((lane & 3) == 0) {
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                float *d = part + ((2 * h_pair + n) * KSH + h_ks) * 16;
                d[g4] = lo[n]; d[g4 + 8] = hi[n];
            }
        }
    };
    // one peer per warp: warp w sends this CTA's whole slice to CTA w of the cluster with one store instruction, lanes at
    // consecutive pieces (a store whose lanes address several CTAs at once is much slower).  The hidden layer, which
    // many threads consume, goes by asynchronous stores that count their bytes on the receiver's barrier of that buffer
    // (nobody polls the data); the logits, which one warp consumes, as tagged values that this warp polls.
    unsigned q_snd[2], l_snd[2], q_bar[2];
#pragma unroll
    for (int par2 = 0; par2 < 2; ++par2) {
        const unsigned peer = warp < CS ? warp : 0;
        q_snd[par2] = map_to_rank(smem_addr(qbuf + (size_t)par2 * K + rank * HR + 2 * (lane < HR / 2 ? lane : 0)), peer);
        l_snd[par2] = map_to_rank(smem_addr(lbuf + (size_t)par2 * 128 + (rank * LR) / 2 + (lane < LR / 2 ? lane : 0)), peer);
        q_bar[par2] = map_to_rank(smem_addr(&xbar[par2]), peer);
    }
    // bounded wait for all bytes of one buffer (use k of a buffer completes barrier phase k)
    auto wait_arrival = [&](int which, unsigned use, int step, int phase) {
        const unsigned bar = smem_addr(&xbar[which]);
        unsigned long long t0 = 0; unsigned cnt = 0;
        while (!mbar_try_parity(bar, use & 1u))
            if ((++cnt & 1023u) == 0 && wt.expired(t0, step, phase)) return false;
        return true;
    };
    // ---- prologue: the recurrent products of step 0 from the initial state, coarse gates of step 0
    if (h_on) hidden_products(wMA, splC);
    __syncthreads();
    if (h_fin && lane < 16 && 16 * warp + lane >= HR && 16 * warp + lane - HR < NR) {
        float v = 0.f;
#pragma unroll
        for (int sp = 0; sp < KSH; ++sp) v += part[(warp * KSH + sp) * 16 + lane];
        a_part[16 * warp + lane - HR] = v;
    }
    __syncthreads();
    if (h_on) hidden_products(wMB, splF);
    __syncthreads();
    if (h_fin && lane < 16 && 16 * warp + lane >= HR && 16 * warp + lane - HR < NR) {
        float v = 0.f;
#pragma unroll
        for (int sp = 0; sp < KSH; ++sp) v += part[(warp * KSH + sp) * 16 + lane];
        a_full[16 * warp + lane - HR] = a_part[16 * warp + lane - HR] + v;
    }
    __syncthreads();

    // Gates of Eq. 2 for this CTA's units of one half of the state, then publish them to the chip.
    // half_g = 0: coarse units (c_s does not reach them: their I* column is zero), 1: fine units.
    // The gate pre-activations up to the one input that is only known after the draw (c_s for the fine units, f_{s-1} for
    // the coarse units of the next step): computed while the logits are still on their way.
    struct GatePre { float pu, pr, pe, ae, ku[NP], kr[NP], ke[NP]; };
    auto gates_prepare = [&](int half_g, const float (&gv)[3]) {
        GatePre q;
        const int rb = half_g ? 3 * UC : 0;
        const float *Iu = sI + NIN * (rb + lane), *Ir = sI + NIN * (rb + UC + lane), *Ie = sI + NIN * (rb + 2 * UC + lane);
        // fine units: inputs (c_{s-1}, f_{s-1}) known, c_s pending (last column group); coarse units: c_{s-1} known,
        // f_{s-1} pending (middle column group)
        float su = gv[0], sr = gv[1], se = gv[2];
#pragma unroll
        for (int k = 0; k < NP; ++k) {
            const float x = xin(c_prev, k);
            su = fmaf(Iu[k], x, su); sr = fmaf(Ir[k], x, sr); se = fmaf(Ie[k], x, se);
        }
        if (half_g) {
#pragma unroll
            for (int k = 0; k < NP; ++k) {
                const float x = xin(f_prev, k);
                su = fmaf(Iu[NP + k], x, su); sr = fmaf(Ir[NP + k], x, sr); se = fmaf(Ie[NP + k], x, se);
            }
        }
        q.pu = a_full[rb + lane] + su;
        q.pr = a_full[rb + UC + lane] + sr;
        q.pe = se;
        q.ae = a_full[rb + 2 * UC + lane];
        const int pend = half_g ? 2 * NP : NP;
#pragma unroll
        for (int k = 0; k < NP; ++k) { q.ku[k] = Iu[pend + k]; q.kr[k] = Ir[pend + k]; q.ke[k] = Ie[pend + k]; }
        return q;
    };
    // Gates of Eq. 2 for this CTA's units of one half of the state, then publish them to the chip.
    // half_g = 0: coarse units (c_s does not reach them: their I* column is zero), 1: fine units.
    const int skip_at = cta == p.skip_cta ? (int)p.skip_step : -1;      // self-test: the step at which this CTA withholds its publication
    auto gates_and_publish = [&](int half_g, long long s, int drawn, const GatePre &q) {
        float pu = q.pu, pr = q.pr, pe = q.pe;
#pragma unroll
        for (int k = 0; k < NP; ++k) {
            const float xk = xin(drawn, k);              // the pending input
            pu = fmaf(q.ku[k], xk, pu); pr = fmaf(q.kr[k], xk, pr); pe = fmaf(q.ke[k], xk, pe);
        }
        const float u = sigmoidf_fast(pu), r = sigmoidf_fast(pr);
        const float e = tanhf_fast(fmaf(r, q.ae, pe));
        const float hn = fmaf(u, half_g ? hF : hC, (1.0f - u) * e);
        if (half_g) hF = hn; else hC = hn;
        const int j = cta * UC + lane, jj = (half_g ? K : 0) + j;
        if ((int)s != skip_at)
            st_relaxed_u64(p.slots + (size_t)((half_g ? 2 : 0) + (s & 1)) * K + j,
                           ((unsigned long long)(unsigned)(s + 1) << 32) | __float_as_uint(hn));
        if (p.dbg_gates) { float *d = p.dbg_gates + (size_t)s * 3 * H; d[jj] = u; d[H + jj] = r; d[2 * H + jj] = e; }
        if (p.dbg_h) p.dbg_h[(size_t)s * H + jj] = hn;
    };
    auto load_g = [&](int half_g, long long s, float (&gv)[3]) {
        const long long fr = ((p.step0 + s) * p.row_stride + (long long)p.stream0 * p.row_offset_mul) / p.hop - p.frame_shift;
        const float *g = p.g + (size_t)fr * 3 * H + (half_g ? K : 0) + cta * UC + lane;
#pragma unroll
        for (int gate = 0; gate < 3; ++gate) gv[gate] = __ldg(g + gate * H);
    };
    if (warp == 0 && lane < UC) {
        float gv[3];
        load_g(0, 0, gv);
        gates_and_publish(0, 0, f_prev, gates_prepare(0, gv));
    }

    // The step is two structurally identical halves (Fig. 1).  Half-step n = 2 s + 1 is the "coarse" half of
    // step s (input y_c(s): coarse head -> c_s; R[:, :Hh] y_c(s) kept for step s+1; then the fine gates of
    // step s); n = 2 s is the "fine" half (input y_f(s-1): fine head -> f_{s-1}; R[:, Hh:] y_f(s-1) completes
    // R h_{s-1}; then the coarse gates of step s).  One loop body serves both so that the code stays small.
    const long long T = p.n_steps;
#pragma unroll 1
    for (long long n = 1; n <= 2 * T; ++n) {
        const int half = (int)(n & 1);                 // 1: coarse half, 0: fine half
        const long long s = n >> 1;
        const bool last = n == 2 * T;                  // final fine half: draw f_{T-1} only
        const unsigned tag = (unsigned)n, par = (unsigned)((n - 1) & 1);   // cluster-exchange tag / buffer of this half
        const uint4 *M = half ? wMA : wMB, *L = half ? wO2 : wO4;
        const float *bh = half ? sb1 : sb3, *bl = half ? sb2 : sb4;
        float *vec = half ? vecC : vecF;
        __nv_bfloat16 *spl = half ? splC : splF;

        const unsigned use = (unsigned)((n - 1) >> 1);          // how often this half's buffers were used before
        if (tid == 0) mbar_arrive_expect(smem_addr(&xbar[par]), (unsigned)K * 4u);      // this half's arrivals: K hidden values
        // everything that does not depend on the chain is fetched / computed before the first wait
        float gv[3] = {0.f, 0.f, 0.f}, u01 = 0.f;
        int forced = -1;
        if (warp == 0) {
            if (lane < UC && !last) load_g(half, s, gv);          // gates evaluated at the end of this half
            if (FUSED) {
                if (half) { if (p.a_forced) forced = p.a_forced[s]; }
                else      { if (p.b_forced) forced = p.b_forced[s - 1]; }
                u01 = uniform24(p.seed, p.stream0, (unsigned long long)(p.step0 + (half ? s : s - 1)), (half ? 0u : 4u) + (unsigned)(lane >> 3));
            } else {
                if (half) { if (p.c_forced) forced = p.c_forced[s]; }
                else      { if (p.f_forced) forced = p.f_forced[s - 1]; }
                u01 = uniform24(p.seed, p.stream0, (unsigned long long)(p.step0 + (half ? s : s - 1)), half ? 0u : 1u);
            }
        }

        // ---- 1. input half-vector from the whole chip (y_c(s) carries tag s+1; y_f(s-1) carries tag s)
        {
            const unsigned long long *slots = p.slots + (size_t)(half ? (s & 1) : 2 + ((s - 1) & 1)) * K;
            const unsigned ytag = (unsigned)(half ? s + 1 : s);
            // two adjacent slots per polling thread (one 16-byte load): half as many requests queue at the L2 slices
#pragma unroll 1
            for (int i = tid; i < K / 2; i += blockDim.x) {
                unsigned long long v0, v1, t0 = 0; unsigned cnt = 0;
                while (true) {
                    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v0), "=l"(v1) : "l"(slots + 2 * i) : "memory");
                    if ((unsigned)(v0 >> 32) == ytag && (unsigned)(v1 >> 32) == ytag) break;
                    if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
                }
                const float x0 = __uint_as_float((unsigned)v0), x1 = __uint_as_float((unsigned)v1);
                vec[2 * i] = x0; vec[2 * i + 1] = x1;
                store_split2_pair(spl, 2 * i, x0, x1);
            }
            if (__syncthreads_or(my_bad)) break;
        }
        STAMP(0 + 6 * half);

        // ---- 2. hidden layer of the head + this CTA's R rows against the same input
        if (h_on) hidden_products(M, spl);
        __syncthreads();
        STAMP(12 + half);
        // warp w finishes the whole hidden-layer slice of this CTA itself (two rows per lane: K-split partials, bias,
        // relu) and sends it to CTA w of the cluster: one store instruction per peer, no further CTA barrier
        if (warp < CS && lane < HR / 2) {
            const int r0 = 2 * lane, tile = r0 >> 4, rr = r0 & 15;
            float v0 = bh[r0], v1 = bh[r0 + 1];
#pragma unroll
            for (int sp = 0; sp < KSH; ++sp) { v0 += part[(tile * KSH + sp) * 16 + rr]; v1 += part[(tile * KSH + sp) * 16 + rr + 1]; }
            st_async_v2(q_snd[par], fmaxf(v0, 0.f), fmaxf(v1, 0.f), q_bar[par]);
        }
        if (h_fin && lane < 16) {
            // R rows of this tile (rows >= HR of the stacked matrix) stay in this CTA
            const int row = 16 * warp + lane;
            if (row >= HR && row - HR < NR) {
                float v = 0.f;
#pragma unroll
                for (int sp = 0; sp < KSH; ++sp) v += part[(warp * KSH + sp) * 16 + lane];
                if (half) a_part[row - HR] = v;                                    // R[:, :Hh] y_c(s): kept for step s+1
                else a_full[row - HR] = a_part[row - HR] + v;                      // R h_{s-1} complete
            }
        }
        STAMP(1 + 6 * half);

        // ---- 3. the cluster's hidden layer -> logits rows of this CTA
        if (tid < K / 2) {
            if (!wait_arrival(par, use, (int)s, 2 + 4 * half)) my_bad = true;
            const float2 v = reinterpret_cast<const float2 *>(qbuf + (size_t)par * K)[tid];
            store_split2_pair(splQ, 2 * tid, v.x, v.y);
        }
        if (__syncthreads_or(my_bad)) break;
        STAMP(2 + 6 * half);
        if (l_on) {
            float lo[1], hi[1];
            mma_tiles<NKL, 1>(L + (size_t)l_tile * tile_u4, tile_u4, l_kt0, splQ, lane, lo, hi);
            if ((lane & 3) == 0) { part[warp * 16 + g4] = lo[0]; part[warp * 16 + g4 + 8] = hi[0]; }
        }
        __syncthreads();
        STAMP(14 + half);
        if (warp < CS && lane < LR / 2) {
            const int r0 = 2 * lane, tile = r0 >> 4, rr = r0 & 15;
            float v0 = bl[r0], v1 = bl[r0 + 1];
#pragma unroll
            for (int sp = 0; sp < KSL; ++sp) { v0 += part[(tile * KSL + sp) * 16 + rr]; v1 += part[(tile * KSL + sp) * 16 + rr + 1]; }
            st_cluster_ll(l_snd[par], v0, v1, tag);
        }
        STAMP(3 + 6 * half);

        // ---- 4. warp 0: the cluster's 256 logits -> draw; then the gates of the other half of the state
        if (warp == 0) {
            GatePre gp = {};
            if (lane < UC && !last) gp = gates_prepare(half, gv);
            int drawn;
            float l[FUSED ? 2 : 8];
            if (FUSED) {
                // 64 logits: one slot (two logits) per lane
                const unsigned a = smem_addr(lbuf + (size_t)par * 128 + lane);
                uint4 v0;
                unsigned long long t0 = 0; unsigned cnt = 0;
                while (true) {
                    v0 = ld_shared_volatile_v4(a);
                    if (v0.y == tag && v0.w == tag) break;
                    if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 3 + 4 * half)) { my_bad = true; break; }
                }
                my_bad = __any_sync(FULL, my_bad);
                STAMP(4 + 6 * half);
                l[0] = __uint_as_float(v0.x); l[1] = __uint_as_float(v0.z);
                const int nib = group16_softmax_draw(l[0], l[1], u01, lane);
                drawn = (__shfl_sync(FULL, nib, 0) << 12) | (__shfl_sync(FULL, nib, 8) << 8) | (__shfl_sync(FULL, nib, 16) << 4) | __shfl_sync(FULL, nib, 24);
            } else {
                {
                    // the four slots of this lane are loaded together and re-read until all of them carry this half-step's tag
                    const unsigned a = smem_addr(lbuf + (size_t)par * 128 + 4 * lane);
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
                drawn = warp_softmax_draw_fast(reinterpret_cast<const float (&)[8]>(l), u01, lane);
            }
            // The chip waits for the slowest CTA's state: publish first, the writer's bookkeeping (which only CTA 0 has)
            // comes after it and overlaps the next exchange.
            const int fed = forced >= 0 ? forced : drawn;
            if (lane < UC && !last && !my_bad) gates_and_publish(half, s, fed, gp);
            if (writer) {
                constexpr int NL = FUSED ? 2 : 8, NLOG2 = FUSED ? 64 : 256;
                if (p.dbg_logits) {
                    float *d = p.dbg_logits + (size_t)(n - 1) * NLOG2 + NL * lane;
#pragma unroll
                    for (int k = 0; k < NL; ++k) d[k] = l[k];
                }
                if (lane == 0) {
                    if (FUSED) {
                        if (half) { if (p.a_out) p.a_out[s] = (uint16_t)drawn; }
                        else      { if (p.b_out) p.b_out[s - 1] = (uint16_t)drawn; }
                        // the two streams side by side: out[0][s] = a_s, out[1][s] = the sample part B emits in step s
                        if (p.out) p.out[(half ? 0 : T) + (half ? s : s - 1)] = (int16_t)(fed - 32768);
                    } else {
                        if (half) { if (p.c_out) p.c_out[s] = (uint8_t)drawn; }
                        else      { if (p.f_out) p.f_out[s - 1] = (uint8_t)drawn; }
                        if (!half && p.out) p.out[s - 1] = (int16_t)(256 * c_prev + fed - 32768);
                    }
                }
            }
            if (half) c_prev = fed; else f_prev = fed;
        }
        STAMP(5 + 6 * half);
    }
    if (prof_on && lane == 0) for (int i = 0; i < 16; ++i) p.prof[i] = s_prof[i];

    // final state (vecC holds y_c(T-1); vecF was refreshed by the last fine half)
    const int any_bad = __syncthreads_or(my_bad);
    if (writer && !any_bad) {
        if (p.h_out) for (int i = tid; i < K; i += blockDim.x) { p.h_out[i] = vecC[i]; p.h_out[K + i] = vecF[i]; }
        if (tid == 0) {
            if (FUSED) {
                if (p.a_st_out) p.a_st_out[0] = (uint16_t)c_prev;
                if (p.b_st_out) p.b_st_out[0] = (uint16_t)f_prev;
            } else {
                if (p.c_st_out) p.c_st_out[0] = (uint8_t)c_prev;
                if (p.f_st_out) p.f_st_out[0] = (uint8_t)f_prev;
            }
        }
    }
    cluster.sync();     // nobody leaves while a peer may still write into its shared memory
}


// ---------------------------------------------------------------------------------------------
// Two streams at once on the same resident weights (Section 5.1 reports a batch of four streams on the paper's kernel).
// The MMAs of the single-stream kernel use three of their eight B columns (the hi / mid / lo parts of one input
// vector); here the parts of a second stream take three more, so both streams advance for the tensor-pipe time of
// one.  Everything per stream is doubled: state vectors, split images (eight columns per piece), exchange slots, the
// drawing warp (warp s draws and gates stream s).  Same schedule, same waits, same weights layout as above.
//
// Columns of a B fragment: 0, 1 = hi, mid of stream 0; 2, 3 = hi, mid of stream 1; 4 = lo of stream 0; 6 = lo of stream 1
// (5, 7 zero): lane (g, t) of a D fragment holds columns 2 t, 2 t + 1, so one shuffle (xor 2) leaves the sums of stream
// t & 1 in the lanes with t < 2.
__host__ __device__ __forceinline__ int split2s_pos(int i, int col)
{
    const int c = i & 15, kt = i >> 4;
    const int t = (c & 7) >> 1, j = c & 1, hi = c >> 3;
    return ((((((kt >> 1) * 8 + col) * 4 + t) << 1) + (kt & 1)) << 2) + 2 * hi + j;
}
__device__ __forceinline__ void store_split2s(__nv_bfloat16 *split, int stream, int i, float x)
{
    const __nv_bfloat16 b0 = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(b0);
    const __nv_bfloat16 b1 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(b1);
    const __nv_bfloat16 b2 = __float2bfloat16_rn(r2);
    split[split2s_pos(i, 2 * stream)] = b0;
    split[split2s_pos(i, 2 * stream + 1)] = b1;
    split[split2s_pos(i, 4 + 2 * stream)] = b2;
}
// two adjacent elements (i even) of one stream: one 32-bit store per part
__device__ __forceinline__ void store_split2s_pair(__nv_bfloat16 *split, int stream, int i, float x0, float x1)
{
    unsigned w[3];
    float r0 = x0, r1 = x1;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const __nv_bfloat16 a = __float2bfloat16_rn(r0), b = __float2bfloat16_rn(r1);
        w[k] = (unsigned)__bfloat16_as_ushort(a) | ((unsigned)__bfloat16_as_ushort(b) << 16);
        r0 -= __bfloat162float(a); r1 -= __bfloat162float(b);
    }
    unsigned *s32 = reinterpret_cast<unsigned *>(split);
    s32[split2s_pos(i, 2 * stream) >> 1] = w[0];
    s32[split2s_pos(i, 2 * stream + 1) >> 1] = w[1];
    s32[split2s_pos(i, 4 + 2 * stream) >> 1] = w[2];
}
// NK consecutive k-tiles (even count, from the even k-tile kt0) of NT 16-row tiles times the two-stream split vector.
// On return lane (g, t), t < 2, holds the partial totals of rows g (lo[n]) and g + 8 (hi[n]) of tile n for stream t.
template <int NK, int NT>
__device__ __forceinline__ void mma_tiles_pair(const uint4 *A, size_t tile_u4, int kt0, const __nv_bfloat16 *split, int lane, float (&lo)[NT], float (&hi)[NT])
{
    const int g = lane >> 2, t = lane & 3;
    const uint4 *bsrc = reinterpret_cast<const uint4 *>(split) + ((kt0 >> 1) * 8 + g) * 4 + t;
    uint4 av[NT][NK];
    uint4 bv[NK / 2];
#pragma unroll
    for (int i = 0; i < NK / 2; ++i) bv[i] = bsrc[32 * i];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int i = 0; i < NK; ++i) av[n][i] = A[n * tile_u4 + (size_t)(kt0 + i) * 32 + lane];
    float acc[NT][2][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[n][c][i] = 0.f;
#pragma unroll
    for (int i = 0; i < NK; ++i)
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            float *c = acc[n][i & 1];
            const unsigned b0 = (i & 1) ? bv[i >> 1].z : bv[i >> 1].x, b1 = (i & 1) ? bv[i >> 1].w : bv[i >> 1].y;
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                         : "r"(av[n][i].x), "r"(av[n][i].y), "r"(av[n][i].z), "r"(av[n][i].w), "r"(b0), "r"(b1));
        }
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        const float c0 = acc[n][0][0] + acc[n][1][0], c1 = acc[n][0][1] + acc[n][1][1];
        const float c2 = acc[n][0][2] + acc[n][1][2], c3 = acc[n][0][3] + acc[n][1][3];
        float s_lo = t < 2 ? c0 + c1 : c0, s_hi = t < 2 ? c2 + c3 : c2;     // t >= 2: the lo part sits in the even column only
        s_lo += __shfl_xor_sync(FULL, s_lo, 2);
        s_hi += __shfl_xor_sync(FULL, s_hi, 2);
        lo[n] = s_lo; hi[n] = s_hi;
    }
}

struct PairParams {
    ResidentParams r;                        // fields of the single-stream kernel; pointers address row 0 of the pair
    int n_batch;                             // rows of the whole call (row pitch of the diagnostic dumps)
    const float *g1;                         // gate offsets of the second row (r.g: of the first)
    unsigned long long *slots2;              // [2 halves][2 parities][2 streams][K]
    long long row_pitch;                     // samples between the two rows of out / c_out / f_out / forced arrays
};

__global__ void __launch_bounds__(512, 1) resident_pair_kernel(const PairParams pp)
{
    constexpr int KSH = 7, NKH = 4, KSL = 7, NKL = 4;
    const ResidentParams &p = pp.r;
    extern __shared__ __align__(16) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int cta = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = p.K, NKT = p.NKT, NMT = p.NMT, NLT = p.NLT, UC = p.UC, HR = p.HR, LR = p.LR, CS = p.CS, H = p.H;
    const int NR = p.n_rrows;

    // ---- shared memory carve-up (must match resident_pair_smem_bytes)
    const size_t tile_u4 = (size_t)NKT * 32;
    const uint4 *wMA = reinterpret_cast<const uint4 *>(smem);
    const uint4 *wMB = wMA + (size_t)NMT * tile_u4;
    const uint4 *wO2 = wMB + (size_t)NMT * tile_u4;
    const uint4 *wO4 = wO2 + (size_t)NLT * tile_u4;
    const float *sI = reinterpret_cast<const float *>(smem + p.w_bytes);       // [NR][3]
    const float *sb1 = sI + NR * 3, *sb3 = sb1 + HR, *sb2 = sb3 + HR, *sb4 = sb2 + LR;
    float *vecC = reinterpret_cast<float *>(smem + p.blob_bytes);              // [2][K]
    float *vecF = vecC + 2 * K;                                                // [2][K]
    float *a_part = vecF + 2 * K;                                              // [2][NR]
    float *a_full = a_part + 2 * NR;                                           // [2][NR]
    float *part = a_full + 2 * NR;                                             // [2 streams][32 slots][16]
    __nv_bfloat16 *splC = reinterpret_cast<__nv_bfloat16 *>(part + 1024);      // two-stream split images, 8 K bf16 each
    __nv_bfloat16 *splF = splC + 8 * K;
    __nv_bfloat16 *splQ = splF + 8 * K;
    float *qbuf = reinterpret_cast<float *>(splQ + 8 * K);                    // [2 parities][2 streams][K]
    uint4 *lbuf = reinterpret_cast<uint4 *>(qbuf + 4 * K);                     // [2 parities][2 streams][128]
    __shared__ __align__(8) unsigned long long xbar[2];

    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.blob + (size_t)cta * p.blob_bytes);
        uint4 *dst = reinterpret_cast<uint4 *>(smem);
        for (size_t i = tid; i < p.blob_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
        for (int i = tid; i < 4 * K + 2048; i += blockDim.x) qbuf[i] = 0.f;             // qbuf and lbuf are adjacent
        if (tid == 0) {
            for (int i = 0; i < 2; ++i) mbar_init_cluster(smem_addr(&xbar[i]), 1);
            mbar_fence_init();
        }
        for (int i = tid; i < 24 * K / 8; i += blockDim.x) reinterpret_cast<uint4 *>(splC)[i] = make_uint4(0, 0, 0, 0);
        __syncthreads();
        for (int i = tid; i < 2 * K; i += blockDim.x) {
            const int st = i / K, j = i - st * K;
            const float c = p.h_in ? p.h_in[(size_t)st * H + j] : 0.f, f = p.h_in ? p.h_in[(size_t)st * H + K + j] : 0.f;
            vecC[i] = c; vecF[i] = f;
            store_split2s(splC, st, j, c);
            store_split2s(splF, st, j, f);
        }
    }
    __syncthreads();
    cluster.sync();

    Waiter wt{p.status, p.limit_ns};
    bool my_bad = false;
    const bool writer = (cta == 0);
    const int g4 = lane >> 2, t4 = lane & 3;
    // optional phase timing (CTA 0, warp 0), the slots of the single-stream kernel
    const bool prof_on = p.prof != nullptr && cta == 0 && warp == 0;
    __shared__ long long s_prof[16];
    if (tid < 16) s_prof[tid] = 0;
    __syncthreads();
    long long prof_t = clock64();
#define STAMP(i) do { if (prof_on) { const long long now_ = clock64(); if (lane == 0) s_prof[i] += now_ - prof_t; prof_t = now_; } } while (0)
    const int ws = warp & 1;                           // the stream a drawing warp (0, 1) serves

    // warps 0 and 1 keep the scalar state of streams 0 and 1
    int c_prev = 128, f_prev = 0;
    float hC = 0.f, hF = 0.f;
    if (warp < 2) {
        c_prev = p.c_in ? p.c_in[ws] : 128; f_prev = p.f_in ? p.f_in[ws] : 0;
        if (lane < UC) { hC = vecC[ws * K + cta * UC + lane]; hF = vecF[ws * K + cta * UC + lane]; }
    }

    const int h_pair = warp / KSH, h_ks = warp % KSH, h_kt0 = h_ks * NKH;
    const int l_tile = warp / KSL, l_ks = warp % KSL, l_kt0 = l_ks * NKL;
    const bool h_on = warp < (NMT / 2) * KSH, l_on = warp < NLT * KSL;
    // partial sums: part[stream][tile * K-splits + split][16]
    auto hidden_products = [&](const uint4 *Mx, const __nv_bfloat16 *sp) {
        float lo[2], hi[2];
        mma_tiles_pair<NKH, 2>(Mx + (size_t)(2 * h_pair) * tile_u4, tile_u4, h_kt0, sp, lane, lo, hi);
        if (t4 < 2) {
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                float *d = part + t4 * 512 + ((2 * h_pair + n) * KSH + h_ks) * 16;
                d[g4] = lo[n]; d[g4 + 8] = hi[n];
            }
        }
    };
    // one peer per warp; lanes [0, 16) serve stream 0, lanes [16, 32) stream 1
    const int ls = lane >> 4, ll = lane & 15;
    unsigned q_snd[2], l_snd[2], q_bar[2];
#pragma unroll
    for (int par2 = 0; par2 < 2; ++par2) {
        const unsigned peer = warp < CS ? warp : 0;
        q_snd[par2] = map_to_rank(smem_addr(qbuf + (size_t)(par2 * 2 + ls) * K + rank * HR + 2 * (ll < HR / 2 ? ll : 0)), peer);
        l_snd[par2] = map_to_rank(smem_addr(lbuf + (size_t)(par2 * 2 + ls) * 128 + (rank * LR) / 2 + (ll < LR / 2 ? ll : 0)), peer);
        q_bar[par2] = map_to_rank(smem_addr(&xbar[par2]), peer);
    }
    auto wait_arrival = [&](int which, unsigned use, int step, int phase) {
        const unsigned bar = smem_addr(&xbar[which]);
        unsigned long long t0 = 0; unsigned cnt = 0;
        while (!mbar_try_parity(bar, use & 1u))
            if ((++cnt & 1023u) == 0 && wt.expired(t0, step, phase)) return false;
        return true;
    };
    // R rows of tile `tile` for stream `st`: sums of the K-split partials stay in this CTA
    auto keep_r_rows = [&](int tile, int st, bool completes) {
        const int row = 16 * tile + ll;
        if (row >= HR && row - HR < NR) {
            float v = 0.f;
#pragma unroll
            for (int sp = 0; sp < KSH; ++sp) v += part[st * 512 + (tile * KSH + sp) * 16 + ll];
            if (completes) a_full[st * NR + row - HR] = a_part[st * NR + row - HR] + v;
            else a_part[st * NR + row - HR] = v;
        }
    };

    // ---- prologue: the recurrent products of step 0 from the initial state, coarse gates of step 0
    if (h_on) hidden_products(wMA, splC);
    __syncthreads();
    if (warp < NMT) keep_r_rows(warp, ls, false);
    __syncthreads();
    if (h_on) hidden_products(wMB, splF);
    __syncthreads();
    if (warp < NMT) keep_r_rows(warp, ls, true);
    __syncthreads();

    struct GatePre { float pu, pr, pe, ae, ku, kr, ke; };
    auto gates_prepare = [&](int half_g, const float (&gv)[3]) {
        GatePre q;
        const int rb = half_g ? 3 * UC : 0;
        const float x0 = scale8(c_prev), x1 = scale8(f_prev);
        const float *Iu = sI + 3 * (rb + lane), *Ir = sI + 3 * (rb + UC + lane), *Ie = sI + 3 * (rb + 2 * UC + lane);
        const float *af = a_full + ws * NR;
        q.pu = af[rb + lane] + fmaf(Iu[0], x0, half_g ? fmaf(Iu[1], x1, gv[0]) : gv[0]);
        q.pr = af[rb + UC + lane] + fmaf(Ir[0], x0, half_g ? fmaf(Ir[1], x1, gv[1]) : gv[1]);
        q.pe = fmaf(Ie[0], x0, half_g ? fmaf(Ie[1], x1, gv[2]) : gv[2]);
        q.ae = af[rb + 2 * UC + lane];
        q.ku = half_g ? Iu[2] : Iu[1]; q.kr = half_g ? Ir[2] : Ir[1]; q.ke = half_g ? Ie[2] : Ie[1];
        return q;
    };
    const int skip_at = cta == p.skip_cta ? (int)p.skip_step : -1;      // self-test: the step at which this CTA withholds its publication
    auto gates_and_publish = [&](int half_g, long long s, int drawn, const GatePre &q) {
        const float xk = scale8(drawn);
        const float u = sigmoidf_fast(fmaf(q.ku, xk, q.pu)), r = sigmoidf_fast(fmaf(q.kr, xk, q.pr));
        const float e = tanhf_fast(fmaf(r, q.ae, fmaf(q.ke, xk, q.pe)));
        const float hn = fmaf(u, half_g ? hF : hC, (1.0f - u) * e);
        if (half_g) hF = hn; else hC = hn;
        const int j = cta * UC + lane, jj = (half_g ? K : 0) + j;
        if ((int)s != skip_at)
            st_relaxed_u64(pp.slots2 + ((size_t)((half_g ? 2 : 0) + (s & 1)) * 2 + ws) * K + j,
                           ((unsigned long long)(unsigned)(s + 1) << 32) | __float_as_uint(hn));
        if (p.dbg_gates) { float *d = p.dbg_gates + ((size_t)s * pp.n_batch + ws) * 3 * H; d[jj] = u; d[H + jj] = r; d[2 * H + jj] = e; }
        if (p.dbg_h) p.dbg_h[((size_t)s * pp.n_batch + ws) * H + jj] = hn;
    };
    auto load_g = [&](int half_g, long long s, float (&gv)[3]) {
        const long long fr = ((p.step0 + s) * p.row_stride + (long long)(p.stream0 + (unsigned)ws) * p.row_offset_mul) / p.hop - p.frame_shift;
        const float *g = (ws ? pp.g1 : p.g) + (size_t)fr * 3 * H + (half_g ? K : 0) + cta * UC + lane;
#pragma unroll
        for (int gate = 0; gate < 3; ++gate) gv[gate] = __ldg(g + gate * H);
    };
    if (warp < 2 && lane < UC) {
        float gv[3];
        load_g(0, 0, gv);
        gates_and_publish(0, 0, f_prev, gates_prepare(0, gv));
    }

    const long long T = p.n_steps;
#pragma unroll 1
    for (long long n = 1; n <= 2 * T; ++n) {
        const int half = (int)(n & 1);
        const long long s = n >> 1;
        const bool last = n == 2 * T;
        const unsigned tag = (unsigned)n, par = (unsigned)((n - 1) & 1);
        const uint4 *M = half ? wMA : wMB, *L = half ? wO2 : wO4;
        const float *bh = half ? sb1 : sb3, *bl = half ? sb2 : sb4;
        float *vec = half ? vecC : vecF;
        __nv_bfloat16 *spl = half ? splC : splF;

        const unsigned use = (unsigned)((n - 1) >> 1);
        if (tid == 0) mbar_arrive_expect(smem_addr(&xbar[par]), (unsigned)K * 8u);      // this half's hidden layers: 2 x K values
        float gv[3] = {0.f, 0.f, 0.f}, u01 = 0.f;
        int forced = -1;
        if (warp < 2) {
            if (lane < UC && !last) load_g(half, s, gv);
            const long long o = (long long)ws * pp.row_pitch + (half ? s : s - 1);
            if (half) { if (p.c_forced) forced = p.c_forced[o]; }
            else      { if (p.f_forced) forced = p.f_forced[o]; }
            u01 = uniform24(p.seed, p.stream0 + (unsigned)ws, (unsigned long long)(p.step0 + (half ? s : s - 1)), half ? 0u : 1u);
        }

        // ---- 1. the input half-vectors of both streams from the whole chip
        {
            const unsigned long long *slots = pp.slots2 + (size_t)(half ? (s & 1) : 2 + ((s - 1) & 1)) * 2 * K;
            const unsigned ytag = (unsigned)(half ? s + 1 : s);
#pragma unroll 1
            for (int i = tid; i < K; i += blockDim.x) {              // K slot pairs: [stream][K / 2]
                unsigned long long v0, v1, t0 = 0; unsigned cnt = 0;
                while (true) {
                    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v0), "=l"(v1) : "l"(slots + 2 * i) : "memory");
                    if ((unsigned)(v0 >> 32) == ytag && (unsigned)(v1 >> 32) == ytag) break;
                    if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
                }
                const int st = (2 * i) / K, j = 2 * i - st * K;
                const float x0 = __uint_as_float((unsigned)v0), x1 = __uint_as_float((unsigned)v1);
                vec[2 * i] = x0; vec[2 * i + 1] = x1;
                store_split2s_pair(spl, st, j, x0, x1);
            }
            if (__syncthreads_or(my_bad)) break;
        }
        STAMP(0 + 6 * half);

        // ---- 2. hidden layers of the head + this CTA's R rows, both streams in the same MMAs
        if (h_on) hidden_products(M, spl);
        __syncthreads();
        STAMP(12 + half);
        if (warp < CS && ll < HR / 2) {
            const int r0 = 2 * ll, tile = r0 >> 4, rr = r0 & 15;
            const float *pt = part + ls * 512;
            float v0 = bh[r0], v1 = bh[r0 + 1];
#pragma unroll
            for (int sp = 0; sp < KSH; ++sp) { v0 += pt[(tile * KSH + sp) * 16 + rr]; v1 += pt[(tile * KSH + sp) * 16 + rr + 1]; }
            st_async_v2(q_snd[par], fmaxf(v0, 0.f), fmaxf(v1, 0.f), q_bar[par]);
        }
        if (warp < NMT) keep_r_rows(warp, ls, !half);
        STAMP(1 + 6 * half);

        // ---- 3. the cluster's hidden layers -> logits rows of this CTA
        if (tid < K) {
            if (!wait_arrival(par, use, (int)s, 2 + 4 * half)) my_bad = true;
            const int st = (2 * tid) / K, j = 2 * tid - st * K;
            const float2 v = reinterpret_cast<const float2 *>(qbuf + (size_t)par * 2 * K)[tid];
            store_split2s_pair(splQ, st, j, v.x, v.y);
        }
        if (__syncthreads_or(my_bad)) break;
        STAMP(2 + 6 * half);
        if (l_on) {
            float lo[1], hi[1];
            mma_tiles_pair<NKL, 1>(L + (size_t)l_tile * tile_u4, tile_u4, l_kt0, splQ, lane, lo, hi);
            if (t4 < 2) { float *d = part + t4 * 512 + warp * 16; d[g4] = lo[0]; d[g4 + 8] = hi[0]; }
        }
        __syncthreads();
        STAMP(14 + half);
        if (warp < CS && ll < LR / 2) {
            const int r0 = 2 * ll, tile = r0 >> 4, rr = r0 & 15;
            const float *pt = part + ls * 512;
            float v0 = bl[r0], v1 = bl[r0 + 1];
#pragma unroll
            for (int sp = 0; sp < KSL; ++sp) { v0 += pt[(tile * KSL + sp) * 16 + rr]; v1 += pt[(tile * KSL + sp) * 16 + rr + 1]; }
            st_cluster_ll(l_snd[par], v0, v1, tag);
        }
        STAMP(3 + 6 * half);

        // ---- 4. warps 0, 1: the 256 logits of their stream -> draw; then the gates of the other half of its state
        if (warp < 2) {
            GatePre gp = {};
            if (lane < UC && !last) gp = gates_prepare(half, gv);
            float l[8];
            {
                const unsigned a = smem_addr(lbuf + (size_t)(par * 2 + ws) * 128 + 4 * lane);
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
            const int fed = forced >= 0 ? forced : drawn;
            if (lane < UC && !last && !my_bad) gates_and_publish(half, s, fed, gp);
            if (writer) {
                if (p.dbg_logits) {
                    float *d = p.dbg_logits + (((size_t)(half ? s : s - 1) * pp.n_batch + ws) * 2 + (half ? 0 : 1)) * 256 + 8 * lane;
#pragma unroll
                    for (int k = 0; k < 8; ++k) d[k] = l[k];
                }
                if (lane == 0) {
                    const long long o = (long long)ws * pp.row_pitch + (half ? s : s - 1);
                    if (half) { if (p.c_out) p.c_out[o] = (uint8_t)drawn; }
                    else      { if (p.f_out) p.f_out[o] = (uint8_t)drawn; }
                    if (!half && p.out) p.out[o] = (int16_t)(256 * c_prev + fed - 32768);
                }
            }
            if (half) c_prev = fed; else f_prev = fed;
        }
        STAMP(5 + 6 * half);
    }
    if (prof_on && lane == 0) for (int i = 0; i < 16; ++i) p.prof[i] = s_prof[i];
#undef STAMP

    const int any_bad = __syncthreads_or(my_bad);
    if (writer && !any_bad) {
        if (p.h_out)
            for (int i = tid; i < 2 * K; i += blockDim.x) {
                const int st = i / K, j = i - st * K;
                p.h_out[(size_t)st * H + j] = vecC[i]; p.h_out[(size_t)st * H + K + j] = vecF[i];
            }
        if (warp < 2 && lane == 0) {
            if (p.c_st_out) p.c_st_out[ws] = (uint8_t)c_prev;
            if (p.f_st_out) p.f_st_out[ws] = (uint8_t)f_prev;
        }
    }
    cluster.sync();
}

// ---------------------------------------------------------------------------------------------
static int resident_smem_bytes(const ResidentPack &k)
{
    size_t b = k.blob_bytes;
    b += (size_t)2 * k.K * 4;                       // vecC, vecF
    size_t a = (size_t)2 * k.n_rrows;               // a_part, a_full
    a += (a % 4) ? 4 - (a % 4) : 0;
    b += a * 4;
    b += 512 * 4;                                   // partial sums [tiles x K-splits][16]
    b += (size_t)12 * k.K * 2;                      // three split images of 4 K bf16
    b += (size_t)2 * k.K * 4;                       // qbuf [2][K]
    b += 256 * 16;                                  // lbuf [2][128] x 16 B
    return (int)b;
}

static int resident_pair_smem_bytes(const ResidentPack &k)
{
    size_t b = k.blob_bytes;
    b += (size_t)4 * k.K * 4;                       // vecC, vecF of two streams
    b += (size_t)4 * k.n_rrows * 4;                 // a_part, a_full of two streams
    b += 1024 * 4;                                  // partial sums [2 streams][32][16]
    b += (size_t)24 * k.K * 2;                      // three two-stream split images of 8 K bf16
    b += (size_t)4 * k.K * 4;                       // qbuf [2][2][K]
    b += 512 * 16;                                  // lbuf [2][2][128] x 16 B
    return (int)b;
}

static uint16_t bf16_bits_of(float rounded)
{
    uint32_t b;
    std::memcpy(&b, &rounded, 4);
    return (uint16_t)(b >> 16);
}

// dense row `row` of a host block-row matrix -> bf16 bits for columns [c0, c0 + n)
void dense_row_bf16(const BsrHost &M, int row, int c0, int n, uint16_t *dst)
{
    std::fill(dst, dst + n, (uint16_t)0);
    const int br = row / 4, r = row % 4;
    for (int i = M.row_ptr[br]; i < M.row_ptr[br + 1]; ++i) {
        const int cbase = 4 * (int)M.col[i];
        for (int c = 0; c < 4; ++c) {
            const int col = cbase + c;
            if (col >= c0 && col < c0 + n) dst[col - c0] = bf16_bits_of(M.vals[(size_t)i * 16 + 4 * r + c]);
        }
    }
}

// rows[16][K] (bf16 bits, natural column order) -> A fragments [K/16][32 lanes][8] of m16n8k16:
// lane (g, t) holds (row g, k 2t..2t+1), (row g+8, same), (row g, k 2t+8..9), (row g+8, same).
// The vector side stores element 16 kt + c at split2_pos and the B-fragment load reads it back from
// there, so fragment column c of k-tile kt is plain column 16 kt + c of the matrix.
void pack_tile(const std::vector<std::vector<uint16_t>> &rows, int K, uint16_t *dst)
{
    for (int kt = 0; kt < K / 16; ++kt)
        for (int lane = 0; lane < 32; ++lane) {
            const int g = lane >> 2, t = lane & 3;
            uint16_t *o = dst + ((size_t)kt * 32 + lane) * 8;
            const int rsel[4] = {g, g + 8, g, g + 8};
            const int csel[4] = {2 * t, 2 * t, 2 * t + 8, 2 * t + 8};
            for (int q = 0; q < 4; ++q)
                for (int j = 0; j < 2; ++j) o[2 * q + j] = rows[rsel[q]][16 * kt + csel[q] + j];
        }
}

static bool choose_shape(const wrnn_model *m, int CS, ResidentPack *k, std::string *why)
{
    const int H = m->H, Hh = H / 2;
    if (m->dtype != WRNN_BF16) { if (why) *why = "resident kernel stores bf16 weights only"; return false; }
    if (m->sparse) { if (why) *why = "resident dense kernel does not take block masks"; return false; }
    if (H % 32 != 0) { if (why) *why = "H must be a multiple of 32"; return false; }
    if (CS != 8 && CS != 16) { if (why) *why = "cluster size must be 8 or 16"; return false; }
    const bool fused = m->variant == 1;
    const int n_logits = fused ? 64 : 256, n_in = fused ? 12 : 3;
    if (Hh % (2 * CS) != 0 || n_logits % (2 * CS) != 0) { if (why) *why = "H/2 must be a multiple of twice the cluster size"; return false; }
    const int HR = Hh / CS, LR = n_logits / CS;
    int best = 0;
    for (int ncta = CS; ncta <= m->n_sms; ncta += CS) {
        if (Hh % ncta) continue;
        const int uc = Hh / ncta;
        if (uc > 32) continue;
        if ((HR + 6 * uc + 15) / 16 > 16) continue;        // stacked [head rows ; R rows], padded with zero rows to 16-row tiles
        best = ncta;
    }
    if (!best) { if (why) *why = "no CTA count tiles H/2 into 16-row fragments"; return false; }
    k->CS = CS; k->NCTA = best; k->NC = best / CS; k->UC = Hh / best; k->HR = HR; k->LR = LR;
    k->K = Hh; k->NKT = Hh / 16; k->n_rrows = 6 * k->UC;
    k->NMT = (HR + k->n_rrows + 15) / 16; k->NLT = (LR + 15) / 16;
    k->fused = fused;
    k->NMT += k->NMT & 1;                                   // tiles are multiplied in pairs
    k->NW = 16; k->KSH = 7; k->KSL = 7;
    if (k->NKT != 28 || (k->NMT / 2) * k->KSH > k->NW || k->NLT * k->KSL > k->NW || CS > k->NW || k->NMT * k->KSH > 32) {
        if (why) *why = "only the H/2 = 448 tiling (7 K-splits of 4 k-tiles) is instantiated";
        return false;
    }
    k->w_bytes = ((size_t)2 * k->NMT + 2 * k->NLT) * 16 * k->K * 2;
    size_t small = ((size_t)k->n_rrows * n_in + 2 * k->HR + 2 * k->LR) * 4;
    small = (small + 15) / 16 * 16;
    k->blob_bytes = k->w_bytes + small;
    k->smem_bytes = resident_smem_bytes(*k);
    return true;
}

// The one instantiated split: K = 448 as 7 x 4 k-tiles, for pairs of hidden tiles and for single logits tiles.
static void *resident_fn(bool fused)
{
    return fused ? (void *)resident_dense_kernel<7, 4, 7, 4, true> : (void *)resident_dense_kernel<7, 4, 7, 4, false>;
}

int resident_supported(const wrnn_model *m, int batch, std::string *why)
{
    if (batch != 1) { if (why) *why = "resident kernel is single-stream (batch 1)"; return WRNN_ERR_UNSUPPORTED; }
    if (!m->resident) { if (why) *why = "model was not packed for the resident kernel"; return WRNN_ERR_UNSUPPORTED; }
    return WRNN_OK;
}

static void fill_launch(const ResidentPack &k, cudaLaunchConfig_t *cfg, cudaLaunchAttribute *at, cudaStream_t s, bool coop)
{
    std::memset(cfg, 0, sizeof(*cfg));
    cfg->gridDim = dim3(k.NCTA);
    cfg->blockDim = dim3(k.NW * 32);
    cfg->dynamicSmemBytes = k.smem_bytes;
    cfg->stream = s;
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = k.CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative;
    at[1].val.cooperative = 1;
    cfg->attrs = at;
    cfg->numAttrs = coop ? 2 : 1;
}

int resident_prepare(wrnn_model *m)
{
    // A cluster of 16 holds half as many head rows per CTA as a cluster of 8 (fewer weight fragments to stream per
    // step); it needs the non-portable cluster size and enough co-resident clusters, else 8 is used.
    // WRNN_RESIDENT_CS=8 / 16 forces one of them (diagnostic).
    ResidentPack k;
    std::string why;
    cudaDeviceProp prop;
    cudaGetDeviceProperties(&prop, m->device);
    cudaFuncSetAttribute(resident_fn(m->variant == 1), cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    cudaGetLastError();
    const char *force = getenv("WRNN_RESIDENT_CS");
    bool found = false;
    for (int cs : {16, 8}) {
        if (force && atoi(force) != cs) continue;
        ResidentPack c;
        if (!choose_shape(m, cs, &c, &why)) continue;
        if ((size_t)c.smem_bytes > prop.sharedMemPerBlockOptin) { why = "weights do not fit in shared memory"; continue; }
        if (cudaFuncSetAttribute(resident_fn(m->variant == 1), cudaFuncAttributeMaxDynamicSharedMemorySize, c.smem_bytes) != cudaSuccess) {
            cudaGetLastError(); why = "cannot raise the dynamic shared memory limit"; continue;
        }
        cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
        fill_launch(c, &cfg, at, 0, false);
        int max_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&max_clusters, resident_fn(m->variant == 1), &cfg) != cudaSuccess || max_clusters < c.NC) {
            cudaGetLastError(); why = "not enough co-resident clusters on this device"; continue;
        }
        k = c; found = true;
        break;
    }
    if (!found) { m->err = why; return WRNN_ERR_UNSUPPORTED; }
    // the two-stream kernel shares the weights; it needs more shared memory for the doubled vectors and exchange buffers
    if (!k.fused && (4 * k.n_rrows) % 4 == 0) {
        const int ps = resident_pair_smem_bytes(k);
        if ((size_t)ps <= prop.sharedMemPerBlockOptin &&
            cudaFuncSetAttribute(resident_pair_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
            cudaFuncSetAttribute(resident_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ps) == cudaSuccess) {
            cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
            fill_launch(k, &cfg, at, 0, false);
            cfg.dynamicSmemBytes = ps;
            int max_clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&max_clusters, resident_pair_kernel, &cfg) == cudaSuccess && max_clusters >= k.NC) k.pair_smem = ps;
        }
        cudaGetLastError();
    }

    // ---- per-CTA blobs
    const int H = m->H, K = k.K, UC = k.UC, n_in = k.fused ? 12 : 3;
    std::vector<uint8_t> blob((size_t)k.NCTA * k.blob_bytes, 0);
    std::vector<std::vector<uint16_t>> rows(16, std::vector<uint16_t>(K));
    const BsrHost *Oa[2] = {&m->hO1, &m->hO3}, *Ob[2] = {&m->hO2, &m->hO4};
    for (int cta = 0; cta < k.NCTA; ++cta) {
        const int rank = cta % k.CS;
        uint8_t *base = blob.data() + (size_t)cta * k.blob_bytes;
        uint16_t *w = reinterpret_cast<uint16_t *>(base);
        float *sm = reinterpret_cast<float *>(base + k.w_bytes);
        const size_t tile_elems = (size_t)16 * K;
        // stacked matrices MA (part 0: y_c input) and MB (part 1: y_f input): HR head rows then NR rows of R.
        // R row rr = (half * 3 + gate) * UC + u  ->  matrix row gate * H + half * K + cta * UC + u
        for (int part = 0; part < 2; ++part)
            for (int mt = 0; mt < k.NMT; ++mt) {
                for (int r = 0; r < 16; ++r) {
                    const int row = 16 * mt + r;
                    if (row < k.HR) dense_row_bf16(*Oa[part], rank * k.HR + row, 0, K, rows[r].data());
                    else if (row - k.HR < k.n_rrows) {
                        const int rr = row - k.HR;
                        const int half = rr / (3 * UC), gate = (rr / UC) % 3, u = rr % UC;
                        dense_row_bf16(m->hR, gate * H + half * K + cta * UC + u, part * K, K, rows[r].data());
                    }
                    else std::fill(rows[r].begin(), rows[r].end(), (uint16_t)0);       // padding row of the last tile
                }
                pack_tile(rows, K, w + ((size_t)part * k.NMT + mt) * tile_elems);
            }
        uint16_t *wl = w + (size_t)2 * k.NMT * tile_elems;
        for (int h = 0; h < 2; ++h)
            for (int mt = 0; mt < k.NLT; ++mt) {
                for (int r = 0; r < 16; ++r) {
                    if (16 * mt + r < k.LR) dense_row_bf16(*Ob[h], rank * k.LR + 16 * mt + r, 0, K, rows[r].data());
                    else std::fill(rows[r].begin(), rows[r].end(), (uint16_t)0);
                }
                pack_tile(rows, K, wl + ((size_t)h * k.NLT + mt) * tile_elems);
            }
        for (int rr = 0; rr < k.n_rrows; ++rr) {
            const int half = rr / (3 * UC), gate = (rr / UC) % 3, u = rr % UC;
            const int mrow = gate * H + half * K + cta * UC + u;
            for (int c = 0; c < n_in; ++c) sm[rr * n_in + c] = m->hI[(size_t)mrow * n_in + c];
        }
        float *b = sm + k.n_rrows * n_in;
        for (int r = 0; r < k.HR; ++r) { b[r] = m->hb1[rank * k.HR + r]; b[k.HR + r] = m->hb3[rank * k.HR + r]; }
        b += 2 * k.HR;
        for (int r = 0; r < k.LR; ++r) { b[r] = m->hb2[rank * k.LR + r]; b[k.LR + r] = m->hb4[rank * k.LR + r]; }
    }
    ResidentPack *pk = new ResidentPack(k);
    bool ok = cudaMalloc((void **)&pk->d_blob, blob.size()) == cudaSuccess &&
              cudaMemcpy(pk->d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice) == cudaSuccess &&
              cudaMalloc((void **)&pk->d_slots, (size_t)4 * K * 8) == cudaSuccess &&
              cudaMalloc((void **)&pk->d_slots2, (size_t)8 * K * 8) == cudaSuccess &&
              cudaMalloc((void **)&pk->d_prof, 16 * sizeof(long long)) == cudaSuccess &&
              cudaMemset(pk->d_prof, 0, 16 * sizeof(long long)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        cudaFree(pk->d_blob); cudaFree(pk->d_slots); cudaFree(pk->d_slots2); cudaFree(pk->d_prof);
        delete pk;
        m->err = "device allocation for the resident kernel failed";
        return WRNN_ERR_NOMEM;
    }
    // bytes of resident weights read per step: every CTA reads its whole bf16 region once
    pk->weight_bytes_per_step = (int64_t)k.NCTA * (int64_t)k.w_bytes;
    m->resident = pk;
    return WRNN_OK;
}

void resident_destroy(wrnn_model *m)
{
    if (!m->resident) return;
    cudaFree(m->resident->d_blob);
    cudaFree(m->resident->d_slots);
    cudaFree(m->resident->d_prof);
    cudaFree(m->resident->d_slots2);
    delete m->resident;
    m->resident = nullptr;
}

int resident_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes)
{
    (void)batch;
    const ResidentPack &k = *m->resident;
    if (n_ctas) *n_ctas = k.NCTA;
    if (n_threads) *n_threads = k.NW * 32;
    if (smem) *smem = k.smem_bytes;
    if (weight_bytes) *weight_bytes = k.weight_bytes_per_step;
    return WRNN_OK;
}

int resident_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    const ResidentPack &k = *m->resident;
    ResidentParams p;
    std::memset(&p, 0, sizeof(p));
    p.H = m->H; p.K = k.K; p.NKT = k.NKT; p.NMT = k.NMT; p.NLT = k.NLT; p.UC = k.UC; p.HR = k.HR; p.LR = k.LR; p.CS = k.CS;
    p.n_rrows = k.n_rrows;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.blob = k.d_blob; p.blob_bytes = k.blob_bytes; p.w_bytes = k.w_bytes;
    p.g = m->g; p.slots = k.d_slots;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in; p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.frame_shift = a.row_lag > 0 ? a.step0 : 0;          // staggered rows bring one frame per step of the call
    p.a_in = a.a_in; p.b_in = a.b_in; p.a_st_out = a.a_st_out; p.b_st_out = a.b_st_out;
    p.a_forced = a.a_forced; p.b_forced = a.b_forced; p.a_out = a.a_out; p.b_out = a.b_out;
    p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;
    p.prof = m->prof_enabled ? k.d_prof : nullptr;     // phase stamps cost the stamped warp some 50 cycles each: off unless asked for

    if (cudaMemsetAsync(k.d_slots, 0, (size_t)4 * k.K * 8, s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
    // The cooperative attribute makes the driver refuse the launch unless all clusters can be co-resident.
    // WRNN_NO_COOP=1 drops it (co-residency was already checked against the occupancy API at create):
    // a profiler that replays kernels may not accept cooperative cluster launches.
    fill_launch(k, &cfg, at, s, coop_launch_allowed());
    cudaError_t e = k.fused ? cudaLaunchKernelEx(&cfg, resident_dense_kernel<7, 4, 7, 4, true>, p)
                            : cudaLaunchKernelEx(&cfg, resident_dense_kernel<7, 4, 7, 4, false>, p);
    if (e != cudaSuccess) {
        m->err = std::string("resident kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    m->prof_multi = false;
    m->prof_lean = false;
    return WRNN_OK;
}

int resident_pair_supported(const wrnn_model *m, int batch)
{
    return m->resident && m->resident->pair_smem > 0 && (batch == 2 || batch == 4) ? WRNN_OK : WRNN_ERR_UNSUPPORTED;
}

// Rows 2 pair, 2 pair + 1 of the call described by `a` (its conditioning already projected into m->g for all rows).
int resident_pair_run(wrnn_model *m, const StepArgs &a, int pair, cudaStream_t s)
{
    const ResidentPack &k = *m->resident;
    PairParams pp;
    std::memset(&pp, 0, sizeof(pp));
    ResidentParams &p = pp.r;
    const int b0 = 2 * pair, H = m->H;
    const size_t nf = m->cond_dim ? a.n_frames : 1;
    p.H = H; p.K = k.K; p.NKT = k.NKT; p.NMT = k.NMT; p.NLT = k.NLT; p.UC = k.UC; p.HR = k.HR; p.LR = k.LR; p.CS = k.CS;
    p.n_rrows = k.n_rrows;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0 + (unsigned)b0; p.seed = a.seed;
    p.n_frames = (int)nf;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.blob = k.d_blob; p.blob_bytes = k.blob_bytes; p.w_bytes = k.w_bytes;
    p.g = m->g + (size_t)b0 * nf * 3 * H;
    pp.g1 = p.g + nf * 3 * H;
    pp.slots2 = k.d_slots2;
    pp.n_batch = a.batch;
    pp.row_pitch = a.n_steps;
    const size_t ro = (size_t)b0 * a.n_steps;
    p.h_in = a.h_in ? a.h_in + (size_t)b0 * H : nullptr; p.h_out = a.h_out ? a.h_out + (size_t)b0 * H : nullptr;
    p.c_in = a.c_in ? a.c_in + b0 : nullptr; p.f_in = a.f_in ? a.f_in + b0 : nullptr;
    p.c_st_out = a.c_st_out ? a.c_st_out + b0 : nullptr; p.f_st_out = a.f_st_out ? a.f_st_out + b0 : nullptr;
    p.c_forced = a.c_forced ? a.c_forced + ro : nullptr; p.f_forced = a.f_forced ? a.f_forced + ro : nullptr;
    p.c_out = a.c_out ? a.c_out + ro : nullptr; p.f_out = a.f_out ? a.f_out + ro : nullptr;
    p.out = a.out ? a.out + ro : nullptr;
    p.dbg_gates = a.dbg_gates ? a.dbg_gates + (size_t)b0 * 3 * H : nullptr;
    p.dbg_h = a.dbg_h ? a.dbg_h + (size_t)b0 * H : nullptr;
    p.dbg_logits = a.dbg_logits ? a.dbg_logits + (size_t)b0 * 512 : nullptr;
    p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;
    p.prof = m->prof_enabled ? k.d_prof : nullptr;     // phase stamps cost the stamped warp some 50 cycles each: off unless asked for

    if (cudaMemsetAsync(k.d_slots2, 0, (size_t)8 * k.K * 8, s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (pair == 0 && cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
    fill_launch(k, &cfg, at, s, coop_launch_allowed());
    cfg.dynamicSmemBytes = k.pair_smem;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, resident_pair_kernel, pp);
    if (e != cudaSuccess) {
        m->err = std::string("two-stream resident kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    m->prof_multi = false;
    m->prof_lean = false;
    return WRNN_OK;
}

int resident_phase_cycles(const wrnn_model *m, long long *out16)
{
    if (!m->resident) return WRNN_ERR_UNSUPPORTED;
    return cudaMemcpy(out16, m->resident->d_prof, 16 * sizeof(long long), cudaMemcpyDeviceToHost) == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
}

}  // namespace wrnn
