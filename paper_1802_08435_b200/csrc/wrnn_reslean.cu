// Shared-memory-resident persistent sampling kernel for one stream, dense bf16 weights: the lean form.
//
// Same machine as wrnn_resident.cu (Section 2.1 of the paper: one persistent launch per utterance, every weight on chip;
// two chip-wide exchanges per step in the order of Fig. 1; both heads replicated once per 16-CTA cluster and row-sharded
// over its CTAs, so that the drawn symbols never cross the chip), with a shorter dependent chain per half-step:
//   * only the 28 hidden-layer rows of this CTA are multiplied before the hidden layer is sent; the CTA's 24 rows of R
//     (needed by the gates at the end of the half-step, not by the head) are multiplied while the hidden layer
//     crosses the cluster;
//   * K-split partial sums are added by one warp (lane = row) instead of by every sending warp;
//   * the output layer is plain fp32 FMAs on the received hidden layer (no bf16 split, no partial sums, no CTA barrier
//     before it): two rows per warp on eight warps, a lane the element pairs lane, lane + 32, ... of both, six shuffles add up;
//   * both cluster exchanges are asynchronous stores that count their bytes on the receiver's mbarrier;
//   * the uniform, the forced symbol and the gate offsets of a half-step are pinned before its first wait;
//   * the body of a half-step exists once per half, and plain sampling, teacher forcing (forced symbols, dumps), the phase
//     stamps and the self-test predicate each run an instantiation of their own (template parameter MODE).
// Hidden-layer and recurrent products are m16n8k16 bf16 MMAs on A-fragment-packed weights with the fp32 input as an
// exact three-way bf16 split.  Every wait is bounded; a CTA that gives up records where and all CTAs leave through the
// final cluster barrier.
#include <cooperative_groups.h>

#include <type_traits>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "wrnn_cluster.cuh"
#include "wrnn_internal.h"

namespace cg = cooperative_groups;

namespace wrnn {

constexpr int RL_CS = 16;        // CTAs per cluster
constexpr int RL_K = 448;        // H / 2
constexpr int RL_NKT = 28;       // k-tiles of 16
constexpr int RL_HR = 28;        // hidden-layer rows per CTA (= columns of its output-layer slice)
constexpr int RL_UC = 4;         // state units per half per CTA
constexpr int RL_NR = 24;        // rows of R per CTA: (coarse, fine) x (u, r, e) x UC
constexpr int RL_KS = 14;        // K-splits of the hidden / recurrent products: 14 warps x 2 k-tiles
// per variant (FUSED = the Fused Subscale WaveRNN 2x: 64 logits per head as four softmaxes of 4 bits, twelve nibble inputs)
__host__ __device__ constexpr int rl_nlog(bool fused) { return fused ? 64 : 256; }
__host__ __device__ constexpr int rl_lr(bool fused) { return rl_nlog(fused) / RL_CS; }      // output-layer rows per CTA
__host__ __device__ constexpr int rl_nin(bool fused) { return fused ? 12 : 3; }

struct ResLeanPack {
    int NCTA = 0, NC = 0;
    size_t blob_bytes = 0, w_bytes = 0;
    uint8_t *d_blob = nullptr;               // [NCTA][blob_bytes]
    unsigned long long *d_slots = nullptr;   // [2 halves][2 parities][K] (value, tag)
    long long *d_prof = nullptr;             // [16] phase cycle totals of the last call
    int smem_bytes = 0;
    bool checked = false;                    // WRNN_DEBUG=1 at create: the guarded carve-up
    bool fused = false;                      // the Fused Subscale WaveRNN 2x (model variant 1)
    int64_t weight_bytes_per_step = 0;
};

struct ResLeanParams {
    int H;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    long long frame_shift;
    const uint8_t *blob; unsigned long long blob_bytes, w_bytes;
    const float *g;
    unsigned long long *slots;
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
    long long *prof;                         // optional [n CTAs][16] per-phase cycle totals of warp 0 (CTA 0 only unless prof_all)
    int prof_all;
    int chk_poke;                            // checked build only: make one deliberate one-past-the-end write (into a guard)
    unsigned long long smem_bytes;           // dynamic shared memory of the launch (the checked build compares its carve-up with it)
    int poll_gap;                            // >= 0: the pollers of the chip-wide exchange start this many cycles after the CTA's own publication; < 0: at once
};

// byte offsets inside the bf16 part of a CTA's blob
constexpr size_t RL_TILE_U4 = (size_t)RL_NKT * 32;                 // uint4 per 16-row tile over the full K
constexpr size_t RL_HID_BYTES = 2 * RL_TILE_U4 * 16;               // two tiles: 28,672 B
__host__ __device__ constexpr size_t rl_log_bytes(bool f) { return (size_t)rl_lr(f) * RL_K * 2; }          // this CTA's rows of O2 (O4), row-major bf16: 14,336 B
__host__ __device__ constexpr size_t rl_w_bytes(bool f) { return 4 * RL_HID_BYTES + 2 * rl_log_bytes(f); }  // 143,360 B
__host__ __device__ constexpr int rl_small_floats(bool f) { return RL_NR * rl_nin(f) + 2 * 32 + 2 * rl_lr(f); }   // I*, b1, b3 (padded to 32), b2, b4 (this CTA's rows)
__host__ __device__ constexpr size_t rl_blob_bytes(bool f) { return rl_w_bytes(f) + (size_t)rl_small_floats(f) * 4; }
static_assert(rl_blob_bytes(false) % 16 == 0 && rl_blob_bytes(true) % 16 == 0, "blob is copied in 16-byte pieces");

__host__ __device__ constexpr size_t rl_smem_bytes(bool f)
{
    return rl_blob_bytes(f) + (size_t)2 * RL_K * 4 /* vecC, vecF */ + 2 * 24 * 4 /* a_part, a_full */ + 2 * RL_KS * 32 * 4 /* partH, partR */ +
           2 * 4 * RL_K * 2 /* splC, splF */ + 32 * 4 /* q_own */ + 32 * 4 /* lrow */ + (size_t)2 * RL_K * 4 /* qbuf */ + (size_t)2 * rl_nlog(f) * 4 /* lbuf */;
}

// CHK: the checked build (WRNN_DEBUG=1 at create).  Every writable region of the shared-memory carve-up is followed by a
// 16-byte guard (and the first one preceded by one) that is filled at the start and verified at the end, the carve-up's end
// is compared with the size the host allocated, and the index of every published exchange slot is range-checked; a
// violation is recorded in the status word (code 6, step = index of the region or -1 for a slot, phase 99), the access that
// would leave its array is skipped, and the kernel runs to its normal exit.
constexpr int RL_N_GUARDS = 13;
constexpr unsigned RL_GUARD_WORD = 0x5afec0deu;
// MODE 0: plain sampling (no forced symbols, no dumps, no stamps, no self-test predicate: what wrnn_sample runs);
// MODE 1: the instantiation that wrnn_selftest_lost_word runs (one CTA withholds one publication); MODE 2: the one with the
// phase stamps of wrnn_phase_profile; MODE 3: teacher forcing and dumps.  Modes 1 to 3 all take forced symbols and dumps.
template <bool CHK, bool FUSED, int MODE>
__global__ void __launch_bounds__(512, 1) resident_lean_kernel(const ResLeanParams p)
{
    constexpr int RL_NLOG = rl_nlog(FUSED), RL_LR = rl_lr(FUSED), NIN = rl_nin(FUSED), NP = NIN / 3;
    constexpr size_t RL_W_BYTES = rl_w_bytes(FUSED), RL_BLOB_BYTES = rl_blob_bytes(FUSED);
    extern __shared__ __align__(16) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int cta = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int K = RL_K, UC = RL_UC, NR = RL_NR, H = 2 * RL_K;

    // ---- shared memory carve-up (must match RL_SMEM_BYTES)
    const uint4 *wHA = reinterpret_cast<const uint4 *>(smem);                       // O1 rows of this CTA (2 tiles)
    const uint4 *wRA = wHA + 2 * RL_TILE_U4;                                        // R rows x coarse columns (2 tiles)
    const uint4 *wHB = wRA + 2 * RL_TILE_U4;                                        // O3 rows
    const uint4 *wRB = wHB + 2 * RL_TILE_U4;                                        // R rows x fine columns
    const unsigned *wL2 = reinterpret_cast<const unsigned *>(wRB + 2 * RL_TILE_U4);   // this CTA's 16 rows of O2, row-major, two bf16 per word
    const unsigned *wL4 = wL2 + RL_LR * K / 2;
    const float *sI = reinterpret_cast<const float *>(smem + RL_W_BYTES);           // [NR][NIN]
    const float *sb1 = sI + NR * NIN, *sb3 = sb1 + 32, *sb2 = sb3 + 32, *sb4 = sb2 + RL_LR;
    // writable regions, each followed by a guard in the checked build (region index = order below)
    size_t off = RL_BLOB_BYTES;
    unsigned guard_off[RL_N_GUARDS];
    int n_guard = 0;
    auto guard = [&]() { if (CHK) { guard_off[n_guard++] = (unsigned)off; off += 16; } };
    auto carve = [&](size_t bytes) { uint8_t *r = smem + off; off += bytes; guard(); return r; };
    guard();                                                                        // 0: between the weights and the first vector
    float *vecC = reinterpret_cast<float *>(carve((size_t)K * 4));                  // 1: [K] y_c
    float *vecF = reinterpret_cast<float *>(carve((size_t)K * 4));                  // 2: [K] y_f
    float *a_part = reinterpret_cast<float *>(carve(NR * 4));                       // 3: [NR] R[:, :Hh] y_c
    float *a_full = reinterpret_cast<float *>(carve(NR * 4));                       // 4: [NR] R h
    float *partH = reinterpret_cast<float *>(carve(RL_KS * 32 * 4));                // 5: [KS][32] K-split partials of the hidden rows
    float *partR = reinterpret_cast<float *>(carve(RL_KS * 32 * 4));                // 6: [KS][32] ... of the R rows
    __nv_bfloat16 *splC = reinterpret_cast<__nv_bfloat16 *>(carve((size_t)4 * K * 2));   // 7: split images, 4 K bf16 each
    __nv_bfloat16 *splF = reinterpret_cast<__nv_bfloat16 *>(carve((size_t)4 * K * 2));   // 8
    float *q_own = reinterpret_cast<float *>(carve(32 * 4));                        // 9: [32] this CTA's rows of the hidden layer
    float *lrow = reinterpret_cast<float *>(carve(32 * 4));                         // 10: [16 (+16)] this CTA's logits
    float *qbuf = reinterpret_cast<float *>(carve((size_t)2 * K * 4));              // 11: [2 parities][K] hidden layer of the cluster
    float *lbuf = reinterpret_cast<float *>(carve((size_t)2 * RL_NLOG * 4));        // 12: [2 parities][256] logits of the cluster
    auto record_check = [&](int what) {
        if (atomicCAS(&p.status->code, DEV_OK, DEV_CHECK) == DEV_OK) { p.status->cta = blockIdx.x; p.status->step = what; p.status->phase = 99; }
    };
    if (CHK && threadIdx.x == 0 && off != p.smem_bytes) record_check(-2);          // the carve-up and the allocation disagree
    __shared__ __align__(8) unsigned long long xq[2], xl[2];                        // arrival barriers of qbuf[.], lbuf[.]

    // ---- one-time load of this CTA's weights
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.blob + (size_t)cta * p.blob_bytes);
        uint4 *dst = reinterpret_cast<uint4 *>(smem);
        for (size_t i = tid; i < p.blob_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
        if (tid == 0) {
            for (int i = 0; i < 2; ++i) { mbar_init_cluster(smem_addr(&xq[i]), 1); mbar_init_cluster(smem_addr(&xl[i]), 1); }
            mbar_fence_init();
        }
        for (int i = tid; i < 4 * K / 8; i += blockDim.x) {
            reinterpret_cast<uint4 *>(splC)[i] = make_uint4(0, 0, 0, 0);
            reinterpret_cast<uint4 *>(splF)[i] = make_uint4(0, 0, 0, 0);
        }
        if (CHK && tid < n_guard) *reinterpret_cast<uint4 *>(smem + guard_off[tid]) = make_uint4(RL_GUARD_WORD, RL_GUARD_WORD, RL_GUARD_WORD, RL_GUARD_WORD);
        __syncthreads();
        for (int i = tid; i < K; i += blockDim.x) {
            const float c = p.h_in ? p.h_in[i] : 0.f, f = p.h_in ? p.h_in[K + i] : 0.f;
            vecC[i] = c; vecF[i] = f;
            store_split2(splC, i, c);
            store_split2(splF, i, f);
        }
    }
    __syncthreads();
    cluster.sync();     // every peer's barriers are initialised before anyone sends

    Waiter wt{p.status, p.limit_ns};
    bool my_bad = false;
    constexpr bool HOOK = MODE == 1, PROF = MODE == 2 || CHK, DBG = MODE != 0 || CHK;
    const bool prof_on = PROF && p.prof != nullptr && (cta == 0 || p.prof_all) && warp == 0;
    __shared__ long long s_prof[16];
    __shared__ __align__(8) unsigned long long pub_bar;      // one arrival per half-step: this CTA's gate threads have published
    if (tid < 16) s_prof[tid] = 0;
    if (tid == 0) { mbar_init_cluster(smem_addr(&pub_bar), 1); mbar_fence_init(); }
    __syncthreads();
    long long prof_t = clock64();
#define STAMP(i) do { if (PROF && prof_on) { const long long now_ = clock64(); if (lane == 0) s_prof[i] += now_ - prof_t; prof_t = now_; } } while (0)

    const bool writer = (cta == 0);
    const int g4 = lane >> 2;

    // the symbols fed back: the coarse / fine bytes, or (fused) the 16-bit samples of parts A / B
    int c_prev, f_prev;
    if (FUSED) { c_prev = p.a_in ? p.a_in[0] : 0x8000; f_prev = p.b_in ? p.b_in[0] : 0x8000; }
    else { c_prev = p.c_in ? p.c_in[0] : 128; f_prev = p.f_in ? p.f_in[0] : 0; }
    auto xin = [](int v, int k) { return FUSED ? scale4((v >> (12 - 4 * k)) & 15) : scale8(v); };    // scalar k of a symbol as the network sees it
    float hC = 0.f, hF = 0.f;
    if (warp == 0 && lane < UC) { hC = vecC[cta * UC + lane]; hF = vecF[cta * UC + lane]; }

    // K-split products of a pair of 16-row tiles: warp w < 14 takes k-tiles 2 w, 2 w + 1 and leaves 32 partial row sums
    auto tile_pair_products = [&](const uint4 *A, const __nv_bfloat16 *sp, float *dst) {
        float lo[2], hi[2];
        mma_tiles<2, 2>(A, RL_TILE_U4, 2 * warp, sp, lane, lo, hi);
        if ((lane & 3) == 0) {
            float *d = dst + warp * 32;
            d[g4] = lo[0]; d[g4 + 8] = hi[0]; d[16 + g4] = lo[1]; d[24 + g4] = hi[1];
        }
    };
    const bool mma_on = warp < RL_KS;
    // sums of the K-split partials of this CTA's R rows (24 lanes of one warp)
    auto finish_r_rows = [&](bool completes) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < RL_KS; ++w) v += partR[w * 32 + lane];
        if (completes) a_full[lane] = a_part[lane] + v;      // R h complete
        else a_part[lane] = v;                               // R[:, :Hh] y_c: kept for the next half-step
    };
    // warp w sends this CTA's slices (28 hidden values, 16 logits) to CTA w of the cluster, one store instruction each
    // (a store whose lanes address several CTAs at once is several times slower); the stores count their bytes on the
    // receiver's barrier of that buffer
    unsigned q_snd[2], q_bar[2], l_snd[2], l_bar[2];
#pragma unroll
    for (int par2 = 0; par2 < 2; ++par2) {
        q_snd[par2] = map_to_rank(smem_addr(qbuf + (size_t)par2 * K + rank * RL_HR + 2 * (lane < RL_HR / 2 ? lane : 0)), (unsigned)warp);
        q_bar[par2] = map_to_rank(smem_addr(&xq[par2]), (unsigned)warp);
        l_snd[par2] = map_to_rank(smem_addr(lbuf + (size_t)par2 * RL_NLOG + rank * RL_LR + 2 * (lane < RL_LR / 2 ? lane : 0)), (unsigned)warp);
        l_bar[par2] = map_to_rank(smem_addr(&xl[par2]), (unsigned)warp);
    }
    auto wait_arrival = [&](unsigned long long *xb, unsigned use, int step, int phase) {
        const unsigned bar = smem_addr(xb);
        unsigned long long t0 = 0; unsigned cnt = 0;
        while (!mbar_try_parity(bar, use & 1u))
            if ((++cnt & 1023u) == 0 && wt.expired(t0, step, phase)) return false;
        return true;
    };

    // self-test of the checker itself: one word written one past the end of a region (it lands in that region's guard)
    if (CHK && p.chk_poke && cta == 3 && tid == 0) partR[RL_KS * 32] = 1.0f;
    // ---- prologue: R h of the initial state, coarse gates of step 0
    if (mma_on) tile_pair_products(wRA, splC, partR);
    __syncthreads();
    if (warp == 0 && lane < NR) finish_r_rows(false);
    __syncthreads();
    if (mma_on) tile_pair_products(wRB, splF, partR);
    __syncthreads();
    if (warp == 0 && lane < NR) finish_r_rows(true);
    __syncthreads();

    // Gates of Eq. 2 for this CTA's units of one half of the state (half_g = 0: coarse units, 1: fine units): everything
    // up to the one input that the pending draw supplies is prepared while the logits are on their way.
    struct GatePre { float pu, pr, pe, ae, ku[NP], kr[NP], ke[NP]; };
    auto gates_prepare = [&](int half_g, const float (&gv)[3]) {
        GatePre q;
        const int rb = half_g ? 3 * UC : 0;
        const float *Iu = sI + NIN * (rb + lane), *Ir = sI + NIN * (rb + UC + lane), *Ie = sI + NIN * (rb + 2 * UC + lane);
        // fine units: inputs (c_{s-1}, f_{s-1}) known, c_s pending (last column group); coarse units: c_{s-1} known, f_{s-1}
        // pending (middle column group)
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
    const int skip_at = (HOOK && cta == p.skip_cta) ? (int)p.skip_step : -1;      // self-test: the step at which this CTA withholds its publication
    const bool dbg_any = DBG && (p.dbg_gates != nullptr || p.dbg_h != nullptr);
    auto gates_and_publish = [&](int half_g, long long s, int drawn, const GatePre &q) {
        float pu = q.pu, pr = q.pr, pe = q.pe;
#pragma unroll
        for (int k = 0; k < NP; ++k) {
            const float xk = xin(drawn, k);                  // the pending input
            pu = fmaf(q.ku[k], xk, pu); pr = fmaf(q.kr[k], xk, pr); pe = fmaf(q.ke[k], xk, pe);
        }
        const float u = sigmoidf_fast(pu), r = sigmoidf_fast(pr);
        const float e = tanhf_fast(fmaf(r, q.ae, pe));
        const float hn = fmaf(u, half_g ? hF : hC, (1.0f - u) * e);
        if (half_g) hF = hn; else hC = hn;
        const int j = cta * UC + lane, jj = (half_g ? K : 0) + j;
        const size_t slot = (size_t)((half_g ? 2 : 0) + (s & 1)) * K + j;
        if (CHK && slot >= (size_t)4 * K) record_check(-1);                          // an exchange slot outside the slot array: skipped
        else if (!HOOK || (int)s != skip_at)
            st_relaxed_u64(p.slots + slot, ((unsigned long long)(unsigned)(s + 1) << 32) | __float_as_uint(hn));
        if (DBG && dbg_any) {
            if (p.dbg_gates) { float *d = p.dbg_gates + (size_t)s * 3 * H; d[jj] = u; d[H + jj] = r; d[2 * H + jj] = e; }
            if (p.dbg_h) p.dbg_h[(size_t)s * H + jj] = hn;
        }
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
    if (tid == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&pub_bar)) : "memory");

    // Half-step n = 2 s + 1 is the coarse half of step s (input y_c(s): coarse head -> c_s, then the fine gates of step s),
    // n = 2 s the fine half (input y_f(s - 1): fine head -> f_{s-1}, R h_{s-1} completed, then the coarse gates of step s).
    const long long T = p.n_steps;
    // (one copy of the body per half, so that everything chosen by the half is chosen at compile time)
    auto half_step = [&](auto HALF_C, const long long n) -> bool {
        constexpr int half = decltype(HALF_C)::value;
        const long long s = n >> 1;
        const bool last = n == 2 * T;
        constexpr unsigned par = 1u - (unsigned)half;           // (n - 1) & 1
        const uint4 *MH = half ? wHA : wHB, *MR = half ? wRA : wRB;
        const unsigned *L = half ? wL2 : wL4;
        const float *bh = half ? sb1 : sb3, *bl = half ? sb2 : sb4;
        float *vec = half ? vecC : vecF;
        __nv_bfloat16 *spl = half ? splC : splF;

        const unsigned use = (unsigned)((n - 1) >> 1);          // how often this half's buffers were used before
        if (tid == 0) {
            mbar_arrive_expect(smem_addr(&xq[par]), (unsigned)K * 4u);          // this half's arrivals: K hidden values
            mbar_arrive_expect(smem_addr(&xl[par]), (unsigned)RL_NLOG * 4u);    // and 256 logits
        }
        // everything that does not depend on the chain is fetched / computed before the first wait, and pinned there
        float gv[3] = {0.f, 0.f, 0.f}, u01 = 0.f;
        int forced = -1;
        if (warp == 0) {
            if (lane < UC && !last) load_g(half, s, gv);
            if (FUSED) {
                if (DBG) {
                    if (half) { if (p.a_forced) forced = p.a_forced[s]; }
                    else      { if (p.b_forced) forced = p.b_forced[s - 1]; }
                }
                u01 = uniform24(p.seed, p.stream0, (unsigned long long)(p.step0 + (half ? s : s - 1)), (half ? 0u : 4u) + (unsigned)(lane >> 3));
            } else {
                if (DBG) {
                    if (half) { if (p.c_forced) forced = p.c_forced[s]; }
                    else      { if (p.f_forced) forced = p.f_forced[s - 1]; }
                }
                u01 = uniform24(p.seed, p.stream0, (unsigned long long)(p.step0 + (half ? s : s - 1)), half ? 0u : 1u);
            }
            asm volatile("" : "+f"(u01), "+r"(forced), "+f"(gv[0]), "+f"(gv[1]), "+f"(gv[2]));
        }

        // ---- 1. input half-vector from the whole chip (y_c(s) carries tag s + 1; y_f(s - 1) carries tag s)
        {
            const unsigned long long *slots = p.slots + (size_t)(half ? (s & 1) : 2 + ((s - 1) & 1)) * K;
            const unsigned ytag = (unsigned)(half ? s + 1 : s);
            if (warp >= 1 && warp <= 7) {
                const int i = tid - 32;
                unsigned long long v0, v1, t0 = 0; unsigned cnt = 0;
                if (p.poll_gap >= 0) {
                    // Polls that come before the data only load the L2 slices the publishing stores have to get through,
                    // and a poll that just misses the data costs a whole round trip.  The pollers therefore hold back
                    // until this CTA's own gate threads have published (all CTAs publish at about the same time), plus
                    // poll_gap cycles, so that their first poll reaches L2 when the words do.
                    // (waiting on an mbarrier parks the thread in hardware; a spin on a shared-memory word takes issue slots from
                    // the warp that draws)
                    while (!mbar_try_parity(smem_addr(&pub_bar), (unsigned)((n - 1) & 1)))
                        if ((++cnt & 1023u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
                    const long long c0 = clock64();
                    while (clock64() - c0 < p.poll_gap) { }
                    cnt = 0; t0 = 0;
                }
                while (!my_bad) {
                    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v0), "=l"(v1) : "l"(slots + 2 * i) : "memory");
                    if ((unsigned)(v0 >> 32) == ytag && (unsigned)(v1 >> 32) == ytag) break;
                    if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
                }
                const float x0 = __uint_as_float((unsigned)v0), x1 = __uint_as_float((unsigned)v1);
                vec[2 * i] = x0; vec[2 * i + 1] = x1;
                store_split2_pair(spl, 2 * i, x0, x1);
            }
            if (__syncthreads_or(my_bad)) return false;
        }
        STAMP(8 * half + 0);

        // ---- 2. hidden layer of the head: this CTA's 28 rows, K split over 14 warps
        if (mma_on) tile_pair_products(MH, spl, partH);
        __syncthreads();
        STAMP(8 * half + 1);
        // one warp adds the partials (lane = row; rows 28..31 are zero padding), bias, relu
        if (warp == 0) {
            float v = bh[lane];
#pragma unroll
            for (int w = 0; w < RL_KS; ++w) v += partH[w * 32 + lane];
            q_own[lane] = fmaxf(v, 0.f);
        }
        __syncthreads();
        if (lane < RL_HR / 2) {
            const float2 v = reinterpret_cast<const float2 *>(q_own)[lane];
            st_async_v2(q_snd[par], v.x, v.y, q_bar[par]);
        }
        STAMP(8 * half + 2);
        // ---- 3. while the hidden layer crosses the cluster: this CTA's rows of R against the same input
        if (mma_on) tile_pair_products(MR, spl, partR);
        __syncthreads();
        STAMP(8 * half + 3);

        // ---- 4. the cluster's hidden layer -> this CTA's 16 output-layer rows in fp32: warps 8..15 take two rows each, a
        // lane the element pairs lane, lane + 32, ... of both (every shared-memory pass delivers 128 distinct bytes)
        GatePre gp = {};
        if (warp >= 8 && warp < 8 + RL_LR / 2) {
            if (!wait_arrival(&xq[par], use, (int)s, 2 + 4 * half)) my_bad = true;
            const int ra = 2 * (warp - 8);
            const unsigned *wa = L + ra * (K / 2) + lane, *wb = wa + K / 2;
            const float2 *q2 = reinterpret_cast<const float2 *>(qbuf + (size_t)par * K) + lane;
            float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
#pragma unroll
            for (int j = 0; j < 7; ++j) {
                const float2 q = q2[32 * j];
                const unsigned x = wa[32 * j], y = wb[32 * j];
                a0 = fmaf(bf16lo(x), q.x, a0); a1 = fmaf(bf16hi(x), q.y, a1);
                b0 = fmaf(bf16lo(y), q.x, b0); b1 = fmaf(bf16hi(y), q.y, b1);
            }
            const float va = a0 + a1, vb = b0 + b1;
            // both sums across the warp in six shuffles: lanes 0..15 end up with row ra, lanes 16..31 with row ra + 1
            const bool up = (lane & 16) != 0;
            float v = (up ? vb : va) + __shfl_xor_sync(FULL, up ? va : vb, 16);
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
            if ((lane & 15) == 0) lrow[ra + (lane >> 4)] = v + bl[ra + (lane >> 4)];
        } else if (warp == 0) {
            // meanwhile: sums of the recurrent K-split partials, then the gate pre-activations up to the pending symbol
            if (lane < NR) finish_r_rows(!half);
            __syncwarp();
            if (lane < UC && !last) gp = gates_prepare(half, gv);
        }
        STAMP(8 * half + 4);
        if (__syncthreads_or(my_bad)) return false;
        if (lane < RL_LR / 2) {
            const float2 v = reinterpret_cast<const float2 *>(lrow)[lane];
            st_async_v2(l_snd[par], v.x, v.y, l_bar[par]);
        }
        STAMP(8 * half + 5);

        // ---- 5. warp 0: the cluster's 256 logits -> draw; then the gates of the other half of the state
        if (warp == 0) {
            if (!wait_arrival(&xl[par], use, (int)s, 3 + 4 * half)) my_bad = true;
            my_bad = __any_sync(FULL, my_bad);
            STAMP(8 * half + 6);
            constexpr int NL = FUSED ? 2 : 8;
            float l[NL];
            int drawn;
            if (FUSED) {
                // 64 logits: two per lane; lanes [8 k, 8 k + 8) are the softmax of nibble k (most significant first)
                const float2 a = reinterpret_cast<const float2 *>(lbuf + (size_t)par * RL_NLOG)[lane];
                l[0] = a.x; l[1] = a.y;
                const int nib = group16_softmax_draw(l[0], l[1], u01, lane);
                drawn = (__shfl_sync(FULL, nib, 0) << 12) | (__shfl_sync(FULL, nib, 8) << 8) | (__shfl_sync(FULL, nib, 16) << 4) | __shfl_sync(FULL, nib, 24);
            } else {
                const float4 a = reinterpret_cast<const float4 *>(lbuf + (size_t)par * RL_NLOG)[2 * lane];
                const float4 b = reinterpret_cast<const float4 *>(lbuf + (size_t)par * RL_NLOG)[2 * lane + 1];
                l[0] = a.x; l[1] = a.y; l[2] = a.z; l[3] = a.w; l[NL - 4] = b.x; l[NL - 3] = b.y; l[NL - 2] = b.z; l[NL - 1] = b.w;
                drawn = warp_softmax_draw_fast(reinterpret_cast<const float (&)[8]>(l), u01, lane);
            }
            const int fed = (DBG && forced >= 0) ? forced : drawn;
            if (lane < UC && !last && !my_bad) gates_and_publish(half, s, fed, gp);
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&pub_bar)) : "memory");
            if (writer) {
                if (DBG && p.dbg_logits) {
                    float *d = p.dbg_logits + (size_t)(n - 1) * RL_NLOG + NL * lane;
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
        STAMP(8 * half + 7);
        return true;
    };
#pragma unroll 1
    for (long long s2 = 0; s2 < T; ++s2) {
        if (!half_step(std::integral_constant<int, 1>{}, 2 * s2 + 1)) break;
        if (!half_step(std::integral_constant<int, 0>{}, 2 * s2 + 2)) break;
    }
    if (prof_on && lane == 0) for (int i = 0; i < 16; ++i) p.prof[cta * 16 + i] = s_prof[i];
#undef STAMP

    const int any_bad = __syncthreads_or(my_bad);
    if (CHK && tid < n_guard) {
        const uint4 g = *reinterpret_cast<const uint4 *>(smem + guard_off[tid]);
        if (g.x != RL_GUARD_WORD || g.y != RL_GUARD_WORD || g.z != RL_GUARD_WORD || g.w != RL_GUARD_WORD) record_check(tid);
    }
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
static const void *kernel_of(const ResLeanPack &k, int mode)
{
    if (k.checked) return k.fused ? (const void *)resident_lean_kernel<true, true, 0> : (const void *)resident_lean_kernel<true, false, 0>;
    if (mode == 1) return k.fused ? (const void *)resident_lean_kernel<false, true, 1> : (const void *)resident_lean_kernel<false, false, 1>;
    if (mode == 2) return k.fused ? (const void *)resident_lean_kernel<false, true, 2> : (const void *)resident_lean_kernel<false, false, 2>;
    if (mode == 3) return k.fused ? (const void *)resident_lean_kernel<false, true, 3> : (const void *)resident_lean_kernel<false, false, 3>;
    return k.fused ? (const void *)resident_lean_kernel<false, true, 0> : (const void *)resident_lean_kernel<false, false, 0>;
}

static void fill_launch(const ResLeanPack &k, cudaLaunchConfig_t *cfg, cudaLaunchAttribute *at, cudaStream_t s, bool coop)
{
    std::memset(cfg, 0, sizeof(*cfg));
    cfg->gridDim = dim3(k.NCTA);
    cfg->blockDim = dim3(512);
    cfg->dynamicSmemBytes = k.smem_bytes + (k.checked ? RL_N_GUARDS * 16 : 0);
    cfg->stream = s;
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = RL_CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative;
    at[1].val.cooperative = 1;
    cfg->attrs = at;
    cfg->numAttrs = coop ? 2 : 1;
}

int reslean_supported(const wrnn_model *m, int batch)
{
    return (batch == 1 && m->reslean != nullptr) ? WRNN_OK : WRNN_ERR_UNSUPPORTED;
}

int reslean_prepare(wrnn_model *m)
{
    if (m->dtype != WRNN_BF16 || m->sparse || m->H != 2 * RL_K) { m->err = "lean resident kernel: dense bf16 H = 896 only"; return WRNN_ERR_UNSUPPORTED; }
    const bool fused = m->variant == 1;
    const int LR = rl_lr(fused), NIN = rl_nin(fused);
    ResLeanPack k;
    k.fused = fused;
    k.NCTA = RL_K / RL_UC; k.NC = k.NCTA / RL_CS;
    k.blob_bytes = rl_blob_bytes(fused); k.w_bytes = rl_w_bytes(fused); k.smem_bytes = (int)rl_smem_bytes(fused);
    cudaDeviceProp prop;
    cudaGetDeviceProperties(&prop, m->device);
    if (k.NCTA > m->n_sms || (size_t)k.smem_bytes > prop.sharedMemPerBlockOptin) { m->err = "lean resident kernel does not fit this device"; return WRNN_ERR_UNSUPPORTED; }
    { const char *d = getenv("WRNN_DEBUG"); k.checked = d && d[0] == '1'; }
    const void *fn = kernel_of(k, 0);
    for (int mode = 0; mode < 4; ++mode) {
        const void *f = kernel_of(k, mode);
        if (cudaFuncSetAttribute(f, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
            cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem_bytes + (k.checked ? RL_N_GUARDS * 16 : 0)) != cudaSuccess) {
            cudaGetLastError(); m->err = "lean resident kernel: cannot set the launch attributes"; return WRNN_ERR_UNSUPPORTED;
        }
    }
    {
        cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
        fill_launch(k, &cfg, at, 0, false);
        int max_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&max_clusters, fn, &cfg) != cudaSuccess || max_clusters < k.NC) {
            cudaGetLastError(); m->err = "lean resident kernel: not enough co-resident clusters"; return WRNN_ERR_UNSUPPORTED;
        }
    }
    const int H = m->H, K = RL_K, UC = RL_UC;
    std::vector<uint8_t> blob((size_t)k.NCTA * k.blob_bytes, 0);
    std::vector<std::vector<uint16_t>> rows(16, std::vector<uint16_t>(K));
    const BsrHost *Oa[2] = {&m->hO1, &m->hO3}, *Ob[2] = {&m->hO2, &m->hO4};
    const size_t tile_elems = (size_t)16 * K;
    for (int cta = 0; cta < k.NCTA; ++cta) {
        const int rank = cta % RL_CS;
        uint8_t *base = blob.data() + (size_t)cta * k.blob_bytes;
        uint16_t *w = reinterpret_cast<uint16_t *>(base);
        float *sm = reinterpret_cast<float *>(base + k.w_bytes);
        for (int part = 0; part < 2; ++part) {
            uint16_t *wH = w + (size_t)part * 4 * tile_elems, *wR = wH + 2 * tile_elems;
            for (int mt = 0; mt < 2; ++mt) {
                // hidden-layer rows rank * 28 .. + 27 of O1 (O3), four zero rows of padding
                for (int r = 0; r < 16; ++r) {
                    const int row = 16 * mt + r;
                    if (row < RL_HR) dense_row_bf16(*Oa[part], rank * RL_HR + row, 0, K, rows[r].data());
                    else std::fill(rows[r].begin(), rows[r].end(), (uint16_t)0);
                }
                pack_tile(rows, K, wH + (size_t)mt * tile_elems);
                // R row rr = (half * 3 + gate) * UC + u -> matrix row gate * H + half * K + cta * UC + u, columns of input half `part`
                for (int r = 0; r < 16; ++r) {
                    const int rr = 16 * mt + r;
                    if (rr < RL_NR) {
                        const int half = rr / (3 * UC), gate = (rr / UC) % 3, u = rr % UC;
                        dense_row_bf16(m->hR, gate * H + half * K + cta * UC + u, part * K, K, rows[r].data());
                    } else std::fill(rows[r].begin(), rows[r].end(), (uint16_t)0);
                }
                pack_tile(rows, K, wR + (size_t)mt * tile_elems);
            }
        }
        // output layers: this CTA's rows of O2 (O4), row-major
        uint16_t *wl = w + (size_t)8 * tile_elems;
        for (int h = 0; h < 2; ++h)
            for (int r = 0; r < LR; ++r) dense_row_bf16(*Ob[h], rank * LR + r, 0, K, wl + ((size_t)h * LR + r) * K);
        for (int rr = 0; rr < RL_NR; ++rr) {
            const int half = rr / (3 * UC), gate = (rr / UC) % 3, u = rr % UC;
            const int mrow = gate * H + half * K + cta * UC + u;
            for (int c = 0; c < NIN; ++c) sm[rr * NIN + c] = m->hI[(size_t)mrow * NIN + c];
        }
        float *b = sm + RL_NR * NIN;
        for (int r = 0; r < RL_HR; ++r) { b[r] = m->hb1[rank * RL_HR + r]; b[32 + r] = m->hb3[rank * RL_HR + r]; }
        b += 64;
        for (int r = 0; r < LR; ++r) { b[r] = m->hb2[rank * LR + r]; b[LR + r] = m->hb4[rank * LR + r]; }
    }
    ResLeanPack *pk = new ResLeanPack(k);
    bool ok = cudaMalloc((void **)&pk->d_blob, blob.size()) == cudaSuccess &&
              cudaMemcpy(pk->d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice) == cudaSuccess &&
              cudaMalloc((void **)&pk->d_slots, (size_t)4 * K * 8) == cudaSuccess &&
              cudaMalloc((void **)&pk->d_prof, (size_t)k.NCTA * 16 * sizeof(long long)) == cudaSuccess &&
              cudaMemset(pk->d_prof, 0, (size_t)k.NCTA * 16 * sizeof(long long)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        cudaFree(pk->d_blob); cudaFree(pk->d_slots); cudaFree(pk->d_prof);
        delete pk;
        m->err = "device allocation for the lean resident kernel failed";
        return WRNN_ERR_NOMEM;
    }
    pk->weight_bytes_per_step = (int64_t)k.NCTA * (int64_t)k.w_bytes;
    m->reslean = pk;
    return WRNN_OK;
}

void reslean_destroy(wrnn_model *m)
{
    if (!m->reslean) return;
    cudaFree(m->reslean->d_blob); cudaFree(m->reslean->d_slots); cudaFree(m->reslean->d_prof);
    delete m->reslean;
    m->reslean = nullptr;
}

int reslean_launch_info(const wrnn_model *m, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes)
{
    const ResLeanPack &k = *m->reslean;
    if (n_ctas) *n_ctas = k.NCTA;
    if (n_threads) *n_threads = 512;
    if (smem) *smem = k.smem_bytes + (k.checked ? RL_N_GUARDS * 16 : 0);
    if (weight_bytes) *weight_bytes = k.weight_bytes_per_step;
    return WRNN_OK;
}

int reslean_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    const ResLeanPack &k = *m->reslean;
    ResLeanParams p;
    std::memset(&p, 0, sizeof(p));
    p.H = m->H;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.blob = k.d_blob; p.blob_bytes = k.blob_bytes; p.w_bytes = k.w_bytes;
    p.g = m->g; p.slots = k.d_slots;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in; p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.a_in = a.a_in; p.b_in = a.b_in; p.a_st_out = a.a_st_out; p.b_st_out = a.b_st_out;
    p.a_forced = a.a_forced; p.b_forced = a.b_forced; p.a_out = a.a_out; p.b_out = a.b_out;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.frame_shift = a.row_lag > 0 ? a.step0 : 0;
    p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;
    { const char *e = getenv("WRNN_POLL_GAP"); p.poll_gap = e ? atoi(e) : 125; }
    p.prof = m->prof_enabled ? k.d_prof : nullptr;     // phase stamps cost the stamped warp some 50 cycles each: off unless asked for
    { const char *e = getenv("WRNN_PROF_ALL"); p.prof_all = (e && e[0] == '1') ? 1 : 0; }
    if (cudaMemsetAsync(k.d_slots, 0, (size_t)4 * RL_K * 8, s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
    fill_launch(k, &cfg, at, s, coop_launch_allowed());
    p.smem_bytes = cfg.dynamicSmemBytes;
    { const char *d = getenv("WRNN_DEBUG_POKE"); p.chk_poke = (k.checked && d && d[0] == '1') ? 1 : 0; }
    void *args[] = {&p};
    const bool teacher = p.c_forced || p.f_forced || p.a_forced || p.b_forced || p.dbg_gates || p.dbg_h || p.dbg_logits;
    const cudaError_t e = cudaLaunchKernelExC(&cfg, kernel_of(k, m->dbg_skip_cta >= 0 ? 1 : (p.prof ? 2 : (teacher ? 3 : 0))), args);
    if (e != cudaSuccess) {
        m->err = std::string("lean resident kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    m->prof_multi = false;
    m->prof_lean = true;
    return WRNN_OK;
}

int reslean_phase_cycles(const wrnn_model *m, long long *out16)
{
    if (!m->reslean) return WRNN_ERR_UNSUPPORTED;
    // WRNN_PROF_DUMP=<file> (with WRNN_PROF_ALL=1 at launch): the stamps of every CTA's first warp as text, one CTA per line
    if (const char *path = getenv("WRNN_PROF_DUMP")) {
        std::vector<long long> all((size_t)m->reslean->NCTA * 16);
        if (cudaMemcpy(all.data(), m->reslean->d_prof, all.size() * sizeof(long long), cudaMemcpyDeviceToHost) == cudaSuccess)
            if (FILE *f = std::fopen(path, "w")) {
                for (int c = 0; c < m->reslean->NCTA; ++c) {
                    for (int i = 0; i < 16; ++i) std::fprintf(f, "%lld%c", all[(size_t)c * 16 + i], i == 15 ? '\n' : ' ');
                }
                std::fclose(f);
            }
    }
    return cudaMemcpy(out16, m->reslean->d_prof, 16 * sizeof(long long), cudaMemcpyDeviceToHost) == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
}

}  // namespace wrnn
