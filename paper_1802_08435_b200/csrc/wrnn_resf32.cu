// Shared-memory-resident persistent sampling kernel for one stream (batch 1), dense fp32 weights.
//
// fp32 weights are twice the size of bf16 ones, so the hidden layers of the output heads cannot be replicated per
// cluster as in the bf16 kernel (Section 2.1: one persistent operation, parameters loaded on-chip once).  Here R, O1
// and O3 are sharded over the whole chip, nothing replicated; only the two logits matrices O2 / O4 are held once per
// cluster of CS CTAs.  CTA c of NCTA (cluster rank r) owns
//   * UC = Hh / NCTA coarse and UC fine state units: 6 UC rows of R (gates u, r, e), split into the columns that
//     multiply y_c and those that multiply y_f;
//   * UC rows of O1 and of O3 (the same indices as its units);
//   * rows [r LR, (r + 1) LR), LR = 256 / CS, of O2 and of O4.
// A half-step (Fig. 1's order; the two-half schedule of the bf16 kernel) therefore has two chip-wide exchanges -- the
// state half and the hidden layer, each an all-gather of (value, step-tag) words through L2 where arrival of the data
// is the signal -- and one cluster-wide exchange of the logits through distributed shared memory; every CTA then
// draws the sample itself, so the drawn value never travels.  Products are plain fp32 FMAs from shared memory: the 16
// warps form 4 row groups x 4 column quarters, so every weight and (per row group) every input is read once.
//
// Every wait is bounded; a CTA that gives up records where, and the give-up is made CTA-uniform before the CTA leaves.
#include <cooperative_groups.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>

#include "wrnn_cluster.cuh"
#include "wrnn_internal.h"

namespace cg = cooperative_groups;

namespace wrnn {

constexpr int RF_THREADS = 512;           // 16 warps: 4 row groups x 4 column quarters

struct ResF32Pack {
    int NCTA = 0, CS = 0, UC = 0, K = 0, NR = 0, LR = 0, PR = 0;   // NR = 6 UC rows of R per CTA; LR = 256 / CS logit rows; PR = pitch of the partial sums
    size_t blob_bytes = 0, w_bytes = 0;              // per CTA: fp32 weights, then small parameters
    uint8_t *d_blob = nullptr;                       // [NCTA][blob_bytes]
    unsigned long long *d_slots = nullptr;           // y: [2 halves][2][K], q: [2][K]
    long long *d_prof = nullptr;                     // [16] phase cycle totals of the last call (diagnostic)
    int smem_bytes = 0;
    int64_t weight_bytes_per_step = 0;
};

struct ResF32Params {
    int H, K, UC, NR, NCTA, CS, LR, PR;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    const uint8_t *blob; unsigned long long blob_bytes, w_bytes;
    const float *g;
    unsigned long long *yslots, *qslots;
    const float *h_in; float *h_out;
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;
    uint8_t *c_out, *f_out;
    int16_t *out;
    float *dbg_gates, *dbg_h, *dbg_logits;
    DevStatus *status;
    unsigned long long limit_ns;
    int poll_gap;                            // >= 0: the state exchange's pollers start this many cycles after the CTA's own publication
    int skip_cta; long long skip_step;      // self-test: this CTA withholds what it publishes at this step (-1: none)
    long long *prof;                         // [16] per-phase cycle totals of CTA 0, warp 0 (same slots as the bf16 kernel)
};

// MODE 1: the instantiation that wrnn_selftest_lost_word runs (one CTA withholds one publication); MODE 2: the one with the phase
// stamps of wrnn_phase_profile; MODE 0 (production) has no trace of either
template <int MODE>
__global__ void __launch_bounds__(RF_THREADS, 1) resident_f32_kernel(const ResF32Params p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int cta = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = (int)cluster.block_rank();
    const int K = p.K, UC = p.UC, NR = p.NR, H = p.H, LR = p.LR, PR = p.PR, CS = p.CS;
    const int NS = UC + NR;                                                     // rows of one stacked matrix

    // ---- shared memory carve-up (must match resf32_smem_bytes)
    const float *wA = reinterpret_cast<const float *>(smem);                    // [NS][K]: rows [O1 ; R x coarse cols]
    const float *wB = wA + (size_t)NS * K;                                      // [NS][K]: rows [O3 ; R x fine cols]
    const float *wO2 = wB + (size_t)NS * K;                                     // [LR][K]
    const float *wO4 = wO2 + (size_t)LR * K;
    const float *sI = reinterpret_cast<const float *>(smem + p.w_bytes);        // [NR][3]
    const float *sb1 = sI + NR * 3, *sb3 = sb1 + UC, *sb2 = sb3 + UC, *sb4 = sb2 + LR;
    float *vecC = reinterpret_cast<float *>(smem + p.blob_bytes);               // [K] y_c
    float *vecF = vecC + K;                                                     // [K] y_f
    float *qvec = vecF + K;                                                     // [K] hidden layer of the head in flight
    float *part = qvec + K;                                                     // [4 quarters][PR] partial sums
    float *a_part = part + 4 * PR;                                              // [NR] R[:, :Hh] y_c
    float *a_full = a_part + NR;                                                // [NR] R h
    uint4 *lbuf = reinterpret_cast<uint4 *>(a_full + NR + ((4 - (2 * NR) % 4) % 4));   // [2][128] logits of the cluster: {v, tag, v, tag}

    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.blob + (size_t)cta * p.blob_bytes);
        uint4 *dst = reinterpret_cast<uint4 *>(smem);
        for (size_t i = tid; i < p.blob_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
        for (int i = tid; i < K; i += blockDim.x) {
            vecC[i] = p.h_in ? p.h_in[i] : 0.f;
            vecF[i] = p.h_in ? p.h_in[K + i] : 0.f;
        }
        for (int i = tid; i < 256; i += blockDim.x) lbuf[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    cluster.sync();     // peers' exchange buffers are zeroed before anyone writes into them

    constexpr bool HOOK = MODE == 1, PROF = MODE == 2;
    const bool prof_on = PROF && p.prof != nullptr && cta == 0 && warp == 0;
    __shared__ long long s_prof[16];
    __shared__ __align__(8) unsigned long long pub_bar;      // one arrival per half-step: this CTA's gate threads have published
    if (tid == 0) { mbar_init_cluster(smem_addr(&pub_bar), 1); mbar_fence_init(); }
    if (tid < 16) s_prof[tid] = 0;
    __syncthreads();
    long long prof_t = clock64();
#define STAMP(i) do { if (PROF && prof_on) { const long long now_ = clock64(); if (lane == 0) s_prof[i] += now_ - prof_t; prof_t = now_; } } while (0)

    Waiter wt{p.status, p.limit_ns};
    bool my_bad = false;
    const bool writer = (cta == 0);

    // warp 0 keeps the stream's scalar state
    int c_prev = p.c_in ? p.c_in[0] : 128, f_prev = p.f_in ? p.f_in[0] : 0;
    float hC = 0.f, hF = 0.f;
    if (warp == 0 && lane < UC) { hC = vecC[cta * UC + lane]; hF = vecF[cta * UC + lane]; }

    // where this warp sends its share of the logits: peer `warp` of the cluster, this CTA's LR rows of its buffer
    unsigned l_snd[2] = {0u, 0u};
    if (warp < CS) {
        l_snd[0] = map_to_rank(smem_addr(lbuf + rank * (LR / 2)), (unsigned)warp);
        l_snd[1] = map_to_rank(smem_addr(lbuf + 128 + rank * (LR / 2)), (unsigned)warp);
    }

    // W[nrows][K] x[K] -> part[quarter][row]: warp (rg, kq) takes a quarter of the columns of a quarter of the rows,
    // eight rows at a time, its piece of x in registers across them.
    auto rows_times = [&](const float *W, int nrows, const float *x) {
        const int kq = warp & 3, rg = warp >> 2, Q4 = K / 16;                   // Q4 = 16-byte pieces per column quarter
        const int rpg = (nrows + 3) / 4, r_end = min(nrows, (rg + 1) * rpg);
        const float4 *x4 = reinterpret_cast<const float4 *>(x) + kq * Q4;
        for (int r0 = rg * rpg; r0 < r_end; r0 += 8) {
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            const float4 *w4 = reinterpret_cast<const float4 *>(W + (size_t)r0 * K) + kq * Q4;
            for (int c = lane; c < Q4; c += 32) {
                const float4 b = x4[c];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (r0 + j < r_end) {
                        const float4 a = w4[(size_t)j * (K / 4) + c];
                        acc[j] = fmaf(a.x, b.x, fmaf(a.y, b.y, fmaf(a.z, b.z, fmaf(a.w, b.w, acc[j]))));
                    }
            }
            const float v = warp_reduce_scatter<8>(acc, lane);                  // lane l: total of row r0 + (l & 7)
            if (lane < 8 && r0 + lane < r_end) part[kq * PR + r0 + lane] = v;
        }
    };
    // After the barrier: thread i < NS finishes row i of the stacked matrix.  Rows [0, UC) are hidden-layer rows (bias, relu,
    // published to the chip), rows [UC, NS) this CTA's rows of R.
    auto stacked_finish = [&](const float *bias, bool completes, unsigned long long *qdst, unsigned tag) {
        if (tid < NS) {
            const float v = (part[tid] + part[PR + tid]) + (part[2 * PR + tid] + part[3 * PR + tid]);
            if (tid < UC) {
                if (qdst) st_relaxed_u64(qdst + cta * UC + tid, ((unsigned long long)tag << 32) | __float_as_uint(fmaxf(v + bias[tid], 0.f)));
            }
            else if (completes) a_full[tid - UC] = a_part[tid - UC] + v;         // R h complete
            else a_part[tid - UC] = v;                                          // R[:, :Hh] y_c: kept for the next step
        }
    };

    // ---- prologue: the recurrent products of step 0 from the initial state, coarse gates of step 0
    rows_times(wA, NS, vecC);
    __syncthreads();
    stacked_finish(sb1, false, nullptr, 0u);
    __syncthreads();
    rows_times(wB, NS, vecF);
    __syncthreads();
    stacked_finish(sb3, true, nullptr, 0u);
    __syncthreads();

    // The gate pre-activations up to the one input that is only known after the draw (c_s for the fine units, f_{s-1} for
    // the coarse units of the next step): computed while the logits are still on their way.
    struct GatePre { float pu, pr, pe, ae, ku, kr, ke; };
    auto gates_prepare = [&](int half_g, const float (&gv)[3]) {
        GatePre q;
        const int rb = half_g ? 3 * UC : 0;
        const float x0 = scale8(c_prev), x1 = scale8(f_prev);
        const float *Iu = sI + 3 * (rb + lane), *Ir = sI + 3 * (rb + UC + lane), *Ie = sI + 3 * (rb + 2 * UC + lane);
        q.pu = a_full[rb + lane] + fmaf(Iu[0], x0, half_g ? fmaf(Iu[1], x1, gv[0]) : gv[0]);
        q.pr = a_full[rb + UC + lane] + fmaf(Ir[0], x0, half_g ? fmaf(Ir[1], x1, gv[1]) : gv[1]);
        q.pe = fmaf(Ie[0], x0, half_g ? fmaf(Ie[1], x1, gv[2]) : gv[2]);
        q.ae = a_full[rb + 2 * UC + lane];
        q.ku = half_g ? Iu[2] : Iu[1]; q.kr = half_g ? Ir[2] : Ir[1]; q.ke = half_g ? Ie[2] : Ie[1];
        return q;
    };
    // Gates of Eq. 2 for this CTA's units of one half of the state, then publish them to the chip.
    // half_g = 0: coarse units (c_s does not reach them: their I* column is zero), 1: fine units.
    const int skip_at = (HOOK && cta == p.skip_cta) ? (int)p.skip_step : -1;      // self-test: the step at which this CTA withholds its publication
    auto gates_and_publish = [&](int half_g, long long s, int drawn, const GatePre &q) {
        const float xk = scale8(drawn);                  // the pending input
        const float u = sigmoidf_fast(fmaf(q.ku, xk, q.pu)), r = sigmoidf_fast(fmaf(q.kr, xk, q.pr));
        const float e = tanhf_fast(fmaf(r, q.ae, fmaf(q.ke, xk, q.pe)));
        const float hn = fmaf(u, half_g ? hF : hC, (1.0f - u) * e);
        if (half_g) hF = hn; else hC = hn;
        const int j = cta * UC + lane, jj = (half_g ? K : 0) + j;
        if (!HOOK || (int)s != skip_at)
            st_relaxed_u64(p.yslots + (size_t)((half_g ? 2 : 0) + (s & 1)) * K + j,
                           ((unsigned long long)(unsigned)(s + 1) << 32) | __float_as_uint(hn));
        if (p.dbg_gates) { float *d = p.dbg_gates + (size_t)s * 3 * H; d[jj] = u; d[H + jj] = r; d[2 * H + jj] = e; }
        if (p.dbg_h) p.dbg_h[(size_t)s * H + jj] = hn;
    };
    auto load_g = [&](int half_g, long long s, float (&gv)[3]) {
        const long long fr = ((p.step0 + s) * p.row_stride + (long long)p.stream0 * p.row_offset_mul) / p.hop;
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

    // all-gather of n (even) tagged words from the chip into a shared-memory vector: two adjacent slots per polling thread.
    // held_back (the exchange of the state, whose words this CTA's own gate threads publish at about the time every other
    // CTA's do): the drawing warp does not poll, and the pollers wait for the CTA's own publication plus poll_gap cycles, so
    // that the first poll reaches L2 when the words do (a poll that just misses them costs a whole round trip, and early
    // polls slow the publishing stores).  hs = the half-step index (parity of the publication barrier).
    auto gather = [&](const unsigned long long *slots, int n, unsigned want, float *dst, int step, int phase, bool held_back, long long hs) {
        const int first = held_back ? 32 : 0, np = (int)blockDim.x - first;
        if (tid >= first) {
            if (held_back) {
                unsigned cnt = 0; unsigned long long t0 = 0;
                while (!mbar_try_parity(smem_addr(&pub_bar), (unsigned)((hs - 1) & 1)))
                    if ((++cnt & 1023u) == 0 && wt.expired(t0, step, phase)) { my_bad = true; break; }
                const long long c0 = clock64();
                while (clock64() - c0 < p.poll_gap) { }
            }
#pragma unroll 1
            for (int i = tid - first; i < n / 2; i += np) {
                unsigned long long v0 = 0, v1 = 0, t0 = 0; unsigned cnt = 0;
                while (!my_bad) {
                    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v0), "=l"(v1) : "l"(slots + 2 * i) : "memory");
                    if ((unsigned)(v0 >> 32) == want && (unsigned)(v1 >> 32) == want) break;
                    if ((++cnt & 4095u) == 0 && wt.expired(t0, step, phase)) { my_bad = true; break; }
                }
                dst[2 * i] = __uint_as_float((unsigned)v0); dst[2 * i + 1] = __uint_as_float((unsigned)v1);
            }
        }
        return __syncthreads_or(my_bad) != 0;
    };
    const bool hold = p.poll_gap >= 0 && blockDim.x > 32;

    // Half-step n = 2 s + 1 is the "coarse" half of step s (input y_c(s): coarse head -> c_s; R[:, :Hh] y_c(s) kept for
    // step s+1; then the fine gates of step s); n = 2 s is the "fine" half (input y_f(s-1): fine head -> f_{s-1};
    // R[:, Hh:] y_f(s-1) completes R h_{s-1}; then the coarse gates of step s).
    const long long T = p.n_steps;
#pragma unroll 1
    for (long long n = 1; n <= 2 * T; ++n) {
        const int half = (int)(n & 1);
        const long long s = n >> 1;
        const bool last = n == 2 * T;
        const unsigned tag = (unsigned)n, par = (unsigned)((n - 1) & 1);
        float *vec = half ? vecC : vecF;

        float gv[3] = {0.f, 0.f, 0.f}, u01 = 0.f;
        int forced = -1;
        if (warp == 0) {
            if (lane < UC && !last) load_g(half, s, gv);
            if (half) { if (p.c_forced) forced = p.c_forced[s]; }
            else      { if (p.f_forced) forced = p.f_forced[s - 1]; }
            u01 = uniform24(p.seed, p.stream0, (unsigned long long)(p.step0 + (half ? s : s - 1)), half ? 0u : 1u);
        }

        // ---- 1. input half-vector from the whole chip (y_c(s) carries tag s+1; y_f(s-1) carries tag s)
        if (gather(p.yslots + (size_t)(half ? (s & 1) : 2 + ((s - 1) & 1)) * K, K, (unsigned)(half ? s + 1 : s), vec, (int)s, 1 + 4 * half, hold, n)) break;
        STAMP(0 + 6 * half);

        // ---- 2. this CTA's rows of the hidden layer and of R against the same input; publish the hidden-layer rows
        rows_times(half ? wA : wB, NS, vec);
        __syncthreads();
        STAMP(12 + half);
        stacked_finish(half ? sb1 : sb3, !half, p.qslots + (size_t)par * K, tag);
        STAMP(1 + 6 * half);

        // ---- 3. the whole hidden layer -> this CTA's rows of the logits, sent to every CTA of the cluster
        if (gather(p.qslots + (size_t)par * K, K, tag, qvec, (int)s, 2 + 4 * half, false, n)) break;
        STAMP(2 + 6 * half);
        rows_times(half ? wO2 : wO4, LR, qvec);
        __syncthreads();
        STAMP(14 + half);
        if (warp < CS) {
            const float *bl = half ? sb2 : sb4;
            for (int i = lane; i < LR / 2; i += 32) {
                const int r0 = 2 * i;
                const float v0 = bl[r0] + ((part[r0] + part[PR + r0]) + (part[2 * PR + r0] + part[3 * PR + r0]));
                const float v1 = bl[r0 + 1] + ((part[r0 + 1] + part[PR + r0 + 1]) + (part[2 * PR + r0 + 1] + part[3 * PR + r0 + 1]));
                st_cluster_ll(l_snd[par] + 16u * i, v0, v1, tag);
            }
        }
        STAMP(3 + 6 * half);

        // ---- 4. warp 0: the cluster's 256 logits -> draw; then the gates of the other half of the state
        if (warp == 0) {
            GatePre gp = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (lane < UC && !last) gp = gates_prepare(half, gv);
            float l[8];
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
            int drawn = warp_softmax_draw_fast(l, u01, lane);
            if (writer) {
                if (p.dbg_logits) {
                    float *d = p.dbg_logits + (size_t)(n - 1) * 256 + 8 * lane;
#pragma unroll
                    for (int k = 0; k < 8; ++k) d[k] = l[k];
                }
                if (lane == 0) {
                    if (half) { if (p.c_out) p.c_out[s] = (uint8_t)drawn; }
                    else      { if (p.f_out) p.f_out[s - 1] = (uint8_t)drawn; }
                }
            }
            if (forced >= 0) drawn = forced;
            if (!half) {
                if (writer && lane == 0 && p.out) p.out[s - 1] = (int16_t)(256 * c_prev + drawn - 32768);
                f_prev = drawn;
            }
            if (lane < UC && !last && !my_bad) gates_and_publish(half, s, drawn, gp);
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&pub_bar)) : "memory");
            if (half) c_prev = drawn;
        }
        STAMP(5 + 6 * half);
    }
    if (prof_on && lane == 0) for (int i = 0; i < 16; ++i) p.prof[i] = s_prof[i];
#undef STAMP

    // final state (vecC holds y_c(T-1); vecF was refreshed by the last fine half)
    const int any_bad = __syncthreads_or(my_bad);
    if (writer && !any_bad) {
        if (p.h_out) for (int i = tid; i < K; i += blockDim.x) { p.h_out[i] = vecC[i]; p.h_out[K + i] = vecF[i]; }
        if (tid == 0) {
            if (p.c_st_out) p.c_st_out[0] = (uint8_t)c_prev;
            if (p.f_st_out) p.f_st_out[0] = (uint8_t)f_prev;
        }
    }
    cluster.sync();     // nobody leaves while a peer may still write into its shared memory
}

// ---------------------------------------------------------------------------------------------
static size_t r16(size_t x) { return (x + 15) & ~(size_t)15; }

static int resf32_smem_bytes(const ResF32Pack &k)
{
    size_t b = k.blob_bytes;
    b += (size_t)3 * k.K * 4;          // vecC, vecF, qvec
    b += (size_t)4 * k.PR * 4;         // partial sums
    b += r16((size_t)2 * k.NR * 4);    // a_part, a_full
    b += 256 * 16;                     // lbuf [2][128] x 16 B
    return (int)r16(b);
}

// dense row `row` of a host block-row matrix -> fp32 values for columns [c0, c0 + n)
static void dense_row_f32(const BsrHost &M, int row, int c0, int n, float *dst)
{
    std::fill(dst, dst + n, 0.f);
    const int br = row / 4, r = row % 4;
    for (int i = M.row_ptr[br]; i < M.row_ptr[br + 1]; ++i) {
        const int cbase = 4 * (int)M.col[i];
        for (int c = 0; c < 4; ++c) {
            const int col = cbase + c;
            if (col >= c0 && col < c0 + n) dst[col - c0] = M.vals[(size_t)i * 16 + 4 * r + c];
        }
    }
}

static void fill_launch(const ResF32Pack &k, cudaLaunchConfig_t *cfg, cudaLaunchAttribute *at, cudaStream_t s, bool coop)
{
    std::memset(cfg, 0, sizeof(*cfg));
    cfg->gridDim = dim3(k.NCTA);
    cfg->blockDim = dim3(RF_THREADS);
    cfg->dynamicSmemBytes = k.smem_bytes;
    cfg->stream = s;
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = k.CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative;
    at[1].val.cooperative = 1;
    cfg->attrs = at;
    cfg->numAttrs = coop ? 2 : 1;
}

int resf32_supported(const wrnn_model *m, int batch, std::string *why)
{
    if (batch != 1) { if (why) *why = "resident kernel is single-stream (batch 1)"; return WRNN_ERR_UNSUPPORTED; }
    if (!m->resf32) { if (why) *why = "model was not packed for the fp32 resident kernel"; return WRNN_ERR_UNSUPPORTED; }
    return WRNN_OK;
}

// one launch attribute on all three instantiations of the kernel
static cudaError_t rf_set_attr(cudaFuncAttribute a, int v)
{
    cudaError_t e = cudaFuncSetAttribute(resident_f32_kernel<0>, a, v);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(resident_f32_kernel<1>, a, v);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(resident_f32_kernel<2>, a, v);
    return e;
}

int resf32_prepare(wrnn_model *m)
{
    const int H = m->H, K = H / 2;
    if (m->dtype != WRNN_F32 || m->sparse) { m->err = "fp32 resident kernel takes dense fp32 models"; return WRNN_ERR_UNSUPPORTED; }
    if (K % 16 != 0) { m->err = "H/2 must be a multiple of 16"; return WRNN_ERR_UNSUPPORTED; }
    cudaDeviceProp prop;
    cudaGetDeviceProperties(&prop, m->device);
    if (rf_set_attr(cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
        cudaGetLastError(); m->err = "cannot configure the fp32 resident kernel"; return WRNN_ERR_UNSUPPORTED;
    }
    // The largest number of CTAs that divides the half state, keeps a CTA's units within one warp, forms clusters (the
    // larger the cluster, the fewer rows of O2 / O4 each CTA holds), fits shared memory and can be co-resident.
    ResF32Pack k;
    for (int n = std::min(m->n_sms, K); n >= 1 && k.NCTA == 0; --n) {
        if (K % n != 0 || K / n > 32) continue;
        for (int cs = 16; cs >= 1; cs >>= 1) {
            if (n % cs != 0) continue;
            ResF32Pack c;
            c.NCTA = n; c.CS = cs; c.UC = K / n; c.K = K; c.NR = 6 * c.UC; c.LR = 256 / cs;
            c.PR = (std::max(7 * c.UC, c.LR) + 3) / 4 * 4;
            c.w_bytes = ((size_t)2 * 7 * c.UC + 2 * c.LR) * K * 4;
            c.blob_bytes = r16(c.w_bytes + ((size_t)c.NR * 3 + 2 * c.UC + 2 * c.LR) * 4);
            c.smem_bytes = resf32_smem_bytes(c);
            if ((size_t)c.smem_bytes + 1024 > prop.sharedMemPerBlockOptin) continue;
            if (rf_set_attr(cudaFuncAttributeMaxDynamicSharedMemorySize, c.smem_bytes) != cudaSuccess) { cudaGetLastError(); continue; }
            cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
            fill_launch(c, &cfg, at, 0, false);
            int max_clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&max_clusters, resident_f32_kernel<0>, &cfg) != cudaSuccess || max_clusters < n / cs) { cudaGetLastError(); continue; }
            k = c;
            break;
        }
    }
    if (k.NCTA == 0) { m->err = "no CTA count shards this model into the shared memory of the device"; return WRNN_ERR_UNSUPPORTED; }
    if (rf_set_attr(cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem_bytes) != cudaSuccess) {
        cudaGetLastError(); m->err = "cannot raise the dynamic shared memory limit"; return WRNN_ERR_UNSUPPORTED;
    }

    const int UC = k.UC, NR = k.NR, NS = 7 * k.UC, LR = k.LR;
    std::vector<uint8_t> blob((size_t)k.NCTA * k.blob_bytes, 0);
    const BsrHost *Oa[2] = {&m->hO1, &m->hO3}, *Ob[2] = {&m->hO2, &m->hO4};
    for (int cta = 0; cta < k.NCTA; ++cta) {
        const int rank = cta % k.CS;
        uint8_t *base = blob.data() + (size_t)cta * k.blob_bytes;
        float *w = reinterpret_cast<float *>(base);
        // stacked matrices: rows [0, UC) = this CTA's rows of O1 / O3; rows UC + rr, rr = (half * 3 + gate) * UC + u, = row
        // gate * H + half * K + cta * UC + u of R, columns [part * K, part * K + K)
        for (int part = 0; part < 2; ++part)
            for (int row = 0; row < NS; ++row) {
                float *dst = w + ((size_t)part * NS + row) * K;
                if (row < UC) dense_row_f32(*Oa[part], cta * UC + row, 0, K, dst);
                else {
                    const int rr = row - UC, half = rr / (3 * UC), gate = (rr / UC) % 3, u = rr % UC;
                    dense_row_f32(m->hR, gate * H + half * K + cta * UC + u, part * K, K, dst);
                }
            }
        // rows [rank LR, (rank + 1) LR) of the two logits matrices
        float *wl = w + (size_t)2 * NS * K;
        for (int h = 0; h < 2; ++h)
            for (int r = 0; r < LR; ++r) dense_row_f32(*Ob[h], rank * LR + r, 0, K, wl + ((size_t)h * LR + r) * K);
        float *sm = reinterpret_cast<float *>(base + k.w_bytes);
        for (int rr = 0; rr < NR; ++rr) {
            const int half = rr / (3 * UC), gate = (rr / UC) % 3, u = rr % UC;
            const int mrow = gate * H + half * K + cta * UC + u;
            for (int c = 0; c < 3; ++c) sm[rr * 3 + c] = m->hI[(size_t)mrow * 3 + c];
        }
        float *b = sm + NR * 3;
        for (int r = 0; r < UC; ++r) { b[r] = m->hb1[cta * UC + r]; b[UC + r] = m->hb3[cta * UC + r]; }
        b += 2 * UC;
        for (int r = 0; r < LR; ++r) { b[r] = m->hb2[rank * LR + r]; b[LR + r] = m->hb4[rank * LR + r]; }
    }
    ResF32Pack *pk = new ResF32Pack(k);
    const size_t n_slots = (size_t)6 * K;
    bool ok = cudaMalloc((void **)&pk->d_blob, blob.size()) == cudaSuccess &&
              cudaMemcpy(pk->d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice) == cudaSuccess &&
              cudaMalloc((void **)&pk->d_slots, n_slots * 8) == cudaSuccess &&
              cudaMalloc((void **)&pk->d_prof, 16 * sizeof(long long)) == cudaSuccess &&
              cudaMemset(pk->d_prof, 0, 16 * sizeof(long long)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        cudaFree(pk->d_blob); cudaFree(pk->d_slots); cudaFree(pk->d_prof);
        delete pk;
        m->err = "device allocation for the fp32 resident kernel failed";
        return WRNN_ERR_NOMEM;
    }
    // shared-memory bytes of weights read per step over the whole chip: R, O1, O3 once, O2 / O4 once per cluster
    pk->weight_bytes_per_step = ((int64_t)3 * H * H + 2 * (int64_t)K * K + (int64_t)(k.NCTA / k.CS) * 2 * 256 * K) * 4 + (int64_t)3 * H * 3 * 4;
    m->resf32 = pk;
    return WRNN_OK;
}

void resf32_destroy(wrnn_model *m)
{
    if (!m->resf32) return;
    cudaFree(m->resf32->d_blob);
    cudaFree(m->resf32->d_slots);
    cudaFree(m->resf32->d_prof);
    delete m->resf32;
    m->resf32 = nullptr;
}

int resf32_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes)
{
    (void)batch;
    const ResF32Pack &k = *m->resf32;
    if (n_ctas) *n_ctas = k.NCTA;
    if (n_threads) *n_threads = RF_THREADS;
    if (smem) *smem = k.smem_bytes;
    if (weight_bytes) *weight_bytes = k.weight_bytes_per_step;
    return WRNN_OK;
}

int resf32_phase_cycles(const wrnn_model *m, long long *out16)
{
    if (!m->resf32) return WRNN_ERR_UNSUPPORTED;
    return cudaMemcpy(out16, m->resf32->d_prof, 16 * sizeof(long long), cudaMemcpyDeviceToHost) == cudaSuccess ? WRNN_OK : WRNN_ERR_CUDA;
}

int resf32_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    const ResF32Pack &k = *m->resf32;
    ResF32Params p;
    std::memset(&p, 0, sizeof(p));
    p.H = m->H; p.K = k.K; p.UC = k.UC; p.NR = k.NR; p.NCTA = k.NCTA; p.CS = k.CS; p.LR = k.LR; p.PR = k.PR;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.blob = k.d_blob; p.blob_bytes = k.blob_bytes; p.w_bytes = k.w_bytes;
    p.g = m->g;
    p.yslots = k.d_slots; p.qslots = k.d_slots + (size_t)4 * k.K;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in; p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.status = m->status;
    { const char *e = getenv("WRNN_F32_POLL_GAP"); p.poll_gap = e ? atoi(e) : 0; }
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;
    p.prof = m->prof_enabled ? k.d_prof : nullptr;     // phase stamps cost the stamped warp some 50 cycles each: off unless asked for

    if (cudaMemsetAsync(k.d_slots, 0, (size_t)6 * k.K * 8, s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
    // The cooperative attribute makes the driver refuse the launch unless all clusters can be co-resident.
    // WRNN_NO_COOP=1 drops it (co-residency was already checked against the occupancy API at create):
    // a profiler that replays kernels may not accept cooperative cluster launches.
    fill_launch(k, &cfg, at, s, coop_launch_allowed());
    const cudaError_t e = m->dbg_skip_cta >= 0 ? cudaLaunchKernelEx(&cfg, resident_f32_kernel<1>, p)
                          : p.prof          ? cudaLaunchKernelEx(&cfg, resident_f32_kernel<2>, p)
                                            : cudaLaunchKernelEx(&cfg, resident_f32_kernel<0>, p);
    if (e != cudaSuccess) {
        m->err = std::string("fp32 resident kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    return WRNN_OK;
}

}  // namespace wrnn
