// Block-sparse single-stream sampling kernel (Section 3: only the kept 4x4 blocks of R_u, R_r, R_e, O1, O3
// are stored and multiplied): bf16 weights, batch 1, the whole model resident in the shared memory of NC
// thread-block clusters of 16 CTAs (NC = 4 where they can be co-resident).
//
// A pruned model is small (H = 2048 at 96 %: 2.3 MB of blocks, plus the dense O2 / O4).  The compressed block rows of R
// are dealt over all NC x 16 CTAs; the heads are held once per cluster, so that the hidden layer of a head and its
// logits are all-gathers through the distributed shared memory of a cluster (asynchronous stores that count their bytes
// on an mbarrier of the receiver); the two halves of the state cross the chip as tagged words in L2 (arrival of the data is
// the signal).
// Each CTA owns Hh/(16 NC) coarse and as many fine units (their block rows of R, compressed: block column index +
// 16 bf16 per kept block), Hh/16 rows of O1 and O3 (compressed block rows) and 16 rows of the dense O2 and O4
// (row-major bf16, multiplied as fp32 FMAs on the received hidden layer: 16 warps = 4 groups of four rows x 4 quarters of K).
// Sparse rows: four (or eight) lanes share a block row, each lane takes every fourth (eighth) kept block (two 16-byte weight
// loads, four activations, 16 FMAs), a four-value reduce-scatter finishes the rows; the rows are sorted by length and stored
// sliced by warp so that every shared-memory load of a warp is one contiguous run; with four clusters the hidden-layer rows sit
// in the slices of warps 0..3 and the rows of R in those of warps 16..19, which the exchanges do not wait for.
// The step itself is the two-half schedule of the dense resident kernel (Fig. 1's order).
//
// Every wait is bounded; all CTAs leave through the final cluster barrier.
#include <cooperative_groups.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>

#include "wrnn_cluster.cuh"
#include "wrnn_internal.h"

namespace cg = cooperative_groups;

namespace wrnn {

constexpr int SCS = 16;          // cluster size
constexpr int SNW = 20;          // warps per CTA

// Compressed block rows of one phase of one CTA, sliced by warp: the block rows are sorted by their number of kept
// blocks and dealt out in runs to the warps; the longest rows get eight lanes each (four rows per warp), the others
// four (eight rows per warp), as many eight-lane warps as the CTA's lanes allow.  Lane lpr g + l of warp w takes
// blocks l, l + lpr, ... of its row g.  Iteration t of a warp reads slot t * nl + lane of its slice (nl = lanes in
// use): the two 16-byte halves of the block's weights from two planes and the block column, so every load of a warp is
// one contiguous run; rows shorter than the warp's longest are padded with zero blocks.
struct SliceMeta { int voff, coff, T, nl, lpr, pad[3]; int16_t row[8]; };   // offsets in 16-byte / 2-byte units from the phase's arrays

struct SparsePack {
    int H = 0, K = 0, NKT = 0, UC = 0, HR = 0, NBR = 0;   // NBR: block rows per phase = (HR + 6 UC) / rows of a block
    int WH = 0;                       // > 0: split layout (hidden-layer block rows in the slices of warps [0, WH), rows of R in those of warps 16..19)
    int NC = 1;                       // clusters: the rows of R are dealt over NC x 16 CTAs, the heads once per cluster
    unsigned long long *d_slots = nullptr;   // [4][K] exchange slots of the state halves
    int tall = 0;                     // 16 x 1 blocks (else 4 x 4)
    int max_slots = 0;                // block slots per phase per CTA (kept blocks + padding of the sliced layout, maximum)
    size_t blob_bytes = 0;            // per CTA
    size_t off_meta[2], off_col[2], off_val[2], off_o2 = 0, off_o4 = 0, off_small = 0;
    uint8_t *d_blob = nullptr;
    int smem_bytes = 0;
    int64_t weight_bytes_per_step = 0;   // kept blocks + indices + row pointers + dense O2/O4/I, each counted once
};

struct SparseParams {
    int WH;                                  // > 0: split layout, the sending warps do not wait for the rows of R
    int H, K, NKT, UC, HR, NBR, tall;        // tall: blocks are 16 x 1 (16 rows of one column) instead of 4 x 4
    unsigned long long *yslots;              // [2 halves][2 parities][K] (value, tag): the state crosses the chip when there is more than one cluster
    unsigned long long off_meta[2], off_col[2], off_val[2], off_o2, off_o4, off_small, blob_bytes;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    const uint8_t *blob;
    const float *g;
    const float *h_in; float *h_out;
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;
    uint8_t *c_out, *f_out;
    int16_t *out;
    float *dbg_gates, *dbg_h, *dbg_logits;
    DevStatus *status;
    unsigned long long limit_ns;
    int skip_cta; long long skip_step;      // self-test: this CTA withholds what it publishes at this step (-1: none)
    int poll_gap;                           // cycles the state pollers hold back after the CTA's own publication (-1: poll at once, all warps)
};

#ifdef WRNN_PROFILE_SPARSE
__device__ long long g_sprof[16];
#define SSTAMP(i) do { if (warp == 0) { const long long n_ = clock64(); if (lane == 0) s_sprof[i] += n_ - st_; st_ = n_; } } while (0)
#else
#define SSTAMP(i) do { } while (0)
#endif

// NKL: k-tiles of the logits tile per warp (K / 16 / NKL warps split K).
// MODE 0: plain sampling (no forced symbols, no dumps, no self-test predicate: what wrnn_sample runs); MODE 1: the instantiation
// that wrnn_selftest_lost_word runs (one CTA withholds one publication); MODE 3: teacher forcing and dumps (modes 1 and 3 take both)
template <int NKL, int MODE>
__global__ void __launch_bounds__(SNW * 32, 1) sparse_cluster_kernel(const SparseParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();      // owner index of head rows and logits (per cluster)
    const int cta = blockIdx.x;                      // owner index of state units and their rows of R (whole grid)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = p.K, UC = p.UC, HR = p.HR, H = p.H;
    const int NR = 6 * UC;

    // ---- shared memory carve-up (must match sparse_smem_bytes)
    const SliceMeta *smeta[2] = {reinterpret_cast<const SliceMeta *>(smem + p.off_meta[0]), reinterpret_cast<const SliceMeta *>(smem + p.off_meta[1])};
    const uint16_t *bcol[2] = {reinterpret_cast<const uint16_t *>(smem + p.off_col[0]), reinterpret_cast<const uint16_t *>(smem + p.off_col[1])};
    const uint4 *bval[2] = {reinterpret_cast<const uint4 *>(smem + p.off_val[0]), reinterpret_cast<const uint4 *>(smem + p.off_val[1])};
    const unsigned *wO2 = reinterpret_cast<const unsigned *>(smem + p.off_o2), *wO4 = reinterpret_cast<const unsigned *>(smem + p.off_o4);   // [16 rows][K / 2] bf16 pairs
    const float *sI = reinterpret_cast<const float *>(smem + p.off_small);            // [NR][3]
    const float *sb1 = sI + NR * 3, *sb3 = sb1 + HR, *sb2 = sb3 + HR, *sb4 = sb2 + 16;
    float *vecC = reinterpret_cast<float *>(smem + p.blob_bytes);                     // [K] y_c
    float *vecF = vecC + K;                                                           // [K] y_f
    float *qvec = vecF + K;                                                           // [K] hidden layer
    float *a_part = qvec + K;                                                         // [NR]
    float *a_full = a_part + NR;                                                      // [NR]
    float *part = a_full + NR;                                                        // [16 warps][16]
    float *qall = part + 256;                                                         // [2 parities][K] the cluster's hidden layer, written by the peers' asynchronous stores
    // Cluster exchange buffers, one of each: a peer can only write the next half-step's words after it has received
    // words that this CTA sent after reading the current ones (q(n+1) follows y(n+1), which follows this CTA's draw from
    // logits(n); logits(n+1) follow q(n+1)).
    uint4 *qbuf = reinterpret_cast<uint4 *>(qall + 2 * K);                            // [K/2] hidden layer
    float *lall = reinterpret_cast<float *>(qbuf + K / 2);                            // [2 parities][256] logits of the cluster

    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.blob + (size_t)cta * p.blob_bytes);
        uint4 *dst = reinterpret_cast<uint4 *>(smem);
        for (size_t i = tid; i < p.blob_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
        for (int i = tid; i < K; i += blockDim.x) {
            vecC[i] = p.h_in ? p.h_in[i] : 0.f;
            vecF[i] = p.h_in ? p.h_in[K + i] : 0.f;
        }
    }
    __syncthreads();
    cluster.sync();

    constexpr bool HOOK = MODE == 1, DBG = MODE != 0;
    Waiter wt{p.status, p.limit_ns};
    bool my_bad = false;
    const bool writer = (cta == 0);
    __shared__ __align__(8) unsigned long long pub_bar;      // one phase per half-step: this CTA's gate warps have published
    __shared__ __align__(8) unsigned long long xq[2], xl[2]; // arrival barriers of qall[.] and lall[.]: the peers' stores count their bytes here
    if (tid == 0) {
        mbar_init_cluster(smem_addr(&pub_bar), (unsigned)((p.UC + 31) / 32));
        mbar_init_cluster(smem_addr(&xq[0]), 1); mbar_init_cluster(smem_addr(&xq[1]), 1);
        mbar_init_cluster(smem_addr(&xl[0]), 1); mbar_init_cluster(smem_addr(&xl[1]), 1);
        mbar_fence_init();
    }
    __syncthreads();
    cluster.sync();      // every peer's barriers are initialised before anyone sends
#ifdef WRNN_PROFILE_SPARSE
    __shared__ long long s_sprof[16];
    long long st_ = clock64();
#endif

    int c_prev = p.c_in ? p.c_in[0] : 128, f_prev = p.f_in ? p.f_in[0] : 0;

    // ---- sparse phase: block rows [0, NBR) of phase ph (0: input y_c -> [O1 ; R x coarse cols], 1: y_f -> [O3 ; R x fine cols]).
    // Four lanes per block row.  Rows [0, HR) are hidden-layer rows (bias, relu, sent to all peers when send != 0),
    // rows [HR, HR + NR) are this CTA's R rows (ph 1 completes R h, ph 0 keeps the partial for the next step).
    // this warp's slices of the two phases: constants of the whole call, kept in registers
    const SliceMeta &sm0 = smeta[0][warp], &sm1 = smeta[1][warp];
    const int sl_nl0 = sm0.nl, sl_nl1 = sm1.nl, sl_T0 = sm0.T, sl_T1 = sm1.T;
    const uint4 *sl_wv0 = bval[0] + sm0.voff + (lane < sl_nl0 ? lane : 0), *sl_wv1 = bval[1] + sm1.voff + (lane < sl_nl1 ? lane : 0);
    const uint16_t *sl_wc0 = bcol[0] + sm0.coff + (lane < sl_nl0 ? lane : 0), *sl_wc1 = bcol[1] + sm1.coff + (lane < sl_nl1 ? lane : 0);
    const bool tall = p.tall != 0;
    const int lpr_n = tall ? 16 : 4;                                    // lanes per block row, narrow slices
    const bool sl_wide0 = sm0.lpr == 2 * lpr_n, sl_wide1 = sm1.lpr == 2 * lpr_n;   // twice as many lanes per block row
    // the block row this lane finishes (the first lpr_n lanes of a row's lanes hold its sums after the reduction)
    const int sl_sh = tall ? 4 : 2;
    const int sl_row0 = (lane < sl_nl0 && (!sl_wide0 || (lane & lpr_n) == 0)) ? (int)sm0.row[lane >> (sl_sh + (sl_wide0 ? 1 : 0))] : -1;
    const int sl_row1 = (lane < sl_nl1 && (!sl_wide1 || (lane & lpr_n) == 0)) ? (int)sm1.row[lane >> (sl_sh + (sl_wide1 ? 1 : 0))] : -1;

    auto sparse_phase = [&](int ph, const float *x, const float *bias) {
        const int nl = ph ? sl_nl1 : sl_nl0, T = ph ? sl_T1 : sl_T0, l4 = lane & 3;
        if (nl == 0) return;                       // a warp without block rows (few rows per CTA): its slice has no slots to read
        const uint4 *wv = ph ? sl_wv1 : sl_wv0;
        const uint16_t *wc = ph ? sl_wc1 : sl_wc0;
        if (tall) {
            // 16 x 1 blocks (Section 3.2): one activation per block, sixteen row sums per lane
            float a16[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) a16[j] = 0.f;
            uint4 w0 = wv[0], w1 = wv[nl];
            int c = wc[0];
            for (int t = 0; t < T; ++t) {
                const float xs = x[c];
                const int tn = t + 1 < T ? t + 1 : t;
                const uint4 w0n = wv[(2 * tn) * nl], w1n = wv[(2 * tn + 1) * nl];
                const int cn = wc[tn * nl];
                a16[0] = fmaf(bf16lo(w0.x), xs, a16[0]);   a16[1] = fmaf(bf16hi(w0.x), xs, a16[1]);
                a16[2] = fmaf(bf16lo(w0.y), xs, a16[2]);   a16[3] = fmaf(bf16hi(w0.y), xs, a16[3]);
                a16[4] = fmaf(bf16lo(w0.z), xs, a16[4]);   a16[5] = fmaf(bf16hi(w0.z), xs, a16[5]);
                a16[6] = fmaf(bf16lo(w0.w), xs, a16[6]);   a16[7] = fmaf(bf16hi(w0.w), xs, a16[7]);
                a16[8] = fmaf(bf16lo(w1.x), xs, a16[8]);   a16[9] = fmaf(bf16hi(w1.x), xs, a16[9]);
                a16[10] = fmaf(bf16lo(w1.y), xs, a16[10]); a16[11] = fmaf(bf16hi(w1.y), xs, a16[11]);
                a16[12] = fmaf(bf16lo(w1.z), xs, a16[12]); a16[13] = fmaf(bf16hi(w1.z), xs, a16[13]);
                a16[14] = fmaf(bf16lo(w1.w), xs, a16[14]); a16[15] = fmaf(bf16hi(w1.w), xs, a16[15]);
                w0 = w0n; w1 = w1n; c = cn;
            }
            if (ph ? sl_wide1 : sl_wide0) {
#pragma unroll
                for (int j = 0; j < 16; ++j) a16[j] += __shfl_xor_sync(FULL, a16[j], 16);
            }
            // sixteen row sums over sixteen lanes: four transposing steps leave row l in lane l of the row's lanes
            float a8[8], a4[4], a2[2];
            const bool u8 = (lane & 8) != 0, u4 = (lane & 4) != 0, u2 = (lane & 2) != 0, u1 = (lane & 1) != 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) a8[j] = (u8 ? a16[8 + j] : a16[j]) + __shfl_xor_sync(FULL, u8 ? a16[j] : a16[8 + j], 8);
#pragma unroll
            for (int j = 0; j < 4; ++j) a4[j] = (u4 ? a8[4 + j] : a8[j]) + __shfl_xor_sync(FULL, u4 ? a8[j] : a8[4 + j], 4);
#pragma unroll
            for (int j = 0; j < 2; ++j) a2[j] = (u2 ? a4[2 + j] : a4[j]) + __shfl_xor_sync(FULL, u2 ? a4[j] : a4[2 + j], 2);
            const float v = (u1 ? a2[1] : a2[0]) + __shfl_xor_sync(FULL, u1 ? a2[0] : a2[1], 1);
            const int lbr = ph ? sl_row1 : sl_row0;
            if (lbr >= 0) {
                const int row = 16 * lbr + (lane & 15);
                if (row < HR) qvec[row] = fmaxf(v + bias[row], 0.f);
                else if (ph) a_full[row - HR] = a_part[row - HR] + v;
                else a_part[row - HR] = v;
            }
            return;
        }
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        SSTAMP(9);
        // software pipeline: the weights and the column of the next block are in flight while this block's four
        // activations are gathered and multiplied (the last prefetch re-reads the last slot)
        uint4 w0 = wv[0], w1 = wv[nl];
        int c = wc[0];
        for (int t = 0; t < T; ++t) {
            const float4 xv = *reinterpret_cast<const float4 *>(x + 4 * c);
            const int tn = t + 1 < T ? t + 1 : t;
            const uint4 w0n = wv[(2 * tn) * nl], w1n = wv[(2 * tn + 1) * nl];
            const int cn = wc[tn * nl];
            acc[0] = fmaf(bf16lo(w0.x), xv.x, fmaf(bf16hi(w0.x), xv.y, fmaf(bf16lo(w0.y), xv.z, fmaf(bf16hi(w0.y), xv.w, acc[0]))));
            acc[1] = fmaf(bf16lo(w0.z), xv.x, fmaf(bf16hi(w0.z), xv.y, fmaf(bf16lo(w0.w), xv.z, fmaf(bf16hi(w0.w), xv.w, acc[1]))));
            acc[2] = fmaf(bf16lo(w1.x), xv.x, fmaf(bf16hi(w1.x), xv.y, fmaf(bf16lo(w1.y), xv.z, fmaf(bf16hi(w1.y), xv.w, acc[2]))));
            acc[3] = fmaf(bf16lo(w1.z), xv.x, fmaf(bf16hi(w1.z), xv.y, fmaf(bf16lo(w1.w), xv.z, fmaf(bf16hi(w1.w), xv.w, acc[3]))));
            w0 = w0n; w1 = w1n; c = cn;
        }
        SSTAMP(10);
        if (ph ? sl_wide1 : sl_wide0) {
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[j] += __shfl_xor_sync(FULL, acc[j], 4);
        }
        // four row sums over four lanes: two transposing steps leave row l4 in lane l4
        const bool up2 = (l4 & 2) != 0;
        const float s0 = up2 ? acc[0] : acc[2], k0 = up2 ? acc[2] : acc[0];
        const float s1 = up2 ? acc[1] : acc[3], k1 = up2 ? acc[3] : acc[1];
        const float t0 = k0 + __shfl_xor_sync(FULL, s0, 2);
        const float t1 = k1 + __shfl_xor_sync(FULL, s1, 2);
        const bool up1 = (l4 & 1) != 0;
        const float v = (up1 ? t1 : t0) + __shfl_xor_sync(FULL, up1 ? t0 : t1, 1);
        const int lbr = ph ? sl_row1 : sl_row0;
        if (lbr >= 0) {
            const int row = 4 * lbr + l4;
            if (row < HR) qvec[row] = fmaxf(v + bias[row], 0.f);
            else if (ph) a_full[row - HR] = a_part[row - HR] + v;
            else a_part[row - HR] = v;
        }
    };

    // Gates of Eq. 2 for this CTA's UC units of one half, then publish them to the whole grid.  The first GW warps (one
    // per 32 units: the fewer warps poll the logits buffer, the sooner the logits land) each draw the sample
    // redundantly (same logits, same uniform, same instructions -> same value) and then gate UC / GW units each.
    const int GW = (UC + 31) / 32;
    const int UW = UC / GW;
    auto load_g = [&](int half_g, long long s, float (&gv)[3]) {
        const long long fr = ((p.step0 + s) * p.row_stride + (long long)p.stream0 * p.row_offset_mul) / p.hop;
        const float *g = p.g + (size_t)fr * 3 * H + (half_g ? K : 0) + cta * UC + warp * UW + lane;
#pragma unroll
        for (int gate = 0; gate < 3; ++gate) gv[gate] = __ldg(g + gate * H);
    };
    // The gate pre-activations up to the one input that is only known after the draw (c_s for the fine units, f_{s-1} for
    // the coarse units of the next step): computed while the logits are still on their way.
    struct GatePre { float pu, pr, pe, ae, ku, kr, ke, hprev; };
    auto gates_prepare = [&](int half_g, const float (&gv)[3]) {
        GatePre q = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (lane < UW) {
            const int rb = half_g ? 3 * UC : 0, u0 = warp * UW + lane;
            const float x0 = scale8(c_prev), x1 = scale8(f_prev);
            const float *Iu = sI + 3 * (rb + u0), *Ir = sI + 3 * (rb + UC + u0), *Ie = sI + 3 * (rb + 2 * UC + u0);
            q.pu = a_full[rb + u0] + fmaf(Iu[0], x0, half_g ? fmaf(Iu[1], x1, gv[0]) : gv[0]);
            q.pr = a_full[rb + UC + u0] + fmaf(Ir[0], x0, half_g ? fmaf(Ir[1], x1, gv[1]) : gv[1]);
            q.pe = fmaf(Ie[0], x0, half_g ? fmaf(Ie[1], x1, gv[2]) : gv[2]);
            q.ae = a_full[rb + 2 * UC + u0];
            q.ku = half_g ? Iu[2] : Iu[1]; q.kr = half_g ? Ir[2] : Ir[1]; q.ke = half_g ? Ie[2] : Ie[1];
            q.hprev = (half_g ? vecF : vecC)[cta * UC + u0];       // previous value of the unit: still in the fp32 vector of that half
        }
        return q;
    };
    const int skip_at = (HOOK && cta == p.skip_cta) ? (int)p.skip_step : -1;      // self-test: the step at which this CTA withholds its publication
    auto gates = [&](int half_g, long long s, int drawn, const GatePre &q) {
        if (lane < UW) {
            const int u0 = warp * UW + lane;
            const float xk = scale8(drawn);              // the pending input
            const float u = sigmoidf_fast(fmaf(q.ku, xk, q.pu)), r = sigmoidf_fast(fmaf(q.kr, xk, q.pr));
            const float e = tanhf_fast(fmaf(r, q.ae, fmaf(q.ke, xk, q.pe)));
            const float hn = fmaf(u, q.hprev, (1.0f - u) * e);
            // published to the whole chip: arrival of the tagged value is the signal (two-deep by step parity)
            if (!HOOK || (int)s != skip_at)
                st_relaxed_u64(p.yslots + (size_t)((half_g ? 2 : 0) + (s & 1)) * K + cta * UC + u0,
                               ((unsigned long long)(unsigned)(s + 1) << 32) | __float_as_uint(hn));
            const int jj = (half_g ? K : 0) + cta * UC + u0;
            if (DBG && p.dbg_gates) { float *d = p.dbg_gates + (size_t)s * 3 * H; d[jj] = u; d[H + jj] = r; d[2 * H + jj] = e; }
            if (DBG && p.dbg_h) p.dbg_h[(size_t)s * H + jj] = hn;
        }
    };
    // ---- prologue: R h of step 0 from the initial state, coarse gates of step 0
    sparse_phase(0, vecC, sb1);
    __syncthreads();
    sparse_phase(1, vecF, sb3);
    __syncthreads();
    if (warp < GW) {
        float gv0[3] = {0.f, 0.f, 0.f};
        if (lane < UW) load_g(0, 0, gv0);
        gates(0, 0, f_prev, gates_prepare(0, gv0));
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&pub_bar)) : "memory");
    }


#ifdef WRNN_PROFILE_SPARSE
    if (tid < 16) s_sprof[tid] = 0;
    __syncthreads();
    st_ = clock64();
#endif
    const long long T = p.n_steps;
#pragma unroll 1
    for (long long n = 1; n <= 2 * T; ++n) {
        const int half = (int)(n & 1);                 // 1: coarse half (input y_c(s)), 0: fine half (input y_f(s-1))
        const long long s = n >> 1;
        const bool last = n == 2 * T;
        float *vec = half ? vecC : vecF;

        const unsigned par = (unsigned)((n - 1) & 1), use = (unsigned)((n - 1) >> 1);
        if (tid == 0) {
            mbar_arrive_expect(smem_addr(&xq[par]), (unsigned)K * 4u);      // this half-step's arrivals: K hidden values
            mbar_arrive_expect(smem_addr(&xl[par]), 256u * 4u);             // and 256 logits
        }
        float u01 = 0.f, gv[3] = {0.f, 0.f, 0.f};
        int forced = -1;
        if (warp < GW) {
            if (lane < UW && !last) load_g(half, s, gv);
            if (DBG) {
                if (half) { if (p.c_forced) forced = p.c_forced[s]; }
                else      { if (p.f_forced) forced = p.f_forced[s - 1]; }
            }
            u01 = uniform24(p.seed, p.stream0, (unsigned long long)(p.step0 + (half ? s : s - 1)), half ? 0u : 1u);
        }

        // ---- 1. the input half of the state from the whole grid (y_c(s) carries tag s + 1, y_f(s-1) tag s): two adjacent
        // slots per polling thread
        {
            const unsigned long long *slots = p.yslots + (size_t)(half ? (s & 1) : 2 + ((s - 1) & 1)) * K;
            const unsigned ytag = (unsigned)(half ? s + 1 : s);
            // Polls that come before the data only load the L2 slices the publishing stores have to get through, and a poll
            // that just misses the data costs a whole round trip: the pollers (every warp but the drawing ones, which have
            // the longest way to the end of the half-step) hold back until this CTA's own gate warps have published (all
            // CTAs publish at about the same time) plus poll_gap cycles.
            const bool held = p.poll_gap >= 0;
            const int first = held ? 32 * GW : 0, stride = (int)blockDim.x - first;
            if (tid >= first) {
                if (held) {
                    unsigned long long t0 = 0; unsigned cnt = 0;
                    while (!mbar_try_parity(smem_addr(&pub_bar), (unsigned)((n - 1) & 1)))
                        if ((++cnt & 1023u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
                    const long long c0 = clock64();
                    while (clock64() - c0 < p.poll_gap) { }
                }
#pragma unroll 1
                for (int i = tid - first; i < K / 2 && !my_bad; i += stride) {
                    unsigned long long v0, v1, t0 = 0; unsigned cnt = 0;
                    while (true) {
                        asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v0), "=l"(v1) : "l"(slots + 2 * i) : "memory");
                        if ((unsigned)(v0 >> 32) == ytag && (unsigned)(v1 >> 32) == ytag) break;
                        if ((++cnt & 4095u) == 0 && wt.expired(t0, (int)s, 1 + 4 * half)) { my_bad = true; break; }
                    }
                    vec[2 * i] = __uint_as_float((unsigned)v0); vec[2 * i + 1] = __uint_as_float((unsigned)v1);
                }
            }
        }
        if (__syncthreads_or(my_bad)) break;
        SSTAMP(0);

        // ---- 2. hidden layer of the head + this CTA's R rows (compressed block rows)
        sparse_phase(half ? 0 : 1, vec, half ? sb1 : sb3);
        SSTAMP(7);
        // Split layout (WH > 0): the hidden-layer block rows sit in the slices of warps [0, WH), the rows of R in those of warps
        // 16..19, which take no part in the exchanges or the output rows: the sixteen sending warps meet at a barrier of their
        // own while the rows of R, which nobody needs before the gates, are still being computed.  Warp w sends this CTA's HR
        // values to peer w (asynchronous stores that count their bytes on the receiver's barrier of that buffer: no tags,
        // no polling pass; one remote store instruction per warp: a second one from the same warp waits for the first).
        if (p.WH > 0) { if (warp < SCS) asm volatile("bar.sync 1, 512;" ::: "memory"); }
        else __syncthreads();
        SSTAMP(8);
        if (warp < SCS) {
            const unsigned bar = map_to_rank(smem_addr(&xq[par]), warp);
            for (int pr2 = lane; pr2 < HR / 2; pr2 += 32) {
                const unsigned a = map_to_rank(smem_addr(qall + (size_t)par * K + rank * HR + 2 * pr2), warp);
                st_async_v2(a, qvec[2 * pr2], qvec[2 * pr2 + 1], bar);
            }
        }
        SSTAMP(1);

        // ---- 3. the cluster's hidden layer -> 16 logits rows of this CTA
        SSTAMP(2);
        // the 16 output-layer rows in fp32 FMAs on 16 warps: warp w takes rows 4 (w & 3) .. + 3 over quarter w >> 2 of the
        // element pairs; a lane takes pairs lane, lane + 32, ... of its quarter (a pass costs a warp some 75 cycles whatever
        // it computes, so the passes are spread over all warps: four each at K = 1024); every pair of the hidden layer is
        // loaded once per four rows.  The four partial sums of a row meet in `part`.
        if (warp < 16) {
#ifdef WRNN_PROFILE_SPARSE
            const long long rt0_ = clock64();
#endif
            {
                unsigned long long t0 = 0; unsigned cnt = 0;
                while (!mbar_try_parity(smem_addr(&xq[par]), use & 1u))
                    if ((++cnt & 1023u) == 0 && wt.expired(t0, (int)s, 2 + 4 * half)) { my_bad = true; break; }
            }
            const int r0 = 4 * (warp & 3), kq = warp >> 2;
            const int Kp = K / 2, Q = Kp / 4;               // element pairs of a row and of a quarter (Q is a multiple of 64 at K = 1024)
            float a[4][2] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
#ifdef WRNN_PROFILE_SPARSE
            const long long rt1_ = clock64();
            if (warp == 4 && lane == 0) s_sprof[12] += rt1_ - rt0_;
#endif
            // in every run of 64 pairs a lane takes pairs 2 l and 2 l + 1: one 16-byte load of the hidden layer, one 8-byte load
            // of each row's weights (all of them conflict-free), issued for the whole quarter before the first FMA
            {
                const float4 *q4 = reinterpret_cast<const float4 *>(qall + (size_t)par * K) + (size_t)kq * (Q / 2) + lane;
                const uint2 *w2 = reinterpret_cast<const uint2 *>((half ? wO2 : wO4) + (size_t)r0 * Kp + (size_t)kq * Q) + lane;
                for (int c0 = 0; c0 < Q / 64; c0 += 2) {
                    float4 q[2];
                    uint2 x[2][4];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        q[u] = q4[32 * (c0 + u)];
#pragma unroll
                        for (int r = 0; r < 4; ++r) x[u][r] = w2[(size_t)r * (Kp / 2) + 32 * (c0 + u)];
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u)
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            a[r][0] = fmaf(bf16lo(x[u][r].x), q[u].x, a[r][0]); a[r][1] = fmaf(bf16hi(x[u][r].x), q[u].y, a[r][1]);
                            a[r][0] = fmaf(bf16lo(x[u][r].y), q[u].z, a[r][0]); a[r][1] = fmaf(bf16hi(x[u][r].y), q[u].w, a[r][1]);
                        }
                }
            }
#ifdef WRNN_PROFILE_SPARSE
            const long long rt2_ = clock64();
            if (warp == 4 && lane == 0) s_sprof[13] += rt2_ - rt1_;
#endif
            // four sums across the warp: two transposing steps leave row (lane >> 3) & 3 in every lane, three more finish it
            float v4[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) v4[r] = a[r][0] + a[r][1];
            const bool u16 = (lane & 16) != 0, u8 = (lane & 8) != 0;
            const float t0 = (u16 ? v4[2] : v4[0]) + __shfl_xor_sync(FULL, u16 ? v4[0] : v4[2], 16);
            const float t1 = (u16 ? v4[3] : v4[1]) + __shfl_xor_sync(FULL, u16 ? v4[1] : v4[3], 16);
            float v = (u8 ? t1 : t0) + __shfl_xor_sync(FULL, u8 ? t0 : t1, 8);
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
            const int rr = r0 + (u16 ? 2 : 0) + (u8 ? 1 : 0);
            if ((lane & 7) == 0) part[kq * 16 + rr] = v;
#ifdef WRNN_PROFILE_SPARSE
            if (warp == 4 && lane == 0) s_sprof[11] += clock64() - rt0_;
#endif
        }
        if (__syncthreads_or(my_bad)) break;
        SSTAMP(3);
        // 16 logits of this CTA: warp w sums the four partials of two rows per lane and sends the eight pairs to peer w
        if (warp < SCS && lane < 8) {
            const int r = 2 * lane;
            const float *bl = half ? sb2 : sb4;
            const float v0 = bl[r] + (part[r] + part[16 + r]) + (part[32 + r] + part[48 + r]);
            const float v1 = bl[r + 1] + (part[r + 1] + part[17 + r]) + (part[33 + r] + part[49 + r]);
            st_async_v2(map_to_rank(smem_addr(lall + (size_t)par * 256 + rank * 16 + r), warp), v0, v1, map_to_rank(smem_addr(&xl[par]), warp));
        }

        // ---- 4. warps 0..GW-1: the cluster's 256 logits -> draw; then the gates of the other half, published to the cluster
        if (warp < GW) {
            const GatePre gp = gates_prepare(half, gv);
            float l[8];
            {
                unsigned long long t0 = 0; unsigned cnt = 0;
                while (!mbar_try_parity(smem_addr(&xl[par]), use & 1u))
                    if ((++cnt & 1023u) == 0 && wt.expired(t0, (int)s, 3 + 4 * half)) { my_bad = true; break; }
                const float4 a = reinterpret_cast<const float4 *>(lall + (size_t)par * 256)[2 * lane];
                const float4 b = reinterpret_cast<const float4 *>(lall + (size_t)par * 256)[2 * lane + 1];
                l[0] = a.x; l[1] = a.y; l[2] = a.z; l[3] = a.w; l[4] = b.x; l[5] = b.y; l[6] = b.z; l[7] = b.w;
            }
            my_bad = __any_sync(FULL, my_bad);
            SSTAMP(4);
            int drawn = warp_softmax_draw_scan(l, u01, lane);
            if (writer && warp == 0) {
                if (DBG && p.dbg_logits) {
                    float *d = p.dbg_logits + (size_t)(n - 1) * 256 + 8 * lane;
#pragma unroll
                    for (int k = 0; k < 8; ++k) d[k] = l[k];
                }
                if (lane == 0) {
                    if (half) { if (p.c_out) p.c_out[s] = (uint8_t)drawn; }
                    else      { if (p.f_out) p.f_out[s - 1] = (uint8_t)drawn; }
                }
            }
            if (DBG && forced >= 0) drawn = forced;
            if (!half) {
                if (writer && warp == 0 && lane == 0 && p.out) p.out[s - 1] = (int16_t)(256 * c_prev + drawn - 32768);
                f_prev = drawn;
            }
            SSTAMP(5);
            if (!last && !my_bad) gates(half, s, drawn, gp);
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&pub_bar)) : "memory");
            if (half) c_prev = drawn;
            SSTAMP(6);
        }
    }

#ifdef WRNN_PROFILE_SPARSE
    if (blockIdx.x == 0 && tid == 0) for (int i = 0; i < 16; ++i) g_sprof[i] += s_sprof[i];
#endif
    const int any_bad = __syncthreads_or(my_bad);
    if (writer && !any_bad) {
        if (p.h_out) for (int i = tid; i < K; i += blockDim.x) { p.h_out[i] = vecC[i]; p.h_out[K + i] = vecF[i]; }
        if (tid == 0) {
            if (p.c_st_out) p.c_st_out[0] = (uint8_t)c_prev;
            if (p.f_st_out) p.f_st_out[0] = (uint8_t)f_prev;
        }
    }
    cluster.sync();
}

// ---------------------------------------------------------------------------------------------
static size_t a16(size_t x) { return (x + 15) & ~(size_t)15; }

static int sparse_smem_bytes(const SparsePack &k)
{
    size_t b = k.blob_bytes;
    b += (size_t)3 * k.K * 4;                      // vecC, vecF, qvec
    b += (size_t)2 * 6 * k.UC * 4;                 // a_part, a_full
    b += 256 * 4;                                  // part
    b += (size_t)2 * k.K * 4;                      // the cluster's hidden layer (K floats in use)
    b += (size_t)k.K * 8;                          // qbuf: [K/2] x 16 B
    b += 128 * 16;                                 // lall: [2][256] floats
    return (int)b;
}

static uint16_t bf16_bits_s(float rounded)
{
    uint32_t b;
    std::memcpy(&b, &rounded, 4);
    return (uint16_t)(b >> 16);
}

int sparse_supported(const wrnn_model *m, int batch, std::string *why)
{
    if (batch != 1) { if (why) *why = "single-stream kernel"; return WRNN_ERR_UNSUPPORTED; }
    if (!m->sparse_pack) { if (why) *why = "model was not packed for the sparse cluster kernel"; return WRNN_ERR_UNSUPPORTED; }
    return WRNN_OK;
}

static void *sparse_fn(int mode) { return mode == 1 ? (void *)sparse_cluster_kernel<8, 1> : mode == 3 ? (void *)sparse_cluster_kernel<8, 3> : (void *)sparse_cluster_kernel<8, 0>; }

static void sparse_fill_launch(const SparsePack &k, cudaLaunchConfig_t *cfg, cudaLaunchAttribute *at, cudaStream_t s, bool coop)
{
    std::memset(cfg, 0, sizeof(*cfg));
    cfg->gridDim = dim3(SCS * k.NC);
    cfg->blockDim = dim3(SNW * 32);
    cfg->dynamicSmemBytes = k.smem_bytes;
    cfg->stream = s;
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = SCS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative;
    at[1].val.cooperative = 1;
    cfg->attrs = at;
    cfg->numAttrs = coop ? 2 : 1;
}

int sparse_prepare(wrnn_model *m)
{
    const int H = m->H, Hh = H / 2;
    if (m->dtype != WRNN_BF16) { m->err = "sparse cluster kernel stores bf16 weights"; return WRNN_ERR_UNSUPPORTED; }
    if (!m->sparse) { m->err = "model has no block masks"; return WRNN_ERR_UNSUPPORTED; }
    const bool tall = m->mask_br == 16 && m->mask_bc == 1;
    if (!tall && (m->mask_br != 4 || m->mask_bc != 4)) { m->err = "sparse cluster kernel takes 4 x 4 or 16 x 1 blocks"; return WRNN_ERR_UNSUPPORTED; }
    if (Hh != 1024) { m->err = "only H/2 = 1024 is instantiated (8 warps x 8 k-tiles for the logits tile)"; return WRNN_ERR_UNSUPPORTED; }
    // The rows of R are dealt over NC clusters of 16 (the heads are held once per cluster); more clusters mean fewer block
    // rows per CTA in the phase that dominates the step, at the price of the state crossing the chip through L2 instead
    // of the cluster's shared memory.  The largest count that divides the units and can be co-resident is taken.
    // WRNN_SPARSE_CLUSTERS = 1 / 2 / 4 forces one (diagnostic).
    SparsePack k;
    std::vector<uint8_t> blob;
    int64_t kept_bytes = 0;
    auto pack = [&](int nc) -> int {
    k = SparsePack();
        k.NC = nc;
        const int NCTA = nc * SCS;
        k.H = H; k.K = Hh; k.NKT = Hh / 16; k.UC = Hh / NCTA; k.HR = Hh / SCS;
        const int BRH = tall ? 16 : 4;                                 // rows of one block
        k.tall = tall ? 1 : 0;
        k.NBR = (k.HR + 6 * k.UC) / BRH;
        const int UC = k.UC, HR = k.HR, NBR = k.NBR, Kb = Hh / 4;      // Kb: 4-wide block columns per half
        if (Hh % NCTA != 0 || HR % BRH != 0 || UC % BRH != 0 || UC % 4 != 0) { m->err = "block height does not divide the rows of one CTA"; return WRNN_ERR_UNSUPPORTED; }

        // kept blocks of each phase of each CTA.  A block is 16 weights: a 4 x 4 block row-major, or the 16 rows of one column;
        // col is the block column (4 x 4) or the column (16 x 1) inside the phase's input half.
        struct Blk { uint16_t col; float v[16]; };
        std::vector<std::vector<std::vector<Blk>>> rows(NCTA * 2);      // [cta * 2 + phase][local block row] -> blocks
        const BsrHost *Oa[2] = {&m->hO1, &m->hO3};
        for (int cta = 0; cta < NCTA; ++cta)
            for (int ph = 0; ph < 2; ++ph) {
                const int rank = cta % SCS;                            // head rows go by the rank inside the cluster
                auto &R = rows[cta * 2 + ph];
                R.assign(NBR, {});
                for (int lbr = 0; lbr < NBR; ++lbr) {
                    // the 4-row block rows of the source matrix under this block row, and the range of its 4-wide block columns
                    const BsrHost *M;
                    int br0, bc_lo, bc_hi;
                    if (lbr < HR / BRH) {
                        M = Oa[ph];
                        br0 = (rank * HR + lbr * BRH) / 4; bc_lo = 0; bc_hi = Kb;
                    } else {
                        const int q = lbr - HR / BRH;                  // (half * 3 + gate) * (UC / BRH) + u
                        const int half = q / (3 * (UC / BRH)), gate = (q / (UC / BRH)) % 3, u = q % (UC / BRH);
                        M = &m->hR;
                        br0 = (gate * H + half * Hh + cta * UC + u * BRH) / 4; bc_lo = ph * Kb; bc_hi = bc_lo + Kb;
                    }
                    if (!tall) {
                        for (int i = M->row_ptr[br0]; i < M->row_ptr[br0 + 1]; ++i) {
                            const int bc = M->col[i];
                            if (bc < bc_lo || bc >= bc_hi) continue;
                            Blk b;
                            b.col = (uint16_t)(bc - bc_lo);
                            std::memcpy(b.v, &M->vals[(size_t)i * 16], sizeof(b.v));
                            R[lbr].push_back(b);
                        }
                    } else {
                        // columns with a nonzero weight in any of the 16 rows, in ascending order
                        std::vector<int> slot((size_t)4 * Kb, -1);
                        std::vector<Blk> found;
                        for (int r4 = 0; r4 < 4; ++r4)
                            for (int i = M->row_ptr[br0 + r4]; i < M->row_ptr[br0 + r4 + 1]; ++i) {
                                const int bc = M->col[i];
                                if (bc < bc_lo || bc >= bc_hi) continue;
                                for (int c = 0; c < 4; ++c) {
                                    bool any = false;
                                    for (int r = 0; r < 4; ++r) any = any || M->vals[(size_t)i * 16 + 4 * r + c] != 0.f;
                                    if (!any) continue;
                                    const int col = 4 * (bc - bc_lo) + c;
                                    if (slot[col] < 0) { slot[col] = (int)found.size(); Blk b; b.col = (uint16_t)col; std::memset(b.v, 0, sizeof(b.v)); found.push_back(b); }
                                    for (int r = 0; r < 4; ++r) found[slot[col]].v[4 * r4 + r] = M->vals[(size_t)i * 16 + 4 * r + c];
                                }
                            }
                        std::sort(found.begin(), found.end(), [](const Blk &a, const Blk &b) { return a.col < b.col; });
                        R[lbr] = found;
                    }
                }
            }
        // slice every (CTA, phase): block rows sorted by length (longest first, stable), dealt to the warps in runs; the
        // first w8 warps take four rows with eight lanes each, the others up to eight rows with four lanes each
        struct Slice { std::vector<int> rows; int T = 0, lpr = 4; };
        const int lpr_n = tall ? 16 : 4, cap_n = 32 / lpr_n, cap_w = cap_n / 2;     // lanes per row and rows per warp, narrow / wide slices
        int w8 = (cap_n * SNW - NBR) / (cap_n - cap_w);                              // warps that can afford wide rows
        if (w8 < 0) { m->err = "too many block rows for the warps of one CTA"; return WRNN_ERR_UNSUPPORTED; }
        if (w8 > SNW) w8 = SNW;
        if (w8 * cap_w > NBR) w8 = NBR / cap_w;
        std::vector<std::vector<Slice>> slices(NCTA * 2);              // [cta * 2 + phase][warp]
        int max_slots = 0;
        for (int cp = 0; cp < NCTA * 2; ++cp) {
            const auto &R = rows[cp];
            std::vector<int> order(NBR);
            for (int i = 0; i < NBR; ++i) order[i] = i;
            // hidden-layer block rows first (their warps send while the others still work on the rows of R), each kind longest first
            const int HRB = HR / BRH;
            std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
                const bool ha = a < HRB, hb = b < HRB;
                if (ha != hb) return ha;
                return R[a].size() > R[b].size();
            });
            slices[cp].assign(SNW, {});
            int next = 0, slots = 0;
            // split layout: hidden-layer rows (first in `order`) wide on warps [0, wh), the rows of R narrow on warps 16..19
            const int n_r = NBR - HRB, wh_split = (HRB + cap_w - 1) / cap_w;
            const bool split = SNW > SCS && wh_split <= SCS && n_r <= cap_n * (SNW - SCS);
            for (int w = 0; w < SNW; ++w) {
                Slice &sl = slices[cp][w];
                int nr;
                if (split) {
                    if (w < wh_split) { sl.lpr = 2 * lpr_n; nr = std::min(cap_w, HRB - next); }
                    else if (w < SCS) { sl.lpr = lpr_n; nr = 0; }
                    else { sl.lpr = lpr_n; const int left = NBR - next, warps_left = SNW - w; nr = (left + warps_left - 1) / warps_left; }
                } else {
                    sl.lpr = w < w8 ? 2 * lpr_n : lpr_n;
                    const int cap = 32 / sl.lpr;
                    // rows still to place, spread evenly over the remaining four-lane warps
                    nr = cap;
                    if (w >= w8) { const int left = NBR - next, warps_left = SNW - w; nr = (left + warps_left - 1) / warps_left; }
                    if (nr > cap) nr = cap;
                }
                if (nr > NBR - next) nr = NBR - next;
                size_t longest = 0;
                for (int i = 0; i < nr; ++i) { sl.rows.push_back(order[next + i]); longest = std::max(longest, R[order[next + i]].size()); }
                next += nr;
                sl.T = (int)((longest + sl.lpr - 1) / sl.lpr);
                if (sl.T < 1) sl.T = 1;                                  // the loop's first loads are unconditional
                slots += sl.lpr * nr * sl.T;
            }
            if (split) k.WH = wh_split;
            if (next != NBR) { m->err = "too many block rows for the warps of one CTA"; return WRNN_ERR_UNSUPPORTED; }
            max_slots = std::max(max_slots, slots);

        }
        k.max_slots = (max_slots + 7) & ~7;

        size_t off = 0;
        for (int ph = 0; ph < 2; ++ph) {
            k.off_meta[ph] = off; off = a16(off + (size_t)SNW * sizeof(SliceMeta));
            k.off_col[ph] = off; off = a16(off + (size_t)k.max_slots * 2);
            k.off_val[ph] = off; off = a16(off + (size_t)k.max_slots * 32);
        }
        const size_t frag = (size_t)k.NKT * 512;
        k.off_o2 = off; off += frag;
        k.off_o4 = off; off += frag;
        k.off_small = off; off = a16(off + ((size_t)6 * UC * 3 + 2 * HR + 32) * 4);
        k.blob_bytes = off;
        k.smem_bytes = sparse_smem_bytes(k);

        cudaDeviceProp prop;
        cudaGetDeviceProperties(&prop, m->device);
        if ((size_t)k.smem_bytes > prop.sharedMemPerBlockOptin) { m->err = "pruned model does not fit the shared memory of the clusters"; return WRNN_ERR_UNSUPPORTED; }
        bool attr_ok = true;
        for (int mode : {0, 1, 3})
            attr_ok = attr_ok && cudaFuncSetAttribute(sparse_fn(mode), cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
                      cudaFuncSetAttribute(sparse_fn(mode), cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem_bytes) == cudaSuccess;
        if (!attr_ok) {
            cudaGetLastError(); m->err = "cannot configure the 16-CTA cluster kernel"; return WRNN_ERR_UNSUPPORTED;
        }
        cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
        sparse_fill_launch(k, &cfg, at, 0, false);
        int max_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&max_clusters, sparse_fn(0), &cfg) != cudaSuccess || max_clusters < nc) {
            cudaGetLastError(); m->err = "the 16-CTA clusters cannot all be co-resident on this device"; return WRNN_ERR_UNSUPPORTED;
        }

        blob.assign((size_t)NCTA * k.blob_bytes, 0);
        const BsrHost *Ob[2] = {&m->hO2, &m->hO4};
        kept_bytes = 0;
        for (int cta = 0; cta < NCTA; ++cta) {
            const int rank = cta % SCS;
            uint8_t *base = blob.data() + (size_t)cta * k.blob_bytes;
            for (int ph = 0; ph < 2; ++ph) {
                SliceMeta *meta = reinterpret_cast<SliceMeta *>(base + k.off_meta[ph]);
                uint16_t *col = reinterpret_cast<uint16_t *>(base + k.off_col[ph]);
                uint16_t *val = reinterpret_cast<uint16_t *>(base + k.off_val[ph]);       // [slot plane][8 bf16]
                const auto &R = rows[cta * 2 + ph];
                int slot0 = 0, n = 0, n_r = 0;
                for (int w = 0; w < SNW; ++w) {
                    const Slice &sl = slices[cta * 2 + ph][w];
                    const int nl = sl.lpr * (int)sl.rows.size();
                    meta[w].voff = 2 * slot0; meta[w].coff = slot0; meta[w].T = sl.T; meta[w].nl = nl; meta[w].lpr = sl.lpr;
                    for (int g = 0; g < 8; ++g) meta[w].row[g] = g < (int)sl.rows.size() ? (int16_t)sl.rows[g] : (int16_t)-1;
                    for (int g = 0; g < (int)sl.rows.size(); ++g) {
                        const auto &blocks = R[sl.rows[g]];
                        for (int i = 0; i < (int)blocks.size(); ++i) {
                            const int t = i / sl.lpr, lane = sl.lpr * g + i % sl.lpr;
                            col[slot0 + t * nl + lane] = blocks[i].col;
                            for (int h = 0; h < 2; ++h)                  // plane h holds rows 2 h, 2 h + 1 of the block
                                for (int e = 0; e < 8; ++e)
                                    val[((size_t)2 * slot0 + (size_t)(2 * t + h) * nl + lane) * 8 + e] = bf16_bits_s(blocks[i].v[8 * h + e]);
                            ++n;
                            if (sl.rows[g] >= HR / BRH) ++n_r;
                        }
                    }
                    slot0 += nl * sl.T;
                }
                // every kept block of R once; the heads once (cluster 0 stands for all)
                kept_bytes += cta < SCS ? (int64_t)n * 34 + (int64_t)(NBR + 1) * 4 : (int64_t)n_r * 34;
            }
            // dense O2 / O4: 16 rows of this CTA, row-major bf16
            for (int h = 0; h < 2; ++h) {
                uint16_t *dst = reinterpret_cast<uint16_t *>(base + (h ? k.off_o4 : k.off_o2));
                std::vector<uint16_t> dense((size_t)16 * Hh, 0);
                const BsrHost &M = *Ob[h];
                for (int r = 0; r < 16; ++r) {
                    const int row = rank * 16 + r, br = row / 4, rr = row % 4;
                    for (int i = M.row_ptr[br]; i < M.row_ptr[br + 1]; ++i)
                        for (int c = 0; c < 4; ++c) dense[(size_t)r * Hh + 4 * M.col[i] + c] = bf16_bits_s(M.vals[(size_t)i * 16 + 4 * rr + c]);
                }
                std::memcpy(dst, dense.data(), dense.size() * 2);
            }
            float *sm = reinterpret_cast<float *>(base + k.off_small);
            for (int rr = 0; rr < 6 * UC; ++rr) {
                const int half = rr / (3 * UC), gate = (rr / UC) % 3, u = rr % UC;
                const int mrow = gate * H + half * Hh + cta * UC + u;
                for (int c = 0; c < 3; ++c) sm[rr * 3 + c] = m->hI[(size_t)mrow * 3 + c];
            }
            float *b = sm + 6 * UC * 3;
            for (int r = 0; r < HR; ++r) { b[r] = m->hb1[rank * HR + r]; b[HR + r] = m->hb3[rank * HR + r]; }
            b += 2 * HR;
            for (int r = 0; r < 16; ++r) { b[r] = m->hb2[rank * 16 + r]; b[16 + r] = m->hb4[rank * 16 + r]; }
        }
        return WRNN_OK;
    };
    {
        const char *force = getenv("WRNN_SPARSE_CLUSTERS");
        int rc = WRNN_ERR_UNSUPPORTED;
        for (int nc : {4, 2, 1}) {
            if (force && atoi(force) != nc) continue;
            rc = pack(nc);
            if (rc == WRNN_OK) break;
        }
        if (rc != WRNN_OK) return rc;
    }
    SparsePack *pk = new SparsePack(k);
    if (cudaMalloc((void **)&pk->d_blob, blob.size()) != cudaSuccess ||
        cudaMemcpy(pk->d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError(); cudaFree(pk->d_blob); delete pk;
        m->err = "device allocation for the sparse cluster kernel failed";
        return WRNN_ERR_NOMEM;
    }
    if (cudaMalloc((void **)&pk->d_slots, (size_t)4 * Hh * 8) != cudaSuccess) {
        cudaGetLastError(); cudaFree(pk->d_blob); delete pk;
        m->err = "device allocation for the sparse cluster kernel failed";
        return WRNN_ERR_NOMEM;
    }
    pk->weight_bytes_per_step = kept_bytes + (int64_t)2 * 256 * Hh * 2 + (int64_t)3 * H * 3 * 4;
    m->sparse_pack = pk;
    return WRNN_OK;
}

void sparse_destroy(wrnn_model *m)
{
    if (!m->sparse_pack) return;
    cudaFree(m->sparse_pack->d_blob);
    cudaFree(m->sparse_pack->d_slots);
    delete m->sparse_pack;
    m->sparse_pack = nullptr;
}

int sparse_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes)
{
    (void)batch;
    const SparsePack &k = *m->sparse_pack;
    if (n_ctas) *n_ctas = SCS * k.NC;
    if (n_threads) *n_threads = SNW * 32;
    if (smem) *smem = k.smem_bytes;
    if (weight_bytes) *weight_bytes = k.weight_bytes_per_step;
    return WRNN_OK;
}

int sparse_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    const SparsePack &k = *m->sparse_pack;
    SparseParams p;
    std::memset(&p, 0, sizeof(p));
    p.H = k.H; p.K = k.K; p.NKT = k.NKT; p.UC = k.UC; p.HR = k.HR; p.NBR = k.NBR; p.tall = k.tall; p.WH = k.WH;
    for (int ph = 0; ph < 2; ++ph) { p.off_meta[ph] = k.off_meta[ph]; p.off_col[ph] = k.off_col[ph]; p.off_val[ph] = k.off_val[ph]; }
    p.off_o2 = k.off_o2; p.off_o4 = k.off_o4; p.off_small = k.off_small; p.blob_bytes = k.blob_bytes;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.blob = k.d_blob; p.g = m->g; p.yslots = k.d_slots;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in; p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;
    { const char *e = getenv("WRNN_SPARSE_POLL_GAP"); p.poll_gap = e ? atoi(e) : 0; }

    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(k.d_slots, 0, (size_t)4 * k.K * 8, s) != cudaSuccess) return WRNN_ERR_CUDA;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
    sparse_fill_launch(k, &cfg, at, s, coop_launch_allowed());
    void *args[] = {&p};
    const bool teacher = p.c_forced || p.f_forced || p.dbg_gates || p.dbg_h || p.dbg_logits;
    cudaError_t e = cudaLaunchKernelExC(&cfg, sparse_fn(m->dbg_skip_cta >= 0 ? 1 : (teacher ? 3 : 0)), args);
    if (e != cudaSuccess) {
        m->err = std::string("sparse cluster kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    return WRNN_OK;
}

}  // namespace wrnn

#ifdef WRNN_PROFILE_SPARSE
extern "C" int wrnn_debug_sparse_prof(long long *out16, int reset)
{
    if (reset) { long long z[16] = {0}; return cudaMemcpyToSymbol(wrnn::g_sprof, z, sizeof(z)) == cudaSuccess ? 0 : 4; }
    return cudaMemcpyFromSymbol(out16, wrnn::g_sprof, 16 * sizeof(long long)) == cudaSuccess ? 0 : 4;
}
#endif
